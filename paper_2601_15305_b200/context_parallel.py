"""Context-parallel prefill: one long sequence split over the ranks of a process group by query rows.

Row t of the indexer (Eq. 7) and of the attention (Eq. 11) reads only keys s <= t, and rows do not depend on
one another, so the path shards by query rows with ONE exchange: every rank needs the indexer keys k^I, the
keys K and the gated values V' (Eq. 9) of every position up to its own last row.  Each rank therefore gates
its own shard of V, the ranks all-gather the three key-side tensors into their own memory (a plain
all_gather of torch.distributed: NCCL on GPUs, gloo on CPUs; the kernels only ever read local memory), and
each rank then runs the unchanged single-GPU path on its row blocks: a block of rows [t0, t1) of a causal
prefill is the library's chunked-prefill geometry Lq = t1 - t0, Lk = t1.

Rows cost differently (row t scores t + 1 keys), so contiguous shards would leave the last rank with almost
twice the mean work.  The sequence is cut into 2 * world * pairs chunks and rank r takes, of every group of
2 * world consecutive chunks, chunk r and chunk 2 * world - 1 - r (an early one and a late one): row counts
are equal and the sums of visible keys agree to within a fraction of a per cent.

This module is host-side plumbing: partition arithmetic, the exchange, the loop over blocks.  Every step of
the path itself runs in the library's kernels (`forward_block` defaults to the C-ABI binding and fails
loudly without the CUDA library).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Dict, List, Optional, Sequence

import torch
import torch.distributed as dist

from .inputs import GsaConfig

KEY_SIDE = ("kI", "K", "Vg")            # what is exchanged: indexer keys, keys, gated values
QUERY_SIDE = ("Q", "qI", "w", "g1")     # what stays on the rank that owns the rows


@dataclass(frozen=True)
class RowBlock:
    t0: int          # first row (= first key position) of the block
    t1: int          # one past its last row

    @property
    def rows(self) -> int:
        return self.t1 - self.t0


def chunk_bounds(L: int, world: int, pairs: int = 1) -> List[int]:
    """Boundaries of the 2 * world * pairs chunks the sequence is cut into (sizes differ by at most one row)."""
    n = 2 * world * pairs
    if L < n:
        raise ValueError(f"a sequence of {L} rows cannot be cut into {n} chunks")
    return [(L * c) // n for c in range(n + 1)]


def chunk_owner(c: int, world: int) -> int:
    """Rank that owns chunk c: within every group of 2 * world chunks, rank r has chunks r and 2 * world - 1 - r."""
    m = c % (2 * world)
    return m if m < world else 2 * world - 1 - m


def plan_row_blocks(L: int, world: int, rank: int, pairs: int = 1) -> List[RowBlock]:
    """The row blocks of `rank`, in position order."""
    b = chunk_bounds(L, world, pairs)
    return [RowBlock(b[c], b[c + 1]) for c in range(len(b) - 1) if chunk_owner(c, world) == rank]


def visible_pairs(blocks: Sequence[RowBlock]) -> int:
    """Sum over the blocks' rows of the number of visible keys, t + 1: the indexer's work."""
    return sum((blk.t1 * (blk.t1 + 1) - blk.t0 * (blk.t0 + 1)) // 2 for blk in blocks)


def shard(x: Dict[str, torch.Tensor], blocks: Sequence[RowBlock]) -> Dict[str, torch.Tensor]:
    """The rows of a rank, concatenated in block order, of full [1, L, ...] tensors (what a rank would hold)."""
    return {k: torch.cat([v[:, blk.t0:blk.t1] for blk in blocks], dim=1).contiguous() for k, v in x.items()}


def all_gather_keys(local: Dict[str, torch.Tensor], L: int, world: int, rank: int, pairs: int = 1,
                    group=None) -> Dict[str, torch.Tensor]:
    """All-gather the key-side tensors ([1, local rows, ...] each, block order) into full [1, L, ...] tensors
    in position order, in this rank's own memory.  Shards may differ by a row or two, so they travel padded to
    the longest one."""
    plans = [plan_row_blocks(L, world, r, pairs) for r in range(world)]
    longest = max(sum(b.rows for b in p) for p in plans)
    full = {}
    for name in KEY_SIDE:
        mine = local[name]
        pad = torch.zeros((1, longest) + tuple(mine.shape[2:]), dtype=mine.dtype, device=mine.device)
        pad[:, : mine.shape[1]] = mine
        if world > 1:
            parts = [torch.empty_like(pad) for _ in range(world)]
            dist.all_gather(parts, pad, group=group)
        else:
            parts = [pad]
        out = torch.empty((1, L) + tuple(mine.shape[2:]), dtype=mine.dtype, device=mine.device)
        for r in range(world):
            at = 0
            for blk in plans[r]:
                out[:, blk.t0:blk.t1] = parts[r][:, at:at + blk.rows]
                at += blk.rows
        full[name] = out
    return full


def _forward_block_cuda(cfg: GsaConfig, blk: RowBlock, q: Dict[str, torch.Tensor], keys: Dict[str, torch.Tensor],
                        bI: Optional[torch.Tensor]):
    """One row block through gsa_forward: chunked-prefill geometry, values already gated (g2_logits = NULL)."""
    from . import binding as gsa
    c = cfg.with_(B=1, Lq=blk.rows, Lk=blk.t1)
    p = gsa.make_params(c)
    out = torch.empty_like(q["Q"])
    kt = torch.empty((1, blk.rows), dtype=torch.int32, device=out.device)
    ws = torch.empty(gsa.gsa_workspace_bytes(p, 0), dtype=torch.uint8, device=out.device)
    gsa.gsa_forward(p, q["Q"], keys["K"][:, : blk.t1], keys["Vg"][:, : blk.t1], q["qI"], keys["kI"][:, : blk.t1], q["w"], bI,
                    q["g1"], None, out, None, kt, None, 0, ws)
    if gsa.gsa_device_status(ws) != 0:
        raise gsa.GsaError("gsa_forward reported a device-side condition in a context-parallel block")
    return out, kt


def _value_gate_cuda(V: torch.Tensor, g2: torch.Tensor) -> torch.Tensor:
    from . import binding as gsa
    Vg = torch.empty_like(V)
    gsa.gsa_value_gate(V, g2, Vg)
    return Vg


def forward_context_parallel(cfg: GsaConfig, local: Dict[str, torch.Tensor], world: int, rank: int, pairs: int = 1,
                             group=None, bI: Optional[torch.Tensor] = None,
                             forward_block: Optional[Callable] = None, value_gate: Optional[Callable] = None,
                             gathered_keys: Optional[Dict[str, torch.Tensor]] = None):
    """GSA forward of a causal prefill (B = 1, Lq = Lk = cfg.Lk) for the rows of `rank`.

    local: this rank's rows of Q, K, V, qI, kI, w, g1, g2 as [1, local rows, ...] tensors in block order
    (see `shard`).  Returns (out [1, local rows, n_h, d_h], kt [1, local rows]) in the same order.
    `forward_block` / `value_gate` default to the library's CUDA entry points.  `gathered_keys` (full kI, K, Vg
    in position order) skips the exchange: for a caller that already holds them, or runs the ranks' shares one
    after another in a single process."""
    if cfg.B != 1 or cfg.Lq != cfg.Lk:
        raise ValueError("context-parallel prefill takes one sequence with Lq == Lk")
    forward_block = forward_block or _forward_block_cuda
    value_gate = value_gate or _value_gate_cuda
    L = cfg.Lk
    blocks = plan_row_blocks(L, world, rank, pairs)
    if gathered_keys is not None:
        keys = gathered_keys
    else:
        # Eq. 9 on the rank's own shard, then the one exchange of the path
        keys_local = {"kI": local["kI"], "K": local["K"], "Vg": value_gate(local["V"], local["g2"])}
        keys = all_gather_keys(keys_local, L, world, rank, pairs, group)
    outs, kts, at = [], [], 0
    for blk in blocks:
        q = {k: local[k][:, at:at + blk.rows].contiguous() for k in QUERY_SIDE}
        o, kt = forward_block(cfg, blk, q, keys, bI)
        outs.append(o)
        kts.append(kt)
        at += blk.rows
    return torch.cat(outs, dim=1), torch.cat(kts, dim=1)
