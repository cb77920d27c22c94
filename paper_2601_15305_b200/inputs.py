"""Seeded synthetic inputs for the GSA forward path.

This module only draws random tensors and plants "needle" keys.  It holds none of
the method's arithmetic (no indexer score, no budget, no softmax): both the CPU
oracle tests and the CUDA path read the tensors it makes, and nothing else is
shared between the two.

Layouts (all contiguous, token-major):
    Q   [B, Lq, n_h,  d_h]  bf16   queries, already projected / rotated
    K   [B, Lk, n_kv, d_h]  bf16
    V   [B, Lk, n_kv, d_h]  bf16
    qI  [B, Lq, HI,   dI ]  bf16   indexer queries  q^I_{t,j}
    kI  [B, Lk, dI]         bf16   shared indexer key k^I_s
    w   [B, Lq, HI]         fp32   indexer head weights, already in (0,1)
    g1  [B, Lq, n_h,  d_h]  bf16   output-gate logits (pre-sigmoid)
    g2  [B, Lk, n_kv, d_h]  bf16   value-gate logits  (pre-sigmoid)

Recipe: base tensors are i.i.d. N(0,1)/sqrt(d) rounded to bf16; in every block of
128 key positions 8 positions are turned into needles: each is paired with a query
position t >= s drawn uniformly ("random depth") and overwritten with
0.8 * (the paired query vector) + 0.6 * noise / sqrt(d), for the indexer key
(against one random indexer head of the paired query) and for every KV head's key
(against the first query head of that KV group).  This imitates the structure of a
long-context retrieval workload without using any item of a published suite.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict

import torch


@dataclass(frozen=True)
class GsaConfig:
    name: str
    B: int
    Lq: int
    Lk: int
    n_h: int
    n_kv: int
    d_h: int
    HI: int
    dI: int
    k_base: int
    k_min: int
    k_max: int
    seed: int
    # v_bar: the caller-owned running mean of score variance (Eq. 8).  The values
    # stored here were written by oracle/calibrate_vbar.py (median row variance of
    # the generated data), so that k_t centres on k_base.
    v_bar: float
    sharp_mix: bool = False      # per-128-row-block sharpness scale on qI (config 3)
    needles_per_block: int = 8
    block: int = 128

    @property
    def decode(self) -> bool:
        return self.Lq != self.Lk

    def with_(self, **kw) -> "GsaConfig":
        return replace(self, **kw)


# The five workloads.  Shapes follow the 1.7B-model layer the metric is quoted on
# (hidden 2048, 16 query heads, d_h 128) with 8 KV heads, 8 indexer heads of width 64.
CONFIGS: Dict[str, GsaConfig] = {
    "tiny": GsaConfig("tiny", 1, 512, 512, 4, 1, 64, 4, 32, 64, 16, 128, seed=0,
                      v_bar=1.9326e-03),
    "l8k": GsaConfig("l8k", 1, 8192, 8192, 16, 8, 128, 8, 64, 2048, 512, 4096, seed=1,
                     v_bar=2.0198e-03),
    "l32k": GsaConfig("l32k", 1, 32768, 32768, 16, 8, 128, 8, 64, 2048, 512, 4096, seed=2,
                      v_bar=1.4700e-03, sharp_mix=True),
    "l128k": GsaConfig("l128k", 1, 131072, 131072, 16, 8, 128, 8, 64, 2048, 512, 4096, seed=3,
                       v_bar=2.0780e-03),
    "decode": GsaConfig("decode", 32, 1, 131072, 16, 8, 128, 8, 64, 2048, 512, 4096, seed=4,
                        v_bar=1.5521e-03),
}


def _randn(gen: torch.Generator, *shape: int) -> torch.Tensor:
    return torch.randn(*shape, generator=gen, dtype=torch.float32)


def make_inputs(cfg: GsaConfig, batch_slice: slice | None = None) -> Dict[str, torch.Tensor]:
    """Draw the tensors of one workload on the CPU.

    `batch_slice` restricts generation to some batch elements (each batch element has
    its own generator stream, so slices are consistent with the full draw); used by
    the decode workload to bound host memory.
    """
    bs = range(cfg.B)[batch_slice] if batch_slice is not None else range(cfg.B)
    outs = [_make_one(cfg, b) for b in bs]
    return {k: torch.stack([o[k] for o in outs], dim=0) for k in outs[0]}


def _make_one(cfg: GsaConfig, b: int) -> Dict[str, torch.Tensor]:
    gen = torch.Generator(device="cpu")
    gen.manual_seed(cfg.seed * 1000003 + b)
    Lq, Lk = cfg.Lq, cfg.Lk
    G = cfg.n_h // cfg.n_kv

    Q = _randn(gen, Lq, cfg.n_h, cfg.d_h) / cfg.d_h ** 0.5
    K = _randn(gen, Lk, cfg.n_kv, cfg.d_h) / cfg.d_h ** 0.5
    V = _randn(gen, Lk, cfg.n_kv, cfg.d_h) / cfg.d_h ** 0.5
    qI = _randn(gen, Lq, cfg.HI, cfg.dI) / cfg.dI ** 0.5
    kI = _randn(gen, Lk, cfg.dI) / cfg.dI ** 0.5
    w = torch.sigmoid(_randn(gen, Lq, cfg.HI))
    g1 = _randn(gen, Lq, cfg.n_h, cfg.d_h)
    g2 = _randn(gen, Lk, cfg.n_kv, cfg.d_h)

    if cfg.sharp_mix:
        # sharp rows (wide score spread) and flat rows (narrow spread), block by block
        nblk = (Lq + cfg.block - 1) // cfg.block
        expo = torch.rand(nblk, generator=gen, dtype=torch.float32) * 2.0 - 1.0
        scale = torch.pow(torch.tensor(2.0), expo).repeat_interleave(cfg.block)[:Lq]
        qI = qI * scale[:, None, None]

    # the vectors needles are built from are the bf16-rounded queries
    Q = Q.to(torch.bfloat16)
    qI = qI.to(torch.bfloat16)

    # needles: `needles_per_block` distinct key positions per block of `block` keys
    nblk_k = Lk // cfg.block
    if nblk_k > 0 and cfg.needles_per_block > 0:
        npb = cfg.needles_per_block
        perm = torch.rand(nblk_k, cfg.block, generator=gen).argsort(dim=1)[:, :npb]
        s_pos = (perm + torch.arange(nblk_k)[:, None] * cfg.block).reshape(-1)       # [N]
        N = s_pos.numel()
        off = Lk - Lq                       # query t sees keys s <= off + t
        t_lo = torch.clamp(s_pos - off, min=0)
        u = torch.rand(N, generator=gen)
        t_pos = (t_lo + (u * (Lq - t_lo).to(torch.float32)).to(torch.int64)).clamp(max=Lq - 1)
        j_star = torch.randint(0, cfg.HI, (N,), generator=gen)
        noise_i = _randn(gen, N, cfg.dI) / cfg.dI ** 0.5
        noise_k = _randn(gen, N, cfg.n_kv, cfg.d_h) / cfg.d_h ** 0.5
        if cfg.decode:
            # one needle per block is paired with the (single) decode query; the others
            # are paired with queries that are not part of this step: random vectors.
            ghost_qI = (_randn(gen, N, cfg.dI) / cfg.dI ** 0.5)
            ghost_Q = (_randn(gen, N, cfg.n_kv, cfg.d_h) / cfg.d_h ** 0.5)
            real = torch.zeros(N, dtype=torch.bool)
            real[::npb] = True
            src_i = torch.where(real[:, None], qI[t_pos, j_star].float(), ghost_qI)
            src_k = torch.where(real[:, None, None], Q[t_pos][:, ::G, :].float(), ghost_Q)
        else:
            src_i = qI[t_pos, j_star].float()
            src_k = Q[t_pos][:, ::G, :].float()
        kI[s_pos] = 0.8 * src_i + 0.6 * noise_i
        K[s_pos] = 0.8 * src_k + 0.6 * noise_k

    return {
        "Q": Q.contiguous(),
        "K": K.to(torch.bfloat16).contiguous(),
        "V": V.to(torch.bfloat16).contiguous(),
        "qI": qI.contiguous(),
        "kI": kI.to(torch.bfloat16).contiguous(),
        "w": w.contiguous(),
        "g1": g1.to(torch.bfloat16).contiguous(),
        "g2": g2.to(torch.bfloat16).contiguous(),
    }


def sample_rows(cfg: GsaConfig, n: int, seed: int = 0) -> torch.Tensor:
    """Query positions for sampled parity checks: the edge rows (first row, the rows
    around k_min / k_max visible keys, the last row) plus `n` stratified rows."""
    off = cfg.Lk - cfg.Lq
    edge = [0, cfg.Lq - 1]
    for k in (cfg.k_min, cfg.k_max):
        for d in (-2, -1, 0):
            t = k + d - off
            if 0 <= t < cfg.Lq:
                edge.append(t)
    gen = torch.Generator().manual_seed(seed + 17)
    if n > 0:
        strata = torch.linspace(0, cfg.Lq, n + 1)
        lo, hi = strata[:-1], strata[1:]
        r = (lo + torch.rand(n, generator=gen) * (hi - lo)).to(torch.int64).clamp(0, cfg.Lq - 1)
        edge.extend(r.tolist())
    return torch.tensor(sorted(set(edge)), dtype=torch.int64)
