"""Context-parallel prefill (paper_2601_15305_b200/context_parallel.py): the partition arithmetic, and, with two
gloo ranks on the CPU, the exchange and the per-block geometry.  The per-block compute is stood in for by the
CPU oracle here (the product default is the CUDA library): what is tested is that the rows of the two ranks,
each computed from gathered keys in the chunked-prefill geometry Lq = block rows, Lk = block end, concatenate
to what the oracle gives for the whole sequence in one piece."""
import os
import sys
import tempfile

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2601_15305_b200 import context_parallel as cp
from paper_2601_15305_b200.inputs import CONFIGS, make_inputs


def test_every_row_has_exactly_one_owner_and_work_is_balanced():
    for L, world, pairs in ((131072, 2, 1), (131072, 4, 1), (131072, 8, 1), (131072, 8, 4), (32768, 4, 2),
                            (1000, 3, 2), (777, 2, 5), (64, 8, 1)):
        owner = np.full(L, -1)
        plans = [cp.plan_row_blocks(L, world, r, pairs) for r in range(world)]
        for r, plan in enumerate(plans):
            assert len(plan) == 2 * pairs
            assert all(a.t1 <= b.t0 for a, b in zip(plan, plan[1:]))          # position order, disjoint
            for blk in plan:
                assert (owner[blk.t0:blk.t1] == -1).all()
                owner[blk.t0:blk.t1] = r
        assert (owner >= 0).all()
        work = np.array([cp.visible_pairs(p) for p in plans], dtype=np.float64)
        assert work.sum() == L * (L + 1) / 2
        # closed form against a direct count
        assert cp.visible_pairs(plans[0]) == sum(t + 1 for blk in plans[0] for t in range(blk.t0, blk.t1))
        rows = np.array([sum(b.rows for b in p) for p in plans])
        assert rows.max() - rows.min() <= 2 * pairs
        if L >= 1000 * world:
            assert np.abs(work / work.mean() - 1).max() <= 0.01
    # contiguous shards, for contrast: the last of 8 ranks would carry 1.87 times the mean work
    L, world = 131072, 8
    last = cp.visible_pairs([cp.RowBlock(L - L // world, L)])
    assert last / (L * (L + 1) / 2 / world) > 1.8


def _oracle_block(cfg, blk, q, keys, bI):
    """Stand-in for the CUDA path of one block: the oracle in the block's chunked-prefill geometry, values
    already gated (gate logits of +40: sigmoid is exactly 1 in fp64)."""
    import oracle
    c = cfg.with_(B=1, Lq=blk.rows, Lk=blk.t1)
    p = oracle.OracleParams.from_config(c, v_bar=float(np.float32(c.v_bar)))
    K, Vg, kI = keys["K"][:, : blk.t1], keys["Vg"][:, : blk.t1], keys["kI"][:, : blk.t1]
    o = oracle.forward(p, q["Q"], K, Vg, q["qI"], kI, q["w"], q["g1"], torch.full_like(Vg, 40.0), bI,
                       rows_t=np.arange(blk.rows))
    return torch.from_numpy(o["out"])[None], torch.from_numpy(o["keff"].astype(np.int32))[None]


def _gate(V, g2):
    return V.float() * torch.sigmoid(g2.double()).float()


def _rank_main(rank: int, world: int, init_file: str, out_dir: str, pairs: int):
    dist.init_process_group("gloo", init_method=f"file://{init_file}", rank=rank, world_size=world)
    try:
        cfg = CONFIGS["tiny"].with_(Lq=509, Lk=509)              # chunks of unequal size: shards travel padded
        x = make_inputs(cfg)                                     # same seed on every rank; each keeps its rows only
        local = cp.shard(x, cp.plan_row_blocks(cfg.Lk, world, rank, pairs))
        out, kt = cp.forward_context_parallel(cfg, local, world, rank, pairs, forward_block=_oracle_block,
                                              value_gate=_gate)
        torch.save((out, kt), os.path.join(out_dir, f"r{rank}.pt"))
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_rank_oracle():
    import oracle
    world, pairs = 2, 2
    cfg = CONFIGS["tiny"].with_(Lq=509, Lk=509)
    x = make_inputs(cfg)
    p = oracle.OracleParams.from_config(cfg, v_bar=float(np.float32(cfg.v_bar)))
    want = oracle.forward(p, **x, rows_t=np.arange(cfg.Lq))
    with tempfile.TemporaryDirectory() as td:
        mp.spawn(_rank_main, args=(world, os.path.join(td, "rendezvous"), td, pairs), nprocs=world, join=True)
        seen = np.zeros(cfg.Lq, bool)
        for r in range(world):
            out, kt = torch.load(os.path.join(td, f"r{r}.pt"))
            at = 0
            for blk in cp.plan_row_blocks(cfg.Lk, world, r, pairs):
                got = out[0, at:at + blk.rows].numpy()
                assert np.abs(got - want["out"][blk.t0:blk.t1]).max() <= 1e-6      # fp32 V' against the fp64 product
                assert (kt[0, at:at + blk.rows].numpy() == want["keff"][blk.t0:blk.t1]).all()
                seen[blk.t0:blk.t1] = True
                at += blk.rows
        assert seen.all()


def test_exchange_restores_position_order_single_process():
    """world = 1 needs no process group: both chunks belong to rank 0 and the gather is the identity."""
    cfg = CONFIGS["tiny"]
    x = make_inputs(cfg)
    local = cp.shard(x, cp.plan_row_blocks(cfg.Lk, 1, 0, 3))
    keys = cp.all_gather_keys({"kI": local["kI"], "K": local["K"], "Vg": local["V"]}, cfg.Lk, 1, 0, 3)
    assert torch.equal(keys["K"], x["K"]) and torch.equal(keys["kI"], x["kI"]) and torch.equal(keys["Vg"], x["V"])
