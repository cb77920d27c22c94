"""gsa_sparse_gated_attn_fwd_static: the entry point for callers that cannot allocate device memory
(fixed memory budgets, latency-critical or callback contexts where cudaMalloc must not be entered).
Its scratch is an array inside the library image, so the call allocates nothing.

Checked here, through the C ABI, against the regular entry point and against the CPU oracle on the same
inputs: two calls in a row on different problems (the second must not see anything the first left in the
shared array), a problem whose keys span several key ranges (softmax state carried from range to range
inside the array, range-cut table behind it), a problem that fills the array to the last byte the limit
allows, and the refusal of problems larger than that.  Collected last on purpose (file name), so a run
that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_15305_b200 import binding as gsa
from paper_2601_15305_b200.inputs import CONFIGS, make_inputs

import gpu_util as U

pytestmark = pytest.mark.gpu


def _random_index_sets(cfg, seed):
    """Valid ascending index sets with varying sizes (the attention stage takes them as given)."""
    g = torch.Generator().manual_seed(seed)
    idx = torch.full((cfg.B, cfg.Lq, cfg.k_max), -1, dtype=torch.int32)
    kt = torch.empty((cfg.B, cfg.Lq), dtype=torch.int32)
    off = cfg.Lk - cfg.Lq
    for b in range(cfg.B):
        for t in range(cfg.Lq):
            n = off + t + 1
            k = min(n, int(torch.randint(cfg.k_min, cfg.k_max + 1, (1,), generator=g)))
            sel = torch.randperm(n, generator=g)[:k].sort().values
            idx[b, t, :k] = sel.to(torch.int32)
            kt[b, t] = k
    return idx.cuda(), kt.cuda()


def _both_paths(cfg, seed):
    x = make_inputs(cfg)
    d = U.to_dev(x)
    idx, kt = _random_index_sets(cfg, seed)
    p = gsa.make_params(cfg)
    want = U.run_attn(cfg, d, idx, kt)                       # regular entry point, caller's workspace
    got = torch.full_like(d["Q"], float("nan"))
    gsa.gsa_sparse_gated_attn_fwd_static(p, d["Q"], d["K"], d["V"], d["g1"], d["g2"], idx, kt, got)
    assert gsa.gsa_device_status(None) == 0          # the status word of the built-in array
    # the oracle on the same index sets (every row, or a spread of them when there are many)
    R = cfg.Lq
    rows_t = np.arange(R) if cfg.B * R <= 400 else np.unique(np.linspace(0, R - 1, 200).astype(np.int64))
    rt, rb = np.tile(rows_t, cfg.B), np.repeat(np.arange(cfg.B), len(rows_t))
    o = oracle.attn(U.oracle_params(cfg), x["Q"], x["K"], x["V"], x["g1"], x["g2"],
                    idx.cpu().numpy()[rb, rt], kt.cpu().numpy()[rb, rt], rt, rb)
    U.check_out(got.float().cpu().numpy()[rb, rt], o)
    return got.float().cpu().numpy(), want.float().cpu().numpy()


def _assert_same(got, want):
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= U.OUT_MAX_ABS_TOL
    rowmax = np.abs(want).max(axis=-1, keepdims=True)
    assert (np.abs(got - want) <= U.OUT_REL_TO_ROWMAX_TOL * rowmax + 1e-6).all()


def test_static_scratch_matches_regular_entry_point_twice():
    # call 1: a problem that fills a good part of the array; call 2: a different, smaller one
    cfg1 = CONFIGS["l8k"].with_(name="noalloc1", B=2, Lq=96, Lk=2000, k_base=300, k_min=40, k_max=512, seed=21)
    cfg2 = CONFIGS["tiny"].with_(name="noalloc2", B=1, Lq=200, Lk=333, seed=22)
    for cfg, seed in ((cfg1, 1), (cfg2, 2)):
        got, want = _both_paths(cfg, seed)
        _assert_same(got, want)


def test_static_scratch_with_several_key_ranges():
    """Enough query rows for one launch per key range: the softmax state is carried between the ranges inside
    the built-in array and the table of range cuts sits behind it (about 13 MB of the array in all)."""
    cfg = CONFIGS["l8k"].with_(name="noalloc_ranges", B=1, Lq=640, Lk=4096, k_base=300, k_min=40, k_max=512, seed=23)
    gsa.gsa_debug_set_attn_range_keys(1024)
    try:
        n0 = gsa.gsa_launch_count()
        got, want = _both_paths(cfg, 3)
        # each path: value gate, range cuts, one attention launch per range the rows can see (4), finalize passes
        assert gsa.gsa_launch_count() - n0 >= 2 * (1 + 1 + 4 + 1)
    finally:
        gsa.gsa_debug_set_attn_range_keys(0)
    _assert_same(got, want)


def _scratch_need(cfg):
    """Bytes of the built-in array the call needs: the documented limit formula."""
    p = gsa.make_params(cfg)
    return cfg.B * cfg.Lk * cfg.n_kv * cfg.d_h * 2 + gsa.gsa_attn_workspace_bytes(p, False) - 256


def test_static_scratch_accepts_up_to_the_limit_and_not_beyond():
    """One decode-shaped query over the longest cache the array can hold: accepted (and correct) there,
    refused one token above."""
    base = CONFIGS["l8k"].with_(name="noalloc_limit", B=1, Lq=1, Lk=16000, k_base=300, k_min=40, k_max=512, seed=24)
    Lk = 16000
    while _scratch_need(base.with_(Lk=Lk + 1)) <= gsa.STATIC_SCRATCH_BYTES:
        Lk += 1
    cfg = base.with_(Lk=Lk)
    assert _scratch_need(cfg) <= gsa.STATIC_SCRATCH_BYTES < _scratch_need(base.with_(Lk=Lk + 1))
    # a cache token costs n_kv * d_h * 2 bytes, so less than one token's worth of the array stays unused
    assert gsa.STATIC_SCRATCH_BYTES - _scratch_need(cfg) < cfg.n_kv * cfg.d_h * 2
    got, want = _both_paths(cfg, 4)
    _assert_same(got, want)
    big = base.with_(Lk=Lk + 1)
    x = make_inputs(big)
    d = U.to_dev(x)
    idx, kt = _random_index_sets(big, 5)
    n0 = gsa.gsa_launch_count()
    with pytest.raises(gsa.GsaError, match="scratch"):
        gsa.gsa_sparse_gated_attn_fwd_static(gsa.make_params(big), d["Q"], d["K"], d["V"], d["g1"], d["g2"], idx, kt,
                                             torch.empty_like(d["Q"]))
    assert gsa.gsa_launch_count() == n0


def test_static_scratch_rejects_oversized_problem():
    # one token more than could ever fit: 16385 tokens * 8 KV heads * 128 * 2 bytes > 32 MiB
    cfg = CONFIGS["l8k"].with_(name="toolarge", B=1, Lq=1, Lk=16385)
    assert cfg.B * cfg.Lk * cfg.n_kv * cfg.d_h * 2 > gsa.STATIC_SCRATCH_BYTES
    p = gsa.make_params(cfg)
    z = lambda *s, dt=torch.bfloat16: torch.zeros(*s, dtype=dt, device="cuda")
    Q, g1, out = (z(1, 1, cfg.n_h, cfg.d_h) for _ in range(3))
    K, V, g2 = (z(1, cfg.Lk, cfg.n_kv, cfg.d_h) for _ in range(3))
    idx, kt = z(1, 1, cfg.k_max, dt=torch.int32), torch.ones((1, 1), dtype=torch.int32, device="cuda")
    n0 = gsa.gsa_launch_count()
    with pytest.raises(gsa.GsaError, match="scratch"):
        gsa.gsa_sparse_gated_attn_fwd_static(p, Q, K, V, g1, g2, idx, kt, out)
    assert gsa.gsa_launch_count() == n0
