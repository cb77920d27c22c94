"""GPU parity of the training-side entry points against the fp64 CPU oracle, through the C ABI:
gsa_sparse_gated_attn_bwd (Eq. 9-12 and Eq. 10 differentiated, index sets fixed), gsa_vbar_update
(running mean of the score variance, Eq. 8), and the indexer's sparse-phase loss (Eq. 14):
gsa_attn_probs_mean (its target) and gsa_indexer_kl_bwd (loss and derivatives).

Tolerance of the gradients: the kernel rounds P, dS, dout*sigmoid(g1) and V' to bf16 (2^-9 each) before
the tensor-core products and every result to bf16 once; sums run in fp32.  As for the forward outputs
the bound is 2.5e-2 of the tensor's largest magnitude (not of the row's: where the exact derivative
cancels to zero, as dQ does for a row with a single key, the roundings of the two cancelling terms
remain), and the error over a whole tensor must stay below 1 % in the Frobenius norm.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_15305_b200 import binding as gsa
from paper_2601_15305_b200.inputs import CONFIGS, make_inputs

import gpu_util as U

pytestmark = pytest.mark.gpu

GRAD_REL_TO_MAX_TOL = 2.5e-2
GRAD_FROBENIUS_TOL = 1e-2


def _index_sets(cfg, q0, q1, seed, k_lo=None, k_hi=None):
    """Valid ascending random index sets for rows [q0, q1) of every batch element: [B, R, k_max], [B, R]."""
    g = torch.Generator().manual_seed(seed)
    R = q1 - q0
    idx = torch.full((cfg.B, R, cfg.k_max), -1, dtype=torch.int32)
    kt = torch.empty((cfg.B, R), dtype=torch.int32)
    for b in range(cfg.B):
        for r in range(R):
            n = cfg.Lk - cfg.Lq + q0 + r + 1
            k = min(n, int(torch.randint(k_lo or cfg.k_min, (k_hi or cfg.k_max) + 1, (1,), generator=g)))
            idx[b, r, :k] = torch.randperm(n, generator=g)[:k].sort().values.to(torch.int32)
            kt[b, r] = k
    return idx, kt


def _run_bwd(cfg, d, idx, kt, dout, q0, q1, key_range=16384, saved_lse=False, **over):
    p = gsa.make_params(cfg, q_begin=q0, q_end=q1, **over)
    out = U.run_attn(cfg, d, idx, kt, q_begin=q0, q_end=q1, **over)
    lse = None
    if saved_lse:                                    # the training-time forward call: same output, plus the statistics
        lse = torch.full((cfg.B, cfg.Lq, cfg.n_h), float("nan"), dtype=torch.float32, device="cuda")
        out2 = torch.full_like(out, float("nan"))
        wsf = torch.empty(gsa.gsa_attn_workspace_bytes(p, True), dtype=torch.uint8, device="cuda")
        gsa.gsa_sparse_gated_attn_fwd_lse(p, d["Q"], d["K"], d["V"], d["g1"], d["g2"], idx, kt, out2, lse, wsf)
        assert torch.equal(out2[:, q0:q1], out[:, q0:q1])
    nan = float("nan")
    dQ, dg1 = torch.full_like(d["Q"], nan), torch.full_like(d["Q"], nan)
    dK, dV, dg2 = (torch.full_like(d["K"], nan) for _ in range(3))
    pbar = torch.full((cfg.B, q1 - q0, cfg.k_max), nan, dtype=torch.float32, device="cuda")
    ws = torch.empty(gsa.gsa_attn_bwd_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    ws.fill_(0xFF)                               # the call must not rely on a cleared workspace
    n0 = gsa.gsa_launch_count()
    gsa.gsa_sparse_gated_attn_bwd(p, d["Q"], d["K"], d["V"], d["g1"], d["g2"], idx, kt, out, dout,
                                  dQ, dK, dV, dg1, dg2, ws, pbar=pbar, lse=lse)
    torch.cuda.synchronize()
    assert gsa.gsa_device_status(ws) == 0
    # value gate, preparation kernel, query-major kernel, count + 3 scan steps, one fill per range of 4096 query rows, key-major
    # kernel, and with several ranges the post-pass
    n_ranges = (q1 - q0 + 4095) // 4096
    key_ranges = (cfg.Lk + key_range - 1) // key_range          # of the query-major half (as in the forward pass)
    extra = (2 if saved_lse else 3) if key_ranges > 1 else 0    # range cuts, statistics launch (unless saved), dQ rounding pass
    assert gsa.gsa_launch_count() - n0 == 8 + n_ranges + (1 if n_ranges > 1 else 0) + extra
    return dict(dQ=dQ, dg1=dg1, dK=dK, dV=dV, dg2=dg2, pbar=pbar, lse=lse)


def _compare(cfg, x, got, idx, kt, dout, q0, q1, **okw):
    R = q1 - q0
    rows_b = np.repeat(np.arange(cfg.B), R)
    rows_t = np.tile(np.arange(q0, q1), cfg.B)
    p = U.oracle_params(cfg, **okw)
    want = oracle.attn_bwd(p, x["Q"], x["K"], x["V"], x["g1"], x["g2"], idx.reshape(cfg.B * R, -1).numpy(),
                           kt.reshape(-1).numpy(), dout[:, q0:q1].reshape(cfg.B * R, cfg.n_h, cfg.d_h),
                           rows_t, rows_b)
    for name in ("dQ", "dg1"):
        g = got[name][:, q0:q1].float().cpu().numpy().reshape(cfg.B * R, cfg.n_h, cfg.d_h)
        w = want[name]
        assert np.isfinite(g).all(), name
        assert (np.abs(g - w) <= GRAD_REL_TO_MAX_TOL * np.abs(w).max() + 1e-7).all(), (name, np.abs(g - w).max(), np.abs(w).max())
        assert np.linalg.norm(g - w) <= GRAD_FROBENIUS_TOL * np.linalg.norm(w), name
        # rows outside the range are left alone (NaN-poisoned)
        if q0 > 0:
            assert torch.isnan(got[name][:, :q0].float()).all()
    for name in ("dK", "dV", "dg2"):
        g = got[name].float().cpu().numpy()
        w = want[name]
        assert np.isfinite(g).all(), name
        assert np.abs(w).max() > 0
        assert (np.abs(g - w) <= GRAD_REL_TO_MAX_TOL * np.abs(w).max() + 1e-7).all(), (name, np.abs(g - w).max(), np.abs(w).max())
        assert np.linalg.norm(g - w) <= GRAD_FROBENIUS_TOL * np.linalg.norm(w), (name, np.linalg.norm(g - w) / np.linalg.norm(w))
        # keys nobody selected get exactly zero
        untouched = np.ones(cfg.B * cfg.Lk, bool)
        for b in range(cfg.B):
            for r in range(R):
                untouched[b * cfg.Lk + idx[b, r, : int(kt[b, r])].numpy()] = False
        assert (g.reshape(cfg.B * cfg.Lk, -1)[untouched] == 0).all(), name
    # the optional by-product: the target of the indexer's loss (same bound as in the test of gsa_attn_probs_mean)
    want_p = oracle.attn_probs_mean(p, x["Q"], x["K"], idx.reshape(cfg.B * R, -1).numpy(), kt.reshape(-1).numpy(),
                                    rows_t, rows_b)
    got_p = got["pbar"].cpu().numpy().reshape(cfg.B * R, -1)
    assert (np.abs(got_p - want_p) <= 2e-3 * want_p + 1e-7).all(), np.abs(got_p - want_p).max()
    return want


def test_attn_backward_tiny_all_rows():
    """Every row of the tiny workload (d_h = 64, four heads on one KV head), budgets from 1 key upwards."""
    cfg = CONFIGS["tiny"]
    x = make_inputs(cfg)
    d = U.to_dev(x)
    idx, kt = _index_sets(cfg, 0, cfg.Lq, seed=31, k_lo=1)
    dout = (torch.randn(d["Q"].shape, generator=torch.Generator().manual_seed(32)) * 0.5).to(torch.bfloat16)
    got = _run_bwd(cfg, d, idx.cuda(), kt.cuda(), dout.cuda(), 0, cfg.Lq)
    _compare(cfg, x, got, idx, kt, dout, 0, cfg.Lq)


def test_attn_backward_l8k_shape_row_range_and_batch():
    """The benchmark's layer shape (d_h = 128, 16 heads on 8 KV heads) on a batch of two, rows [300, 396)
    only; ragged budgets (tiles of 16 keys with a tail), custom softmax scale."""
    cfg = CONFIGS["l8k"].with_(name="bwd", B=2, Lq=396, Lk=1500, k_base=300, k_min=17, k_max=419, seed=33)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    q0, q1 = 300, 396
    idx, kt = _index_sets(cfg, q0, q1, seed=34)
    dout = (torch.randn(d["Q"].shape, generator=torch.Generator().manual_seed(35)) * 0.25).to(torch.bfloat16)
    got = _run_bwd(cfg, d, idx.cuda(), kt.cuda(), dout.cuda(), q0, q1, sm_scale=0.11)
    _compare(cfg, x, got, idx, kt, dout, q0, q1, sm_scale=0.11)


def test_attn_backward_decode_shape_and_wide_groups():
    """One query row per sequence against a longer cache; eight heads per KV head."""
    cfg = CONFIGS["l8k"].with_(name="bwd_dec", B=3, Lq=1, Lk=700, n_h=16, n_kv=2, k_base=100, k_min=30, k_max=256, seed=36)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    idx, kt = _index_sets(cfg, 0, 1, seed=37)
    dout = torch.randn(d["Q"].shape, generator=torch.Generator().manual_seed(38)).to(torch.bfloat16)
    got = _run_bwd(cfg, d, idx.cuda(), kt.cuda(), dout.cuda(), 0, 1)
    _compare(cfg, x, got, idx, kt, dout, 0, 1)


@pytest.mark.parametrize("n_h,n_kv,d_h", [(32, 8, 64), (8, 8, 128), (2, 1, 64), (1, 1, 128), (64, 8, 64)])
def test_attn_backward_head_layouts(n_h, n_kv, d_h):
    """Head counts on either side of the 16-row tile of the key-major kernel: several queries per tile
    (n_h < 16), several head blocks per key (n_h > 16), one head per KV head, eight heads per KV head."""
    cfg = CONFIGS["tiny"].with_(name=f"bwd_h{n_h}", B=2, Lq=70, Lk=150, n_h=n_h, n_kv=n_kv, d_h=d_h,
                                k_base=40, k_min=5, k_max=61, seed=60 + n_h)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    idx, kt = _index_sets(cfg, 0, cfg.Lq, seed=61)
    dout = (torch.randn(d["Q"].shape, generator=torch.Generator().manual_seed(62)) * 0.5).to(torch.bfloat16)
    got = _run_bwd(cfg, d, idx.cuda(), kt.cuda(), dout.cuda(), 0, cfg.Lq)
    _compare(cfg, x, got, idx, kt, dout, 0, cfg.Lq)


def test_attn_backward_several_key_ranges():
    """Keys spanning several L2 ranges (forced small here): the query-major half runs per (range, row, KV head),
    combines the ranges' softmax statistics and sums their parts of dQ.  Rows whose visible keys end inside a
    range, rows with nothing in some range, a batch of two."""
    cfg = CONFIGS["l8k"].with_(name="bwd_kr", B=2, Lq=300, Lk=3500, k_base=200, k_min=9, k_max=333, seed=44)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    q0, q1 = 100, 300
    idx, kt = _index_sets(cfg, q0, q1, seed=45)
    idx[0, 5, : int(kt[0, 5])] = torch.arange(int(kt[0, 5]), dtype=torch.int32) + 1030     # one row inside one range
    dout = (torch.randn(d["Q"].shape, generator=torch.Generator().manual_seed(46)) * 0.25).to(torch.bfloat16)
    gsa.gsa_debug_set_attn_range_keys(1024)
    try:
        got = _run_bwd(cfg, d, idx.cuda(), kt.cuda(), dout.cuda(), q0, q1, key_range=1024)
    finally:
        gsa.gsa_debug_set_attn_range_keys(0)
    _compare(cfg, x, got, idx, kt, dout, q0, q1)


@pytest.mark.parametrize("key_range", [16384, 1024])
def test_attn_backward_with_statistics_saved_by_the_forward(key_range):
    """gsa_sparse_gated_attn_fwd_lse writes the same output as the plain call plus lse = log sum exp of the
    scaled logits over S_t (checked against a library logsumexp); the backward pass given lse skips its
    first sweep and must give the same gradients (one key range, and several)."""
    cfg = CONFIGS["l8k"].with_(name="bwd_lse", B=2, Lq=260, Lk=2600, k_base=200, k_min=9, k_max=300, seed=47)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    q0, q1 = 60, 260
    idx, kt = _index_sets(cfg, q0, q1, seed=48)
    dout = (torch.randn(d["Q"].shape, generator=torch.Generator().manual_seed(49)) * 0.25).to(torch.bfloat16)
    gsa.gsa_debug_set_attn_range_keys(key_range)
    try:
        got = _run_bwd(cfg, d, idx.cuda(), kt.cuda(), dout.cuda(), q0, q1, key_range=key_range, saved_lse=True)
    finally:
        gsa.gsa_debug_set_attn_range_keys(0)
    grp = cfg.n_h // cfg.n_kv
    lse = got["lse"].cpu()
    for b, r in ((0, 0), (1, 77), (1, 199)):
        S = idx[b, r, : int(kt[b, r])].long()
        for h in (0, 5, cfg.n_h - 1):
            z = (x["K"][b, S, h // grp].double() @ x["Q"][b, q0 + r, h].double()) / cfg.d_h ** 0.5
            assert abs(lse[b, q0 + r, h].item() - torch.logsumexp(z, dim=0).item()) <= 2e-3
    assert torch.isnan(lse[:, :q0]).all()
    _compare(cfg, x, got, idx, kt, dout, q0, q1)


def test_attn_backward_several_query_ranges():
    """More than 4096 query rows (here three ranges): the key lists are built and walked range by range and the ranges'
    partial sums meet in fp32 arrays."""
    cfg = CONFIGS["tiny"].with_(name="bwd_ranges", B=1, Lq=8192 + 777, Lk=8192 + 777, n_h=4, n_kv=2, d_h=64,
                                k_base=32, k_min=8, k_max=48, seed=41)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    idx, kt = _index_sets(cfg, 0, cfg.Lq, seed=42)
    dout = (torch.randn(d["Q"].shape, generator=torch.Generator().manual_seed(43)) * 0.5).to(torch.bfloat16)
    got = _run_bwd(cfg, d, idx.cuda(), kt.cuda(), dout.cuda(), 0, cfg.Lq)
    _compare(cfg, x, got, idx, kt, dout, 0, cfg.Lq)


def test_attn_backward_argument_errors_do_not_launch():
    cfg = CONFIGS["tiny"]
    d = U.to_dev(make_inputs(cfg))
    idx, kt = _index_sets(cfg, 0, cfg.Lq, seed=39)
    p = gsa.make_params(cfg)
    z = torch.zeros_like
    small = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    n0 = gsa.gsa_launch_count()
    with pytest.raises(gsa.GsaError, match="workspace"):
        gsa.gsa_sparse_gated_attn_bwd(p, d["Q"], d["K"], d["V"], d["g1"], d["g2"], idx.cuda(), kt.cuda(), z(d["Q"]),
                                      z(d["Q"]), z(d["Q"]), z(d["K"]), z(d["K"]), z(d["Q"]), z(d["K"]), small)
    assert gsa.gsa_launch_count() == n0


def test_vbar_update_matches_oracle():
    g = torch.Generator().manual_seed(40)
    var = (torch.rand(131072 + 77, generator=g) * 4e-3).float()
    for momentum, v0 in ((0.99, 2.0e-3), (0.0, 1.0), (1.0, 0.125), (0.5, 3.3e-3)):
        vb = torch.tensor([v0], dtype=torch.float32, device="cuda")
        mv = torch.zeros(1, dtype=torch.float32, device="cuda")
        gsa.gsa_vbar_update(var.cuda(), momentum, vb, mv)
        new, mean = oracle.vbar_update(float(np.float32(v0)), momentum, var.numpy())
        assert abs(mv.item() - mean) <= 2e-7 * abs(mean)            # one rounding to fp32
        assert abs(vb.item() - new) <= 2e-7 * abs(new)
    # a second step feeds on the first one's result
    vb = torch.tensor([1.0], dtype=torch.float32, device="cuda")
    gsa.gsa_vbar_update(var.cuda(), 0.9, vb)
    first = vb.item()
    gsa.gsa_vbar_update(var.cuda(), 0.9, vb)
    want = oracle.vbar_update(first, 0.9, var.numpy())[0]
    assert abs(vb.item() - want) <= 2e-7 * want


# ------------------------------------------------------------------------- the indexer's loss (Eq. 14)
def _run_probs(cfg, d, idx, kt, q0, q1, **over):
    p = gsa.make_params(cfg, q_begin=q0, q_end=q1, **over)
    pbar = torch.full((cfg.B, q1 - q0, cfg.k_max), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    gsa.gsa_attn_probs_mean(p, d["Q"], d["K"], idx, kt, pbar, ws)
    torch.cuda.synchronize()
    assert gsa.gsa_device_status(ws) == 0
    return pbar


def _run_kl(cfg, d, bI, idx, kt, pbar, q0, q1, **over):
    p = gsa.make_params(cfg, q_begin=q0, q_end=q1, **over)
    nan = float("nan")
    loss = torch.full((cfg.B, q1 - q0), nan, dtype=torch.float32, device="cuda")
    dqI = torch.full_like(d["qI"], nan)
    dkI = torch.full_like(d["kI"], nan)
    dw = torch.full_like(d["w"], nan)
    dbI = torch.full((cfg.HI,), nan, dtype=torch.float32, device="cuda")
    ws = torch.empty(gsa.gsa_indexer_kl_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    ws.fill_(0xFF)
    gsa.gsa_indexer_kl_bwd(p, d["qI"], d["kI"], d["w"], bI, idx, kt, pbar, loss, dqI, dkI, dw, dbI, ws)
    torch.cuda.synchronize()
    assert gsa.gsa_device_status(ws) == 0
    return dict(loss=loss, dqI=dqI, dkI=dkI, dw=dw, dbI=dbI)


def _check_loss_path(cfg, q0, q1, seed, bias=False, act=0, **over):
    """Both entry points against the oracle.  The loss kernel is fed the oracle's target rounded to fp32, so
    its own comparison does not inherit the target kernel's rounding."""
    x = make_inputs(cfg)
    d = U.to_dev(x)
    idx, kt = _index_sets(cfg, q0, q1, seed=seed)
    R = q1 - q0
    rows_b, rows_t = np.repeat(np.arange(cfg.B), R), np.tile(np.arange(q0, q1), cfg.B)
    p = U.oracle_params(cfg, act=act, **over)
    idx2, kt1 = idx.reshape(cfg.B * R, -1).numpy(), kt.reshape(-1).numpy()

    want_p = oracle.attn_probs_mean(p, x["Q"], x["K"], idx2, kt1, rows_t, rows_b)
    got_p = _run_probs(cfg, d, idx.cuda(), kt.cuda(), q0, q1, **over).cpu().numpy().reshape(cfg.B * R, -1)
    # probabilities: fp32 sums of 2^(.) from bf16 products; 2e-3 relative plus a floor for the tiny ones
    assert np.isfinite(got_p).all()
    assert (np.abs(got_p - want_p) <= 2e-3 * want_p + 1e-7).all(), np.abs(got_p - want_p).max()
    assert np.abs(got_p.sum(axis=1) - 1.0).max() <= 1e-4
    for r in range(cfg.B * R):
        assert (got_p[r, kt1[r]:] == 0).all()

    bI = torch.tensor([0.3, -0.2, 0.1, 0.0, -0.4, 0.25, 0.05, -0.1][: cfg.HI]) if bias else None
    _compare_kl(cfg, x, d, p, bI, idx, kt, want_p, q0, q1, act=act, **over)


def _compare_kl(cfg, x, d, p, bI, idx, kt, want_p, q0, q1, **over):
    """gsa_indexer_kl_bwd against the oracle, both fed the oracle's target rounded to fp32."""
    R = q1 - q0
    rows_b, rows_t = np.repeat(np.arange(cfg.B), R), np.tile(np.arange(q0, q1), cfg.B)
    idx2, kt1 = idx.reshape(cfg.B * R, -1).numpy(), kt.reshape(-1).numpy()
    pb32 = want_p.astype(np.float32)
    want = oracle.indexer_kl(p, x["qI"], x["kI"], x["w"], bI, idx2, kt1, pb32.astype(np.float64), rows_t, rows_b)
    got = _run_kl(cfg, d, None if bI is None else bI.cuda(), idx.cuda(), kt.cuda(),
                  torch.from_numpy(pb32).reshape(cfg.B, R, -1).cuda(), q0, q1, **over)
    gl = got["loss"].cpu().numpy().reshape(-1)
    # the loss is a difference of O(log k) terms held in fp32
    assert (np.abs(gl - want["loss"]) <= 2e-3 * np.abs(want["loss"]) + 2e-5).all(), np.abs(gl - want["loss"]).max()
    cmp = dict(dqI=(got["dqI"][:, q0:q1].float().cpu().numpy().reshape(cfg.B * R, cfg.HI, cfg.dI), want["dqI"]),
               dw=(got["dw"][:, q0:q1].cpu().numpy().reshape(cfg.B * R, cfg.HI), want["dw"]),
               dkI=(got["dkI"].float().cpu().numpy(), want["dkI"]),
               dbI=(got["dbI"].cpu().numpy(), want["dbI"]))
    for name, (g, w) in cmp.items():
        assert np.isfinite(g).all(), name
        assert np.abs(w).max() > 0, name
        assert (np.abs(g - w) <= GRAD_REL_TO_MAX_TOL * np.abs(w).max() + 1e-7).all(), (name, np.abs(g - w).max(), np.abs(w).max())
        assert np.linalg.norm(g - w) <= GRAD_FROBENIUS_TOL * np.linalg.norm(w), (name, np.linalg.norm(g - w) / np.linalg.norm(w))
    if q0 > 0:
        assert torch.isnan(got["dqI"][:, :q0].float()).all() and torch.isnan(got["dw"][:, :q0]).all()


def test_indexer_kl_tiny_all_rows():
    _check_loss_path(CONFIGS["tiny"], 0, CONFIGS["tiny"].Lq, seed=51)


def test_indexer_kl_layer_shape_row_range_batch_bias():
    cfg = CONFIGS["l8k"].with_(name="kl", B=2, Lq=396, Lk=1500, k_base=300, k_min=17, k_max=419, seed=52)
    _check_loss_path(cfg, 300, 396, seed=53, bias=True)


def test_indexer_kl_relu_indexer():
    cfg = CONFIGS["l8k"].with_(name="kl_relu", B=1, Lq=200, Lk=900, HI=4, dI=32, k_base=100, k_min=20, k_max=160, seed=54)
    _check_loss_path(cfg, 0, 200, seed=55, bias=True, act=1)


def test_indexer_warmup_loss_on_all_visible_keys():
    """Eq. 13 for a short context: the index sets of the dense fallback (k_mode 3: every visible key) fed to the
    same two entry points."""
    cfg = CONFIGS["tiny"].with_(name="warmup", B=2, Lq=90, Lk=200, k_base=8, k_min=4, k_max=208, seed=56)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    p = gsa.make_params(cfg, k_mode=3)
    out = torch.empty_like(d["Q"])
    idx = torch.empty((cfg.B, cfg.Lq, cfg.k_max), dtype=torch.int32, device="cuda")
    kt = torch.empty((cfg.B, cfg.Lq), dtype=torch.int32, device="cuda")
    ws = torch.empty(gsa.gsa_workspace_bytes(p, 0), dtype=torch.uint8, device="cuda")
    gsa.gsa_forward(p, d["Q"], d["K"], d["V"], None, None, None, None, d["g1"], d["g2"], out, idx, kt, None, 0, ws)
    torch.cuda.synchronize()
    idx_c, kt_c = idx.cpu(), kt.cpu()
    assert (kt_c[0].numpy() == cfg.Lk - cfg.Lq + np.arange(cfg.Lq) + 1).all()
    R = cfg.Lq
    rows_b, rows_t = np.repeat(np.arange(cfg.B), R), np.tile(np.arange(R), cfg.B)
    po = U.oracle_params(cfg)
    idx2, kt1 = idx_c.reshape(cfg.B * R, -1).numpy(), kt_c.reshape(-1).numpy()
    want_p = oracle.attn_probs_mean(po, x["Q"], x["K"], idx2, kt1, rows_t, rows_b)
    got_p = _run_probs(cfg, d, idx, kt, 0, R).cpu().numpy().reshape(cfg.B * R, -1)
    assert (np.abs(got_p - want_p) <= 2e-3 * want_p + 1e-7).all()
    pb32 = want_p.astype(np.float32)
    want = oracle.indexer_kl(po, x["qI"], x["kI"], x["w"], None, idx2, kt1, pb32.astype(np.float64), rows_t, rows_b)
    got = _run_kl(cfg, d, None, idx, kt, torch.from_numpy(pb32).reshape(cfg.B, R, -1).cuda(), 0, R)
    gl = got["loss"].cpu().numpy().reshape(-1)
    assert (np.abs(gl - want["loss"]) <= 2e-3 * np.abs(want["loss"]) + 2e-5).all()
    g, w = got["dkI"].float().cpu().numpy(), want["dkI"]
    assert np.linalg.norm(g - w) <= GRAD_FROBENIUS_TOL * np.linalg.norm(w)


# ------------------------------------------------------------------------- the benchmark's geometry
def test_backward_and_indexer_loss_at_the_benchmark_geometry():
    """The launch plan `bench.py --backward` times, checked against the oracle: the l128k workload with the
    default range sizes (8 key ranges of 16384 keys in the query-major half, 2 query ranges of 4096 rows in
    the key-major half), index sets taken from the real forward pass, gradients of the last 4200 query rows.
    dQ and dg1 on every row of the range; dK, dV, dg2, the loss target and dk^I on every key."""
    cfg = CONFIGS["l128k"]
    x = make_inputs(cfg)
    d = U.to_dev(x)
    _, idx_all, kt_all, _ = U.run_forward(cfg, d)
    q0, q1 = cfg.Lq - 4200, cfg.Lq
    idx = idx_all[:, q0:q1].contiguous()
    kt = kt_all[:, q0:q1].contiguous()
    del idx_all
    g = torch.Generator().manual_seed(71)
    dout = torch.zeros_like(d["Q"])
    dout_rows = (torch.randn((cfg.B, q1 - q0, cfg.n_h, cfg.d_h), generator=g) * 0.25).to(torch.bfloat16)
    dout[:, q0:q1] = dout_rows.cuda()
    got = _run_bwd(cfg, d, idx, kt, dout, q0, q1)
    idx_c, kt_c = idx.cpu(), kt.cpu()
    dout_c = torch.zeros((cfg.B, cfg.Lq, cfg.n_h, cfg.d_h), dtype=torch.bfloat16)
    dout_c[:, q0:q1] = dout_rows
    _compare(cfg, x, got, idx_c, kt_c, dout_c, q0, q1)
    # the same gradients when the forward call saved its softmax statistics (first sweep skipped)
    got2 = _run_bwd(cfg, d, idx, kt, dout, q0, q1, saved_lse=True)
    for name in ("dQ", "dg1"):
        a, b = got[name][:, q0:q1].float(), got2[name][:, q0:q1].float()
        assert (a - b).abs().max().item() <= 2.0 ** -7 * a.abs().max().item(), name
    for name in ("dK", "dV", "dg2"):
        a, b = got[name].float(), got2[name].float()
        assert (a - b).abs().max().item() <= 2.0 ** -7 * a.abs().max().item(), name
    del got2
    # the indexer's loss on the same index sets
    R = q1 - q0
    p = U.oracle_params(cfg)
    want_p = oracle.attn_probs_mean(p, x["Q"], x["K"], idx_c.reshape(cfg.B * R, -1).numpy(), kt_c.reshape(-1).numpy(),
                                    np.tile(np.arange(q0, q1), cfg.B), np.repeat(np.arange(cfg.B), R))
    _compare_kl(cfg, x, d, p, None, idx_c, kt_c, want_p, q0, q1)
