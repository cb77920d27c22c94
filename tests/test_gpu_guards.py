"""What the kernels do when something is wrong, without faulting or hanging the GPU:

* a bounded device-side wait that runs out -- made to run out by leaving out the copy that would complete
  its barrier (the library's test knob), so the wait is for a flag that nothing sets -- must end with the
  status word set, the kernel returned, and the next ordinary call correct;
* an index set with an entry outside [0, Lk) or a budget outside [0, k_max] never becomes an address: the
  call completes, its outputs are finite, and the status word says so.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_15305_b200 import binding as gsa
from paper_2601_15305_b200.inputs import CONFIGS, make_inputs

import gpu_util as U

pytestmark = pytest.mark.gpu

WAIT_CYCLES = 400_000          # about 0.2 ms of SM clock instead of the default second


def test_indexer_wait_runs_out_then_next_call_is_correct():
    cfg = CONFIGS["tiny"]
    x = make_inputs(cfg)
    d = U.to_dev(x)
    p = gsa.make_params(cfg)
    st = U.row_stride(cfg)
    sc = torch.zeros((cfg.B, cfg.Lq, st), device="cuda", dtype=torch.float32)
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    gsa.gsa_debug_set_wait_limit(WAIT_CYCLES, withhold_first_copy=True)
    try:
        gsa.gsa_indexer_scores(p, d["qI"], d["kI"], d["w"], None, sc, st, ws)     # returns: argument checks passed
        status = gsa.gsa_device_status(ws)                                        # waits for the stream
    finally:
        gsa.gsa_debug_set_wait_limit(0, withhold_first_copy=False)
    assert status in (1, 2, 3), status                # which role's wait ran out first
    rc = gsa.lib().gsa_device_status(gsa._dp(ws), gsa._stream(None), None)
    assert rc == -5                                   # GSA_ERR_DEVICE_TIMEOUT
    torch.cuda.synchronize()                          # the context is intact
    # the next ordinary call on the same workspace clears the word and computes the scores
    got = U.run_scores(cfg, d)[0].cpu().numpy()
    rows = np.arange(0, cfg.Lq, 5)
    want = oracle.scores(U.oracle_params(cfg), x["qI"], x["kI"], x["w"], None, rows)
    U.check_scores(got[rows], want, [int(t) + 1 for t in rows])


def test_projection_wait_runs_out_then_next_call_is_correct():
    cfg = CONFIGS["tiny"].with_(name="proj_wait", B=1, Lq=300, Lk=300)
    p = gsa.make_params(cfg)
    d_model = 192
    n_cols = gsa.gsa_project_columns(p)
    g = torch.Generator().manual_seed(81)
    M = cfg.B * cfg.Lq
    H = torch.randn(M, d_model, generator=g).to(torch.bfloat16)
    Wt = (torch.randn(n_cols, d_model, generator=g) / d_model ** 0.5).to(torch.bfloat16)
    dev = lambda *s, dt=torch.bfloat16: torch.zeros(s, dtype=dt, device="cuda")
    qI, kI = dev(cfg.B, cfg.Lq, cfg.HI, cfg.dI), dev(cfg.B, cfg.Lq, cfg.dI)
    w = dev(cfg.B, cfg.Lq, cfg.HI, dt=torch.float32)
    g1, g2 = dev(cfg.B, cfg.Lq, cfg.n_h, cfg.d_h), dev(cfg.B, cfg.Lq, cfg.n_kv, cfg.d_h)
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    Hd, Wd = H.cuda(), Wt.cuda()
    gsa.gsa_debug_set_wait_limit(WAIT_CYCLES, withhold_first_copy=True)
    try:
        gsa.gsa_project(p, d_model, Hd, Wd, qI, kI, w, g1, g2, ws)
        status = gsa.gsa_device_status(ws)
    finally:
        gsa.gsa_debug_set_wait_limit(0, withhold_first_copy=False)
    assert status in (1, 2, 3), status
    torch.cuda.synchronize()
    gsa.gsa_project(p, d_model, Hd, Wd, qI, kI, w, g1, g2, ws)
    assert gsa.gsa_device_status(ws) == 0
    rows = np.arange(0, M, 23)
    o = oracle.project(U.oracle_params(cfg), d_model, H, Wt, rows)
    got = kI.reshape(M, -1)[torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
    assert (np.abs(got - o["kI"]) <= 2.0 ** -8 * np.abs(o["kI"]) + 1e-5).all()
    gw = w.reshape(M, -1)[torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.float64)
    assert np.abs(gw - o["w"]).max() <= 2e-6


def _sets(cfg, seed):
    g = torch.Generator().manual_seed(seed)
    idx = torch.full((cfg.B, cfg.Lq, cfg.k_max), -1, dtype=torch.int32)
    kt = torch.empty((cfg.B, cfg.Lq), dtype=torch.int32)
    for b in range(cfg.B):
        for t in range(cfg.Lq):
            n = cfg.Lk - cfg.Lq + t + 1
            k = min(n, int(torch.randint(cfg.k_min, cfg.k_max + 1, (1,), generator=g)))
            idx[b, t, :k] = torch.randperm(n, generator=g)[:k].sort().values.to(torch.int32)
            kt[b, t] = k
    return idx, kt


@pytest.mark.parametrize("damage", ["position_too_large", "position_negative", "budget_too_large"])
def test_corrupt_index_sets_are_reported_not_followed(damage):
    cfg = CONFIGS["tiny"].with_(name="guards", B=2, Lq=120, Lk=300, seed=83)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    idx, kt = _sets(cfg, 84)
    good_idx, good_kt = idx.clone(), kt.clone()
    if damage == "position_too_large":
        idx[1, 70, 3] = cfg.Lk + 12345
    elif damage == "position_negative":
        idx[0, 5, 0] = -9
    else:
        kt[1, 100] = cfg.k_max + 1000
    p = gsa.make_params(cfg)

    def attn(i, k):
        out = torch.full_like(d["Q"], float("nan"))
        ws = torch.empty(gsa.gsa_attn_workspace_bytes(p, True), dtype=torch.uint8, device="cuda")
        gsa.gsa_sparse_gated_attn_fwd(p, d["Q"], d["K"], d["V"], d["g1"], d["g2"], i.cuda(), k.cuda(), out, ws)
        return out, gsa.gsa_device_status(ws)

    def bwd(i, k, out):
        dout = (torch.randn(d["Q"].shape, generator=torch.Generator().manual_seed(85)) * 0.5).to(torch.bfloat16).cuda()
        gq = [torch.full_like(d["Q"], float("nan")) for _ in range(2)]
        gk = [torch.full_like(d["K"], float("nan")) for _ in range(3)]
        ws = torch.empty(gsa.gsa_attn_bwd_workspace_bytes(p), dtype=torch.uint8, device="cuda")
        gsa.gsa_sparse_gated_attn_bwd(p, d["Q"], d["K"], d["V"], d["g1"], d["g2"], i.cuda(), k.cuda(), out, dout,
                                      gq[0], gk[0], gk[1], gq[1], gk[2], ws)
        return gq + gk, gsa.gsa_device_status(ws)

    def kl(i, k):
        pbar = torch.full((cfg.B, cfg.Lq, cfg.k_max), 1.0 / cfg.k_max, dtype=torch.float32, device="cuda")
        loss = torch.empty((cfg.B, cfg.Lq), dtype=torch.float32, device="cuda")
        dqI, dkI, dw = torch.empty_like(d["qI"]), torch.empty_like(d["kI"]), torch.empty_like(d["w"])
        ws = torch.empty(gsa.gsa_indexer_kl_workspace_bytes(p), dtype=torch.uint8, device="cuda")
        gsa.gsa_indexer_kl_bwd(p, d["qI"], d["kI"], d["w"], None, i.cuda(), k.cuda(), pbar, loss, dqI, dkI, dw, None, ws)
        return gsa.gsa_device_status(ws)

    out, status = attn(idx, kt)
    assert status == 6 and torch.isfinite(out.float()).all()
    grads, status = bwd(idx, kt, out)
    assert status == 6 and all(torch.isfinite(t.float()).all() for t in grads)
    assert kl(idx, kt) == 6
    rc = gsa.lib().gsa_device_status(gsa._dp(torch.full((64,), 6, dtype=torch.int32, device="cuda")), gsa._stream(None), None)
    assert rc == -7                                   # GSA_ERR_INDEX_RANGE
    # the same calls on the undamaged sets report nothing
    out, status = attn(good_idx, good_kt)
    assert status == 0
    assert bwd(good_idx, good_kt, out)[1] == 0 and kl(good_idx, good_kt) == 0
