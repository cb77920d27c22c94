"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the same
seeded inputs.  Per stage (scores within 1e-3 relative; index sets bit-exact on equal fp32 scores;
outputs within 2e-2 max-abs) and end to end."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_15305_b200 import binding as gsa
from paper_2601_15305_b200.inputs import CONFIGS, make_inputs, sample_rows

import gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tiny():
    cfg = CONFIGS["tiny"]
    x = make_inputs(cfg)
    return cfg, x, U.to_dev(x)


@pytest.fixture(scope="module")
def l8k():
    cfg = CONFIGS["l8k"]
    x = make_inputs(cfg)
    return cfg, x, U.to_dev(x)


def _vis(cfg, rows):
    return [cfg.Lk - cfg.Lq + int(t) + 1 for t in rows]


# ------------------------------------------------------------------------------------------ stage 1
@pytest.mark.parametrize("path", [0, 1])
def test_indexer_tiny_all_rows(tiny, path):
    cfg, x, d = tiny
    gsa.gsa_debug_set_indexer_path(path)
    try:
        sc = U.run_scores(cfg, d)[0].cpu().numpy()
    finally:
        gsa.gsa_debug_set_indexer_path(0)
    rows = np.arange(cfg.Lq)
    want = oracle.scores(U.oracle_params(cfg), x["qI"], x["kI"], x["w"], None, rows)
    U.check_scores(sc, want, _vis(cfg, rows))
    # nothing is written past a row's visible keys (buffer was NaN-poisoned)
    for t in (0, 100, 510):
        assert np.isnan(sc[t, t + 1:cfg.Lk]).all()
    # fp32 scores stay inside [0, sum_j w_j] (the paper's (0, H^I))
    wsum = x["w"][0].sum(-1).numpy()
    for t in rows:
        assert (sc[t, :t + 1] >= 0).all() and (sc[t, :t + 1] <= wsum[t] * (1 + 1e-6)).all()


@pytest.mark.parametrize("path", [0, 1])
def test_indexer_bias_and_row_range(tiny, path):
    cfg, x, d = tiny
    bI = torch.tensor([0.5, -1.0, 2.0, 0.0], dtype=torch.float32)
    gsa.gsa_debug_set_indexer_path(path)
    try:
        sc = U.run_scores(cfg, d, q_begin=37, q_end=301, bI=bI.cuda())[0].cpu().numpy()
    finally:
        gsa.gsa_debug_set_indexer_path(0)
    rows = np.arange(37, 301)
    want = oracle.scores(U.oracle_params(cfg), x["qI"], x["kI"], x["w"], bI, rows)
    U.check_scores(sc, want, _vis(cfg, rows))


@pytest.mark.parametrize("path", [0, 1])
def test_indexer_l8k_sampled_rows(l8k, path):
    cfg, x, d = l8k
    gsa.gsa_debug_set_indexer_path(path)
    try:
        sc = U.run_scores(cfg, d)[0]
    finally:
        gsa.gsa_debug_set_indexer_path(0)
    rows = sample_rows(cfg, 48).numpy()
    got = sc[torch.from_numpy(rows).cuda()].cpu().numpy()
    want = oracle.scores(U.oracle_params(cfg), x["qI"], x["kI"], x["w"], None, rows)
    U.check_scores(got, want, _vis(cfg, rows))


def test_indexer_ragged_batch_decode_shapes():
    """Lq not a multiple of any tile, Lk > Lq (chunked prefill), B > 1."""
    cfg = CONFIGS["l8k"].with_(name="ragged", B=2, Lq=203, Lk=459, seed=11)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    for path in (0, 1):
        gsa.gsa_debug_set_indexer_path(path)
        try:
            sc = U.run_scores(cfg, d).cpu().numpy()
        finally:
            gsa.gsa_debug_set_indexer_path(0)
        p = U.oracle_params(cfg)
        for b in range(cfg.B):
            rows = np.arange(cfg.Lq)
            want = oracle.scores(p, x["qI"], x["kI"], x["w"], None, rows, np.full_like(rows, b))
            U.check_scores(sc[b], want, _vis(cfg, rows))


@pytest.mark.parametrize("base,Lq,HI", [("l8k", 1, 8), ("l8k", 3, 8), ("tiny", 2, 4), ("tiny", 4, 2)])
def test_indexer_few_rows_streams_keys(base, Lq, HI):
    """Calls with at most 4 query rows per sequence take the key-streaming kernel (decode geometry)."""
    cfg = CONFIGS[base].with_(name="fewrows", B=3, Lq=Lq, Lk=2117, HI=HI, seed=15)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    bI = torch.linspace(-1.0, 1.5, HI)
    sc = U.run_scores(cfg, d, bI=bI.cuda()).cpu().numpy()
    p = U.oracle_params(cfg)
    for b in range(cfg.B):
        rows = np.arange(cfg.Lq)
        want = oracle.scores(p, x["qI"], x["kI"], x["w"], bI, rows, np.full_like(rows, b))
        U.check_scores(sc[b], want, _vis(cfg, rows))
        for t in rows:                                   # nothing written past the visible keys
            assert np.isnan(sc[b, t, cfg.Lk - cfg.Lq + t + 1:cfg.Lk]).all()


@pytest.mark.parametrize("path", [0, 1])
def test_relu_indexer_scores(tiny, path):
    """act = 1: the ReLU indexer of Eq. 3 (no special-function work; scores are >= 0 and unbounded)."""
    cfg, x, d = tiny
    bI = torch.tensor([0.25, -0.5, 0.0, 1.0], dtype=torch.float32)
    gsa.gsa_debug_set_indexer_path(path)
    try:
        sc = U.run_scores(cfg, d, bI=bI.cuda(), act=1)[0].cpu().numpy()
    finally:
        gsa.gsa_debug_set_indexer_path(0)
    rows = np.arange(cfg.Lq)
    want = oracle.scores(U.oracle_params(cfg, act=1), x["qI"], x["kI"], x["w"], bI, rows)
    for t in rows:
        g, w = sc[t, :t + 1].astype(np.float64), want[t, :t + 1]
        assert (g >= 0).all()
        # relative 1e-3 as for the sigmoid scores, plus an absolute floor because ReLU scores reach 0
        assert (np.abs(g - w) <= U.SCORE_REL_TOL * np.abs(w) + 1e-6).all()
    # few query rows: the key-streaming kernel
    cfg2 = CONFIGS["l8k"].with_(name="relu_rows", B=2, Lq=2, Lk=1500, seed=16)
    x2 = make_inputs(cfg2)
    sc2 = U.run_scores(cfg2, U.to_dev(x2), act=1).cpu().numpy()
    for b in range(cfg2.B):
        want2 = oracle.scores(U.oracle_params(cfg2, act=1), x2["qI"], x2["kI"], x2["w"], None, np.arange(2), np.full(2, b))
        for t in range(2):
            n = cfg2.Lk - cfg2.Lq + t + 1
            assert (np.abs(sc2[b, t, :n] - want2[t, :n]) <= U.SCORE_REL_TOL * np.abs(want2[t, :n]) + 1e-6).all()


def test_forward_relu_indexer_fixed_budget(l8k):
    """The 'sparse only' indexer setting of the paper's comparison (ReLU scores, fixed k) through the whole path."""
    cfg, x, d = l8k
    rows = sample_rows(cfg, 16).numpy()
    mism, kt = _forward_and_compare(cfg, x, d, rows, act=1, k_mode=2)
    assert (kt[0].cpu().numpy() == np.minimum(cfg.k_base, np.arange(cfg.Lq) + 1)).all()


# ------------------------------------------------------------------------------------------ stage 2
def _select_and_compare(cfg, sc_dev, rows=None, k_mode=0, **over):
    """sc_dev: [B, Lq, stride] fp32 on the GPU; compares every (or the listed) row of batch 0."""
    idx, kt, var = U.run_topk(cfg, sc_dev, k_mode=k_mode, **over)
    rows = np.arange(cfg.Lq) if rows is None else np.asarray(rows)
    sel = torch.from_numpy(rows).cuda()
    sc_rows = sc_dev[0][sel].cpu().numpy()
    p = U.oracle_params(cfg, k_mode=k_mode, **over)
    o = oracle.select_f32(p, sc_rows, rows)

    def again(i, k):
        p2 = U.oracle_params(cfg, k_mode=2, **{**over, "k_base": k, "k_min": 1, "k_max": p.k_max})
        return oracle.select_f32(p2, sc_rows[i:i + 1], rows[i:i + 1])["idx"][0]

    U.check_selection_exact(o, idx[0][sel].cpu().numpy(), kt[0][sel].cpu().numpy(), again)
    np.testing.assert_allclose(var[0][sel].cpu().numpy(), o["var"], rtol=2e-6, atol=1e-12)
    return o, kt[0][sel].cpu().numpy()


@pytest.mark.parametrize("k_mode", [0, 1, 2])
def test_topk_bit_exact_tiny(tiny, k_mode):
    cfg, x, d = tiny
    sc = U.run_scores(cfg, d, poison=True)
    o, kt = _select_and_compare(cfg, sc, k_mode=k_mode)
    if k_mode == 0:
        assert len(set(kt.tolist())) > 5          # budgets really vary
    if k_mode == 2:
        assert (kt == np.minimum(cfg.k_base, np.arange(cfg.Lq) + 1)).all()


def test_topk_bit_exact_on_oracle_scores_with_ties():
    """Scores quantised to a few levels: thousands of exact ties; lower position must win."""
    cfg = CONFIGS["tiny"].with_(Lq=700, Lk=700, k_base=100, k_min=30, k_max=333)
    g = torch.Generator().manual_seed(5)
    lv = torch.randint(0, 7, (1, cfg.Lq, U.row_stride(cfg)), generator=g).float() * 0.125 + 0.5
    lv[0, 500:520] = 1.25                         # constant rows: variance 0
    sc = lv.cuda()
    for k_mode in (0, 1, 2):
        _select_and_compare(cfg, sc, k_mode=k_mode, v_bar=0.05)


def test_topk_wide_dynamic_range_and_negatives():
    """Keys spanning many binades (three radix rounds) and negative values."""
    cfg = CONFIGS["tiny"].with_(Lq=1500, Lk=1500, k_base=200, k_min=10, k_max=1000)
    g = torch.Generator().manual_seed(6)
    e = torch.randint(-20, 3, (1, cfg.Lq, U.row_stride(cfg)), generator=g).float()
    sc = (torch.rand(e.shape, generator=g) + 1.0) * torch.pow(2.0, e)
    sc[0, 1000:1100] *= -1.0
    sc[0, 1200:1300, ::3] *= -1.0
    _select_and_compare(cfg, sc.cuda(), k_mode=2)
    _select_and_compare(cfg, sc.cuda(), k_mode=0, v_bar=0.3)


def test_topk_l8k_rows_cached_and_global_paths(l8k):
    cfg, x, d = l8k
    sc = U.run_scores(cfg, d)
    rows = sample_rows(cfg, 64).numpy()
    _select_and_compare(cfg, sc, rows=rows)


def test_topk_long_rows_take_the_uncached_path():
    """Rows longer than the shared-memory cache (n > ~46K) are re-read from global memory."""
    cfg = CONFIGS["l8k"].with_(name="long", B=1, Lq=8, Lk=70000, seed=12)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    sc = U.run_scores(cfg, d)
    _select_and_compare(cfg, sc)


def test_topk_long_rows_that_defeat_the_sample():
    """Long rows on which the sampled candidate threshold is useless: a handful of score levels (huge
    ties), scores increasing with position (every top score sits at the end of the row), a constant row.
    The kernel must notice (list overflow / too few candidates) and still return the exact set."""
    cfg = CONFIGS["l8k"].with_(name="degenerate", B=1, Lq=6, Lk=20011, k_base=700, k_min=100, k_max=3000)
    st = U.row_stride(cfg)
    g = torch.Generator().manual_seed(7)
    sc = torch.zeros((1, cfg.Lq, st), dtype=torch.float32)
    sc[0, 0] = torch.randint(0, 5, (st,), generator=g).float() * 0.25 + 1.0        # 5 levels
    sc[0, 1] = torch.arange(st).float() * 1e-4 + 1.0                                # increasing
    sc[0, 2] = 2.5                                                                  # constant
    sc[0, 3] = torch.arange(st).float().flip(0) * 1e-4 + 1.0                        # decreasing
    sc[0, 4] = torch.rand(st, generator=g) + (torch.arange(st) > st - 3000).float() * 3.0   # a late cluster
    sc[0, 5] = torch.rand(st, generator=g)
    for k_mode, v_bar in ((2, 1.0), (0, 0.05), (1, 0.05)):
        _select_and_compare(cfg, sc.cuda(), k_mode=k_mode, v_bar=v_bar)


def test_topk_long_rows_with_a_tie_cut_and_rows_beyond_the_bitmap():
    """The two cases in which a long row's set is written by walking the candidate table instead of through
    the position bitmap: the budget cuts a group of equal scores (scores quantised to 4096 levels: a few equal
    scores per level, the candidate list does not overflow), and a row of more than 131072 visible scores."""
    cfg = CONFIGS["l8k"].with_(name="tiecut", B=1, Lq=5, Lk=30011, k_base=900, k_min=100, k_max=3000)
    st = U.row_stride(cfg)
    g = torch.Generator().manual_seed(10)
    sc = torch.floor(torch.rand((1, cfg.Lq, st), generator=g) * 4096.0) / 4096.0
    for k_mode, v_bar in ((2, 1.0), (0, 0.08)):
        _select_and_compare(cfg, sc.cuda(), k_mode=k_mode, v_bar=v_bar)
    cfg = CONFIGS["l8k"].with_(name="beyond_bitmap", B=1, Lq=3, Lk=131072 + 4099, k_base=1500, k_min=100, k_max=4096)
    st = U.row_stride(cfg)
    sc = torch.rand((1, cfg.Lq, st), generator=g) ** 3
    for k_mode, v_bar in ((2, 1.0), (0, 0.05)):
        _select_and_compare(cfg, sc.cuda(), k_mode=k_mode, v_bar=v_bar)


def test_topk_row_lengths_around_the_chunk_and_list_boundaries():
    """Visible lengths n just below / at / above the short-row limit (8192) and multiples of the 512-score
    chunk, and rows whose last chunk holds a single score."""
    cfg = CONFIGS["l8k"].with_(name="edges", B=1, Lq=1540, Lk=9730, k_base=900, k_min=64, k_max=2048)
    st = U.row_stride(cfg)
    g = torch.Generator().manual_seed(8)
    sc = (torch.rand((1, cfg.Lq, st), generator=g) ** 4).cuda()          # long right tail
    # rows t = 0 .. 1539 see n = 8191 .. 9730 keys: 8191, 8192, 8193 and 8704 = 17 * 512, 9216, 9217, 9728
    rows = np.array([0, 1, 2, 3, 511, 512, 513, 514, 1024, 1025, 1026, 1027, 1535, 1536, 1537, 1538, 1539])
    for k_mode, v_bar in ((0, 0.07), (2, 1.0)):
        _select_and_compare(cfg, sc, rows=rows, k_mode=k_mode, v_bar=v_bar)


def test_topk_rows_longer_than_the_candidate_table():
    """Rows of more than 2048 * 512 visible scores are not listed: they take the whole-row path."""
    cfg = CONFIGS["l8k"].with_(name="verylong", B=1, Lq=2, Lk=1048576 + 777, k_base=1500, k_min=100, k_max=4096)
    st = U.row_stride(cfg)
    g = torch.Generator().manual_seed(9)
    sc = (torch.randn((1, cfg.Lq, st), generator=g) * 0.05 + 1.0).cuda()
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    for k_mode, v_bar in ((0, 0.0025), (2, 1.0)):
        _select_and_compare(cfg, sc, k_mode=k_mode, v_bar=v_bar)


# ------------------------------------------------------------------------------------------ stage 3
def _oracle_idx(cfg, x, rows, **kw):
    p = U.oracle_params(cfg, **kw)
    return p, oracle.forward(p, **x, rows_t=rows, want_scores=True)


def test_attn_given_oracle_indices_tiny(tiny):
    cfg, x, d = tiny
    rows = np.arange(cfg.Lq)
    p, o = _oracle_idx(cfg, x, rows)
    idx = torch.from_numpy(o["idx"]).cuda()[None]
    kt = torch.from_numpy(o["keff"]).cuda()[None]
    for use_prepass in (True, False):
        out = U.run_attn(cfg, d, idx, kt, prepass=use_prepass)
        U.check_out(out[0].float().cpu().numpy(), o["out"])


@pytest.mark.parametrize("n_h,n_kv,d_h", [(8, 8, 128), (1, 1, 128), (16, 2, 128), (2, 1, 64), (32, 8, 64), (64, 8, 64)])
def test_attn_head_layouts(n_h, n_kv, d_h):
    """One, two, four and eight query heads per KV head at both head widths, with the value gate as a pre-pass
    and inside the gather; index sets are the oracle's (budgets from k_min up to everything visible)."""
    cfg = CONFIGS["tiny"].with_(name=f"attn_h{n_h}_{n_kv}_{d_h}", B=2, Lq=70, Lk=150, n_h=n_h, n_kv=n_kv, d_h=d_h,
                                k_base=40, k_min=5, k_max=61, seed=90 + n_h)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    p = U.oracle_params(cfg)
    rows_t = np.tile(np.arange(cfg.Lq), cfg.B)
    rows_b = np.repeat(np.arange(cfg.B), cfg.Lq)
    o = oracle.forward(p, **x, rows_t=rows_t, rows_b=rows_b)
    idx = torch.from_numpy(o["idx"]).reshape(cfg.B, cfg.Lq, -1).cuda()
    kt = torch.from_numpy(o["keff"]).reshape(cfg.B, cfg.Lq).cuda()
    for use_prepass in (True, False):
        out = U.run_attn(cfg, d, idx, kt, prepass=use_prepass)
        U.check_out(out.reshape(cfg.B * cfg.Lq, n_h, d_h).float().cpu().numpy(), o["out"])


@pytest.mark.parametrize("Lq", [40, 2])
def test_attn_empty_index_sets_give_zero_rows(Lq):
    """kt = 0 for some rows (an empty S_t): their outputs are zeros, the other rows are unaffected; with many
    query rows (one launch per key range) and with few (parallel segments merged at the end)."""
    cfg = CONFIGS["tiny"].with_(name="attn_empty", B=2, Lq=Lq, Lk=200, k_base=40, k_min=5, k_max=61, seed=95)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    p = U.oracle_params(cfg)
    rows_t = np.tile(np.arange(cfg.Lq), cfg.B)
    rows_b = np.repeat(np.arange(cfg.B), cfg.Lq)
    o = oracle.forward(p, **x, rows_t=rows_t, rows_b=rows_b)
    idx = torch.from_numpy(o["idx"]).reshape(cfg.B, cfg.Lq, -1).clone()
    kt = torch.from_numpy(o["keff"]).reshape(cfg.B, cfg.Lq).clone()
    empty = [(0, 0), (1, cfg.Lq - 1)]
    for b, t in empty:
        kt[b, t] = 0
        idx[b, t] = -1
    for use_prepass in (True, False):
        out = U.run_attn(cfg, d, idx.cuda(), kt.cuda(), prepass=use_prepass).float().cpu().numpy()
        want = o["out"].reshape(cfg.B, cfg.Lq, cfg.n_h, cfg.d_h).copy()
        for b, t in empty:
            assert (out[b, t] == 0.0).all()
            want[b, t] = 0.0
        U.check_out(out.reshape(-1, cfg.n_h, cfg.d_h), want.reshape(-1, cfg.n_h, cfg.d_h))


def test_attn_pregated_values_and_custom_scale(tiny):
    cfg, x, d = tiny
    rows = np.arange(0, cfg.Lq, 7)
    p = U.oracle_params(cfg, sm_scale=0.2)
    o = oracle.forward(p, **x, rows_t=rows)
    # rows subset through q_begin/q_end is contiguous; use the full range and compare the subset
    po, oa = _oracle_idx(cfg, x, np.arange(cfg.Lq))
    idx = torch.from_numpy(oa["idx"]).cuda()[None]
    kt = torch.from_numpy(oa["keff"]).cuda()[None]
    out = U.run_attn(cfg, d, idx, kt, sm_scale=0.2)
    U.check_out(out[0, rows].float().cpu().numpy(), o["out"])
    # g2 = NULL means V is already gated: feed V' = V*sigmoid(g2) rounded to bf16
    d2 = dict(d)
    d2["V"] = (d["V"].float() * torch.sigmoid(d["g2"].float())).to(torch.bfloat16)
    out2 = U.run_attn(cfg, d2, idx, kt, use_g2=False, sm_scale=0.2)
    U.check_out(out2[0, rows].float().cpu().numpy(), o["out"])


def test_attn_l8k_sampled_rows(l8k):
    cfg, x, d = l8k
    rows = sample_rows(cfg, 24).numpy()
    p, o = _oracle_idx(cfg, x, rows)
    q0, q1 = int(rows.min()), int(rows.max()) + 1
    # place the oracle's index sets into a full [R, k_max] table (other rows: a valid dummy set)
    R = q1 - q0
    idx = torch.zeros((1, R, cfg.k_max), dtype=torch.int32)
    kt = torch.ones((1, R), dtype=torch.int32)
    idx[0, rows - q0] = torch.from_numpy(o["idx"])
    kt[0, rows - q0] = torch.from_numpy(o["keff"])
    out = U.run_attn(cfg, d, idx.cuda(), kt.cuda(), q_begin=q0, q_end=q1)
    U.check_out(out[0, rows].float().cpu().numpy(), o["out"])
    # rows outside [q_begin, q_end) are untouched (NaN-poisoned)
    if q0 > 0:
        assert torch.isnan(out[0, :q0].float()).all()


def test_attn_saturated_gates_is_plain_attention(tiny):
    """Gate logits +40: sigmoid is 1.0 in fp32 too, the layer is ungated sparse attention."""
    cfg, x, d = tiny
    x2 = dict(x)
    x2["g1"] = torch.full_like(x["g1"], 40.0)
    x2["g2"] = torch.full_like(x["g2"], 40.0)
    rows = np.arange(cfg.Lq)
    p, o = _oracle_idx(cfg, x2, rows)
    d2 = U.to_dev(x2)
    out = U.run_attn(cfg, d2, torch.from_numpy(o["idx"]).cuda()[None], torch.from_numpy(o["keff"]).cuda()[None])
    U.check_out(out[0].float().cpu().numpy(), o["out"])
    # and g1 = -40 closes the output gate
    d2["g1"] = torch.full_like(d["g1"], -40.0)
    out = U.run_attn(cfg, d2, torch.from_numpy(o["idx"]).cuda()[None], torch.from_numpy(o["keff"]).cuda()[None])
    assert out.float().abs().max().item() < 1e-12


# ------------------------------------------------------------------------------------------ end to end
def _forward_and_compare(cfg, x, d, rows, slab_rows=0, **kw):
    out, idx, kt, var = U.run_forward(cfg, d, slab_rows=slab_rows, **kw)
    rows = np.asarray(rows)
    sel = torch.from_numpy(rows).cuda()
    p = U.oracle_params(cfg, **kw)
    o = oracle.forward(p, **x, rows_t=rows, want_scores=True)
    mism = U.check_forward_rows(p, x, o, out[0][sel].float().cpu().numpy(), idx[0][sel].cpu().numpy(),
                                kt[0][sel].cpu().numpy(), rows, None, _vis(cfg, rows))
    assert not torch.isnan(out.float()).any()
    return mism, kt


@pytest.mark.parametrize("slab_rows", [0, 32, 96])
def test_forward_tiny_all_rows(tiny, slab_rows):
    cfg, x, d = tiny
    mism, kt = _forward_and_compare(cfg, x, d, np.arange(cfg.Lq), slab_rows=slab_rows)
    assert mism <= 5


def test_forward_l8k_sampled_rows(l8k):
    cfg, x, d = l8k
    mism, kt = _forward_and_compare(cfg, x, d, sample_rows(cfg, 40).numpy())
    k = kt[0, cfg.k_max:].float()
    assert k.min() >= cfg.k_min and k.max() <= cfg.k_max and k.mean() > 1200 and k.mean() < 3000


def test_forward_large_budget_equals_dense_gated_attention():
    """k_min >= L: S_t is everything visible; the output is dense gated attention (oracle's dense limit)."""
    cfg = CONFIGS["tiny"].with_(Lq=200, Lk=200, k_base=256, k_min=256, k_max=256)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    out, idx, kt, var = U.run_forward(cfg, d)
    assert (kt[0].cpu().numpy() == np.arange(1, 201)).all()
    for t in (0, 1, 57, 199):
        assert idx[0, t, :t + 1].tolist() == list(range(t + 1)) and (idx[0, t, t + 1:] == -1).all()
    o = oracle.forward(U.oracle_params(cfg), **x, rows_t=np.arange(200))
    U.check_out(out[0].float().cpu().numpy(), o["out"])


def test_forward_dense_fallback_mode_needs_no_indexer_inputs():
    """k_mode 3: every visible key, no indexer and no selection launches, indexer inputs may be absent."""
    cfg = CONFIGS["tiny"].with_(name="dense", B=2, Lq=150, Lk=333, k_base=8, k_min=4, k_max=336)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    p = gsa.make_params(cfg, k_mode=3)
    out = torch.full_like(d["Q"], float("nan"))
    idx = torch.full((cfg.B, cfg.Lq, cfg.k_max), -7, dtype=torch.int32, device="cuda")
    kt = torch.full((cfg.B, cfg.Lq), -7, dtype=torch.int32, device="cuda")
    ws = torch.empty(gsa.gsa_workspace_bytes(p, 0), dtype=torch.uint8, device="cuda")
    ws.fill_(0xFF)
    n0 = gsa.gsa_launch_count()
    gsa.gsa_forward(p, d["Q"], d["K"], d["V"], None, None, None, None, d["g1"], d["g2"], out, idx, kt, None, 0, ws)
    torch.cuda.synchronize()
    assert gsa.gsa_device_status(ws) == 0
    n_vis = cfg.Lk - cfg.Lq + np.arange(cfg.Lq) + 1
    assert (kt.cpu().numpy() == n_vis[None]).all()
    for t in (0, 77, 149):
        assert idx[1, t, : n_vis[t]].tolist() == list(range(n_vis[t])) and (idx[1, t, n_vis[t]:] == -1).all()
    rows_t = np.tile(np.arange(cfg.Lq), cfg.B)
    rows_b = np.repeat(np.arange(cfg.B), cfg.Lq)
    o = oracle.forward(U.oracle_params(cfg, k_mode=3), **x, rows_t=rows_t, rows_b=rows_b)
    U.check_out(out.float().cpu().numpy().reshape(cfg.B * cfg.Lq, cfg.n_h, cfg.d_h), o["out"])
    # k_max below Lk cannot hold every key: refused before any launch
    n1 = gsa.gsa_launch_count()
    with pytest.raises(gsa.GsaError):
        gsa.gsa_forward(gsa.make_params(cfg.with_(k_max=256), k_mode=3), d["Q"], d["K"], d["V"], None, None, None, None,
                        d["g1"], d["g2"], out, None, kt, None, 0, ws)
    assert gsa.gsa_launch_count() == n1
    assert n1 - n0 <= 6          # all-visible, value gate, range cuts, attention, finalize
    # the per-stage selection call in the same mode: whatever the scores, every visible key, in order
    sc = torch.rand((cfg.B, cfg.Lq, U.row_stride(cfg)), device="cuda")
    idx2, kt2, _ = U.run_topk(cfg, sc, k_mode=3)
    assert torch.equal(idx2, idx) and torch.equal(kt2, kt)


def test_forward_batched_chunked_prefill():
    """B = 3, Lk > Lq, ragged sizes, k_max not a multiple of the 16-key tile."""
    cfg = CONFIGS["l8k"].with_(name="chunk", B=3, Lq=150, Lk=1111, k_base=300, k_min=50, k_max=777, seed=13,
                               v_bar=2.0e-3)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    out, idx, kt, var = U.run_forward(cfg, d, slab_rows=64)
    p = U.oracle_params(cfg)
    for b in range(cfg.B):
        rows = np.arange(0, cfg.Lq, 5)
        o = oracle.forward(p, **x, rows_t=rows, rows_b=np.full_like(rows, b), want_scores=True)
        U.check_forward_rows(p, x, o, out[b][rows].float().cpu().numpy(), idx[b][rows].cpu().numpy(),
                             kt[b][rows].cpu().numpy(), rows, np.full_like(rows, b), _vis(cfg, rows))


def test_forward_small_decode_batch():
    """Decode geometry (Lq = 1) with the value gate applied inside the gather."""
    cfg = CONFIGS["decode"].with_(name="dec_small", B=5, Lk=9000, seed=14)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    out, idx, kt, var = U.run_forward(cfg, d)
    p = U.oracle_params(cfg)
    rows_b = np.arange(cfg.B)
    o = oracle.forward(p, **x, rows_t=np.zeros(cfg.B, np.int32), rows_b=rows_b, want_scores=True)
    U.check_forward_rows(p, x, o, out[:, 0].float().cpu().numpy(), idx[:, 0].cpu().numpy(), kt[:, 0].cpu().numpy(),
                         np.zeros(cfg.B, np.int64), rows_b, [cfg.Lk] * cfg.B)


@pytest.mark.parametrize("which", ["tiny", "l8k"])
def test_forward_is_deterministic(which, request):
    cfg, x, d = request.getfixturevalue(which)
    a = U.run_forward(cfg, d)
    b = U.run_forward(cfg, d)
    assert torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])
    assert torch.equal(a[0].view(torch.int16), b[0].view(torch.int16))


def test_forward_host_buffers_match_device_call(tiny):
    cfg, x, d = tiny
    p = gsa.make_params(cfg)
    out_dev, _, kt_dev, _ = U.run_forward(cfg, d)
    pin = {k: v.pin_memory() for k, v in x.items()}
    out_h = torch.empty_like(x["Q"]).pin_memory()
    kt_h = torch.empty((cfg.B, cfg.Lq), dtype=torch.int32).pin_memory()
    arena = torch.empty(gsa.gsa_forward_host_arena_bytes(p, 0), dtype=torch.uint8, device="cuda")
    gsa.gsa_forward_host(p, pin["Q"], pin["K"], pin["V"], pin["qI"], pin["kI"], pin["w"], None, pin["g1"], pin["g2"],
                         out_h, kt_h, 0, arena)
    assert torch.equal(out_h.view(torch.int16), out_dev.cpu().view(torch.int16))
    assert torch.equal(kt_h, kt_dev.cpu())


def test_forward_many_key_ranges_device_and_host_paths():
    """Key ranges of 1024 keys on a 3000-token sequence: three attention launches with carried softmax
    state, rows finalised range by range; the host-buffer call streams finished rows back early."""
    cfg = CONFIGS["tiny"].with_(name="ranges", B=2, Lq=3000, Lk=3000, k_base=300, k_min=64, k_max=600, seed=17,
                               v_bar=2.0e-3)
    x = make_inputs(cfg)
    d = U.to_dev(x)
    gsa.gsa_debug_set_attn_range_keys(1024)
    try:
        out, idx, kt, var = U.run_forward(cfg, d)
        p = gsa.make_params(cfg)
        pin = {k: v.pin_memory() for k, v in x.items()}
        out_h = torch.empty_like(x["Q"]).pin_memory()
        kt_h = torch.empty((cfg.B, cfg.Lq), dtype=torch.int32).pin_memory()
        arena = torch.empty(gsa.gsa_forward_host_arena_bytes(p, 0), dtype=torch.uint8, device="cuda")
        gsa.gsa_forward_host(p, pin["Q"], pin["K"], pin["V"], pin["qI"], pin["kI"], pin["w"], None, pin["g1"],
                             pin["g2"], out_h, kt_h, 0, arena)
    finally:
        gsa.gsa_debug_set_attn_range_keys(0)
    assert torch.equal(out_h.view(torch.int16), out.cpu().view(torch.int16))
    assert torch.equal(kt_h, kt.cpu())
    po = U.oracle_params(cfg)
    for b in range(cfg.B):
        rows = np.array([0, 5, 1023, 1024, 1500, 2047, 2048, 2999])
        o = oracle.forward(po, **x, rows_t=rows, rows_b=np.full_like(rows, b), want_scores=True)
        U.check_forward_rows(po, x, o, out[b][rows].float().cpu().numpy(), idx[b][rows].cpu().numpy(),
                             kt[b][rows].cpu().numpy(), rows, np.full_like(rows, b), _vis(cfg, rows))


def test_context_parallel_row_blocks_match_the_whole_sequence(l8k):
    """The context-parallel split on one GPU: the shares of two ranks (four row blocks in the chunked-prefill
    geometry Lq = block rows, Lk = block end, values gated by gsa_value_gate before the exchange) computed one
    after another from the gathered keys, against gsa_forward over the whole sequence and against the oracle."""
    from paper_2601_15305_b200 import context_parallel as cp
    cfg, x, d = l8k
    out_full, idx_full, kt_full, _ = U.run_forward(cfg, d)
    Vg = torch.empty_like(d["V"])
    gsa.gsa_value_gate(d["V"], d["g2"], Vg)
    keys = {"kI": d["kI"], "K": d["K"], "Vg": Vg}
    world = 2
    n0 = gsa.gsa_launch_count()
    for rank in range(world):
        blocks = cp.plan_row_blocks(cfg.Lk, world, rank)
        local = cp.shard(d, blocks)
        out, kt = cp.forward_context_parallel(cfg, local, world, rank, gathered_keys=keys)
        at = 0
        for blk in blocks:
            assert torch.equal(kt[0, at:at + blk.rows], kt_full[0, blk.t0:blk.t1])
            a, b = out[0, at:at + blk.rows].float(), out_full[0, blk.t0:blk.t1].float()
            assert (a - b).abs().max().item() <= 2.0 ** -8 * b.abs().max().item()       # one bf16 ulp of the largest value
            at += blk.rows
    assert gsa.gsa_launch_count() - n0 >= 4 * 4          # per block: indexer, selection, attention, finalize at least
    rows = sample_rows(cfg, 16).numpy()
    o = oracle.forward(U.oracle_params(cfg), **x, rows_t=rows, want_scores=True)
    sel = torch.from_numpy(rows).cuda()
    U.check_forward_rows(U.oracle_params(cfg), x, o, out_full[0][sel].float().cpu().numpy(), idx_full[0][sel].cpu().numpy(),
                         kt_full[0][sel].cpu().numpy(), rows, None, _vis(cfg, rows))


def test_argument_errors_do_not_launch(tiny):
    cfg, x, d = tiny
    p = gsa.make_params(cfg)
    n0 = gsa.gsa_launch_count()
    out = torch.empty_like(d["Q"])
    small_ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(gsa.GsaError, match="workspace"):
        gsa.gsa_forward(p, d["Q"], d["K"], d["V"], d["qI"], d["kI"], d["w"], None, d["g1"], d["g2"], out, ws=small_ws)
    with pytest.raises(gsa.GsaError, match="invalid"):
        gsa.gsa_indexer_scores(p, d["qI"], d["kI"], d["w"], None, torch.empty(10, device="cuda"), 100, small_ws)
    assert gsa.gsa_launch_count() == n0


# ------------------------------------------------------------------------------------------ full sizes
# The workloads of the benchmark at their full sizes, in the launch configuration bench.py times
# (default slab, default key ranges), checked on sampled rows the oracle computes one by one.
@pytest.fixture(scope="module")
def l128k():
    cfg = CONFIGS["l128k"]
    x = make_inputs(cfg)
    return cfg, x, U.to_dev(x)


def test_forward_l32k_sampled_rows_budgets_span_the_clamp_range():
    cfg = CONFIGS["l32k"]
    x = make_inputs(cfg)
    d = U.to_dev(x)
    mism, kt = _forward_and_compare(cfg, x, d, sample_rows(cfg, 256).numpy())
    k = kt[0, cfg.k_max:].cpu().numpy()
    assert k.min() == cfg.k_min and k.max() == cfg.k_max          # heterogeneous variance: both clamps are hit
    assert ((k > cfg.k_min) & (k < cfg.k_max)).mean() > 0.3


def test_stages_l128k_sampled_rows(l128k):
    """Stage by stage at L = 131072: scores of a block of late rows, bit-exact selection on those fp32 scores."""
    cfg, x, d = l128k
    for q0 in (9000, 40000, 70000, 101000, cfg.Lq - 48):      # 5 blocks x 16 rows = 80 rows
        q1 = q0 + 48
        sc = U.run_scores(cfg, d, q_begin=q0, q_end=q1)
        rows = q0 + np.arange(0, 48, 3)
        rows[-1] = q1 - 1
        got = sc[0][torch.from_numpy(rows - q0).cuda()].cpu().numpy()
        want = oracle.scores(U.oracle_params(cfg), x["qI"], x["kI"], x["w"], None, rows)
        U.check_scores(got, want, _vis(cfg, rows))
        idx, kt, var = U.run_topk(cfg, sc, q_begin=q0, q_end=q1)
        o = oracle.select_f32(U.oracle_params(cfg), got, rows)
        sel = torch.from_numpy(rows - q0).cuda()
        U.check_selection_exact(o, idx[0][sel].cpu().numpy(), kt[0][sel].cpu().numpy(), None)


def test_forward_l128k_sampled_rows(l128k):
    cfg, x, d = l128k
    mism, kt = _forward_and_compare(cfg, x, d, sample_rows(cfg, 256).numpy())
    k = kt[0, cfg.k_max:].float()
    assert k.min() >= cfg.k_min and k.max() <= cfg.k_max and 1500 < k.mean() < 3000


def test_forward_decode_full_size():
    """B = 32 single-token queries over 131072-token caches; sequences are generated and uploaded one
    at a time, the oracle checks a sample of them."""
    cfg = CONFIGS["decode"]
    p = gsa.make_params(cfg)
    dev = {}
    checked = (0, 5, 13, 22, 31)
    host = {}
    for b in range(cfg.B):
        xb = make_inputs(cfg, slice(b, b + 1))
        for k, v in xb.items():
            if k not in dev:
                dev[k] = torch.empty((cfg.B,) + tuple(v.shape[1:]), dtype=v.dtype, device="cuda")
            dev[k][b].copy_(v[0])
        if b in checked:
            host[b] = xb
    out, idx, kt, var = U.run_forward(cfg, dev)
    cfg1 = cfg.with_(B=1)
    for b in checked:
        o = oracle.forward(U.oracle_params(cfg1), **host[b], rows_t=np.zeros(1, np.int32), want_scores=True)
        U.check_forward_rows(U.oracle_params(cfg1), host[b], o, out[b].float().cpu().numpy(), idx[b].cpu().numpy(),
                             kt[b].cpu().numpy(), np.zeros(1, np.int64), None, [cfg.Lk])
    assert (kt >= cfg.k_min).all() and (kt <= cfg.k_max).all()


# ------------------------------------------------------------------------------------------ projections
@pytest.mark.parametrize("base,L,d_model", [("tiny", 300, 192), ("l8k", 1000, 2048)])
def test_project_matches_oracle(base, L, d_model):
    """gsa_project (tcgen05 GEMM + routing epilogue) against the fp64 oracle: ragged token count and a
    last column tile that is only partly used."""
    cfg = CONFIGS[base].with_(name="proj", B=2, Lq=L, Lk=L)
    p = gsa.make_params(cfg)
    n_cols = gsa.gsa_project_columns(p)
    g = torch.Generator().manual_seed(23)
    M = cfg.B * L
    H = torch.randn(M, d_model, generator=g).to(torch.bfloat16)
    Wt = (torch.randn(n_cols, d_model, generator=g) / d_model ** 0.5).to(torch.bfloat16)
    dev = lambda *s, dt=torch.bfloat16: torch.full(s, float("nan"), dtype=dt, device="cuda")
    qI, kI = dev(cfg.B, L, cfg.HI, cfg.dI), dev(cfg.B, L, cfg.dI)
    w = dev(cfg.B, L, cfg.HI, dt=torch.float32)
    g1, g2 = dev(cfg.B, L, cfg.n_h, cfg.d_h), dev(cfg.B, L, cfg.n_kv, cfg.d_h)
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    gsa.gsa_project(p, d_model, H.cuda(), Wt.cuda(), qI, kI, w, g1, g2, ws)
    assert gsa.gsa_device_status(ws) == 0
    rows = np.unique(np.concatenate([np.arange(0, M, 37), [0, 127, 128, M - 1]]))
    o = oracle.project(U.oracle_params(cfg), d_model, H, Wt, rows)
    sel = torch.from_numpy(rows).cuda()

    def close_bf16(got, want):          # fp32 accumulation rounded to bf16 once: half an ulp = 2^-9 relative
        got = got.reshape(M, -1)[sel].float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        assert (np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 1e-5).all()

    close_bf16(qI, o["qI"]); close_bf16(kI, o["kI"]); close_bf16(g1, o["g1"]); close_bf16(g2, o["g2"])
    gw = w.reshape(M, -1)[sel].cpu().numpy().astype(np.float64)
    assert np.abs(gw - o["w"]).max() <= 2e-6          # fp32 sigmoid of an fp32-accumulated logit
    for t in (qI, kI, w, g1, g2):                      # every element written
        assert not torch.isnan(t.float()).any()


def test_output_projection_matches_oracle():
    cfg = CONFIGS["l8k"].with_(name="wo", B=1, Lq=777, Lk=777)
    p = gsa.make_params(cfg)
    d_model = 2048
    g = torch.Generator().manual_seed(29)
    K = cfg.n_h * cfg.d_h
    X = torch.randn(cfg.B, cfg.Lq, cfg.n_h, cfg.d_h, generator=g).to(torch.bfloat16)
    Wt = (torch.randn(d_model, K, generator=g) / K ** 0.5).to(torch.bfloat16)
    u = torch.full((cfg.B, cfg.Lq, d_model), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    gsa.gsa_output_projection(p, d_model, X.cuda(), Wt.cuda(), u, ws)
    assert gsa.gsa_device_status(ws) == 0
    rows = np.unique(np.concatenate([np.arange(0, cfg.Lq, 41), [127, 128, cfg.Lq - 1]]))
    want = oracle.out_project(X.reshape(-1, K), Wt, rows)
    got = u.reshape(-1, d_model)[torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
    assert (np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 1e-5).all()     # fp32 accumulate, one bf16 rounding
    assert not torch.isnan(u.float()).any()
