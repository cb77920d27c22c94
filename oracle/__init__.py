"""Python face of the fp64 CPU oracle (oracle/gsa_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline / reference legs.  Nothing here touches the CUDA library,
and the CUDA package never imports this module.

The wrappers only marshal arguments: torch / numpy arrays are widened (exactly) to
contiguous fp32 and handed to the C functions, which do all arithmetic in double.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gsa_oracle.c")
_LIB = os.path.join(_HERE, "libgsa_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over query rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _P(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "Lq", "Lk", "n_h", "n_kv", "d_h", "HI", "dI", "k_base", "k_min", "k_max", "k_mode")] + \
               [("v_bar", ctypes.c_double), ("sm_scale", ctypes.c_double), ("act", ctypes.c_int32)]


@dataclass
class OracleParams:
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
    k_mode: int = 0
    v_bar: float = 1.0
    sm_scale: float = 0.0
    act: int = 0          # 0: sigmoid indexer (Eq. 7), 1: ReLU indexer (Eq. 3)

    @classmethod
    def from_config(cls, cfg, **kw) -> "OracleParams":
        base = dict(B=cfg.B, Lq=cfg.Lq, Lk=cfg.Lk, n_h=cfg.n_h, n_kv=cfg.n_kv, d_h=cfg.d_h, HI=cfg.HI,
                    dI=cfg.dI, k_base=cfg.k_base, k_min=cfg.k_min, k_max=cfg.k_max, v_bar=cfg.v_bar)
        base.update(kw)
        return cls(**base)

    def c(self) -> _P:
        return _P(self.B, self.Lq, self.Lk, self.n_h, self.n_kv, self.d_h, self.HI, self.dI,
                  self.k_base, self.k_min, self.k_max, self.k_mode, float(self.v_bar), float(self.sm_scale),
                  int(self.act))

    def visible(self, t: int) -> int:
        return self.Lk - self.Lq + t + 1


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.gsa_oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().gsa_oracle_num_threads())


def _f32(x) -> np.ndarray:
    """exact widening of bf16 / fp32 data to contiguous float32 numpy"""
    if x is None:
        return None
    if hasattr(x, "detach"):
        import torch
        x = x.detach().to("cpu").to(torch.float32).numpy()
    return np.ascontiguousarray(x, dtype=np.float32)


def _i32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().to("cpu").numpy()
    return np.ascontiguousarray(x, dtype=np.int32)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _rows(p: OracleParams, rows_t, rows_b=None):
    rows_t = _i32(rows_t).reshape(-1)
    rows_b = np.zeros_like(rows_t) if rows_b is None else _i32(rows_b).reshape(-1)
    assert rows_t.shape == rows_b.shape
    assert rows_t.min(initial=0) >= 0 and rows_t.max(initial=0) < p.Lq
    assert rows_b.min(initial=0) >= 0 and rows_b.max(initial=0) < p.B
    return rows_b, rows_t


def scores(p: OracleParams, qI, kI, w, bI=None, rows_t: Sequence[int] = (), rows_b=None) -> np.ndarray:
    """Eq. 7 for the listed rows.  Returns [n_rows, Lk] float64; entries past the row's
    causal limit are NaN."""
    rows_b, rows_t = _rows(p, rows_t, rows_b)
    qI, kI, w, bI = _f32(qI), _f32(kI), _f32(w), _f32(bI)
    assert qI.size == p.B * p.Lq * p.HI * p.dI and kI.size == p.B * p.Lk * p.dI and w.size == p.B * p.Lq * p.HI
    out = np.full((len(rows_t), p.Lk), np.nan, dtype=np.float64)
    c = p.c()
    lib().gsa_oracle_scores_rows(ctypes.byref(c), _ptr(qI), _ptr(kI), _ptr(w), _ptr(bI), _ptr(rows_b),
                                 _ptr(rows_t), ctypes.c_int(len(rows_t)), _ptr(out))
    return out


def select_f32(p: OracleParams, score_rows, rows_t):
    """Eq. 8 + Eq. 4 on supplied fp32 score rows (row r belongs to query rows_t[r]).
    Returns dict(idx [n,k_max] ascending / -1 padded, kt, keff, var, r)."""
    rows_t = _i32(rows_t).reshape(-1)
    sc = _f32(score_rows)
    assert sc.ndim == 2 and sc.shape[0] == len(rows_t)
    n = len(rows_t)
    idx = np.empty((n, p.k_max), dtype=np.int32)
    kt = np.empty(n, dtype=np.int32)
    keff = np.empty(n, dtype=np.int32)
    var = np.empty(n, dtype=np.float64)
    r = np.empty(n, dtype=np.float64)
    c = p.c()
    lib().gsa_oracle_select_rows_f32(ctypes.byref(c), _ptr(sc), ctypes.c_int64(sc.shape[1]), _ptr(rows_t),
                                     ctypes.c_int(n), _ptr(idx), _ptr(kt), _ptr(keff), _ptr(var), _ptr(r))
    return dict(idx=idx, kt=kt, keff=keff, var=var, r=r)


def attn(p: OracleParams, Q, K, V, g1, g2, idx, keff, rows_t, rows_b=None) -> np.ndarray:
    """Eq. 9-12 and Eq. 10 for the listed rows with given index sets.  [n, n_h, d_h] float64."""
    rows_b, rows_t = _rows(p, rows_t, rows_b)
    Q, K, V, g1, g2 = _f32(Q), _f32(K), _f32(V), _f32(g1), _f32(g2)
    idx, keff = _i32(idx), _i32(keff).reshape(-1)
    assert idx.shape == (len(rows_t), p.k_max) and keff.shape == (len(rows_t),)
    for r in range(len(rows_t)):
        assert (idx[r, :keff[r]] >= 0).all() and (idx[r, :keff[r]] < p.Lk).all()
    out = np.empty((len(rows_t), p.n_h, p.d_h), dtype=np.float64)
    c = p.c()
    lib().gsa_oracle_attn_rows(ctypes.byref(c), _ptr(Q), _ptr(K), _ptr(V), _ptr(g1), _ptr(g2), _ptr(rows_b),
                               _ptr(rows_t), ctypes.c_int(len(rows_t)), _ptr(idx), _ptr(keff), _ptr(out))
    return out


def forward(p: OracleParams, Q, K, V, qI, kI, w, g1, g2, bI=None, rows_t: Sequence[int] = (), rows_b=None,
            want_scores: bool = False):
    """The whole path for the listed rows.  Returns dict(out, idx, kt, keff, var, r[, scores])."""
    rows_b, rows_t = _rows(p, rows_t, rows_b)
    Q, K, V, g1, g2 = _f32(Q), _f32(K), _f32(V), _f32(g1), _f32(g2)
    qI, kI, w, bI = _f32(qI), _f32(kI), _f32(w), _f32(bI)
    n = len(rows_t)
    out = np.empty((n, p.n_h, p.d_h), dtype=np.float64)
    idx = np.empty((n, p.k_max), dtype=np.int32)
    kt = np.empty(n, dtype=np.int32)
    keff = np.empty(n, dtype=np.int32)
    var = np.empty(n, dtype=np.float64)
    r = np.empty(n, dtype=np.float64)
    sc = np.full((n, p.Lk), np.nan, dtype=np.float64) if want_scores else None
    c = p.c()
    lib().gsa_oracle_forward_rows(ctypes.byref(c), _ptr(Q), _ptr(K), _ptr(V), _ptr(qI), _ptr(kI), _ptr(w),
                                  _ptr(bI), _ptr(g1), _ptr(g2), _ptr(rows_b), _ptr(rows_t), ctypes.c_int(n),
                                  _ptr(out), _ptr(idx), _ptr(kt), _ptr(keff), _ptr(var), _ptr(r), _ptr(sc))
    res = dict(out=out, idx=idx, kt=kt, keff=keff, var=var, r=r)
    if want_scores:
        res["scores"] = sc
    return res


def project_rows_total(p: OracleParams) -> int:
    """Rows of the stacked, transposed weight matrix: q^I, k^I, 8 head-weight rows, g1, g2."""
    return p.HI * p.dI + p.dI + 8 + p.n_h * p.d_h + p.n_kv * p.d_h


def project(p: OracleParams, d_model: int, H, Wt, rows_m: Sequence[int]):
    """Upstream projections (text below Eq. 7, Eq. 9, Eq. 10) of the listed token rows of H [M, d_model].
    Returns dict(qI [n, HI*dI], kI [n, dI], w [n, HI] (after the sigmoid), g1 [n, n_h*d_h], g2 [n, n_kv*d_h]), fp64."""
    H, Wt = _f32(H), _f32(Wt)
    rows_m = _i32(rows_m).reshape(-1)
    assert H.ndim == 2 and H.shape[1] == d_model and Wt.shape == (project_rows_total(p), d_model)
    assert rows_m.min(initial=0) >= 0 and rows_m.max(initial=0) < H.shape[0]
    n = len(rows_m)
    out = dict(qI=np.empty((n, p.HI * p.dI)), kI=np.empty((n, p.dI)), w=np.empty((n, p.HI)),
               g1=np.empty((n, p.n_h * p.d_h)), g2=np.empty((n, p.n_kv * p.d_h)))
    c = p.c()
    lib().gsa_oracle_project_rows(ctypes.byref(c), ctypes.c_int(d_model), _ptr(H), _ptr(Wt), _ptr(rows_m),
                                  ctypes.c_int(n), _ptr(out["qI"]), _ptr(out["kI"]), _ptr(out["w"]),
                                  _ptr(out["g1"]), _ptr(out["g2"]))
    return out


def out_project(X, Wt, rows_m: Sequence[int]) -> np.ndarray:
    """Output projection (concatenated heads times W_O) of the listed token rows: X [M, K], Wt [N, K] -> [n, N] fp64."""
    X, Wt = _f32(X), _f32(Wt)
    rows_m = _i32(rows_m).reshape(-1)
    assert X.ndim == 2 and Wt.ndim == 2 and X.shape[1] == Wt.shape[1]
    assert rows_m.min(initial=0) >= 0 and rows_m.max(initial=0) < X.shape[0]
    u = np.empty((len(rows_m), Wt.shape[0]))
    lib().gsa_oracle_out_project_rows(ctypes.c_int(X.shape[1]), ctypes.c_int(Wt.shape[0]), _ptr(X), _ptr(Wt),
                                      _ptr(rows_m), ctypes.c_int(len(rows_m)), _ptr(u))
    return u


def attn_bwd(p: OracleParams, Q, K, V, g1, g2, idx, keff, dout, rows_t, rows_b=None):
    """Backward of Eq. 9-12 and Eq. 10 for the listed rows with given index sets: derivatives of
    sum_r <dout[r], out[r]>.  dout: [n, n_h, d_h].  Returns dict(dQ, dg1: [n, n_h, d_h];
    dK, dV, dg2: [B, Lk, n_kv, d_h] summed over the listed rows), all float64."""
    rows_b, rows_t = _rows(p, rows_t, rows_b)
    Q, K, V, g1, g2, dout = _f32(Q), _f32(K), _f32(V), _f32(g1), _f32(g2), _f32(dout)
    idx, keff = _i32(idx), _i32(keff).reshape(-1)
    n = len(rows_t)
    assert idx.shape == (n, p.k_max) and keff.shape == (n,) and dout.shape == (n, p.n_h, p.d_h)
    for r in range(n):
        assert (idx[r, :keff[r]] >= 0).all() and (idx[r, :keff[r]] < p.Lk).all()
    dQ = np.empty((n, p.n_h, p.d_h), dtype=np.float64)
    dg1 = np.empty_like(dQ)
    dK = np.empty((p.B, p.Lk, p.n_kv, p.d_h), dtype=np.float64)
    dV = np.empty_like(dK)
    dg2 = np.empty_like(dK)
    c = p.c()
    lib().gsa_oracle_attn_bwd_rows(ctypes.byref(c), _ptr(Q), _ptr(K), _ptr(V), _ptr(g1), _ptr(g2), _ptr(rows_b),
                                   _ptr(rows_t), ctypes.c_int(n), _ptr(idx), _ptr(keff), _ptr(dout),
                                   _ptr(dQ), _ptr(dg1), _ptr(dK), _ptr(dV), _ptr(dg2))
    return dict(dQ=dQ, dg1=dg1, dK=dK, dV=dV, dg2=dg2)


def vbar_update(v_bar: float, momentum: float, var) -> tuple:
    """(new v_bar, batch-mean variance): EMA of the score variance across the batch (text below Eq. 8)."""
    v = _f32(var).reshape(-1)
    f = lib().gsa_oracle_vbar_update
    f.restype = ctypes.c_double
    m = ctypes.c_double(0.0)
    new = f(ctypes.c_double(v_bar), ctypes.c_double(momentum), _ptr(v), ctypes.c_int64(v.size), ctypes.byref(m))
    return float(new), float(m.value)


def attn_probs_mean(p: OracleParams, Q, K, idx, keff, rows_t, rows_b=None) -> np.ndarray:
    """Target of the indexer's sparse-phase loss (Eq. 14): the attention distribution of Eq. 11 on S_t,
    averaged over the heads.  [n, k_max] float64, zeros past keff."""
    rows_b, rows_t = _rows(p, rows_t, rows_b)
    Q, K = _f32(Q), _f32(K)
    idx, keff = _i32(idx), _i32(keff).reshape(-1)
    n = len(rows_t)
    assert idx.shape == (n, p.k_max) and keff.shape == (n,)
    out = np.empty((n, p.k_max), dtype=np.float64)
    c = p.c()
    lib().gsa_oracle_attn_probs_mean_rows(ctypes.byref(c), _ptr(Q), _ptr(K), _ptr(rows_b), _ptr(rows_t),
                                          ctypes.c_int(n), _ptr(idx), _ptr(keff), _ptr(out))
    return out


def indexer_kl(p: OracleParams, qI, kI, w, bI, idx, keff, pbar, rows_t, rows_b=None):
    """Eq. 14 for the listed rows with the target distribution pbar [n, k_max] given, and its derivatives.
    Returns dict(loss [n], dqI [n, HI, dI], dw [n, HI], dkI [B, Lk, dI], dbI [HI]), all float64."""
    rows_b, rows_t = _rows(p, rows_t, rows_b)
    qI, kI, w, bI = _f32(qI), _f32(kI), _f32(w), _f32(bI)
    idx, keff = _i32(idx), _i32(keff).reshape(-1)
    pbar = np.ascontiguousarray(pbar, dtype=np.float64)
    n = len(rows_t)
    assert idx.shape == (n, p.k_max) and keff.shape == (n,) and pbar.shape == (n, p.k_max)
    loss = np.empty(n, dtype=np.float64)
    dqI = np.empty((n, p.HI, p.dI), dtype=np.float64)
    dw = np.empty((n, p.HI), dtype=np.float64)
    dkI = np.empty((p.B, p.Lk, p.dI), dtype=np.float64)
    dbI = np.empty(p.HI, dtype=np.float64)
    c = p.c()
    lib().gsa_oracle_indexer_kl_rows(ctypes.byref(c), _ptr(qI), _ptr(kI), _ptr(w), _ptr(bI), _ptr(rows_b),
                                     _ptr(rows_t), ctypes.c_int(n), _ptr(idx), _ptr(keff), _ptr(pbar),
                                     _ptr(loss), _ptr(dqI), _ptr(dw), _ptr(dkI), _ptr(dbI))
    return dict(loss=loss, dqI=dqI, dw=dw, dkI=dkI, dbI=dbI)
