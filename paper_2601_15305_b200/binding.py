"""Thin ctypes binding of libgsa_b200.so: same names as include/gsa.h, argument
marshalling only.  torch is used for device memory and streams; every step of the path
runs inside the library's CUDA kernels.  There is no fallback: if the shared library
is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from .inputs import GsaConfig

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libgsa_b200.so")

EXPORTS = (
    "gsa_workspace_bytes", "gsa_indexer_scores", "gsa_adaptive_topk", "gsa_sparse_gated_attn_fwd",
    "gsa_forward", "gsa_forward_host_arena_bytes", "gsa_forward_host", "gsa_device_status",
    "gsa_launch_count", "gsa_debug_set_indexer_path", "gsa_profile_set_events", "gsa_status_string",
    "gsa_sparse_gated_attn_fwd_static", "gsa_attn_workspace_bytes", "gsa_debug_set_attn_range_keys",
    "gsa_select_fallback_rows", "gsa_project", "gsa_project_columns", "gsa_output_projection",
    "gsa_attn_bwd_workspace_bytes", "gsa_sparse_gated_attn_bwd", "gsa_vbar_update",
    "gsa_attn_probs_mean", "gsa_indexer_kl_workspace_bytes", "gsa_indexer_kl_bwd", "gsa_sparse_gated_attn_fwd_lse",
    "gsa_profile_set_timeline", "gsa_probe_gather", "gsa_probe_ex2", "gsa_debug_set_wait_limit", "gsa_value_gate",
)

STATIC_SCRATCH_BYTES = 32 << 20     # GSA_STATIC_SCRATCH_BYTES of include/gsa.h


class GsaError(RuntimeError):
    pass


class gsa_params_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "Lq", "Lk", "n_h", "n_kv", "d_h", "HI", "dI", "k_base", "k_min", "k_max", "k_mode")] + \
               [("v_bar", ctypes.c_float), ("sm_scale", ctypes.c_float),
                ("q_begin", ctypes.c_int32), ("q_end", ctypes.c_int32), ("act", ctypes.c_int32)]


def make_params(cfg: GsaConfig = None, *, k_mode: int = 0, sm_scale: float = 0.0, q_begin: int = 0,
                q_end: int = 0, act: int = 0, **over) -> gsa_params_t:
    f = dict(B=1, Lq=1, Lk=1, n_h=1, n_kv=1, d_h=64, HI=1, dI=32, k_base=1, k_min=1, k_max=1, v_bar=1.0)
    if cfg is not None:
        f.update(B=cfg.B, Lq=cfg.Lq, Lk=cfg.Lk, n_h=cfg.n_h, n_kv=cfg.n_kv, d_h=cfg.d_h, HI=cfg.HI, dI=cfg.dI,
                 k_base=cfg.k_base, k_min=cfg.k_min, k_max=cfg.k_max, v_bar=cfg.v_bar)
    f.update(over)
    return gsa_params_t(f["B"], f["Lq"], f["Lk"], f["n_h"], f["n_kv"], f["d_h"], f["HI"], f["dI"], f["k_base"],
                        f["k_min"], f["k_max"], k_mode, float(f["v_bar"]), float(sm_scale), q_begin, q_end, act)


_lib = None


def lib() -> ctypes.CDLL:
    """Load the shared library (built by paper_2601_15305_b200.build).  Raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise GsaError(f"{LIB_PATH} not found: build it with `python -m paper_2601_15305_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        L.gsa_status_string.restype = ctypes.c_char_p
        L.gsa_launch_count.restype = ctypes.c_int64
        for name in EXPORTS:
            getattr(L, name)
        _lib = L
    return _lib


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise GsaError(f"{what} failed: {lib().gsa_status_string(rc).decode()} ({rc})")


def _dp(t: Optional[torch.Tensor], dtype=None, cuda: bool = True):
    if t is None:
        return ctypes.c_void_p(0)
    if dtype is not None and t.dtype != dtype:
        raise GsaError(f"expected dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise GsaError("tensor must be contiguous")
    if cuda and not t.is_cuda:
        raise GsaError("tensor must live on the GPU")
    if not cuda and t.is_cuda:
        raise GsaError("tensor must live on the host")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream]) -> ctypes.c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


BF16, F32, I32 = torch.bfloat16, torch.float32, torch.int32


def gsa_workspace_bytes(p: gsa_params_t, slab_rows: int = 0) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().gsa_workspace_bytes(ctypes.byref(p), ctypes.c_int32(slab_rows), ctypes.byref(n)), "gsa_workspace_bytes")
    return n.value


def gsa_attn_workspace_bytes(p: gsa_params_t, with_value_gate_prepass: bool = True) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().gsa_attn_workspace_bytes(ctypes.byref(p), ctypes.c_int32(1 if with_value_gate_prepass else 0),
                                          ctypes.byref(n)), "gsa_attn_workspace_bytes")
    return n.value


def gsa_debug_set_attn_range_keys(keys: int) -> None:
    lib().gsa_debug_set_attn_range_keys(ctypes.c_int32(keys))


def gsa_indexer_scores(p, qI, kI, w, bI, scores, row_stride: int, ws, stream=None) -> None:
    _check(lib().gsa_indexer_scores(ctypes.byref(p), _dp(qI, BF16), _dp(kI, BF16), _dp(w, F32), _dp(bI, F32),
                                    _dp(scores, F32), ctypes.c_int64(row_stride), _dp(ws),
                                    ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)),
           "gsa_indexer_scores")


def gsa_project_columns(p: gsa_params_t) -> int:
    n = ctypes.c_int32(0)
    _check(lib().gsa_project_columns(ctypes.byref(p), ctypes.byref(n)), "gsa_project_columns")
    return n.value


def gsa_project(p, d_model: int, H, Wt, qI, kI, w, g1, g2, ws, stream=None) -> None:
    _check(lib().gsa_project(ctypes.byref(p), ctypes.c_int32(d_model), _dp(H, BF16), _dp(Wt, BF16), _dp(qI, BF16),
                             _dp(kI, BF16), _dp(w, F32), _dp(g1, BF16), _dp(g2, BF16), _dp(ws),
                             ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)), "gsa_project")


def gsa_output_projection(p, d_model: int, attn_out, Wo_t, u, ws, stream=None) -> None:
    _check(lib().gsa_output_projection(ctypes.byref(p), ctypes.c_int32(d_model), _dp(attn_out, BF16), _dp(Wo_t, BF16),
                                       _dp(u, BF16), _dp(ws), ctypes.c_size_t(ws.numel() * ws.element_size()),
                                       _stream(stream)), "gsa_output_projection")


def gsa_adaptive_topk(p, scores, row_stride: int, idx, kt, var=None, ws=None, stream=None) -> None:
    _check(lib().gsa_adaptive_topk(ctypes.byref(p), _dp(scores, F32), ctypes.c_int64(row_stride), _dp(idx, I32),
                                   _dp(kt, I32), _dp(var, F32), _dp(ws),
                                   ctypes.c_size_t(0 if ws is None else ws.numel() * ws.element_size()),
                                   _stream(stream)), "gsa_adaptive_topk")


def gsa_sparse_gated_attn_fwd(p, Q, K, V, g1, g2, idx, kt, out, ws=None, stream=None) -> None:
    _check(lib().gsa_sparse_gated_attn_fwd(ctypes.byref(p), _dp(Q, BF16), _dp(K, BF16), _dp(V, BF16), _dp(g1, BF16),
                                           _dp(g2, BF16), _dp(idx, I32), _dp(kt, I32), _dp(out, BF16), _dp(ws),
                                           ctypes.c_size_t(0 if ws is None else ws.numel() * ws.element_size()),
                                           _stream(stream)), "gsa_sparse_gated_attn_fwd")


def gsa_attn_bwd_workspace_bytes(p) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().gsa_attn_bwd_workspace_bytes(ctypes.byref(p), ctypes.byref(n)), "gsa_attn_bwd_workspace_bytes")
    return int(n.value)


def gsa_sparse_gated_attn_bwd(p, Q, K, V, g1, g2, idx, kt, out, dout, dQ, dK, dV, dg1, dg2, ws, stream=None,
                              pbar=None, lse=None) -> None:
    _check(lib().gsa_sparse_gated_attn_bwd(ctypes.byref(p), _dp(Q, BF16), _dp(K, BF16), _dp(V, BF16), _dp(g1, BF16),
                                           _dp(g2, BF16), _dp(idx, I32), _dp(kt, I32), _dp(out, BF16),
                                           _dp(dout, BF16), _dp(dQ, BF16), _dp(dK, BF16), _dp(dV, BF16),
                                           _dp(dg1, BF16), _dp(dg2, BF16), _dp(pbar, F32), _dp(lse, F32), _dp(ws),
                                           ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)),
           "gsa_sparse_gated_attn_bwd")


def gsa_attn_probs_mean(p, Q, K, idx, kt, pbar, ws, stream=None) -> None:
    _check(lib().gsa_attn_probs_mean(ctypes.byref(p), _dp(Q, BF16), _dp(K, BF16), _dp(idx, I32), _dp(kt, I32),
                                     _dp(pbar, F32), _dp(ws), ctypes.c_size_t(ws.numel() * ws.element_size()),
                                     _stream(stream)), "gsa_attn_probs_mean")


def gsa_indexer_kl_workspace_bytes(p) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().gsa_indexer_kl_workspace_bytes(ctypes.byref(p), ctypes.byref(n)), "gsa_indexer_kl_workspace_bytes")
    return int(n.value)


def gsa_indexer_kl_bwd(p, qI, kI, w, bI, idx, kt, pbar, loss, dqI, dkI, dw, dbI, ws, stream=None) -> None:
    _check(lib().gsa_indexer_kl_bwd(ctypes.byref(p), _dp(qI, BF16), _dp(kI, BF16), _dp(w, F32), _dp(bI, F32),
                                    _dp(idx, I32), _dp(kt, I32), _dp(pbar, F32), _dp(loss, F32), _dp(dqI, BF16),
                                    _dp(dkI, BF16), _dp(dw, F32), _dp(dbI, F32), _dp(ws),
                                    ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)),
           "gsa_indexer_kl_bwd")


def gsa_vbar_update(var, momentum: float, v_bar, mean_var=None, stream=None) -> None:
    """v_bar (one fp32 on the device) <- momentum * v_bar + (1 - momentum) * mean(var)."""
    _check(lib().gsa_vbar_update(_dp(var, F32), ctypes.c_int64(var.numel()), ctypes.c_float(momentum),
                                 _dp(v_bar, F32), _dp(mean_var, F32), _stream(stream)), "gsa_vbar_update")


def gsa_value_gate(V, g2, V_gated, stream=None) -> None:
    _check(lib().gsa_value_gate(_dp(V, BF16), _dp(g2, BF16), _dp(V_gated, BF16), ctypes.c_int64(V.numel()), _stream(stream)),
           "gsa_value_gate")


def gsa_sparse_gated_attn_fwd_lse(p, Q, K, V, g1, g2, idx, kt, out, lse, ws, stream=None) -> None:
    _check(lib().gsa_sparse_gated_attn_fwd_lse(ctypes.byref(p), _dp(Q, BF16), _dp(K, BF16), _dp(V, BF16),
                                               _dp(g1, BF16), _dp(g2, BF16), _dp(idx, I32), _dp(kt, I32),
                                               _dp(out, BF16), _dp(lse, F32), _dp(ws),
                                               ctypes.c_size_t(ws.numel() * ws.element_size()), _stream(stream)),
           "gsa_sparse_gated_attn_fwd_lse")


def gsa_sparse_gated_attn_fwd_static(p, Q, K, V, g1, g2, idx, kt, out, stream=None) -> None:
    """Sparse gated attention with the library's built-in scratch array: nothing is allocated, so it
    suits callers that cannot call cudaMalloc or hand over a workspace.  Problems whose gated values
    exceed STATIC_SCRATCH_BYTES are refused; calls on one GPU must not overlap (one shared array)."""
    _check(lib().gsa_sparse_gated_attn_fwd_static(ctypes.byref(p), _dp(Q, BF16), _dp(K, BF16), _dp(V, BF16),
                                                  _dp(g1, BF16), _dp(g2, BF16), _dp(idx, I32), _dp(kt, I32),
                                                  _dp(out, BF16), _stream(stream)),
           "gsa_sparse_gated_attn_fwd_static")


def gsa_forward(p, Q, K, V, qI, kI, w, bI, g1, g2, out, idx_out=None, kt_out=None, var_out=None, slab_rows: int = 0,
                ws=None, stream=None) -> None:
    _check(lib().gsa_forward(ctypes.byref(p), _dp(Q, BF16), _dp(K, BF16), _dp(V, BF16), _dp(qI, BF16), _dp(kI, BF16),
                             _dp(w, F32), _dp(bI, F32), _dp(g1, BF16), _dp(g2, BF16), _dp(out, BF16),
                             _dp(idx_out, I32), _dp(kt_out, I32), _dp(var_out, F32), ctypes.c_int32(slab_rows),
                             _dp(ws), ctypes.c_size_t(0 if ws is None else ws.numel() * ws.element_size()),
                             _stream(stream)), "gsa_forward")


def gsa_forward_host_arena_bytes(p: gsa_params_t, slab_rows: int = 0) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().gsa_forward_host_arena_bytes(ctypes.byref(p), ctypes.c_int32(slab_rows), ctypes.byref(n)),
           "gsa_forward_host_arena_bytes")
    return n.value


def gsa_forward_host(p, Q, K, V, qI, kI, w, bI, g1, g2, out, kt_out, slab_rows: int, arena, stream=None) -> None:
    """All tensors but `arena` are HOST tensors (pinned recommended); returns after the result is on the host."""
    h = lambda t, dt: _dp(t, dt, cuda=False)
    _check(lib().gsa_forward_host(ctypes.byref(p), h(Q, BF16), h(K, BF16), h(V, BF16), h(qI, BF16), h(kI, BF16),
                                  h(w, F32), h(bI, F32), h(g1, BF16), h(g2, BF16), h(out, BF16), h(kt_out, I32),
                                  ctypes.c_int32(slab_rows), _dp(arena),
                                  ctypes.c_size_t(arena.numel() * arena.element_size()), _stream(stream)),
           "gsa_forward_host")


def gsa_device_status(ws, stream=None) -> int:
    """Waits for the stream and returns the device status word (0 = ok) of `ws`; ws=None reads the
    one of gsa_sparse_gated_attn_fwd_static."""
    v = ctypes.c_int32(0)
    rc = lib().gsa_device_status(_dp(ws), _stream(stream), ctypes.byref(v))
    if rc not in (0, -5, -7):
        _check(rc, "gsa_device_status")
    return v.value


def gsa_select_fallback_rows(ws, stream=None) -> int:
    v = ctypes.c_int32(0)
    _check(lib().gsa_select_fallback_rows(_dp(ws), _stream(stream), ctypes.byref(v)), "gsa_select_fallback_rows")
    return v.value


def gsa_launch_count() -> int:
    return int(lib().gsa_launch_count())


def gsa_debug_set_indexer_path(path: int) -> None:
    lib().gsa_debug_set_indexer_path(ctypes.c_int32(path))


def gsa_debug_set_wait_limit(cycles: int = 0, withhold_first_copy: bool = False) -> None:
    lib().gsa_debug_set_wait_limit(ctypes.c_int64(cycles), ctypes.c_int32(1 if withhold_first_copy else 0))


STAGE_NAMES = ("indexer", "select", "value_gate", "range_cuts", "sparse_attn", "finalize")
_timeline_keep = None        # the arrays the library writes into must outlive the calls


def gsa_profile_set_timeline(events=None):
    """events: list of torch.cuda.Event(enable_timing=True), each recorded once already (so its handle exists),
    or None to switch the hook off.  Returns a function that, after a synchronize, gives the list of
    (stage name, milliseconds) intervals of the last gsa_forward."""
    global _timeline_keep
    if not events:
        lib().gsa_profile_set_timeline(None, ctypes.c_int32(0), None, None)
        _timeline_keep = None
        return None
    n = len(events)
    handles = (ctypes.c_void_p * n)(*[e.cuda_event for e in events])
    stages = (ctypes.c_int32 * n)()
    count = ctypes.c_int32(0)
    _timeline_keep = (handles, stages, count, events)
    lib().gsa_profile_set_timeline(handles, ctypes.c_int32(n), stages, ctypes.byref(count))

    def read():
        return [(STAGE_NAMES[stages[i]], events[i].elapsed_time(events[i + 1])) for i in range(count.value)]
    return read


def gsa_probe_gather(table, n_rows: int, row_bytes: int, piece_bytes: int, row_idx, sink, stream=None) -> None:
    _check(lib().gsa_probe_gather(_dp(table), ctypes.c_int32(n_rows), ctypes.c_int64(row_bytes), ctypes.c_int32(piece_bytes),
                                  _dp(row_idx, I32), ctypes.c_int64(row_idx.numel()), _dp(sink), _stream(stream)),
           "gsa_probe_gather")


def gsa_probe_ex2(iters: int, sink, stream=None) -> int:
    """Enqueues the exp2 probe; returns the number of 2^x it evaluates."""
    ops = ctypes.c_int64(0)
    _check(lib().gsa_probe_ex2(ctypes.c_int32(iters), ctypes.byref(ops), _dp(sink), _stream(stream)), "gsa_probe_ex2")
    return ops.value


def gsa_profile_set_events(ev_begin=None, ev_selected=None, ev_end=None) -> None:
    """torch.cuda.Event objects (already recorded once, so their handles exist) or None."""
    h = lambda e: ctypes.c_void_p(0 if e is None else e.cuda_event)
    lib().gsa_profile_set_events(h(ev_begin), h(ev_selected), h(ev_end))
