#!/usr/bin/env python
"""Benchmark of the GSA forward path: tokens/s of gsa_forward at L = 128K on one B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload l128k] [--impl reference]

A step is one gsa_forward over the whole workload (value gate, indexer, budget, top-k,
sparse attention, output gate).  Inputs are seeded synthetic tensors, resident in HBM before
the timed region; `e2e` repeats the measurement through gsa_forward_host with pinned host
buffers, so host<->device copies are inside its timed region.  N > 1 runs N independent
replicas (the path has no exchange step) and reports the aggregate.
`--impl reference` times the CPU oracle, as it stands, on a bounded sample of the same
workload (rank 0 only).
Prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2601_15305_b200 import cost_model
from paper_2601_15305_b200.inputs import CONFIGS, make_inputs, sample_rows

METRIC = "gsa_fwd_tokens_per_s"
UNIT = "tokens/s"
# special-function operations the indexer's epilogue spends per sigmoid: one exp2 each and one reciprocal
# shared by the eight heads of a query
SFU_OPS_PER_SIGMOID = 1.125
# DRAM bytes (read + written) of the sparse-attention launches of one forward, per workload, from the one-pass
# ncu capture summarised in profiles/gsa_sparse_attn_kernel_l128k_dram.md (taken with the current kernel,
# default slab and key ranges); a workload without a capture reports null
ATTN_DRAM_TRAFFIC = {"l128k": 47.06e9}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 200 ms.  The sampler is started before the warm-up
    steps (nvidia-smi takes a moment to produce its first line); mark() is called when the timed region starts
    and only the samples from then on are summarised.  A timed region shorter than the sampling period has none:
    the last sample before it (taken under the warm-up's load) is reported then, and `samples` stays 0."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.gpu, self.first = [], None, gpu_index, 0

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.gpu)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def mark(self):
        self.first = len(self.rows)

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=2)
        rows = self.rows[self.first:]
        in_region = len(rows)
        if not rows:
            rows = self.rows[-1:]
        sm = [float(r[1]) for r in rows if len(r) >= 9 and r[1].replace(".", "").isdigit()]
        mx = [float(r[2]) for r in rows if len(r) >= 9 and r[2].replace(".", "").isdigit()]
        reasons = set()
        for r in rows:
            if len(r) >= 9:
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm) if in_region else 0}


def aggregate_over_ranks(ms_local: float, units_local: float):
    """max time over ranks, sum of units: the whole-job throughput of N independent replicas."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return ms_local, units_local
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    u = torch.tensor([units_local], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def attention_bytes(cfg, kt_sum: int) -> float:
    """Algorithmic bytes of one sparse-attention launch: per selected (t, s) one K row and one V' row of
    all KV heads (2 * n_kv * d_h * 2 B) and one 4-byte index; per token Q, g1 and out (3 * n_h * d_h * 2 B)."""
    per_pair = 2 * cfg.n_kv * cfg.d_h * 2 + 4
    per_tok = 3 * cfg.n_h * cfg.d_h * 2 + 4
    return float(kt_sum) * per_pair + float(cfg.B * cfg.Lq) * per_tok


def measure_rates(gsa, stream):
    """Ceilings no vendor figure gives, measured here with the library's probe kernels (CUDA events on the
    launching stream, one warm-up launch, best of three): the rate at which 256-byte and 2048-byte row pieces
    picked by a random index list are gathered out of a 64 MB table (L2-resident, like one key range of K and
    V' rows) and out of a 2 GB table (HBM), and the special-function unit's exp2 rate."""
    gen = torch.Generator(device="cuda").manual_seed(7)
    sink = torch.zeros(64, dtype=torch.int32, device="cuda")
    out = {}

    def best_ms(fn, reps=3):
        fn()
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            fn()
            e1.record(stream)
            e1.synchronize()
            ts.append(e0.elapsed_time(e1))
        return min(ts)

    row_bytes = 2048
    for label, table_bytes in (("l2_64MB", 64 << 20), ("hbm_2GB", 2 << 30)):
        n_rows = table_bytes // row_bytes
        table = torch.empty(table_bytes, dtype=torch.uint8, device="cuda")
        table.random_(0, 255, generator=gen)
        for piece in (256, 2048):
            n_idx = (2 << 30) // piece
            idx = torch.randint(0, n_rows, (n_idx,), generator=gen, device="cuda", dtype=torch.int32)
            ms = best_ms(lambda: gsa.gsa_probe_gather(table, n_rows, row_bytes, piece, idx, sink, stream))
            out[f"gather_{label}_piece{piece}_gbs"] = n_idx * piece / (ms * 1e-3) / 1e9
            del idx
        del table
    ops = [0]

    def ex2():
        ops[0] = gsa.gsa_probe_ex2(4096, sink, stream)
    ms = best_ms(ex2)
    out["ex2_per_s"] = ops[0] / (ms * 1e-3)
    out["how"] = ("gsa_probe_gather: random rows of a 2048-byte-row table, first 256 / 2048 bytes of each, plain 32-byte "
                  "loads, 4 in flight per thread at 2048 threads per SM, 2 GiB gathered per launch; gsa_probe_ex2: 8 independent ex2.approx "
                  "chains per thread, 2048 threads per SM; best of 3 launches after a warm-up")
    return out


def oracle_sample_rate(cfg, x, n_rows: int):
    """tokens/s of the fp64 oracle on a stratified sample of query rows (mean row cost = mean over the sequence)."""
    import oracle
    p = oracle.OracleParams.from_config(cfg, v_bar=float(np.float32(cfg.v_bar)))
    if cfg.decode:
        rows_b = np.arange(min(cfg.B, n_rows), dtype=np.int32)
        rows_t = np.zeros_like(rows_b)
    else:
        strata = np.linspace(0, cfg.Lq, n_rows + 1)
        rows_t = ((strata[:-1] + strata[1:]) / 2).astype(np.int32)
        rows_b = np.zeros_like(rows_t)
    f32 = {k: oracle._f32(v) for k, v in x.items()}          # widening is not part of the timed work
    t0 = time.perf_counter()
    oracle.forward(p, **f32, rows_t=rows_t, rows_b=rows_b)
    dt = time.perf_counter() - t0
    return len(rows_t) / dt, dt, len(rows_t), oracle.num_threads()


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    x = make_inputs(cfg, slice(0, min(cfg.B, 4)) if cfg.decode else None)
    cores = oracle.num_threads()
    n_rows = 1024          # about 10 s of the oracle on 16 host cores
    rates = []
    for i in range(args.warmup + args.steps):
        r, dt, n, cores = oracle_sample_rate(cfg.with_(B=x["Q"].shape[0]), x, n_rows)
        if i >= args.warmup:
            rates.append((r, dt))
    value = float(np.mean([r for r, _ in rates]))
    ms = float(np.mean([dt for _, dt in rates]) * 1e3)
    sample = f"{n_rows} stratified query rows of {cfg.name} per step, full visible context each, fp64, OpenMP"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(cfg),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def workload_config(cfg):
    return {"workload": f"{cfg.name}: GSA layer fwd, B={cfg.B}, Lq={cfg.Lq}, Lk={cfg.Lk}, causal, n_h={cfg.n_h}, "
                        f"n_kv={cfg.n_kv}, d_h={cfg.d_h}, H^I={cfg.HI}, d^I={cfg.dI}, k_base={cfg.k_base}, "
                        f"k in [{cfg.k_min},{cfg.k_max}], planted needles, seed {cfg.seed}",
            "global_batch_tokens": cfg.B * cfg.Lq, "seq_len": cfg.Lk, "parallelism": "replicas",
            "l2": "inputs (>= 1 GB) exceed the 126 MB L2; no flush between steps"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="l128k", choices=sorted(CONFIGS))
    ap.add_argument("--impl", default="gsa_b200", choices=["gsa_b200", "reference"])
    ap.add_argument("--slab-rows", type=int, default=0)
    ap.add_argument("--act", default="sigmoid", choices=["sigmoid", "relu"], help="indexer activation (Eq. 7 / Eq. 3)")
    ap.add_argument("--k-mode", type=int, default=0, choices=[0, 1, 2, 3],
                    help="0 Eq. 8, 1 inverse, 2 fixed k = k_base, 3 every visible key (needs k_max >= Lk)")
    ap.add_argument("--k-base", type=int, default=0, help="override the base budget (k sweep)")
    ap.add_argument("--lq", type=int, default=0, help="only the last LQ query rows (chunked prefill; smaller ncu captures)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (smaller ncu captures)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-projection", action="store_true", help="skip timing the upstream projection GEMM")
    ap.add_argument("--backward", action="store_true", help="(kept for old command lines: the backward leg is on by default)")
    ap.add_argument("--no-backward", action="store_true",
                    help="skip timing gsa_sparse_gated_attn_bwd and the indexer loss on the workload's own index sets")
    ap.add_argument("--no-rates", action="store_true", help="skip the gather-rate and exp2-rate probes")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "gsa_b200" else args.warmup
    cfg = CONFIGS[args.workload]
    if args.batch > 0:
        cfg = cfg.with_(B=args.batch, name=f"{cfg.name}-b{args.batch}")
    if args.lq > 0:
        cfg = cfg.with_(Lq=args.lq, name=f"{cfg.name}-lq{args.lq}")
    if args.k_base > 0:
        cfg = cfg.with_(k_base=args.k_base, name=f"{cfg.name}-k{args.k_base}")
    variant = dict(act=1 if args.act == "relu" else 0, k_mode=args.k_mode)
    if variant != dict(act=0, k_mode=0):
        cfg = cfg.with_(name=f"{cfg.name}-{args.act}-kmode{args.k_mode}")

    if args.impl == "reference":
        run_reference(args, cfg)
        return

    from paper_2601_15305_b200 import binding as gsa
    gsa.lib()                                   # fails loudly if the CUDA library is missing
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    if cfg.B > 4:
        # many long sequences (decode): generate and upload one batch element at a time
        x, d = None, {}
        for b in range(cfg.B):
            xb = make_inputs(cfg, slice(b, b + 1))
            for k, v in xb.items():
                if k not in d:
                    d[k] = torch.empty((cfg.B,) + tuple(v.shape[1:]), dtype=v.dtype, device="cuda")
                d[k][b].copy_(v[0])
        args.no_e2e = True            # the host-buffer leg would pin tens of GB
        x_cpu_sample = make_inputs(cfg, slice(0, min(cfg.B, 4)))
    else:
        x = make_inputs(cfg)
        d = {k: v.cuda() for k, v in x.items()}
        x_cpu_sample = x
    p = gsa.make_params(cfg, **variant)
    out = torch.empty_like(d["Q"])
    kt = torch.empty((cfg.B, cfg.Lq), dtype=torch.int32, device="cuda")
    ws = torch.empty(gsa.gsa_workspace_bytes(p, args.slab_rows), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        gsa.gsa_forward(p, d["Q"], d["K"], d["V"], d["qI"], d["kI"], d["w"], None, d["g1"], d["g2"], out, None, kt,
                        None, args.slab_rows, ws, stream)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert gsa.gsa_device_status(ws) == 0
    kt_sum = int(kt.sum().item())
    fallback_rows = gsa.gsa_select_fallback_rows(ws)

    # per-step stage events (recorded by the library on the launching stream)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    for tri in evs:
        for e in tri:
            e.record(stream)
    t_beg, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.mark()
    n0 = gsa.gsa_launch_count()
    t_beg.record(stream)
    for i in range(args.steps):
        gsa.gsa_profile_set_events(*evs[i])
        step()
    t_end.record(stream)
    barrier()
    launches = gsa.gsa_launch_count() - n0
    clocks = sampler.stop()
    gsa.gsa_profile_set_events(None, None, None)
    assert gsa.gsa_device_status(ws) == 0
    # one more step, outside the timed region, with an event behind every launch: per-kernel times
    tl_events = [torch.cuda.Event(enable_timing=True) for _ in range(256)]
    for e in tl_events:
        e.record(stream)
    read_timeline = gsa.gsa_profile_set_timeline(tl_events)
    step()
    torch.cuda.synchronize()
    timeline = read_timeline()
    gsa.gsa_profile_set_timeline(None)
    stage_ms = {}
    for name, ms in timeline:
        stage_ms[name] = stage_ms.get(name, 0.0) + ms
    stage_launches = {name: sum(1 for n, _ in timeline if n == name) for name in stage_ms}
    ms_local = t_beg.elapsed_time(t_end)
    ms_total, tokens_total = aggregate_over_ranks(ms_local, float(cfg.B * cfg.Lq * args.steps))
    value = tokens_total / (ms_total * 1e-3)
    sel_ms = float(np.mean([tri[0].elapsed_time(tri[1]) for tri in evs]))
    attn_ms = float(np.mean([tri[1].elapsed_time(tri[2]) for tri in evs]))

    peaks = measured_peaks()
    rates = None if args.no_rates else measure_rates(gsa, stream)
    ab = attention_bytes(cfg, kt_sum)
    achieved = ab / (attn_ms * 1e-3) / 1e9
    hbm_src = f"{peaks['source']} (MEASURED_PEAKS.json hbm_gbs)" if peaks["source"] == "measured" else "fallback 6650 GB/s"
    # The gather of sparse attention is served by the L2 (key ranges of 16384 keys keep a range's K and V' rows
    # resident), so the ceiling that binds is the L2's gather rate for 256-byte pieces, measured by the probe
    # above; the fraction of the HBM copy bandwidth is kept beside it.  `traffic`: DRAM bytes of the launch from
    # an ncu capture of this kernel (ATTN_DRAM_TRAFFIC), null for workloads without one.
    l2_peak = rates["gather_l2_64MB_piece256_gbs"] if rates else None
    roofline = {"kernel": "gsa_sparse_attn_kernel", "bound": "l2" if rates else "hbm", "achieved": achieved,
                "peak": l2_peak if rates else peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / (l2_peak if rates else peaks["hbm_gbs"]), "traffic": ATTN_DRAM_TRAFFIC.get(cfg.name)
                if args.slab_rows == 0 else None,
                "peak_source": "measured in this run: gsa_probe_gather, random 256-byte pieces of a 64 MB table (L2-resident)"
                if rates else hbm_src,
                "l2_gather_gbs": l2_peak, "frac_l2": achieved / l2_peak if rates else None,
                "hbm_gbs": peaks["hbm_gbs"], "frac_hbm": achieved / peaks["hbm_gbs"], "hbm_source": hbm_src,
                "hbm_gather_gbs": rates["gather_hbm_2GB_piece256_gbs"] if rates else None,
                "algorithmic_bytes_per_launch": ab, "launch_ms": attn_ms,
                "note": "one 'launch' = the sparse-attention stage of a forward (range cuts, one kernel launch per 16384-key "
                        "range, finalize).  The 126 MB L2, not HBM, serves the gather, so frac is taken against the L2's "
                        "measured gather rate; frac_hbm (against the HBM copy bandwidth) exceeds 1 for the same reason"}
    causal_pairs = cfg.B * sum(cfg.Lk - cfg.Lq + t + 1 for t in (0, cfg.Lq - 1)) * cfg.Lq / 2.0
    stages = {"indexer_plus_topk_ms": sel_ms, "sparse_attn_ms": attn_ms,
              "indexer_causal_tflop": 2.0 * cfg.HI * cfg.dI * causal_pairs / 1e12,
              "mean_k_t": kt_sum / float(cfg.B * cfg.Lq), "select_fallback_rows": fallback_rows,
              "paper_cost_model_speedup_vs_dense": cost_model.theoretical_speedup(cfg.Lk, cfg.n_h * cfg.d_h, cfg.dI, cfg.HI,
                                                                                 cfg.k_base)}

    # ---- one object per kernel of the forward, from the per-launch events of the profiling step ----
    def per_kernel(name):
        return stage_ms.get(name, 0.0), stage_launches.get(name, 0)
    roofline_all = {}
    ms, n = per_kernel("indexer")
    if n:
        flop = 2.0 * cfg.HI * cfg.dI * causal_pairs
        sig = cfg.HI * causal_pairs
        tf = flop / (ms * 1e-3) / 1e12
        roofline_all["indexer"] = {
            "kernel": "gsa_indexer_tc_kernel" if cfg.Lq > 4 else "gsa_indexer_rows_kernel", "ms": ms, "launches": n,
            "tflops_causal": tf, "bound": "tensor (nominal)", "peak_tflops": peaks["bf16_tflops_sustained"],
            "frac": tf / peaks["bf16_tflops_sustained"],
            "sigmoids_per_s": sig / (ms * 1e-3), "sfu_ops_per_sigmoid": SFU_OPS_PER_SIGMOID if variant["act"] == 0 else 0.0,
            "ex2_per_s_measured": rates["ex2_per_s"] if rates else None,
            "frac_sfu": (SFU_OPS_PER_SIGMOID * sig / (ms * 1e-3) / rates["ex2_per_s"]) if (rates and variant["act"] == 0) else None,
            "note": "flops of causal pairs only (2 * H^I * d^I each); the epilogue's H^I sigmoids per pair run on the "
                    "special-function unit (one exp2 each and one reciprocal shared by the heads), which binds before the tensor pipe"}
    ms, n = per_kernel("select")
    if n:
        gbs = 4.0 * causal_pairs / (ms * 1e-3) / 1e9
        roofline_all["select"] = {"kernel": "gsa_select_kernel", "ms": ms, "launches": n, "bound": "hbm",
                                  "achieved_gbs": gbs, "peak_gbs": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"],
                                  "note": "4 bytes per causal pair read once; index sets written"}
    ms, n = per_kernel("value_gate")
    if n:
        gbs = 3.0 * 2 * cfg.B * cfg.Lk * cfg.n_kv * cfg.d_h / (ms * 1e-3) / 1e9
        roofline_all["value_gate"] = {"kernel": "gsa_value_gate_kernel", "ms": ms, "launches": n, "bound": "hbm",
                                      "achieved_gbs": gbs, "peak_gbs": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"]}
    ms, n = per_kernel("sparse_attn")
    if n:
        gb = float(kt_sum) * (2 * cfg.n_kv * cfg.d_h * 2 + 4)
        gbs = gb / (ms * 1e-3) / 1e9
        roofline_all["sparse_attn"] = {"kernel": "gsa_sparse_attn_kernel", "ms": ms, "launches": n,
                                       "bound": "l2" if rates else "hbm", "achieved_gbs": gbs,
                                       "peak_gbs": l2_peak if rates else peaks["hbm_gbs"],
                                       "frac": gbs / (l2_peak if rates else peaks["hbm_gbs"]),
                                       "frac_hbm": gbs / peaks["hbm_gbs"],
                                       "tflops": float(kt_sum) * cfg.n_h * cfg.d_h * 4 / (ms * 1e-3) / 1e12,
                                       "note": "gathered K and V' rows (+ indices) of the selected pairs; the kernel launches only"}
    ms, n = per_kernel("finalize")
    if n:
        slots = 1
        state = cfg.B * cfg.Lq * cfg.n_h * (cfg.d_h + 2) * 4.0 * slots
        gbs = (state + 2.0 * 2 * cfg.B * cfg.Lq * cfg.n_h * cfg.d_h) / (ms * 1e-3) / 1e9
        roofline_all["finalize"] = {"kernel": "gsa_attn_finalize_kernel", "ms": ms, "launches": n, "bound": "hbm",
                                    "achieved_gbs": gbs, "peak_gbs": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"],
                                    "note": "fp32 softmax state + g1 read, bf16 out written (one state slot per row counted)"}
    ms, n = per_kernel("range_cuts")
    if n:
        roofline_all["range_cuts"] = {"kernel": "gsa_range_cuts_kernel", "ms": ms, "launches": n}
    roofline_all["profiled_step_ms"] = sum(ms for _, ms in timeline)

    # ---- the upstream projection GEMM (outside the timed step: its outputs are the step's inputs) ----
    projection = None
    if not args.no_projection and cfg.Lq == cfg.Lk:
        d_model = 2048
        n_cols = gsa.gsa_project_columns(p)
        M = cfg.B * cfg.Lk
        gen = torch.Generator(device="cuda").manual_seed(5)
        Hs = torch.randn(M, d_model, generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        Wt = (torch.randn(n_cols, d_model, generator=gen, device="cuda", dtype=torch.float32) / d_model ** 0.5).to(torch.bfloat16)
        po = {k: torch.empty_like(d[k]) for k in ("qI", "kI", "w", "g1", "g2")}
        ws_p = torch.zeros(1024, dtype=torch.uint8, device="cuda")
        run_p = lambda: gsa.gsa_project(p, d_model, Hs, Wt, po["qI"], po["kI"], po["w"], po["g1"], po["g2"], ws_p, stream)
        for _ in range(3):
            run_p()
        pe0, pe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pe0.record(stream)
        for _ in range(5):
            run_p()
        pe1.record(stream)
        torch.cuda.synchronize()
        assert gsa.gsa_device_status(ws_p) == 0
        p_ms = pe0.elapsed_time(pe1) / 5
        tf = 2.0 * M * d_model * n_cols / (p_ms * 1e-3) / 1e12
        projection = {"kernel": "gsa_project_kernel", "ms": p_ms, "tflops": tf, "bound": "tensor",
                      "peak": peaks["bf16_tflops"], "frac": tf / peaks["bf16_tflops"],
                      "shape": f"M={M} tokens, K={d_model}, N={n_cols} stacked output columns"}
        del Hs, Wt, po

    # ---- backward of the sparse gated attention stage, on the index sets this workload selects ----
    backward = None
    if not args.no_backward and world == 1 and not cfg.decode:
        idx_b = torch.empty((cfg.B, cfg.Lq, cfg.k_max), dtype=torch.int32, device="cuda")
        gsa.gsa_forward(p, d["Q"], d["K"], d["V"], d["qI"], d["kI"], d["w"], None, d["g1"], d["g2"], out, idx_b, kt,
                        None, args.slab_rows, ws, stream)
        gen = torch.Generator(device="cuda").manual_seed(6)
        dout = torch.randn(d["Q"].shape, generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        gq = {k: torch.empty_like(d["Q"]) for k in ("dQ", "dg1")}
        gk = {k: torch.empty_like(d["K"]) for k in ("dK", "dV", "dg2")}
        ws_b = torch.empty(gsa.gsa_attn_bwd_workspace_bytes(p), dtype=torch.uint8, device="cuda")
        pbar = torch.empty((cfg.B, cfg.Lq, cfg.k_max), dtype=torch.float32, device="cuda")
        run_b = lambda: gsa.gsa_sparse_gated_attn_bwd(p, d["Q"], d["K"], d["V"], d["g1"], d["g2"], idx_b, kt, out, dout,
                                                      gq["dQ"], gk["dK"], gk["dV"], gq["dg1"], gk["dg2"], ws_b, stream,
                                                      pbar=pbar)
        # the training-time forward call of the attention stage saves the softmax statistics for the backward
        lse = torch.empty((cfg.B, cfg.Lq, cfg.n_h), dtype=torch.float32, device="cuda")
        ws_f = torch.empty(gsa.gsa_attn_workspace_bytes(p, True), dtype=torch.uint8, device="cuda")
        gsa.gsa_sparse_gated_attn_fwd_lse(p, d["Q"], d["K"], d["V"], d["g1"], d["g2"], idx_b, kt, out, lse, ws_f, stream)
        del ws_f
        run_b_lse = lambda: gsa.gsa_sparse_gated_attn_bwd(p, d["Q"], d["K"], d["V"], d["g1"], d["g2"], idx_b, kt, out, dout,
                                                          gq["dQ"], gk["dK"], gk["dV"], gq["dg1"], gk["dg2"], ws_b, stream,
                                                          pbar=pbar, lse=lse)
        run_b(); run_b_lse()
        torch.cuda.synchronize()
        assert gsa.gsa_device_status(ws_b) == 0
        be = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        n_b = 2
        be[0].record(stream)
        for _ in range(n_b):
            run_b_lse()
        be[1].record(stream)
        run_b()
        be[2].record(stream)
        torch.cuda.synchronize()
        b_ms = be[0].elapsed_time(be[1]) / n_b
        b_ms_recompute = be[1].elapsed_time(be[2])
        # algorithmic bytes (statistics saved by the forward): the query-major kernel gathers K and V' once per selected (query, key) pair
        # and KV head (d_h * 2 bytes each); the key-major kernel gathers Q and dout * sigmoid(g1) of every
        # head once per pair (n_h * d_h * 2 bytes each); plus the index sets and their inverse (4 + 4 bytes)
        gather = float(kt_sum) * (2 * cfg.n_kv * cfg.d_h * 2 + 2 * cfg.n_h * cfg.d_h * 2 + 8)
        backward = {"kernels": "gsa_sparse_attn_bwd_kernel + gsa_sparse_attn_bwd_keys_kernel", "ms": b_ms,
                    "bound": "hbm", "algorithmic_bytes": gather, "achieved_gbs": gather / (b_ms * 1e-3) / 1e9,
                    "peak_gbs": peaks["hbm_gbs"], "frac": gather / (b_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                    "ms_recomputing_statistics": b_ms_recompute,
                    "tokens_per_s": cfg.B * cfg.Lq / (b_ms * 1e-3), "vs_forward": b_ms / (ms_total / args.steps),
                    "note": "value gate pre-pass, query-major kernel (dQ, dg1, and the indexer loss's target as a "
                            "by-product), index-set inversion, key-major kernel (dK, dV, dg2)"}
        del dout, gq, gk, ws_b, lse
        # the indexer's sparse-phase loss (Eq. 14) on the same index sets: its target, then loss + derivatives
        loss_rows = torch.empty((cfg.B, cfg.Lq), dtype=torch.float32, device="cuda")
        dqI, dkI, dw = torch.empty_like(d["qI"]), torch.empty_like(d["kI"]), torch.empty_like(d["w"])
        dbI = torch.empty((cfg.HI,), dtype=torch.float32, device="cuda")
        ws_s = torch.zeros(1024, dtype=torch.uint8, device="cuda")
        ws_k = torch.empty(gsa.gsa_indexer_kl_workspace_bytes(p), dtype=torch.uint8, device="cuda")
        run_t = lambda: gsa.gsa_attn_probs_mean(p, d["Q"], d["K"], idx_b, kt, pbar, ws_s, stream)
        run_k = lambda: gsa.gsa_indexer_kl_bwd(p, d["qI"], d["kI"], d["w"], None, idx_b, kt, pbar, loss_rows, dqI, dkI,
                                               dw, dbI, ws_k, stream)
        run_t(); run_k()
        torch.cuda.synchronize()
        assert gsa.gsa_device_status(ws_s) == 0 and gsa.gsa_device_status(ws_k) == 0
        le = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        le[0].record(stream)
        for _ in range(n_b):
            run_t()
        le[1].record(stream)
        for _ in range(n_b):
            run_k()
        le[2].record(stream)
        torch.cuda.synchronize()
        backward["indexer_loss"] = {"target_ms": le[0].elapsed_time(le[1]) / n_b, "loss_and_grads_ms": le[1].elapsed_time(le[2]) / n_b,
                                    "mean_loss": float(loss_rows.double().mean().item()),
                                    "note": "target_ms: gsa_attn_probs_mean on its own (the backward call above already "
                                            "emits the same target); gsa_indexer_kl_bwd gathers k^I, dk^I by fp32 vector reductions"}
        backward["train_step_ms"] = ms_total / args.steps + b_ms + backward["indexer_loss"]["loss_and_grads_ms"]
        backward["train_step_note"] = "forward + attention backward (statistics saved, loss target as by-product) + indexer loss and derivatives"
        del idx_b, pbar, loss_rows, dqI, dkI, dw, ws_k

    # ---- end to end through the host-buffer entry point ------------------------------------
    e2e = None
    if not args.no_e2e:
        pin = {k: v.pin_memory() for k, v in x.items()}
        out_h = torch.empty_like(x["Q"]).pin_memory()
        kt_h = torch.empty((cfg.B, cfg.Lq), dtype=torch.int32).pin_memory()
        del ws
        arena = torch.empty(gsa.gsa_forward_host_arena_bytes(p, args.slab_rows), dtype=torch.uint8, device="cuda")
        h2d = sum(v.numel() * v.element_size() for v in pin.values())
        d2h = out_h.numel() * 2 + kt_h.numel() * 4

        def step_host():
            gsa.gsa_forward_host(p, pin["Q"], pin["K"], pin["V"], pin["qI"], pin["kI"], pin["w"], None, pin["g1"],
                                 pin["g2"], out_h, kt_h, args.slab_rows, arena, stream)

        step_host()
        barrier()
        e_steps = max(1, min(args.steps, 3))
        t0 = time.perf_counter()
        for _ in range(e_steps):
            step_host()                      # returns after the result is on the host
        barrier()
        e_ms, e_tok = aggregate_over_ranks((time.perf_counter() - t0) * 1e3, float(cfg.B * cfg.Lq * e_steps))
        e2e = {"value": e_tok / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "steps": e_steps, "api": "gsa_forward_host (pinned host buffers)"}
        assert torch.equal(out_h.view(torch.int16), out.cpu().view(torch.int16)), "host and device paths disagree"

    # ---- the oracle on the host cores, bounded sample (rank 0, N = 1 only) ------------------
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        cores = oracle.num_threads()
        n_rows = 1024          # about 10 s of the oracle on 16 host cores
        r, dt, n, cores = oracle_sample_rate(cfg.with_(B=x_cpu_sample["Q"].shape[0]), x_cpu_sample, n_rows)
        cpu_baseline = {"value": r, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"{n} stratified query rows of {cfg.name} (full visible context each), {dt:.1f} s"}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": workload_config(cfg), "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
                "roofline": roofline, "roofline_all": roofline_all, "measured_rates": rates,
                "cpu_baseline": cpu_baseline, "stages": stages,
                "upstream_projection": projection, "backward": backward}
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
