"""Writes the v_bar constants stored in paper_2601_15305_b200/inputs.py.

V-bar in Eq. 8 is a running mean of score variance that the caller owns.  For the
synthetic workloads it is set once to the median row variance of the generated
data (rows with at least k_max visible keys), so that k_t centres on k_base.
This script calls only the oracle (Eq. 7 then the variance of Eq. 8) on sampled rows
and prints the constants; paste them into CONFIGS.

    python -m oracle.calibrate_vbar [config ...]
"""
import sys

import numpy as np

import oracle
from paper_2601_15305_b200.inputs import CONFIGS, make_inputs, sample_rows


def calibrate(name: str, n_rows: int = 96) -> float:
    cfg = CONFIGS[name]
    bsl = slice(0, min(cfg.B, 4))
    x = make_inputs(cfg, bsl)
    nb = x["Q"].shape[0]
    p = oracle.OracleParams.from_config(cfg, B=nb)
    if cfg.decode:
        rows_t = np.zeros(nb, dtype=np.int32)
        rows_b = np.arange(nb, dtype=np.int32)
    else:
        rows_t = sample_rows(cfg, n_rows).numpy().astype(np.int32)
        rows_t = rows_t[rows_t + 1 >= min(cfg.k_max, cfg.Lq // 2)]
        rows_b = np.zeros_like(rows_t)
    sc = oracle.scores(p, x["qI"], x["kI"], x["w"], None, rows_t, rows_b)
    var = np.array([np.var(sc[i, : p.visible(int(t))]) for i, t in enumerate(rows_t)])
    return float(np.median(var))


if __name__ == "__main__":
    for n in (sys.argv[1:] or list(CONFIGS)):
        print(f"{n}: v_bar={calibrate(n):.4e}", flush=True)
