"""The paper's own cost model (Theorem 1, Corollary 2 and Appendix A), as arithmetic on the hyper-parameters:
dense attention costs L^2 d per layer, GSA costs the indexer's L^2 d^I H^I plus L k d for attention over the
selected keys.  Used by the benchmark to print, beside the measured numbers, what the model predicts for the
workload's shape; nothing on the compute path depends on it."""
from __future__ import annotations


def indexer_to_attention_ratio(d: int, n_h: int, dI: int, HI: int) -> float:
    """Per (query, key) pair, the indexer's cost over dense attention's: d^I H^I / (d n_h) (Appendix A)."""
    return dI * HI / float(d * n_h)


def dense_cost(L: int, d: int) -> float:
    return float(L) * L * d


def gsa_cost(L: int, d: int, dI: int, HI: int, k: int) -> float:
    """Indexer over every pair plus attention over k selected keys per query (Theorem 1)."""
    return float(L) * L * dI * HI + float(L) * k * d


def theoretical_speedup(L: int, d: int, dI: int, HI: int, k: int) -> float:
    """dense / GSA = (d / (d^I H^I)) / (1 + k d / (L d^I H^I))  (Corollary 2)."""
    return dense_cost(L, d) / gsa_cost(L, d, dI, HI, k)
