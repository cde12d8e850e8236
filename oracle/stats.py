"""Closed-form memory metrics of Section 3.1 (test infrastructure only).

adapter_sparsity: S_i = sum_l (E_i - e_i^(l)) / (L * E_i), E_i = max_l e_i^(l).
fragmentation:    F_mem = L (M + N E_max) / sum_l (M + sum_i e_i^(l)).
Both also accept the summary form the paper's Table 1 prints (maximum and average experts per layer).
"""
import numpy as np


def adapter_sparsity(e_per_layer) -> float:
    e = np.asarray(e_per_layer, np.float64)
    E = e.max()
    return float((E - e).sum() / (e.shape[0] * E))


def adapter_sparsity_from_summary(max_experts: float, avg_experts: float) -> float:
    # sum_l (E - e_l) / (L E) = 1 - mean(e) / E
    return 1.0 - avg_experts / max_experts


def fragmentation(M: int, e_max: int, e) -> float:
    """e: [N, L] experts tuned per adapter per layer."""
    e = np.asarray(e, np.float64)
    N, L = e.shape
    return float(L * (M + N * e_max) / (L * M + e.sum()))


def fragmentation_from_summary(M: int, e_max: int, avg_experts) -> float:
    avg = np.asarray(avg_experts, np.float64)
    return float((M + len(avg) * e_max) / (M + avg.sum()))
