"""CPU oracle for the vocabulary-size selection that precedes the trimmed head.  TEST INFRASTRUCTURE ONLY.

Plain numpy in fp64 / int64, one function per definition of the paper's Method section:

  frequencies     f(v) = occurrences of token v in the (already assistant-masked) stream      Section 2.2
  ranking         ids by f descending; equal f by ascending id (the paper leaves ties open)   Section 2.1
  coverage        C(k) = sum_{v in top-k} f(v) / sum_v f(v)                                    Eq. 2
  reduction       R(k) = 1 - (F_fixed + 2 d k) / (F_fixed + 2 d V)                             Eq. 3
  utility         U(k) = alpha C(k) + (1 - alpha) R(k)                                         Eq. 4
  penalised       U~(k) = U(k) if C(k) >= c_min else -1                                        Eq. 5
  selection       k* = argmax_{k in [k_min, k_max]} U~(k), the smallest k among equal maxima   Eq. 1
  unique coverage fraction of the DISTINCT ids of the stream that the top-k keeps               Table 4 caption

The paper searches k with 100 TPE trials; an exhaustive scan over every k gives the exact optimum of the
same objective and is what both this oracle and the CUDA path compute.  It shares no code with the CUDA path.
"""
from __future__ import annotations

import numpy as np


def frequencies(token_ids: np.ndarray, V: int) -> np.ndarray:
    f = np.zeros(V, dtype=np.int64)
    for t in np.asarray(token_ids).ravel():      # the definition, one occurrence at a time
        if 0 <= t < V:
            f[t] += 1
    return f


def frequencies_fast(token_ids: np.ndarray, V: int) -> np.ndarray:
    """Same counts through numpy's bincount (library primitive), for streams too long for the loop."""
    t = np.asarray(token_ids).ravel()
    t = t[(t >= 0) & (t < V)]
    return np.bincount(t, minlength=V).astype(np.int64)


def ranking(f: np.ndarray) -> np.ndarray:
    V = len(f)
    return np.lexsort((np.arange(V), -f.astype(np.int64))).astype(np.int32)


def coverage_curve(f: np.ndarray, order: np.ndarray) -> np.ndarray:
    """C(k) for k = 1..V as fp64 (index k-1)."""
    cum = np.cumsum(f[order].astype(np.int64))
    return cum.astype(np.float64) / np.float64(cum[-1])


def unique_coverage_curve(f: np.ndarray, order: np.ndarray) -> np.ndarray:
    """Unique coverage for k = 1..V (index k-1): of the distinct ids that occur in the stream (f > 0), the
    fraction that lies in the top-k.  Table 4 reports it beside the frequency-weighted coverage of Eq. 2."""
    occurs = (f[order] > 0).astype(np.int64)
    distinct = int(occurs.sum())
    return np.cumsum(occurs).astype(np.float64) / np.float64(distinct)


def fixed_flops(d: int, attention: float, feed_forward: float) -> float:
    """F_fixed: feature fusion (3d -> d projection, 2 * 3d * d FLOPs) + attention + feed-forward (Table 1 gives the last two)."""
    return 2.0 * (3 * d) * d + attention + feed_forward


def reduction(k, d: int, V: int, F_fixed: float):
    k = np.asarray(k, dtype=np.float64)
    return 1.0 - (F_fixed + 2.0 * d * k) / (F_fixed + 2.0 * d * V)


def utility(C, R, alpha: float):
    return alpha * np.asarray(C, dtype=np.float64) + (1.0 - alpha) * np.asarray(R, dtype=np.float64)


def penalised(U, C, c_min: float):
    return np.where(np.asarray(C) >= c_min, U, -1.0)


def select(token_ids: np.ndarray, V: int, d: int, F_fixed: float, alpha: float, c_min: float, k_min: int, k_max: int,
           fast_counts: bool = True) -> dict:
    f = frequencies_fast(token_ids, V) if fast_counts else frequencies(token_ids, V)
    order = ranking(f)
    C = coverage_curve(f, order)
    ks = np.arange(1, V + 1)
    R = reduction(ks, d, V, F_fixed)
    U = utility(C, R, alpha)
    Ut = penalised(U, C, c_min)
    lo, hi = max(1, k_min), min(V, k_max)
    window = Ut[lo - 1:hi]
    k_star = lo + int(np.argmax(window))          # argmax returns the first (smallest k) of equal maxima
    return {"f": f, "order": order, "sorted_counts": f[order], "C": C, "R": R, "U": U, "U_pen": Ut, "k_star": k_star,
            "C_star": float(C[k_star - 1]), "R_star": float(R[k_star - 1]), "U_star": float(Ut[k_star - 1]),
            "unique_star": float(unique_coverage_curve(f, order)[k_star - 1])}
