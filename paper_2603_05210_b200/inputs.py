"""Seeded synthetic inputs for the trimmed-vocabulary draft head.

This module only *draws* inputs: bf16 weights and hidden states, a Zipf token
stream over a permuted vocabulary, and the frequency ranking that turns the
stream into ``keep_ids`` / ``d2t``.  It contains none of the head's arithmetic
(no dot products, no softmax, no top-k, no coverage count) and is the single
piece of code that both the CUDA path's callers and the CPU oracle's callers
import.  Everything is numpy on the host, so the same seed gives the same bits
with or without a GPU.

The shapes follow the paper's draft models: the Llama-3 vocabulary of 128,256
ids (Section 2.3), hidden sizes 2048-5120, and draft vocabularies made of the
most frequent ids of a token sample (Section 2.1).
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np

V_LLAMA3 = 128256  # full target vocabulary (Section 2.3)

_BLOCK = 1 << 22  # elements drawn per independent sub-stream


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (round-to-nearest-even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to fp32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal_block(args):
    seed, block, n, std = args
    g = np.random.Generator(np.random.Philox(np.random.SeedSequence([int(seed), 1, int(block)])))
    x = g.standard_normal(n, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return f32_to_bf16_bits(x)


def normal_bf16(shape, std: float, seed: int, threads: int | None = None) -> np.ndarray:
    """bf16 bit patterns of N(0, std^2) samples, drawn in fixed-size blocks.

    Each block of ``_BLOCK`` elements has its own Philox stream keyed by
    ``(seed, 1, block index)``, so the result does not depend on the thread count.  Hidden states
    use the key ``(seed, 2)`` and token streams ``(seed, 3)``: no two generators share a stream.
    """
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    jobs = [(seed, b, min(_BLOCK, n - b * _BLOCK), float(std)) for b in range((n + _BLOCK - 1) // _BLOCK)]
    threads = threads or min(16, os.cpu_count() or 1)
    if len(jobs) <= 1 or threads <= 1:
        parts = map(_normal_block, jobs)
    else:
        pool = ThreadPoolExecutor(max_workers=threads)
        parts = pool.map(_normal_block, jobs)
    for j, part in zip(jobs, parts):
        out[j[1] * _BLOCK: j[1] * _BLOCK + j[2]] = part
    return out.reshape(shape)


def hidden_states_bf16(M: int, d: int, seed: int, row_scale: tuple[float, float] | None = None) -> np.ndarray:
    """``h`` [M, d]: N(0,1) rows, optionally each multiplied by a U(lo, hi) scale, as bf16 bits."""
    g = np.random.Generator(np.random.Philox(np.random.SeedSequence([int(seed), 2])))
    x = g.standard_normal((M, d), dtype=np.float32)
    if row_scale is not None:
        lo, hi = row_scale
        x *= g.uniform(lo, hi, size=(M, 1)).astype(np.float32)
    return f32_to_bf16_bits(x).reshape(M, d)


def zipf_token_stream(V: int, s: float, N: int, seed: int) -> np.ndarray:
    """``N`` token ids: rank r in 1..V drawn with p(r) proportional to r^-s, id = perm[r-1].

    ``perm`` is a seeded permutation of the ids, so frequent tokens are scattered
    over the id range the way a tokenizer's frequent ids are.
    """
    g = np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), 3])))
    perm = g.permutation(V).astype(np.int32)
    w = np.arange(1, V + 1, dtype=np.float64) ** (-float(s))
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    u = g.random(N)
    ranks = np.searchsorted(cdf, u, side="right")
    np.minimum(ranks, V - 1, out=ranks)
    return perm[ranks]


def frequency_ranking(token_ids: np.ndarray, V: int) -> tuple[np.ndarray, np.ndarray]:
    """All ids ordered by (count descending, id ascending), and the counts in that order.

    Ids that never occur follow in id order, so every prefix length up to ``V``
    is a well-defined draft vocabulary (Section 2.1: the top-k most frequent tokens).
    """
    counts = np.bincount(token_ids, minlength=V).astype(np.int64)
    order = np.lexsort((np.arange(V), -counts)).astype(np.int32)
    return order, counts[order]


def smallest_prefix_with_coverage(sorted_counts: np.ndarray, num: int, den: int) -> int:
    """Smallest K with ``den * (first K counts) >= num * total`` in exact integers (C(K) >= num/den)."""
    cum = np.cumsum(sorted_counts.astype(np.int64))
    total = int(cum[-1])
    K = int(np.searchsorted(cum * den, num * total, side="left")) + 1
    return min(K, len(sorted_counts))


@dataclass
class HeadCase:
    """One synthetic workload for the draft head; arrays are host numpy, bf16 as uint16 bits."""
    name: str
    d: int
    V_full: int
    V_trim: int
    M: int
    k: int
    W_full: np.ndarray          # [V_full, d] uint16
    h: np.ndarray               # [M, d] uint16
    keep_ids: np.ndarray        # [V_trim] int32, frequency-rank order
    d2t: np.ndarray             # [V_trim] int32 (== keep_ids: absolute target ids)
    token_ids: np.ndarray | None = None   # the stream keep_ids came from
    extra: dict = field(default_factory=dict)


def make_case(name: str, d: int, V_trim: int | None, M: int, k: int, seed: int, *, V_full: int = V_LLAMA3,
              zipf_s: float = 1.1, n_tokens: int = 1_000_000, row_scale=None, coverage_target=None,
              w_std: float = 0.02, keep_stream: bool = False, W_full: np.ndarray | None = None,
              ranking: tuple[np.ndarray, np.ndarray] | None = None) -> HeadCase:
    """Build a workload: weights, hidden states and a frequency-ranked draft vocabulary.

    ``coverage_target=(num, den)`` replaces ``V_trim`` by the smallest frequency-ranked
    prefix whose coverage of the stream is at least ``num/den``.  ``W_full`` and
    ``ranking`` may be passed in to share them between cases of a sweep.
    """
    tokens = None
    if ranking is None:
        tokens = zipf_token_stream(V_full, zipf_s, n_tokens, seed)
        ranking = frequency_ranking(tokens, V_full)
    order, sorted_counts = ranking
    extra = {}
    if coverage_target is not None:
        V_trim = smallest_prefix_with_coverage(sorted_counts, *coverage_target)
        extra["coverage_target"] = coverage_target
    assert V_trim is not None and 1 <= V_trim <= V_full
    keep = np.ascontiguousarray(order[:V_trim])
    if W_full is None:
        W_full = normal_bf16((V_full, d), w_std, seed)
    h = hidden_states_bf16(M, d, seed, row_scale)
    return HeadCase(name, d, V_full, int(V_trim), M, k, W_full, h, keep, keep.copy(),
                    tokens if keep_stream else None, extra)
