"""CPU oracle for the draft model's feature-fusion projection (Section 2.3, component 1; Table 1's first row:
2 * 3d * d FLOPs).  TEST INFRASTRUCTURE ONLY.

  y[m, i] = sum_j h3[m, j] * W_fuse[i, j]          h3 [M, 3d]: the concatenated hidden states, W_fuse [d, 3d]

Inputs are bf16 bit patterns, decoded exactly to fp64; every product of two bf16 values is exact in fp64 and the
sum is numpy's fp64 matrix product (a library primitive; its rounding is ~1e-16 relative).  The result is rounded
ONCE, to nearest-even, onto the bf16 grid - the paper does not state the precision of the fused feature; one
rounding of an exactly accumulated sum is the reading used here.  It shares no code with the CUDA path.
"""
from __future__ import annotations

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def f64_to_bf16_bits_rne(x: np.ndarray) -> np.ndarray:
    """Round fp64 to the nearest bf16 (ties to even) directly, without passing through fp32.
    Zeros and values in bf16's normal range only (what the fused features of the workloads here are)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    b = x.view(np.uint64)
    sign = (b >> np.uint64(63)).astype(np.uint32)
    exp = ((b >> np.uint64(52)) & np.uint64(0x7FF)).astype(np.int64)
    mant = b & np.uint64((1 << 52) - 1)
    m7 = (mant >> np.uint64(45)).astype(np.int64)
    rem = mant & np.uint64((1 << 45) - 1)
    half = np.uint64(1 << 44)
    up = (rem > half) | ((rem == half) & ((m7 & 1) == 1))
    m7 = m7 + up.astype(np.int64)
    e = exp - 1023 + 127
    carry = m7 == 128
    m7 = np.where(carry, 0, m7)
    e = e + carry.astype(np.int64)
    zero = (exp == 0) & (mant == 0)
    if not np.all(zero | ((e >= 1) & (e <= 254))):
        raise ValueError("value outside bf16's normal range")
    out = (sign << np.uint32(15)) | np.where(zero, 0, (e.astype(np.uint32) << np.uint32(7)) | m7.astype(np.uint32)).astype(np.uint32)
    return out.astype(np.uint16)


def fuse_features_f64(h3_bits: np.ndarray, W_fuse_bits: np.ndarray) -> np.ndarray:
    """The projection before rounding: fp64 [M, d_out]."""
    return bf16_bits_to_f64(h3_bits) @ bf16_bits_to_f64(W_fuse_bits).T


def fuse_features(h3_bits: np.ndarray, W_fuse_bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns [M, d_out] of the fused feature."""
    return f64_to_bf16_bits_rne(fuse_features_f64(h3_bits, W_fuse_bits))
