"""Pins for the CPU oracle: each test ties one oracle function to something other than itself.

Brute force is done in exact rational arithmetic (``fractions.Fraction``) on the exact values of
the bf16 inputs, closed forms come from the mathematics, and the invariants are the ones that
vocabulary trimming fixes: a trimmed head is the full head restricted to the kept rows
(Section 2.1), probabilities over the kept rows sum to one, and coverage is the kept share of
token occurrences (Eq. 2).
"""
import math
from fractions import Fraction

import numpy as np
import pytest

from paper_2603_05210_b200 import inputs


# ----------------------------------------------------------------------------- helpers (test-local)
def bf16_fraction(bits: int) -> Fraction:
    """Exact value of a finite bf16 pattern from its fields: (-1)^s * 2^(e-127) * (1 + m/128)."""
    s = -1 if bits >> 15 else 1
    e = (bits >> 7) & 0xFF
    m = bits & 0x7F
    assert e != 0xFF
    if e == 0:
        return s * Fraction(m, 128) * Fraction(2) ** (-126)
    return s * (1 + Fraction(m, 128)) * Fraction(2) ** (e - 127)


def bits_of(values) -> np.ndarray:
    """bf16 patterns of values that are exactly representable (checked)."""
    a = np.asarray(values, dtype=np.float32)
    b = inputs.f32_to_bf16_bits(a).reshape(a.shape)
    assert np.array_equal(inputs.bf16_bits_to_f32(b).reshape(a.shape), a), "value not exact in bf16"
    return b


def exact_logits(h_bits, W_bits):
    M, d = h_bits.shape
    Vt = W_bits.shape[0]
    return [[sum(bf16_fraction(int(h_bits[m, j])) * bf16_fraction(int(W_bits[i, j])) for j in range(d))
             for i in range(Vt)] for m in range(M)]


def topk_by_scans(row, k):
    """k passes of a linear max scan; strict '>' keeps the lowest index among equals."""
    taken, out = set(), []
    for _ in range(k):
        best = None
        for i, v in enumerate(row):
            if i in taken:
                continue
            if best is None or v > row[best]:
                best = i
        taken.add(best)
        out.append(best)
    return out


# ----------------------------------------------------------------------------- bf16 decode
@pytest.mark.parametrize("bits,value", [
    (0x3F80, 1.0), (0xBF80, -1.0), (0x4000, 2.0), (0xC040, -3.0), (0x3F00, 0.5), (0x0000, 0.0),
    (0x3FC0, 1.5), (0x4049, 3.140625), (0x7F7F, (2 - 2 ** -7) * 2.0 ** 127), (0x0080, 2.0 ** -126),
    (0x0001, 2.0 ** -133), (0x3CA4, 0.02001953125),
])
def test_bf16_decode_known_patterns(oracle, bits, value):
    assert oracle.bf16_to_f64(bits) == value


def test_bf16_decode_all_finite_patterns_match_field_formula(oracle):
    for bits in list(range(0, 0x7F80, 97)) + list(range(0x8000, 0xFF80, 89)):
        assert Fraction(oracle.bf16_to_f64(bits)) == bf16_fraction(bits), hex(bits)


# ----------------------------------------------------------------------------- logits
def test_logits_hand_example_dyadic(oracle):
    # d=3, V_trim=5, M=2; every entry is a small dyadic, so every logit is an exact dyadic too.
    h = bits_of([[1.0, -2.0, 0.5], [0.25, 0.0, -1.5]])
    W = bits_of([[2.0, 1.0, -1.0], [0.5, 0.5, 0.5], [-2.0, 0.25, 1.0], [0.0, -1.0, 2.0], [1.5, -0.5, -2.0]])
    x = oracle.logits(h, W)
    expect = np.array([[2 - 2 - 0.5, 0.5 - 1 + 0.25, -2 - 0.5 + 0.5, 0 + 2 + 1, 1.5 + 1 - 1],
                       [0.5 + 0 + 1.5, 0.125 + 0 - 0.75, -0.5 + 0 - 1.5, 0 + 0 - 3, 0.375 + 0 + 3]])
    assert x.shape == (2, 5)
    assert np.array_equal(x, expect)


@pytest.mark.parametrize("M,d,Vt,seed", [(3, 16, 7, 1), (1, 40, 5, 2), (5, 8, 11, 3)])
def test_logits_vs_exact_rational_brute_force(oracle, M, d, Vt, seed):
    rng = np.random.default_rng(seed)
    h = inputs.f32_to_bf16_bits(rng.standard_normal((M, d)).astype(np.float32)).reshape(M, d)
    W = inputs.f32_to_bf16_bits((0.02 * rng.standard_normal((Vt, d))).astype(np.float32)).reshape(Vt, d)
    x = oracle.logits(h, W)
    ex = exact_logits(h, W)
    for m in range(M):
        for i in range(Vt):
            scale = sum(abs(bf16_fraction(int(h[m, j])) * bf16_fraction(int(W[i, j]))) for j in range(d))
            assert abs(Fraction(x[m, i]) - ex[m][i]) <= Fraction(d, 2 ** 52) * scale


def test_logits_one_hot_hidden_state_reads_a_weight_column(oracle):
    rng = np.random.default_rng(5)
    d, Vt = 24, 9
    W = inputs.f32_to_bf16_bits(rng.standard_normal((Vt, d)).astype(np.float32)).reshape(Vt, d)
    for j in (0, 7, d - 1):
        e = np.zeros((1, d), dtype=np.float32)
        e[0, j] = 1.0
        x = oracle.logits(bits_of(e), W)
        assert np.array_equal(x[0], inputs.bf16_bits_to_f32(W[:, j]).astype(np.float64))


def test_zero_hidden_state_gives_uniform_distribution_and_index_zero(oracle):
    d, Vt, k = 16, 37, 4
    rng = np.random.default_rng(6)
    W = inputs.f32_to_bf16_bits(rng.standard_normal((Vt, d)).astype(np.float32)).reshape(Vt, d)
    h = np.zeros((2, d), dtype=np.uint16)
    r = oracle.draft_head(h, W, np.arange(Vt, dtype=np.int32), k, want_logits=True)
    assert np.all(r["logits"] == 0.0)
    assert np.array_equal(r["draft_ids"], np.tile(np.arange(k, dtype=np.int32), (2, 1)))
    assert np.allclose(r["logprobs"], -math.log(Vt), rtol=0, atol=1e-14)


def test_logits_power_of_two_scaling_is_exact(oracle):
    rng = np.random.default_rng(7)
    M, d, Vt = 2, 64, 13
    hf = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(rng.standard_normal((M, d)).astype(np.float32))).reshape(M, d)
    W = inputs.f32_to_bf16_bits(rng.standard_normal((Vt, d)).astype(np.float32)).reshape(Vt, d)
    x1 = oracle.logits(bits_of(hf), W)
    x2 = oracle.logits(bits_of(2.0 * hf), W)
    x4 = oracle.logits(bits_of(-0.25 * hf), W)
    assert np.array_equal(x2, 2.0 * x1)
    assert np.array_equal(x4, -0.25 * x1)


# ----------------------------------------------------------------------------- log-softmax
def test_log_softmax_probabilities_sum_to_one(oracle):
    rng = np.random.default_rng(8)
    x = rng.standard_normal((4, 1000)) * 3.0
    lp, lse = oracle.log_softmax(x)
    assert np.allclose(np.exp(lp).sum(axis=1), 1.0, rtol=0, atol=1e-12)
    assert np.allclose(lp, x - lse[:, None], rtol=0, atol=0)


def test_log_softmax_shift_invariance_and_large_values(oracle):
    rng = np.random.default_rng(9)
    x = rng.standard_normal((3, 257))
    lp0, lse0 = oracle.log_softmax(x)
    for c in (1000.0, -750.0):
        lp, lse = oracle.log_softmax(x + c)
        assert np.all(np.isfinite(lp))
        assert np.allclose(lp, lp0, rtol=0, atol=1e-9)
        assert np.allclose(lse, lse0 + c, rtol=0, atol=1e-9)


def test_log_softmax_closed_forms(oracle):
    lp, lse = oracle.log_softmax(np.full((1, 50), 3.25))
    assert np.allclose(lp, -math.log(50), atol=1e-15) and abs(lse[0] - (3.25 + math.log(50))) < 1e-14
    for delta in (0.0, 0.5, 7.0, 40.0):
        lp, _ = oracle.log_softmax(np.array([[delta, 0.0]]))
        assert abs(lp[0, 0] + math.log1p(math.exp(-delta))) < 1e-14
        assert abs(lp[0, 1] + delta + math.log1p(math.exp(-delta))) < 1e-13
    # a spread far beyond exp's range: only the row maximum may be factored out
    lp, lse = oracle.log_softmax(np.array([[1000.0, 0.0, -1000.0], [-2000.0, -900.0, -901.0]]))
    assert np.all(np.isfinite(lse)) and lse[0] == 1000.0 and lp[0, 0] == 0.0 and lp[0, 2] == -2000.0
    assert abs(lse[1] - (-900.0 + math.log1p(math.exp(-1.0)))) < 1e-12
    # three classes, hand value: log(1 + 2 + 4) with logits log 1, log 2, log 4
    lp, lse = oracle.log_softmax(np.log(np.array([[1.0, 2.0, 4.0]])))
    assert abs(lse[0] - math.log(7.0)) < 1e-14
    assert np.allclose(np.exp(lp[0]), [1 / 7, 2 / 7, 4 / 7], atol=1e-15)


# ----------------------------------------------------------------------------- top-k
@pytest.mark.parametrize("Vt,k,seed", [(50, 1, 0), (50, 8, 1), (33, 33, 2), (200, 10, 3)])
def test_topk_matches_k_pass_max_scan(oracle, Vt, k, seed):
    rng = np.random.default_rng(seed)
    x = np.round(rng.standard_normal((3, Vt)) * 4) / 4     # coarse grid: many exact ties
    idx = oracle.topk(x, k)
    for m in range(3):
        assert list(idx[m]) == topk_by_scans(list(x[m]), k)
    if k == 1:
        assert np.array_equal(idx[:, 0], np.argmax(x, axis=1))
    if k == Vt:
        assert all(sorted(idx[m]) == list(range(Vt)) for m in range(3))


def test_topk_ties_break_to_lowest_index_and_k_bounds(oracle):
    x = np.array([[1.0, 5.0, 5.0, 2.0, 5.0, -1.0]])
    assert list(oracle.topk(x, 4)[0]) == [1, 2, 4, 3]
    with pytest.raises(ValueError):
        oracle.topk(x, 7)
    with pytest.raises(ValueError):
        oracle.topk(x, 0)


def test_planted_winner_rows_rank_first(oracle):
    rng = np.random.default_rng(11)
    M, d, Vt = 3, 32, 101
    hf = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(rng.standard_normal((M, d)).astype(np.float32))).reshape(M, d)
    Wf = (0.02 * rng.standard_normal((Vt, d))).astype(np.float32)
    planted = [17, 0, 100]
    for m, r in enumerate(planted):
        Wf[r] = 4.0 * hf[m]          # exact in bf16: power-of-two multiple of bf16 values
    r = oracle.draft_head(bits_of(hf), inputs.f32_to_bf16_bits(Wf).reshape(Vt, d),
                          np.arange(Vt, dtype=np.int32)[::-1].copy(), 3)
    assert list(r["draft_ids"][:, 0]) == planted
    assert list(r["target_ids"][:, 0]) == [Vt - 1 - p for p in planted]


# ----------------------------------------------------------------------------- trimming invariants
def test_trimmed_head_equals_full_head_restricted_to_keep_ids(oracle):
    rng = np.random.default_rng(12)
    V, d, M, Vt, k = 300, 48, 4, 77, 5
    W_full = inputs.f32_to_bf16_bits((0.02 * rng.standard_normal((V, d))).astype(np.float32)).reshape(V, d)
    h = inputs.f32_to_bf16_bits(rng.standard_normal((M, d)).astype(np.float32)).reshape(M, d)
    keep = rng.permutation(V)[:Vt].astype(np.int32)
    W_trim = oracle.compact(W_full, keep)
    assert np.array_equal(W_trim, W_full[keep])
    x_full = oracle.logits(h, W_full)
    r = oracle.draft_head(h, W_trim, keep, k, want_logits=True)
    assert np.array_equal(r["logits"], x_full[:, keep])               # bit-for-bit in fp64
    # top-k of the trimmed head = top-k of the full head among kept ids, as target ids
    for m in range(M):
        kept_sorted = sorted(range(Vt), key=lambda i: (-x_full[m, keep[i]], i))[:k]
        assert list(r["draft_ids"][m]) == kept_sorted
        assert list(r["target_ids"][m]) == [int(keep[i]) for i in kept_sorted]
        full_arg = int(np.argmax(x_full[m]))
        if full_arg in set(keep.tolist()):
            assert r["target_ids"][m, 0] == full_arg
    # log-probs are normalised over the kept rows only
    lse_trim = np.log(np.exp(x_full[:, keep]).sum(axis=1))
    assert np.allclose(r["lse"], lse_trim, atol=1e-12)
    assert np.allclose(r["logprobs"], np.take_along_axis(x_full[:, keep], r["draft_ids"], 1) - lse_trim[:, None], atol=1e-12)


def test_untrimmed_vocabulary_reproduces_full_head(oracle):
    rng = np.random.default_rng(13)
    V, d, M = 211, 40, 3
    W_full = inputs.f32_to_bf16_bits(rng.standard_normal((V, d)).astype(np.float32)).reshape(V, d)
    h = inputs.f32_to_bf16_bits(rng.standard_normal((M, d)).astype(np.float32)).reshape(M, d)
    ident = np.arange(V, dtype=np.int32)
    r = oracle.draft_head(h, oracle.compact(W_full, ident), ident, 1, want_logits=True)
    assert np.array_equal(r["target_ids"], r["draft_ids"])
    assert np.array_equal(r["target_ids"][:, 0], np.argmax(oracle.logits(h, W_full), axis=1))
    assert np.allclose(np.exp(r["logits"] - r["lse"][:, None]).sum(axis=1), 1.0, atol=1e-12)


def test_compact_with_inverse_permutation_is_identity_and_remap_is_a_gather(oracle):
    rng = np.random.default_rng(14)
    V, d = 64, 8
    W = rng.integers(0, 2 ** 16, size=(V, d), dtype=np.uint16)
    perm = rng.permutation(V).astype(np.int32)
    inv = np.argsort(perm).astype(np.int32)
    assert np.array_equal(oracle.compact(oracle.compact(W, perm), inv), W)
    d2t = rng.integers(0, 10 ** 6, size=V).astype(np.int32)
    idx = rng.integers(0, V, size=(5, 3)).astype(np.int32)
    out = oracle.remap(idx, d2t)
    assert all(out[a, b] == d2t[idx[a, b]] for a in range(5) for b in range(3))


def test_draft_head_is_the_composition_of_its_steps(oracle):
    rng = np.random.default_rng(15)
    M, d, Vt, k = 3, 24, 90, 6
    W = inputs.f32_to_bf16_bits(rng.standard_normal((Vt, d)).astype(np.float32)).reshape(Vt, d)
    h = inputs.f32_to_bf16_bits(rng.standard_normal((M, d)).astype(np.float32)).reshape(M, d)
    d2t = rng.permutation(1000)[:Vt].astype(np.int32)
    r = oracle.draft_head(h, W, d2t, k)
    x = oracle.logits(h, W)
    lp, lse = oracle.log_softmax(x)
    idx = oracle.topk(x, k)
    assert np.array_equal(r["draft_ids"], idx)
    assert np.array_equal(r["target_ids"], oracle.remap(idx, d2t))
    assert np.allclose(r["logprobs"], np.take_along_axis(lp, idx, 1), atol=1e-13)
    assert np.all(np.diff(r["logprobs"], axis=1) <= 0)


# ----------------------------------------------------------------------------- coverage (Eq. 2)
def test_coverage_vs_brute_force_membership(oracle):
    rng = np.random.default_rng(16)
    V = 50
    tok = rng.integers(0, V, size=400).astype(np.int32)
    keep = rng.permutation(V)[:13].astype(np.int32)
    covered, frac = oracle.coverage(tok, keep, V)
    brute = sum(1 for t in tok for kk in keep if t == kk)
    assert covered == brute and frac == brute / 400
    assert oracle.coverage(tok, np.arange(V, dtype=np.int32), V) == (400, 1.0)
    never = np.setdiff1d(np.arange(V + 10), np.arange(V))[:3].astype(np.int32)   # ids no token has
    assert oracle.coverage(tok, never, V + 10)[0] == 0
    with pytest.raises(ValueError):
        oracle.coverage(np.zeros(0, dtype=np.int32), keep, V)


def test_coverage_equals_eq2_from_independent_histogram(oracle):
    V = 5000
    tok = inputs.zipf_token_stream(V, 1.1, 60_000, seed=3)
    order, sorted_counts = inputs.frequency_ranking(tok, V)
    f = np.bincount(tok, minlength=V)
    for k in (1, 10, 321, 4999, 5000):
        covered, frac = oracle.coverage(tok, order[:k], V)
        assert covered == int(f[order[:k]].sum()) == int(sorted_counts[:k].sum())
        assert frac == covered / 60_000
    # out-of-range ids stay in the denominator and are never covered
    tok2 = np.concatenate([tok[:100], np.array([-1, V, V + 7], dtype=np.int32)])
    c_in, _ = oracle.coverage(tok[:100], order[:50], V)
    c2, frac2 = oracle.coverage(tok2, order[:50], V)
    assert c2 == c_in and frac2 == c_in / 103


def test_zipf_coverage_band_for_llama3_vocabulary(oracle):
    V = inputs.V_LLAMA3
    tok = inputs.zipf_token_stream(V, 1.1, 1_000_000, seed=1)
    order, sorted_counts = inputs.frequency_ranking(tok, V)
    # analytic Zipf(1.1) mass of the first k ranks; ranking by the sample's own counts runs slightly higher
    w = np.arange(1, V + 1, dtype=np.float64) ** -1.1
    for k in (4096, 8192, 16384, 32000):
        expect = w[:k].sum() / w.sum()
        _, frac = oracle.coverage(tok, order[:k], V)
        assert expect - 0.003 <= frac <= expect + 0.02, (k, expect, frac)


def test_smallest_prefix_reaching_95_percent_is_monotone_boundary(oracle):
    V = 20000
    tok = inputs.zipf_token_stream(V, 1.05, 300_000, seed=4)
    order, sorted_counts = inputs.frequency_ranking(tok, V)
    K = inputs.smallest_prefix_with_coverage(sorted_counts, 19, 20)
    c_K, _ = oracle.coverage(tok, order[:K], V)
    c_Km1, _ = oracle.coverage(tok, order[:K - 1], V)
    assert 20 * c_K >= 19 * len(tok) > 20 * c_Km1
