"""Pins of the two small oracles added beside the head: the index buffers of Section 1 and the feature-fusion
projection of Section 2.3 (component 1; Table 1, first row).  CPU only."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import vt_fuse_oracle as fo
from oracle import vt_maps_oracle as mo
from paper_2603_05210_b200 import inputs


def test_offsets_and_mask_invert_each_other():
    rng = np.random.default_rng(1)
    V = 500
    keep = rng.permutation(V)[:123].astype(np.int32)
    off = mo.d2t_offsets(keep)
    # target id = draft index + offset reproduces keep_ids, for every draft index, in any order
    idx = rng.permutation(123).astype(np.int32)
    assert np.array_equal(mo.remap_offsets(idx, off), keep[idx])
    assert np.array_equal(np.arange(123) + off, keep)
    mask = mo.t2d_mask(keep, V)
    assert mask.sum() == 123 and set(np.nonzero(mask)[0].tolist()) == set(keep.tolist())
    # identity vocabulary: zero offsets, full mask (untrimmed draft)
    ident = np.arange(V, dtype=np.int32)
    assert not mo.d2t_offsets(ident).any() and mo.t2d_mask(ident, V).all()
    # a frequency-ranked prefix sorted by id has non-decreasing offsets (each skipped id adds one)
    srt = np.sort(keep)
    assert np.all(np.diff(mo.d2t_offsets(srt)) >= 0)


def test_bf16_rounding_of_fp64_is_nearest_even_without_double_rounding():
    # every bf16 value rounds to itself
    bits = np.arange(0x0080, 0x7F80, 7, dtype=np.uint16)
    bits = np.concatenate([bits, bits | np.uint16(0x8000), np.array([0, 0x8000], dtype=np.uint16)])
    assert np.array_equal(fo.f64_to_bf16_bits_rne(fo.bf16_bits_to_f64(bits)), bits)
    # exact midpoints go to the even neighbour; a hair above / below goes up / down
    lo = fo.bf16_bits_to_f64(np.array([0x3F80, 0x3F81, 0x4000, 0xBF81], dtype=np.uint16))      # 1.0, 1.0078125, 2.0, -1.0078125
    hi = fo.bf16_bits_to_f64(np.array([0x3F81, 0x3F82, 0x4001, 0xBF82], dtype=np.uint16))
    mid = (lo + hi) / 2
    assert fo.f64_to_bf16_bits_rne(mid).tolist() == [0x3F80, 0x3F82, 0x4000, 0xBF82]
    assert fo.f64_to_bf16_bits_rne(mid + np.sign(mid) * 1e-12).tolist() == [0x3F81, 0x3F82, 0x4001, 0xBF82]
    assert fo.f64_to_bf16_bits_rne(mid - np.sign(mid) * 1e-12).tolist() == [0x3F80, 0x3F81, 0x4000, 0xBF81]
    # a value that double rounding (fp64 -> fp32 -> bf16) gets wrong: just above a bf16 midpoint by less than half an fp32 ulp
    x = np.array([1.0 + 2.0 ** -8 + 2.0 ** -30])
    assert fo.f64_to_bf16_bits_rne(x)[0] == 0x3F81
    assert np.float32(x[0]) == np.float32(1.0 + 2.0 ** -8)                  # fp32 lands exactly on the midpoint ...
    # mantissa carry into the exponent
    assert fo.f64_to_bf16_bits_rne(np.array([1.99999]))[0] == 0x4000


@pytest.mark.parametrize("M,d", [(1, 8), (3, 24), (5, 40)])
def test_fused_features_vs_exact_rational_arithmetic(M, d):
    h3 = inputs.hidden_states_bf16(M, 3 * d, 11)
    W = inputs.normal_bf16((d, 3 * d), 0.02, 12)
    y = fo.fuse_features_f64(h3, W)
    hf = [[Fraction(float(v)) for v in row] for row in fo.bf16_bits_to_f64(h3)]
    wf = [[Fraction(float(v)) for v in row] for row in fo.bf16_bits_to_f64(W)]
    for m in range(M):
        for i in range(d):
            exact = sum(a * b for a, b in zip(hf[m], wf[i]))
            assert abs(Fraction(float(y[m, i])) - exact) <= abs(exact) * Fraction(1, 10 ** 13) + Fraction(1, 10 ** 18)
    out = fo.fuse_features(h3, W)
    assert out.shape == (M, d) and out.dtype == np.uint16
    # one-hot rows of W_fuse copy a column of h3 through unchanged (a bf16 value rounds to itself)
    W1 = np.zeros((d, 3 * d), dtype=np.uint16)
    cols = np.random.default_rng(0).permutation(3 * d)[:d]
    W1[np.arange(d), cols] = 0x3F80
    assert np.array_equal(fo.fuse_features(h3, W1), h3[:, cols])
    # linearity under an exact power-of-two scale
    h2 = inputs.f32_to_bf16_bits(inputs.bf16_bits_to_f32(h3) * np.float32(4.0))
    assert np.array_equal(fo.fuse_features_f64(h2, W), 4.0 * y)


def test_fusion_flops_match_table1():
    # Table 1, first row: a 3d -> d projection costs 2 * 3d * d FLOPs = 100.7M at d = 4096
    text = open(__file__.replace("test_aux_oracle_pins.py", "golden/table1_flops.txt")).read()
    assert "100.7" in text
    assert round(2 * (3 * 4096) * 4096 / 1e6, 1) == 100.7


def test_tree_selection_vs_repeated_argmax_and_closed_cases():
    """The tree-step oracle against T passes of "take the best remaining pair" written out with Python floats, on
    tie-rich scores; with equal parents it reduces to the head's own order; one dominant parent takes every slot."""
    from oracle import vt_tree_oracle as to
    rng = np.random.default_rng(9)
    M, k, T = 6, 5, 11
    lp = (rng.integers(-6, 0, size=(M, k)) * 0.5).astype(np.float32)
    lp = -np.sort(-lp, axis=1)                                     # each row descends, like the head's output
    parent = (rng.integers(-4, 1, size=M) * 0.5).astype(np.float32)
    tid = rng.integers(0, 1000, size=(M, k)).astype(np.int32)
    got = to.tree_select(lp, tid, parent, T)
    score = [[float(np.float32(parent[m]) + np.float32(lp[m, j])) for j in range(k)] for m in range(M)]
    taken = set()
    for t in range(T):
        best = None
        for m in range(M):
            for j in range(k):
                if (m, j) in taken:
                    continue
                if best is None or score[m][j] > score[best[0]][best[1]]:      # strict: the first of equals stays
                    best = (m, j)
        taken.add(best)
        assert (got["rows"][t], got["slots"][t]) == best
        assert got["tokens"][t] == tid[best] and got["scores"][t] == np.float32(score[best[0]][best[1]])
    # equal parents: row 0's slots first among equals, scores never increase
    same = to.tree_select(lp, tid, np.zeros(M, dtype=np.float32), M * k)
    assert np.all(np.diff(same["scores"]) <= 0) and sorted(zip(same["rows"], same["slots"])) == [(m, j) for m in range(M) for j in range(k)]
    # one parent far above the rest takes its k slots first, in slot order
    p2 = np.full(M, -100.0, dtype=np.float32)
    p2[3] = 0.0
    dom = to.tree_select(lp, tid, p2, k)
    assert dom["rows"].tolist() == [3] * k and dom["slots"].tolist() == sorted(range(k), key=lambda j: (-lp[3, j], j))
