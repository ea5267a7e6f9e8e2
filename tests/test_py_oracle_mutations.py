"""The pins of the Python oracles (selection, index buffers, feature fusion, tree selection) must notice a mistake:
each plausible slip is planted in a copy of the oracle's source (on the CPU, never in the CUDA path) and the pin
files are run against that copy in a child process; they have to fail."""
import os
import shutil
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PIN_FILES = {"vt_select_oracle.py": "test_select_oracle_pins.py", "vt_maps_oracle.py": "test_aux_oracle_pins.py",
             "vt_fuse_oracle.py": "test_aux_oracle_pins.py", "vt_tree_oracle.py": "test_aux_oracle_pins.py"}

# name: (file, text in the oracle, the slip)
MUTANTS = {
    "ranking_ties_to_higher_id": ("vt_select_oracle.py", "np.lexsort((np.arange(V), -f.astype(np.int64)))", "np.lexsort((-np.arange(V), -f.astype(np.int64)))"),
    "ranking_ascending": ("vt_select_oracle.py", "np.lexsort((np.arange(V), -f.astype(np.int64)))", "np.lexsort((np.arange(V), f.astype(np.int64)))"),
    "coverage_denominator": ("vt_select_oracle.py", "cum.astype(np.float64) / np.float64(cum[-1])", "cum.astype(np.float64) / np.float64(cum[-1] + 1)"),
    "coverage_off_by_one": ("vt_select_oracle.py", "cum = np.cumsum(f[order].astype(np.int64))\n    return", "cum = np.cumsum(f[order].astype(np.int64))\n    cum = np.concatenate(([0], cum[:-1] + 0))\n    cum[-1] = np.sum(f)\n    return"),
    "reduction_without_factor_two": ("vt_select_oracle.py", "1.0 - (F_fixed + 2.0 * d * k)", "1.0 - (F_fixed + 1.0 * d * k)"),
    "reduction_not_complemented": ("vt_select_oracle.py", "return 1.0 - (F_fixed + 2.0 * d * k) / (F_fixed + 2.0 * d * V)", "return (F_fixed + 2.0 * d * k) / (F_fixed + 2.0 * d * V)"),
    "reduction_ignores_fixed_cost": ("vt_select_oracle.py", "1.0 - (F_fixed + 2.0 * d * k) / (F_fixed + 2.0 * d * V)", "1.0 - (2.0 * d * k) / (2.0 * d * V)"),
    "utility_weights_swapped": ("vt_select_oracle.py", "alpha * np.asarray(C, dtype=np.float64) + (1.0 - alpha) * np.asarray(R, dtype=np.float64)",
                                "(1.0 - alpha) * np.asarray(C, dtype=np.float64) + alpha * np.asarray(R, dtype=np.float64)"),
    "penalty_strict": ("vt_select_oracle.py", "np.where(np.asarray(C) >= c_min, U, -1.0)", "np.where(np.asarray(C) > c_min, U, -1.0)"),
    "penalty_value": ("vt_select_oracle.py", "np.where(np.asarray(C) >= c_min, U, -1.0)", "np.where(np.asarray(C) >= c_min, U, 0.0)"),
    "window_starts_one_late": ("vt_select_oracle.py", "window = Ut[lo - 1:hi]", "window = Ut[lo:hi + 1]"),
    "k_star_off_by_one": ("vt_select_oracle.py", "k_star = lo + int(np.argmax(window))", "k_star = lo - 1 + int(np.argmax(window))"),
    "largest_k_among_equal_maxima": ("vt_select_oracle.py", "k_star = lo + int(np.argmax(window))", "k_star = lo + int(len(window) - 1 - np.argmax(window[::-1]))"),
    "unique_counts_repeated_ids_only": ("vt_select_oracle.py", "occurs = (f[order] > 0).astype(np.int64)", "occurs = (f[order] > 1).astype(np.int64)"),
    "unique_over_whole_vocabulary": ("vt_select_oracle.py", "distinct = int(occurs.sum())", "distinct = len(f)"),
    "fusion_flops_of_a_square_projection": ("vt_select_oracle.py", "2.0 * (3 * d) * d + attention + feed_forward", "2.0 * d * d + attention + feed_forward"),
    "counts_drop_id_zero": ("vt_select_oracle.py", "if 0 <= t < V:\n            f[t] += 1", "if 0 < t < V:\n            f[t] += 1"),
    "offset_sign": ("vt_maps_oracle.py", "out[i] = int(v) - i", "out[i] = i - int(v)"),
    "mask_skips_first_id": ("vt_maps_oracle.py", "for v in keep_ids:\n        if 0 <= int(v) < V_full:", "for v in keep_ids[1:]:\n        if 0 <= int(v) < V_full:"),
    "remap_subtracts": ("vt_maps_oracle.py", "out[t] = int(i) + int(offsets[int(i)])", "out[t] = int(i) - int(offsets[int(i)])"),
    "remap_offset_of_position": ("vt_maps_oracle.py", "out[t] = int(i) + int(offsets[int(i)])", "out[t] = int(i) + int(offsets[t % len(offsets)])"),
    "bf16_decode_shift": ("vt_fuse_oracle.py", "astype(np.uint32) << np.uint32(16)", "astype(np.uint32) << np.uint32(15)"),
    "rounding_ties_away": ("vt_fuse_oracle.py", "up = (rem > half) | ((rem == half) & ((m7 & 1) == 1))", "up = rem >= half"),
    "rounding_truncates": ("vt_fuse_oracle.py", "up = (rem > half) | ((rem == half) & ((m7 & 1) == 1))", "up = rem > (half << np.uint64(1))"),
    "exponent_bias": ("vt_fuse_oracle.py", "e = exp - 1023 + 127", "e = exp - 1023 + 126"),
    "mantissa_carry_lost": ("vt_fuse_oracle.py", "e = e + carry.astype(np.int64)", "e = e + 0 * carry.astype(np.int64)"),
    "fuse_reversed_columns": ("vt_fuse_oracle.py", "return bf16_bits_to_f64(h3_bits) @ bf16_bits_to_f64(W_fuse_bits).T", "return bf16_bits_to_f64(h3_bits)[:, ::-1] @ bf16_bits_to_f64(W_fuse_bits).T"),
    "tree_ties_to_higher_index": ("vt_tree_oracle.py", "key=lambda e: (-float(flat[e]), e)", "key=lambda e: (-float(flat[e]), -e)"),
    "tree_ascending": ("vt_tree_oracle.py", "key=lambda e: (-float(flat[e]), e)", "key=lambda e: (float(flat[e]), e)"),
    "tree_ignores_parent": ("vt_tree_oracle.py", "score = (np.asarray(parent, dtype=np.float32)[:, None] + lp).astype(np.float32)", "score = (0 * np.asarray(parent, dtype=np.float32)[:, None] + lp).astype(np.float32)"),
    "tree_row_and_slot_swapped": ("vt_tree_oracle.py", '"rows": (order // k).astype(np.int32), "slots": (order % k).astype(np.int32)', '"rows": (order % k).astype(np.int32), "slots": (order // k).astype(np.int32)'),
    "tree_one_too_few": ("vt_tree_oracle.py", "[:T]", "[:max(T - 1, 0)]"),
}

CHILD = """
import sys
sys.path.insert(0, {tmp!r})
import oracle, oracle.vt_select_oracle, oracle.vt_maps_oracle, oracle.vt_fuse_oracle, oracle.vt_tree_oracle
assert oracle.__file__.startswith({tmp!r}), oracle.__file__
sys.path.insert(1, {root!r})
import pytest
sys.exit(pytest.main([{pins!r}, "-x", "-q", "-p", "no:cacheprovider"]))
"""


def run_pins(tmp, fname):
    pins = os.path.join(ROOT, "tests", PIN_FILES[fname])
    code = CHILD.format(tmp=str(tmp), root=ROOT, pins=pins)
    return subprocess.run([sys.executable, "-c", code], cwd=ROOT, capture_output=True, text=True, timeout=600)


def copy_oracle(tmp_path):
    dst = tmp_path / "oracle"
    dst.mkdir()
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            shutil.copy(os.path.join(ROOT, "oracle", f), dst / f)
    return dst


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_catch_planted_mistake(name, tmp_path):
    fname, old, new = MUTANTS[name]
    dst = copy_oracle(tmp_path)
    text = (dst / fname).read_text()
    assert text.count(old) == 1, f"mutation site for {name} not found exactly once"
    (dst / fname).write_text(text.replace(old, new))
    r = run_pins(tmp_path, fname)
    assert r.returncode != 0, f"the pins passed with the mistake '{name}' planted:\n{r.stdout[-1500:]}"
    assert "passed" in r.stdout or "failed" in r.stdout or "error" in r.stdout.lower(), r.stdout[-800:] + r.stderr[-800:]


@pytest.mark.parametrize("fname", sorted(set(PIN_FILES)))
def test_unmodified_copy_passes(fname, tmp_path):
    copy_oracle(tmp_path)
    r = run_pins(tmp_path, fname)
    assert r.returncode == 0, r.stdout[-1500:] + r.stderr[-800:]
