"""The pins must notice a mistake: each plausible slip is planted in a copy of the oracle's C source (on the
CPU, never in the CUDA path), compiled, and the pin suite is run against that copy; it has to fail."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "vt_oracle.c")

MUTANTS = {
    "bf16_shift": ("(uint32_t)b << 16", "(uint32_t)b << 15"),
    "dropped_first_term": ("for (int64_t j = 0; j < d; ++j)\n                acc +=", "for (int64_t j = 1; j < d; ++j)\n                acc +="),
    "hidden_state_index_reversed": ("vto_bf16_to_f64(h[m * d + j]) *", "vto_bf16_to_f64(h[m * d + (d - 1 - j)]) *"),
    "softmax_without_max": ("s += exp(row[i] - mx);", "s += exp(row[i]);"),
    "lse_sign": ("double l = mx + log(s);", "double l = mx - log(s);"),
    "max_becomes_min": ("if (row[i] > mx) mx = row[i];", "if (row[i] < mx) mx = row[i];"),
    "topk_ascending": ("if (p->x > q->x) return -1;       /* larger logit first */\n    if (p->x < q->x) return 1;",
                       "if (p->x > q->x) return 1;       /* larger logit first */\n    if (p->x < q->x) return -1;"),
    "tie_to_higher_index": ("return (p->i > q->i) - (p->i < q->i);", "return (p->i < q->i) - (p->i > q->i);"),
    "remap_identity": ("target_ids[t] = d2t[draft_idx[t]];", "target_ids[t] = draft_idx[t];"),
    "coverage_drops_first_keep_id": ("for (int64_t i = 0; i < V_trim; ++i)\n        if (keep_ids[i] >= 0", "for (int64_t i = 1; i < V_trim; ++i)\n        if (keep_ids[i] >= 0"),
    "compact_reversed_rows": ("W_full[(int64_t)keep_ids[i] * d + j]", "W_full[(int64_t)keep_ids[V_trim - 1 - i] * d + j]"),
    "logprob_sign": ("x[m * V_trim + idx[m * k + j]] - lse[m];", "x[m * V_trim + idx[m * k + j]] + lse[m];"),
}


def run_pins(lib_path):
    env = dict(os.environ, VT_ORACLE_LIB=lib_path)
    return subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"), "-x", "-q",
                           "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_catch_planted_mistake(name, tmp_path):
    old, new = MUTANTS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation site for {name} not found exactly once"
    src = tmp_path / "mutant.c"
    src.write_text(text.replace(old, new))
    lib = tmp_path / "libmutant.so"
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", "-std=c11", "-o", str(lib),
                           str(src), "-lm"])
    r = run_pins(str(lib))
    assert r.returncode != 0, f"the pins passed with the mistake '{name}' planted:\n{r.stdout[-1500:]}"


def test_unmodified_copy_passes(tmp_path):
    lib = tmp_path / "libcopy.so"
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", "-std=c11", "-o", str(lib), SRC, "-lm"])
    r = run_pins(str(lib))
    assert r.returncode == 0, r.stdout[-1500:]
