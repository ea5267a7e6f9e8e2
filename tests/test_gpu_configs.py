"""The five benchmark workloads at full size, through the C boundary, in the launch configuration the
bench times (automatic path choice), against the CPU oracle on every output.

Inputs follow the synthetic recipe: Llama-3 vocabulary (128,256 ids, Section 2.3), bf16 weights N(0, 0.02),
bf16 hidden states N(0, 1), draft vocabularies = the most frequent ids of a Zipf token sample
(Section 2.1), d2t = the kept ids in frequency-rank order.
"""
import numpy as np
import pytest
import torch

from paper_2603_05210_b200 import inputs
from tests import parity
from tests.gpu_util import dev_bf16, dev_i32, run_head

pytestmark = pytest.mark.gpu
V = inputs.V_LLAMA3


@pytest.fixture(scope="module")
def vt():
    import paper_2603_05210_b200 as vt
    vt.lib()
    assert torch.cuda.is_available()
    return vt


def full_check(vt, oracle, W_full_dev, W_full, keep, h, k, check_logits=True):
    """compact on the GPU == oracle compact; head outputs and logits within tolerance of the oracle."""
    keep_dev = dev_i32(keep)
    assert vt.vt_validate_keep_ids(keep_dev, V) == vt.VT_OK
    W_trim_dev = vt.vt_compact_head(W_full_dev, keep_dev)
    W_trim = oracle.compact(W_full, keep)
    assert np.array_equal(W_trim_dev.view(torch.int16).cpu().numpy().view(np.uint16), W_trim)
    ora = oracle.draft_head(h, W_trim, keep, k, want_logits=True)
    got = run_head(vt, h, W_trim_dev, keep, k, vt.VT_PATH_AUTO)
    soft = parity.check_head(got, ora, keep, k)
    assert set(got["target_ids"].ravel().tolist()) <= set(keep.tolist())
    if check_logits:
        logits = vt.vt_debug_logits(dev_bf16(h), W_trim_dev).cpu().numpy()
        parity.check_logits(logits, ora["logits"])
    del W_trim_dev
    return got, ora, soft


def test_cfg1_d2048_vtrim4096_m1_argmax(vt, oracle):
    c = inputs.make_case("cfg1", d=2048, V_trim=4096, M=1, k=1, seed=1000)
    full_check(vt, oracle, dev_bf16(c.W_full), c.W_full, c.keep_ids, c.h, 1)


def test_cfg2_d3072_m1_argmax_over_the_vtrim_sweep(vt, oracle):
    tokens = inputs.zipf_token_stream(V, 1.1, 1_000_000, 2000)
    ranking = inputs.frequency_ranking(tokens, V)
    W_full = inputs.normal_bf16((V, 3072), 0.02, 2000)
    W_full_dev = dev_bf16(W_full)
    h = inputs.hidden_states_bf16(1, 3072, 2000)
    tok_dev = dev_i32(tokens)
    last_cov = 0.0
    for i, Vt in enumerate((4096, 4380, 6521, 8192, 13264, 16384, 32000, V)):   # incl. the paper's vocabulary sizes
        keep = np.ascontiguousarray(ranking[0][:Vt])
        got, ora, _ = full_check(vt, oracle, W_full_dev, W_full, keep, h, 1)
        cov = vt.vt_coverage(tok_dev, dev_i32(keep), V)
        assert cov == oracle.coverage(tokens, keep, V)
        assert cov[1] >= last_cov                                        # C(k) grows with k (Eq. 2)
        last_cov = cov[1]
        if Vt == V:                                                      # untrimmed: the full-head argmax
            x_full = oracle.logits(h, W_full)
            assert got["target_ids"][0, 0] == int(np.argmax(x_full[0]))
            assert cov[1] == 1.0


def test_cfg3_d4096_vtrim32000_m8_top8(vt, oracle):
    c = inputs.make_case("cfg3", d=4096, V_trim=32000, M=8, k=8, seed=3000, row_scale=(0.5, 2.0))
    got, ora, _ = full_check(vt, oracle, dev_bf16(c.W_full), c.W_full, c.keep_ids, c.h, 8)
    # probabilities over the trimmed vocabulary sum to one: lse is the log of the partition sum
    assert np.allclose(np.exp(ora["logits"] - got["lse"][:, None].astype(np.float64)).sum(axis=1), 1.0, atol=2e-3)


def test_cfg4_d4096_vtrim16384_m16_64_256_top10(vt, oracle):
    tokens = inputs.zipf_token_stream(V, 1.1, 1_000_000, 4000)
    ranking = inputs.frequency_ranking(tokens, V)
    W_full = inputs.normal_bf16((V, 4096), 0.02, 4000)
    W_full_dev = dev_bf16(W_full)
    keep = np.ascontiguousarray(ranking[0][:16384])
    for i, M in enumerate((16, 64, 256)):
        h = inputs.hidden_states_bf16(M, 4096, 4000 + i)
        full_check(vt, oracle, W_full_dev, W_full, keep, h, 10)


def test_cfg5_d5120_95pct_prefix_m32_top8_next_to_the_untrimmed_head(vt, oracle):
    tokens = inputs.zipf_token_stream(V, 1.05, 10_000_000, 5000)
    order, sorted_counts = inputs.frequency_ranking(tokens, V)
    Vt = inputs.smallest_prefix_with_coverage(sorted_counts, 19, 20)
    keep = np.ascontiguousarray(order[:Vt])
    tok_dev = dev_i32(tokens)
    covered, frac = vt.vt_coverage(tok_dev, dev_i32(keep), V)
    assert (covered, frac) == oracle.coverage(tokens, keep, V)
    covered_m1, _ = vt.vt_coverage(tok_dev, dev_i32(keep[:-1]), V)
    assert 20 * covered >= 19 * tokens.size > 20 * covered_m1              # smallest prefix with C >= 0.95
    assert 30_000 < Vt < 90_000

    W_full = inputs.normal_bf16((V, 5120), 0.02, 5000)
    W_full_dev = dev_bf16(W_full)
    h = inputs.hidden_states_bf16(32, 5120, 5000)
    got_t, ora_t, _ = full_check(vt, oracle, W_full_dev, W_full, keep, h, 8)
    ident = np.arange(V, dtype=np.int32)
    got_f, ora_f, _ = full_check(vt, oracle, W_full_dev, W_full, ident, h, 8, check_logits=False)
    # the trimmed head is the full head restricted to the kept ids (exact in the oracle, whose logits are
    # bit-identical on both sides; each GPU side was held to its oracle above): every full-head winner that
    # is kept leads the trimmed winners, in the same order, and the full partition sum has more terms
    kept = set(keep.tolist())
    for m in range(32):
        full_kept = [int(t) for t in ora_f["target_ids"][m] if int(t) in kept]
        assert full_kept == [int(t) for t in ora_t["target_ids"][m][:len(full_kept)]]
        assert got_f["lse"][m] - got_t["lse"][m] >= -1e-4
