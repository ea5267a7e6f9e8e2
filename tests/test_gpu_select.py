"""vt_select_vocab (Eq. 1-5 as an exhaustive scan) against the fp64 selection oracle: frequency ranking and
cumulative counts bit-exact, k* exact, C/R/U at k* to the last bit (both sides use IEEE double, no FMA)."""
import numpy as np
import pytest
import torch

from oracle import vt_select_oracle as so
from paper_2603_05210_b200 import inputs

pytestmark = pytest.mark.gpu
F_FIXED_LLAMA3_8B = so.fixed_flops(4096, 436.2e6, 50.3e6)       # Table 1: fusion + attention + feed-forward


@pytest.fixture(scope="module")
def vt():
    import paper_2603_05210_b200 as vt
    vt.lib()
    assert torch.cuda.is_available()
    return vt


def check(vt, tokens, V, d, F, alpha, c_min, k_min, k_max):
    ref = so.select(tokens, V, d, F, alpha, c_min, k_min, k_max)
    got = vt.vt_select_vocab(torch.from_numpy(tokens).cuda(), V, d, F, alpha, c_min, k_min, k_max, want_cum=True)
    assert np.array_equal(got["ranked_ids"].cpu().numpy(), ref["order"])
    assert np.array_equal(got["cum_counts"].cpu().numpy(), np.cumsum(ref["sorted_counts"]))
    assert got["k_star"] == ref["k_star"]
    assert got["C"] == ref["C_star"] and got["R"] == ref["R_star"] and got["U"] == ref["U_star"]
    assert got["unique"] == ref["unique_star"]          # Table 4's unique coverage at k*: a ratio of two integers
    return got, ref


@pytest.mark.parametrize("V,N,seed", [(40, 500, 0), (257, 3000, 1), (5000, 60_000, 2), (1025, 1, 3)])
def test_small_streams(vt, V, N, seed):
    rng = np.random.default_rng(seed)
    tokens = (rng.zipf(1.2, size=N) % (V + 5) - 2).astype(np.int32)       # a few ids outside [0, V)
    if not ((tokens >= 0) & (tokens < V)).any():
        tokens[0] = 0
    for alpha, c_min in ((0.5, 0.9), (1.0, 0.0), (0.0, 0.5), (0.3, 2.0)):
        check(vt, tokens, V, 64, 5e4, alpha, c_min, 1, V)
    check(vt, tokens, V, 64, 5e4, 0.5, 0.0, max(1, V // 3), max(1, V // 2))


def test_coverage_exactly_at_the_threshold_is_admitted(vt):
    # Eq. 5: C(k) >= c_min keeps U(k); counts 5, 3, 2 give C(2) = 8/10 = the double 0.8
    tokens = np.array([0] * 5 + [1] * 3 + [2] * 2, dtype=np.int32)
    got, _ = check(vt, tokens, 3, 4, 10.0, 0.2, 0.8, 1, 3)
    assert got["k_star"] == 2
    got, _ = check(vt, tokens, 3, 4, 10.0, 0.2, float(np.nextafter(0.8, 1.0)), 1, 3)
    assert got["k_star"] == 3


def test_llama3_vocabulary_paper_constants(vt):
    V = inputs.V_LLAMA3
    tokens = inputs.zipf_token_stream(V, 1.1, 1_000_000, seed=11)
    for alpha, c_min in ((0.5, 0.9), (0.8, 0.95), (0.2, 0.6)):
        got, ref = check(vt, tokens, V, 4096, F_FIXED_LLAMA3_8B, alpha, c_min, 1000, 64000)
        assert got["C"] >= c_min or got["U"] == -1.0
    # the selected prefix is a valid keep set for the head: it covers exactly C(k*) of the stream
    got, ref = check(vt, tokens, V, 4096, F_FIXED_LLAMA3_8B, 0.5, 0.9, 1000, 64000)
    keep = got["ranked_ids"][:got["k_star"]].contiguous()
    assert vt.vt_validate_keep_ids(keep, V) == vt.VT_OK
    covered, frac = vt.vt_coverage(torch.from_numpy(tokens).cuda(), keep, V)
    assert frac == got["C"]


def test_ten_million_token_stream(vt):
    V = inputs.V_LLAMA3
    tokens = inputs.zipf_token_stream(V, 1.05, 10_000_000, seed=5000)
    check(vt, tokens, V, 5120, so.fixed_flops(5120, 436.2e6, 50.3e6), 0.6, 0.95, 1, V)


def test_errors(vt):
    tok = torch.zeros(10, dtype=torch.int32, device="cuda")
    with pytest.raises(vt.VtError) as e:
        vt.vt_select_vocab(tok[:0], 100, 64, 1e4, 0.5, 0.9, 1, 100)
    assert e.value.status == vt.VT_ERR_EMPTY
    with pytest.raises(vt.VtError) as e:
        vt.vt_select_vocab(tok - 5, 100, 64, 1e4, 0.5, 0.9, 1, 100)       # no id inside the vocabulary
    assert e.value.status == vt.VT_ERR_EMPTY
    for bad in (dict(k_min=0), dict(k_min=50, k_max=40), dict(k_max=101), dict(alpha=1.5), dict(d=0)):
        a = dict(V_full=100, d=64, F_fixed=1e4, alpha=0.5, c_min=0.9, k_min=1, k_max=100)
        a.update(bad)
        with pytest.raises(vt.VtError) as e:
            vt.vt_select_vocab(tok, **a)
        assert e.value.status == vt.VT_ERR_SHAPE, bad
