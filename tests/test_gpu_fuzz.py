"""Seeded random shapes through every head path against the oracle: draft-row counts across every per-pass
limit (2, 4, 8, 16, 32, 128), vocabulary sizes below and above the CTA count and off every tile size,
k from 1 to VT_MAX_K, hidden sizes that are not multiples of the 64-column k-block."""
import numpy as np
import pytest
import torch

from tests import parity
from tests.gpu_util import dev_bf16, run_head
from tests.test_gpu_small import rand_case

pytestmark = pytest.mark.gpu


def shapes():
    rng = np.random.default_rng(2026)
    out = []
    Ms = [1, 2, 3, 4, 5, 8, 9, 16, 17, 31, 32, 33, 64, 100, 128, 129, 200]
    ds = [8, 24, 72, 128, 200, 520, 1024, 1536, 2048]
    for i in range(44):
        M = int(rng.choice(Ms))
        d = int(rng.choice(ds))
        Vt = int(rng.choice([1, 5, 33, 147, 148, 149, 300, 1000, 2369, 5000, 9999]))
        k = int(min(Vt, rng.choice([1, 2, 7, 8, 9, 16, 17, 32, 33, 64])))
        if M * Vt * d > 6e8:
            Vt = max(k, Vt // 8)
        out.append((M, d, Vt, k))
    return out


@pytest.fixture(scope="module")
def vt():
    import paper_2603_05210_b200 as vt
    vt.lib()
    assert torch.cuda.is_available()
    return vt


@pytest.mark.parametrize("M,d,Vt,k", shapes())
def test_random_shape_both_paths(vt, oracle, M, d, Vt, k):
    h, W, d2t = rand_case(M, d, Vt, seed=M * 31 + d * 7 + Vt + k)
    ora = oracle.draft_head(h, W, d2t, k, want_logits=True)
    Wd = dev_bf16(W)
    paths = (vt.VT_PATH_AUTO, vt.VT_PATH_GEMV, vt.VT_PATH_MMA) + (vt.VT_PATH_MMA_SMALL,)
    for path in paths:
        got = run_head(vt, h, Wd, d2t, k, path)
        parity.check_head(got, ora, d2t, k)


def tall_shapes():
    """Vocabulary sizes on both sides of the tile-count and fold boundaries of a 148-CTA grid (64, 128 rows per
    CTA and beyond), hidden sizes up to 5120 and draft-row counts across the 8 / 16 / 32 / 128 limits."""
    rng = np.random.default_rng(77)
    out = []
    Ms = [1, 2, 3, 8, 9, 16, 17, 32, 33, 64, 65, 128, 129, 300]
    while len(out) < 28:
        M = int(rng.choice(Ms))
        d = int(rng.choice([384, 1000, 2048, 3072, 4096, 5120]))
        Vt = int(rng.choice([4735, 4737, 9472, 9473, 13264, 18944, 18945, 32000, 40000, 57000]))
        k = int(rng.choice([1, 7, 8, 10, 16, 33, 64]))
        while M * Vt * d > 1.5e9:
            if M > 8:
                M = max(8, M // 2)
            else:
                Vt = max(k, Vt // 2)
        out.append((M, d, Vt, k))
    return out


@pytest.mark.parametrize("M,d,Vt,k", tall_shapes())
def test_random_tall_shape_tensor_core_paths(vt, oracle, M, d, Vt, k):
    h, W, d2t = rand_case(M, d, Vt, seed=M * 13 + d + Vt * 3 + k)
    ora = oracle.draft_head(h, W, d2t, k, want_logits=True)
    Wd = dev_bf16(W)
    for path in (vt.VT_PATH_AUTO, vt.VT_PATH_MMA_SMALL):
        got = run_head(vt, h, Wd, d2t, k, path)
        parity.check_head(got, ora, d2t, k)
