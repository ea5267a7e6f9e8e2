"""vt_tree_select against the tree-step oracle: rows, slots and tokens bit-exact, scores bit-exact (both sides
add the parent score and the log-prob once, in fp32), on tie-rich inputs and on real head outputs."""
import numpy as np
import pytest
import torch

from oracle import vt_tree_oracle as to

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def vt():
    import paper_2603_05210_b200 as vt
    vt.lib()
    assert torch.cuda.is_available()
    return vt


@pytest.mark.parametrize("M,k,T,ties", [(1, 1, 1, False), (8, 8, 8, False), (8, 8, 64, True), (64, 10, 60, False), (256, 10, 100, True),
                                        (128, 64, 500, True), (3, 7, 21, True)])
def test_tree_selection_is_bit_exact(vt, M, k, T, ties):
    rng = np.random.default_rng(M * 100 + k)
    if ties:
        lp = (rng.integers(-12, 0, size=(M, k)) * 0.25).astype(np.float32)
        parent = (rng.integers(-8, 1, size=M) * 0.25).astype(np.float32)
    else:
        lp = (-rng.random((M, k)) * 8).astype(np.float32)
        parent = (-rng.random(M) * 5).astype(np.float32)
    lp = -np.sort(-lp, axis=1)
    tid = rng.integers(0, 128256, size=(M, k)).astype(np.int32)
    want = to.tree_select(lp, tid, parent, T)
    rows, slots, tokens, scores = vt.vt_tree_select(torch.from_numpy(lp).cuda(), torch.from_numpy(tid).cuda(),
                                                    torch.from_numpy(parent).cuda(), T)
    assert vt.vt_last_launch_count() == 1
    assert np.array_equal(rows.cpu().numpy(), want["rows"]) and np.array_equal(slots.cpu().numpy(), want["slots"])
    assert np.array_equal(tokens.cpu().numpy(), want["tokens"])
    assert np.array_equal(scores.cpu().numpy().view(np.uint32), want["scores"].view(np.uint32))


def test_argument_checks(vt):
    z = torch.zeros((4, 4), dtype=torch.float32, device="cuda")
    zi = torch.zeros((4, 4), dtype=torch.int32, device="cuda")
    p = torch.zeros(4, dtype=torch.float32, device="cuda")
    with pytest.raises(vt.VtError) as e:
        vt.vt_tree_select(z, zi, p, 17)                       # T > M * k
    assert e.value.status == vt.VT_ERR_SHAPE
    big = torch.zeros((256, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(vt.VtError) as e:
        vt.vt_tree_select(big, torch.zeros((256, 64), dtype=torch.int32, device="cuda"), torch.zeros(256, device="cuda"), 8)
    assert e.value.status == vt.VT_ERR_SHAPE                  # more than 8192 pairs
