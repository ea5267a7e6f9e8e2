"""vt_fuse_features (the feature-fusion projection of Section 2.3, Table 1 first row) against the fusion oracle.

Both sides round the sum ONCE to bf16, the GPU from the tensor cores' fp32 accumulation, the oracle from fp64.  The
contraction itself carries the head's logit tolerance, |GPU sum - oracle sum| <= 2e-3 * max(1, |y|); the rounded
output must therefore be the nearest-even bf16 of SOME value inside that interval around the oracle's fp64 sum:
rne(y - tol) <= fused <= rne(y + tol).  In practice the accumulation error is ~1e-5 and nearly every element agrees
bit for bit, which the test also asks for (> 99 %)."""
import numpy as np
import pytest
import torch

from oracle import vt_fuse_oracle as fo
from paper_2603_05210_b200 import inputs
from tests.gpu_util import dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def vt():
    import paper_2603_05210_b200 as vt
    vt.lib()
    assert torch.cuda.is_available()
    return vt


def check_fused(got_bits, h3, W):
    y = fo.fuse_features_f64(h3, W)
    tol = 2e-3 * np.maximum(1.0, np.abs(y))
    lo = fo.bf16_bits_to_f64(fo.f64_to_bf16_bits_rne(y - tol))
    hi = fo.bf16_bits_to_f64(fo.f64_to_bf16_bits_rne(y + tol))
    gv = fo.bf16_bits_to_f64(got_bits.astype(np.uint16))
    bad = (gv < lo) | (gv > hi)
    assert not bad.any(), f"{int(bad.sum())} fused features outside the rounded tolerance interval; worst |d| = {np.abs(gv - y)[bad].max():.3e}"
    return float((got_bits.astype(np.uint16) == fo.f64_to_bf16_bits_rne(y)).mean())


@pytest.mark.parametrize("M,d_in,d_out", [(1, 24, 8), (3, 192, 100), (8, 3 * 512, 512), (2, 3 * 2048, 2048),
                                          (17, 3 * 256, 999), (64, 3 * 512, 512), (130, 384, 777), (8, 3 * 4096, 4096)])
def test_fused_features_match_the_oracle(vt, M, d_in, d_out):
    h3 = inputs.hidden_states_bf16(M, d_in, 500 + M)
    W = inputs.normal_bf16((d_out, d_in), 0.02, 600 + d_out)
    guard = torch.full((M * d_out + 64,), 0x5A5A, dtype=torch.int16, device="cuda")
    out = guard[32:32 + M * d_out].view(M, d_out)
    ws = vt.new_workspace(vt.vt_workspace_bytes(M, 1))
    vt.vt_fuse_features(dev_bf16(h3), dev_bf16(W), out=out.view(torch.bfloat16), workspace=ws)
    assert vt.vt_last_status(ws) == vt.VT_OK
    assert vt.vt_last_launch_count() >= 1
    g = guard.cpu().numpy()
    assert (g[:32] == 0x5A5A).all() and (g[32 + M * d_out:] == 0x5A5A).all(), "write outside the output"
    exact_share = check_fused(out.cpu().numpy().view(np.uint16), h3, W)
    assert exact_share > 0.99


def test_fusion_then_head_on_one_stream(vt, oracle):
    """The fused feature feeds the head with nothing in between (the order of a draft step): the head's result must be
    the oracle's head on the oracle's fused feature wherever the two fused features agree bit for bit."""
    M, d, Vt, k = 4, 256, 2000, 4
    h3 = inputs.hidden_states_bf16(M, 3 * d, 901)
    Wf = inputs.normal_bf16((d, 3 * d), 0.05, 902)
    W = inputs.normal_bf16((Vt, d), 0.02, 903)
    d2t = np.arange(Vt, dtype=np.int32)
    fused = vt.vt_fuse_features(dev_bf16(h3), dev_bf16(Wf))
    tid, lp = vt.vt_draft_head(fused, dev_bf16(W), torch.from_numpy(d2t).cuda(), k)
    torch.cuda.synchronize()
    fused_bits = fused.view(torch.int16).cpu().numpy().view(np.uint16)
    check_fused(fused_bits, h3, Wf)
    from tests import parity
    ora = oracle.draft_head(fused_bits, W, d2t, k, want_logits=True)       # the head's parity on the GPU's own fused bits
    parity.check_head({"target_ids": tid.cpu().numpy(), "logprobs": lp.cpu().numpy()}, ora, d2t, k)
