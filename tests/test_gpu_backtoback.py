"""Calls enqueued back to back with no synchronisation between them - the launch mode the benchmark times.

Every other GPU test reads the status word (a stream synchronisation) after each call.  Here 64+ calls go
onto one stream in a row, alternating over three distinct input sets (hidden states, a copy of W_trim in its
own row order, its d2t), sharing ONE workspace, each call writing its own output buffers; nothing is
synchronised until all are enqueued.  That is the only mode in which a call's set-up overlaps the previous
call's merge (programmatic dependent launch), the arrival tickets are reset by one call and counted by the
next, and - with VT_HEAD_STATIC_WEIGHTS - weight tiles are requested ahead of the dependency wait.  Each
call's outputs are then compared with the CPU oracle, once for eager launches and once for a replayed CUDA
graph of the same calls.
"""
import numpy as np
import pytest
import torch

from paper_2603_05210_b200 import inputs
from tests import parity
from tests.gpu_util import dev_bf16, dev_i32

pytestmark = pytest.mark.gpu

N_CALLS = 66          # a multiple of the three input sets
D, VT, K = 1024, 9001, 8


@pytest.fixture(scope="module")
def vt():
    import paper_2603_05210_b200 as vt
    vt.lib()
    assert torch.cuda.is_available()
    return vt


def make_sets(M, seed, D=D, VT=VT):
    """Three (h, W_trim, d2t) sets that give three different answers."""
    sets = []
    for s in range(3):
        W = inputs.normal_bf16((VT, D), 0.02, seed + 10 * s)
        h = inputs.hidden_states_bf16(M, D, seed + 10 * s + 1, row_scale=(0.5, 2.0))
        d2t = np.random.default_rng(seed + s).permutation(4 * VT)[:VT].astype(np.int32)
        sets.append((h, W, d2t))
    return sets


def enqueue_all(vt, dev_sets, outs, ws, static_weights):
    for i in range(N_CALLS):
        h, W, d2t = dev_sets[i % 3]
        tid, lp, did, lse = outs[i]
        vt.vt_draft_head(h, W, d2t, K, workspace=ws, target_ids=tid, logprobs=lp, draft_ids=did, lse=lse,
                         static_weights=static_weights)


def check_all(outs, refs, sets, M):
    for i in range(N_CALLS):
        tid, lp, did, lse = outs[i]
        got = {"target_ids": tid.cpu().numpy(), "logprobs": lp.cpu().numpy(), "draft_ids": did.cpu().numpy(),
               "lse": lse.cpu().numpy()}
        parity.check_head(got, refs[i % 3], sets[i % 3][2], K)


def fresh_outs(M):
    return [(torch.full((M, K), -7, dtype=torch.int32, device="cuda"),
             torch.full((M, K), float("nan"), dtype=torch.float32, device="cuda"),
             torch.full((M, K), -7, dtype=torch.int32, device="cuda"),
             torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")) for _ in range(N_CALLS)]


@pytest.mark.parametrize("static_weights", [False, True])
@pytest.mark.parametrize("M", [1, 2, 8, 16, 32, 100, 300])
def test_unsynchronised_calls_on_a_shared_workspace_match_the_oracle(vt, oracle, M, static_weights):
    sets = make_sets(M, 9100 + M)
    refs = [oracle.draft_head(h, W, d2t, K, want_logits=True) for h, W, d2t in sets]
    dev_sets = [(dev_bf16(h), dev_bf16(W), dev_i32(d2t)) for h, W, d2t in sets]
    ws = vt.new_workspace(vt.vt_workspace_bytes(M, K))
    # eager: all calls enqueued, then one synchronisation
    outs = fresh_outs(M)
    torch.cuda.synchronize()
    enqueue_all(vt, dev_sets, outs, ws, static_weights)
    assert vt.vt_last_status(ws) == vt.VT_OK
    check_all(outs, refs, sets, M)
    # the same calls as one captured graph, replayed twice (the second replay starts on the first one's tail)
    outs = fresh_outs(M)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            enqueue_all(vt, dev_sets, outs, ws, static_weights)
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    graph.replay()
    assert vt.vt_last_status(ws) == vt.VT_OK
    check_all(outs, refs, sets, M)


@pytest.mark.parametrize("M", [130, 256])
def test_unsynchronised_calls_many_rows_several_tiles_per_cta(vt, oracle, M):
    # CTA pairs sharing each MMA, passes of 64 draft rows, three tiles per CTA: the rows' records carry over between
    # tiles through the workspace the calls share, and the MMA issuer waits for both CTAs' readers
    sets = make_sets(M, 9300 + M, D=256, VT=40000)
    refs = [oracle.draft_head(h, W, d2t, K, want_logits=True) for h, W, d2t in sets]
    dev_sets = [(dev_bf16(h), dev_bf16(W), dev_i32(d2t)) for h, W, d2t in sets]
    ws = vt.new_workspace(vt.vt_workspace_bytes(M, K))
    outs = fresh_outs(M)
    torch.cuda.synchronize()
    enqueue_all(vt, dev_sets, outs, ws, False)
    assert vt.vt_last_status(ws) == vt.VT_OK
    check_all(outs, refs, sets, M)
    outs = fresh_outs(M)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            enqueue_all(vt, dev_sets, outs, ws, False)
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    graph.replay()
    assert vt.vt_last_status(ws) == vt.VT_OK
    check_all(outs, refs, sets, M)


@pytest.mark.parametrize("M", [1, 8, 16, 64])
def test_compaction_immediately_before_the_head(vt, oracle, M):
    """vt_compact_head writes W_trim and the head reads it with nothing in between, several times over with a
    different kept set each time into the same W_trim buffer (default options: full stream order)."""
    V_full = 20000
    W_full = inputs.normal_bf16((V_full, D), 0.02, 77)
    W_full_dev = dev_bf16(W_full)
    h = inputs.hidden_states_bf16(M, D, 78)
    h_dev = dev_bf16(h)
    rng = np.random.default_rng(79)
    keeps = [np.ascontiguousarray(rng.permutation(V_full)[:VT].astype(np.int32)) for _ in range(4)]
    keep_devs = [dev_i32(kp) for kp in keeps]
    W_trim = torch.empty((VT, D), dtype=torch.bfloat16, device="cuda")
    ws = vt.new_workspace(vt.vt_workspace_bytes(M, K))
    outs = [(torch.empty((M, K), dtype=torch.int32, device="cuda"), torch.empty((M, K), dtype=torch.float32, device="cuda"),
             torch.empty((M, K), dtype=torch.int32, device="cuda"), torch.empty((M,), dtype=torch.float32, device="cuda"))
            for _ in range(12)]
    torch.cuda.synchronize()
    for i in range(12):
        vt.vt_compact_head(W_full_dev, keep_devs[i % 4], out=W_trim)
        tid, lp, did, lse = outs[i]
        vt.vt_draft_head(h_dev, W_trim, keep_devs[i % 4], K, workspace=ws, target_ids=tid, logprobs=lp, draft_ids=did, lse=lse)
    assert vt.vt_last_status(ws) == vt.VT_OK
    refs = [oracle.draft_head(h, oracle.compact(W_full, kp), kp, K, want_logits=True) for kp in keeps]
    for i in range(12):
        tid, lp, did, lse = outs[i]
        got = {"target_ids": tid.cpu().numpy(), "logprobs": lp.cpu().numpy(), "draft_ids": did.cpu().numpy(),
               "lse": lse.cpu().numpy()}
        parity.check_head(got, refs[i % 4], keeps[i % 4], K)


@pytest.mark.parametrize("static_weights", [False, True])
@pytest.mark.parametrize("M", [1, 8, 16, 48])
def test_hidden_states_written_late_by_a_kernel_that_released_its_dependents(vt, oracle, M, static_weights):
    """The producer of h lets the next kernel start before it has written h (programmatic dependent launch with an
    early trigger).  The head must still wait for it: only W_trim may be read early, and only when declared static."""
    W = inputs.normal_bf16((VT, D), 0.02, 501)
    W_dev = dev_bf16(W)
    d2t = np.arange(VT, dtype=np.int32)
    d2t_dev = dev_i32(d2t)
    hs = [inputs.hidden_states_bf16(M, D, 600 + i) for i in range(4)]
    srcs = [dev_bf16(x) for x in hs]
    h_dev = torch.zeros((M, D), dtype=torch.bfloat16, device="cuda")
    ws = vt.new_workspace(vt.vt_workspace_bytes(M, K))
    outs = [(torch.empty((M, K), dtype=torch.int32, device="cuda"), torch.empty((M, K), dtype=torch.float32, device="cuda"))
            for _ in range(8)]
    torch.cuda.synchronize()
    for i in range(8):
        vt.vt_test_late_copy(h_dev, srcs[i % 4], delay_us=30)
        vt.vt_draft_head(h_dev, W_dev, d2t_dev, K, workspace=ws, target_ids=outs[i][0], logprobs=outs[i][1],
                         static_weights=static_weights)
    assert vt.vt_last_status(ws) == vt.VT_OK
    refs = [oracle.draft_head(x, W, d2t, K, want_logits=True) for x in hs]
    for i in range(8):
        got = {"target_ids": outs[i][0].cpu().numpy(), "logprobs": outs[i][1].cpu().numpy()}
        parity.check_head(got, refs[i % 4], d2t, K)
