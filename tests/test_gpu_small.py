"""CUDA kernels vs the CPU oracle, element by element, on shapes the oracle finishes in seconds.

Shapes span several tiles and ragged tails: vocabulary sizes that are not multiples of any tile
(1, 7, 127, 129, 4380, 6521 - the paper's in-domain draft vocabularies, Section 3.2), hidden sizes
from one 16-byte chunk up to 5120, and draft-row counts across the per-pass limits of both paths.
"""
import numpy as np
import pytest
import torch

from paper_2603_05210_b200 import inputs
from tests import parity
from tests.gpu_util import Guarded, dev_bf16, dev_i32, run_head

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def vt():
    import paper_2603_05210_b200 as vt
    vt.lib()
    assert torch.cuda.is_available()
    return vt


def rand_case(M, d, Vt, seed, w_std=0.02, h_std=1.0):
    rng = np.random.default_rng(seed)
    W = inputs.f32_to_bf16_bits((w_std * rng.standard_normal((Vt, d))).astype(np.float32)).reshape(Vt, d)
    h = inputs.f32_to_bf16_bits((h_std * rng.standard_normal((M, d))).astype(np.float32)).reshape(M, d)
    d2t = rng.permutation(max(Vt * 3, 10))[:Vt].astype(np.int32)
    return h, W, d2t


PATHS = [pytest.param(1, id="gemv"), pytest.param(2, id="mma"), pytest.param(3, id="mma_small")]
def skip_unless_path_takes(path, M, d):
    if path == 1 and d > 8192:
        pytest.skip("the GEMV path takes d <= 8192")



# ------------------------------------------------------------------------------ compaction
@pytest.mark.parametrize("V,d,Vt", [(50, 8, 1), (300, 64, 77), (1000, 2048, 129), (5000, 5120, 4380), (257, 24, 257)])
def test_compact_head_bit_exact(vt, oracle, V, d, Vt):
    rng = np.random.default_rng(V + d)
    W = rng.integers(0, 2 ** 16, size=(V, d), dtype=np.uint16)
    keep = rng.permutation(V)[:Vt].astype(np.int32)
    out = Guarded((Vt, d), torch.bfloat16)
    vt.vt_compact_head(dev_bf16(W), dev_i32(keep), out=out.t)
    torch.cuda.synchronize()
    got = out.t.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got, oracle.compact(W, keep))
    assert out.intact()


# ------------------------------------------------------------------------------ coverage (Eq. 2)
@pytest.mark.parametrize("V,N,Vt,offset", [(50, 1, 5, 0), (1000, 4099, 100, 1), (128256, 300_001, 13264, 3),
                                           (128256, 40_850, 4380, 2), (7_000_000, 50_000, 100_000, 0)])
def test_coverage_bit_exact(vt, oracle, V, N, Vt, offset):
    rng = np.random.default_rng(N)
    tok = rng.integers(-3, V + 3, size=N + offset).astype(np.int32)     # a few ids fall outside [0, V)
    keep = rng.permutation(V)[:Vt].astype(np.int32)
    tok_dev = dev_i32(tok)[offset:]                                       # start off a 16-byte boundary
    covered, frac = vt.vt_coverage(tok_dev, dev_i32(keep), V)
    assert (covered, frac) == oracle.coverage(tok[offset:], keep, V)


def test_coverage_in_two_steps_matches_the_one_call_form(vt, oracle):
    """vt_coverage_enqueue + vt_coverage_result: two enqueues back to back on different streams' worth of data,
    each result read from its own workspace; a large stream so that every CTA runs the unrolled loop and its tail."""
    V = 128256
    rng = np.random.default_rng(12)
    toks = [rng.integers(-2, V + 2, size=n).astype(np.int32) for n in (3_000_017, 70_001)]
    keep = rng.permutation(V)[:13264].astype(np.int32)
    keep_dev = dev_i32(keep)
    devs = [dev_i32(t) for t in toks]
    wss = [torch.empty(vt.vt_coverage_workspace_bytes(V), dtype=torch.uint8, device="cuda") for _ in toks]
    for t, ws in zip(devs, wss):
        vt.vt_coverage_enqueue(t, keep_dev, V, ws)
    assert vt.vt_last_launch_count() == 1            # a bitmap this small is built inside the counting kernel
    for t, ws in zip(toks, wss):
        assert vt.vt_coverage_result(ws, t.size) == oracle.coverage(t, keep, V)


def test_coverage_zipf_stream_and_validate(vt, oracle):
    V = inputs.V_LLAMA3
    tok = inputs.zipf_token_stream(V, 1.1, 574_168, seed=2)               # combined size of Table 4's streams
    order, _ = inputs.frequency_ranking(tok, V)
    tok_dev = dev_i32(tok)
    for Vt in (4380, 6521, 13264, V):
        assert vt.vt_coverage(tok_dev, dev_i32(order[:Vt]), V) == oracle.coverage(tok, order[:Vt], V)
    assert vt.vt_validate_keep_ids(dev_i32(order[:13264]), V) == vt.VT_OK
    dup = order[:100].copy()
    dup[57] = dup[3]
    assert vt.vt_validate_keep_ids(dev_i32(dup), V) == vt.VT_ERR_DUP
    oor = order[:100].copy()
    oor[99] = V
    assert vt.vt_validate_keep_ids(dev_i32(oor), V) == vt.VT_ERR_RANGE
    with pytest.raises(vt.VtError) as e:
        vt.vt_coverage(tok_dev[:0], dev_i32(order[:10]), V)
    assert e.value.status == vt.VT_ERR_EMPTY


# ------------------------------------------------------------------------------ remap
def test_remap_bit_exact(vt, oracle):
    rng = np.random.default_rng(3)
    d2t = rng.permutation(128256)[:4380].astype(np.int32)
    idx = rng.integers(0, 4380, size=(17, 10)).astype(np.int32)
    got = vt.vt_remap(dev_i32(idx), dev_i32(d2t)).cpu().numpy()
    assert np.array_equal(got, oracle.remap(idx, d2t))
    bad = idx.copy()
    bad[0, 0], bad[1, 1] = -1, 4380
    got = vt.vt_remap(dev_i32(bad), dev_i32(d2t)).cpu().numpy()
    assert got[0, 0] == -1 and got[1, 1] == -1 and np.array_equal(got[2:], oracle.remap(idx, d2t)[2:])


def test_vocab_maps_bit_exact(vt):
    """The draft-to-target offsets and the target-to-draft mask (Section 1) against the index-buffer oracle."""
    from oracle import vt_maps_oracle as mo
    rng = np.random.default_rng(4)
    V, Vt = 128256, 13264
    keep = rng.permutation(V)[:Vt].astype(np.int32)
    off, mask = vt.vt_vocab_maps(dev_i32(keep), V)
    assert np.array_equal(off.cpu().numpy(), mo.d2t_offsets(keep))
    assert np.array_equal(mask.cpu().numpy(), mo.t2d_mask(keep, V))
    assert int(mask.sum()) == Vt


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M", [1, 8, 40])
def test_head_with_offset_form_d2t(vt, oracle, path, M):
    """VT_HEAD_D2T_OFFSETS: the head takes the offsets vt_vocab_maps wrote (target id = draft index + offset, the
    form an EAGLE-3 style checkpoint stores) and must return the ids the oracle's offset remap gives."""
    from oracle import vt_maps_oracle as mo
    d, Vt, k, V = 512, 3001, 8, 50_000
    h, W, _ = rand_case(M, d, Vt, seed=77 + M)
    keep = np.sort(np.random.default_rng(M).permutation(V)[:Vt]).astype(np.int32)
    off_dev, _ = vt.vt_vocab_maps(dev_i32(keep), V)
    tid = torch.empty((M, k), dtype=torch.int32, device="cuda")
    did = torch.empty((M, k), dtype=torch.int32, device="cuda")
    ws = vt.new_workspace(vt.vt_workspace_bytes(M, k))
    _, lp = vt.vt_draft_head(dev_bf16(h), dev_bf16(W), off_dev, k, workspace=ws, path=path, target_ids=tid, draft_ids=did,
                             d2t_offsets=True)
    assert vt.vt_last_status(ws) == vt.VT_OK
    ora = oracle.draft_head(h, W, keep, k, want_logits=True)
    got = {"target_ids": tid.cpu().numpy(), "logprobs": lp.cpu().numpy(), "draft_ids": did.cpu().numpy()}
    assert np.array_equal(got["target_ids"], mo.remap_offsets(got["draft_ids"], mo.d2t_offsets(keep)))
    parity.check_head(got, ora, keep, k)


# ------------------------------------------------------------------------------ logits
LOGIT_SHAPES = [(1, 8, 1), (1, 64, 7), (3, 64, 127), (8, 2048, 129), (2, 3072, 1000), (4, 4096, 4380),
                (9, 2048, 300), (17, 64, 1025), (3, 5120, 700), (5, 200, 2000), (64, 512, 333), (1, 8192, 150)]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M,d,Vt", LOGIT_SHAPES)
def test_logits_vs_oracle(vt, oracle, path, M, d, Vt):
    skip_unless_path_takes(path, M, d)
    h, W, _ = rand_case(M, d, Vt, seed=M * 1000 + Vt)
    got = vt.vt_debug_logits(dev_bf16(h), dev_bf16(W), path=path).cpu().numpy()
    parity.check_logits(got, oracle.logits(h, W))


# ------------------------------------------------------------------------------ full head
HEAD_SHAPES = [(1, 64, 1, 1), (1, 64, 7, 7), (1, 2048, 4380, 1), (3, 64, 127, 8), (8, 2048, 129, 10),
               (8, 4096, 6521, 8), (2, 3072, 1000, 64), (9, 2048, 300, 10), (17, 128, 1025, 3),
               (4, 5120, 700, 8), (64, 512, 333, 10), (5, 200, 2000, 33), (1, 4096, 13264, 1),
               (16, 256, 40000, 10), (7, 64, 60001, 64), (12, 4096, 3000, 8), (2, 8192, 600, 5),
               (33, 1024, 20000, 10), (64, 4096, 2500, 8), (48, 2048, 9000, 16), (8, 16384, 400, 4),
               (100, 2048, 30000, 10), (128, 512, 1000, 8), (257, 256, 20000, 3),
               # more than 64 draft rows and one tile per CTA: the tensor-core kernel takes the tile 64 draft rows at a
               # time, CTA pairs share each MMA, one launch holds up to 256 draft rows
               (65, 256, 5000, 10), (100, 1024, 16384, 10), (128, 512, 2368, 8), (129, 512, 18944, 4),
               (200, 2048, 9000, 16), (256, 1024, 16384, 10), (300, 256, 10000, 1), (256, 4096, 4736, 8),
               (96, 200, 7000, 5), (256, 64, 18944, 10), (128, 512, 18945, 8), (255, 320, 2367, 10),
               # ... and with several tiles per CTA: the rows' records carry over between the tiles (two tiles; three and
               # four, where the MMA issuer waits for both CTAs' readers before it reuses an accumulator buffer)
               (256, 256, 40000, 10), (200, 512, 60000, 4), (65, 128, 20000, 16), (130, 320, 75000, 8),
               # 9 to 16 draft rows on single-tile CTAs: thread-per-row epilogue, with and without folded k-blocks
               (16, 512, 3000, 10), (13, 256, 16384, 8), (10, 1024, 4096, 16), (16, 4096, 4096, 4), (9, 320, 9000, 9)]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M,d,Vt,k", HEAD_SHAPES)
def test_draft_head_vs_oracle(vt, oracle, path, M, d, Vt, k):
    skip_unless_path_takes(path, M, d)
    h, W, d2t = rand_case(M, d, Vt, seed=M * 77 + Vt + k)
    ora = oracle.draft_head(h, W, d2t, k, want_logits=True)
    try:
        got = run_head(vt, h, dev_bf16(W), d2t, k, path)
    except vt.VtError as e:
        if e.status == vt.VT_ERR_UNSUPPORTED and M > 16:      # a forced kernel may decline a shape; the automatic
            pytest.skip("this kernel declines the shape")     # choice (test_gpu_configs, test_gpu_fuzz) never may
        raise
    parity.check_head(got, ora, d2t, k)


@pytest.mark.parametrize("path", PATHS)
def test_large_logits_keep_softmax_stable(vt, oracle, path):
    # |x| in the hundreds: exp() of a raw logit would overflow fp32, the running max must absorb it
    h, W, d2t = rand_case(4, 256, 900, seed=5, w_std=1.0, h_std=8.0)
    ora = oracle.draft_head(h, W, d2t, 5, want_logits=True)
    assert np.abs(ora["logits"]).max() > 200
    got = run_head(vt, h, dev_bf16(W), d2t, 5, path)
    assert np.all(np.isfinite(got["logprobs"]))
    # at this magnitude fp32 accumulation error scales with |x|; ids must still match where gaps are wide
    x = ora["logits"]
    for m in range(4):
        assert got["draft_ids"][m, 0] == ora["draft_ids"][m, 0] or \
            abs(x[m, got["draft_ids"][m, 0]] - x[m, ora["draft_ids"][m, 0]]) < 2e-3 * np.abs(x[m]).max()
    assert np.max(np.abs(got["lse"] - ora["lse"])) <= 2e-3 * np.abs(ora["lse"]).max()


@pytest.mark.parametrize("path", PATHS)
def test_exact_ties_resolve_to_lowest_draft_index(vt, oracle, path):
    # duplicated weight rows give bit-equal logits on both sides
    rng = np.random.default_rng(8)
    M, d, Vt, k = 3, 256, 600, 10
    base = inputs.f32_to_bf16_bits((0.05 * rng.standard_normal((60, d))).astype(np.float32)).reshape(60, d)
    W = base[rng.integers(0, 60, size=Vt)]
    h = inputs.f32_to_bf16_bits(rng.standard_normal((M, d)).astype(np.float32)).reshape(M, d)
    d2t = np.arange(Vt, dtype=np.int32) + 1000
    ora = oracle.draft_head(h, W, d2t, k, want_logits=True)
    got = run_head(vt, h, dev_bf16(W), d2t, k, path)
    assert np.array_equal(got["draft_ids"], ora["draft_ids"])
    assert np.array_equal(got["target_ids"], ora["target_ids"])
    parity.check_exact_tie_order(got["draft_ids"], ora["logits"])
    # zero hidden state: every logit is 0, the winners are indices 0..k-1, log-prob = -log(Vt)
    h0 = np.zeros((2, d), dtype=np.uint16)
    got0 = run_head(vt, h0, dev_bf16(W), d2t, k, path)
    assert np.array_equal(got0["draft_ids"], np.tile(np.arange(k, dtype=np.int32), (2, 1)))
    assert np.allclose(got0["logprobs"], -np.log(Vt), atol=1e-5)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M,k", [(1, 8), (4, 10), (40, 8), (3, 16)])
def test_all_winners_in_one_ctas_rows(vt, oracle, path, M, k):
    # the k best logits of every draft row sit in adjacent vocabulary rows (one CTA's share): that CTA's list places
    # more winners than the merge keeps in registers per list, the other lists none
    rng = np.random.default_rng(50 + M + k)
    d, Vt = 512, 6000
    Wf = (0.02 * rng.standard_normal((Vt, d))).astype(np.float32)
    hf = rng.standard_normal((M, d)).astype(np.float32)
    hot = 1234 + np.arange(k + 3)
    Wf[hot] = 0.05 * np.sign(hf.sum(axis=0))[None, :] * (1.0 + 0.01 * np.arange(k + 3))[:, None]   # same sign pattern as every row of h below
    W = inputs.f32_to_bf16_bits(Wf).reshape(Vt, d)
    h = inputs.f32_to_bf16_bits(np.abs(hf) * np.sign(hf.sum(axis=0))[None, :]).reshape(M, d)       # every row of h shares that sign pattern
    d2t = np.arange(Vt, dtype=np.int32)[::-1].copy()
    ora = oracle.draft_head(h, W, d2t, k, want_logits=True)
    assert set(ora["draft_ids"][0].tolist()) <= set(hot.tolist())
    got = run_head(vt, h, dev_bf16(W), d2t, k, path)
    parity.check_head(got, ora, d2t, k)


@pytest.mark.parametrize("path", PATHS)
def test_same_input_twice_is_bit_identical_and_workspace_is_reusable(vt, oracle, path):
    h, W, d2t = rand_case(8, 1024, 5000, seed=9)
    Wd = dev_bf16(W)
    ws = vt.new_workspace(vt.vt_workspace_bytes(8, 8))
    a = run_head(vt, h, Wd, d2t, 8, path, workspace=ws)
    b = run_head(vt, h, Wd, d2t, 8, path, workspace=ws)
    for key in a:
        assert np.array_equal(a[key].view(np.int32), b[key].view(np.int32)), key
    # a different, smaller call on the same workspace afterwards
    h2, W2, d2t2 = rand_case(2, 64, 50, seed=10)
    got = run_head(vt, h2, dev_bf16(W2), d2t2, 3, path, workspace=ws)
    parity.check_head(got, oracle.draft_head(h2, W2, d2t2, 3, want_logits=True), d2t2, 3)


def test_all_paths_agree_on_logits(vt):
    h, W, _ = rand_case(8, 4096, 2000, seed=11)
    a = vt.vt_debug_logits(dev_bf16(h), dev_bf16(W), path=1).cpu().numpy()
    b = vt.vt_debug_logits(dev_bf16(h), dev_bf16(W), path=2).cpu().numpy()
    c = vt.vt_debug_logits(dev_bf16(h), dev_bf16(W), path=3).cpu().numpy()
    assert np.max(np.abs(a - b)) <= 2e-3 and np.max(np.abs(a - c)) <= 2e-3


@pytest.mark.parametrize("M,launches", [(1, 1), (8, 1), (12, 1), (13, 2), (16, 2), (17, 2), (64, 2), (65, 2), (256, 2), (300, 3)])
def test_launches_per_call_of_the_automatic_choice(vt, oracle, M, launches):
    # M = 1: GEMV; M <= 12 (16 with several tiles per CTA): one launch, rows merged by the last warp to publish them;
    # beyond: the same kernel in passes of 256 draft rows (one tile per CTA, as here; 128 otherwise) followed by the
    # row-wise merge kernel
    h, W, d2t = rand_case(M, 256, 3000, seed=40 + M)
    got = run_head(vt, h, dev_bf16(W), d2t, 4, vt.VT_PATH_AUTO)
    assert vt.vt_last_launch_count() == launches
    parity.check_head(got, oracle.draft_head(h, W, d2t, 4, want_logits=True), d2t, 4)


def test_trimmed_head_equals_full_head_restricted(vt, oracle):
    # the invariant trimming rests on, end to end on the GPU: compact + head over V_d == full head restricted to V_d
    V, d, M, Vt, k = 3000, 512, 4, 700, 8
    rng = np.random.default_rng(12)
    W_full = inputs.f32_to_bf16_bits((0.02 * rng.standard_normal((V, d))).astype(np.float32)).reshape(V, d)
    h = inputs.f32_to_bf16_bits(rng.standard_normal((M, d)).astype(np.float32)).reshape(M, d)
    keep = rng.permutation(V)[:Vt].astype(np.int32)
    W_trim = vt.vt_compact_head(dev_bf16(W_full), dev_i32(keep))
    got = run_head(vt, h, W_trim, keep, k, 0)
    full = vt.vt_debug_logits(dev_bf16(h), dev_bf16(W_full)).cpu().numpy()
    trim = vt.vt_debug_logits(dev_bf16(h), W_trim).cpu().numpy()
    assert np.array_equal(trim, full[:, keep])                       # same products, same order: bit-equal
    ora = oracle.draft_head(h, oracle.compact(W_full, keep), keep, k, want_logits=True)
    parity.check_head(got, ora, keep, k)
    ident = np.arange(V, dtype=np.int32)
    got_full = run_head(vt, h, dev_bf16(W_full), ident, 1, 0)
    assert np.array_equal(got_full["target_ids"], got_full["draft_ids"])
    assert np.array_equal(got_full["target_ids"][:, 0], np.argmax(oracle.logits(h, W_full), axis=1))


@pytest.mark.parametrize("pinned", [True, False], ids=["pinned", "pageable"])
def test_host_buffer_entry_point(vt, oracle, pinned):
    M, d, Vt, k = 8, 1024, 3000, 8
    h, W, d2t = rand_case(M, d, Vt, seed=13)
    ws = vt.new_workspace(vt.vt_host_workspace_bytes(M, d, k))
    h_host = torch.from_numpy(h.view(np.int16).copy())
    tid = torch.full((M, k), -7, dtype=torch.int32)
    lp = torch.full((M, k), float("nan"), dtype=torch.float32)
    if pinned:      # pinned outputs are written by the kernel itself, pageable ones by copies after it
        h_host, tid, lp = h_host.pin_memory(), tid.pin_memory(), lp.pin_memory()
    Wd, d2td = dev_bf16(W), dev_i32(d2t)
    ora = oracle.draft_head(h, W, d2t, k, want_logits=True)
    for _ in range(2):
        tid.fill_(-7)
        vt.vt_draft_head_host(h_host, Wd, d2td, k, tid, lp, ws)
        parity.check_head({"target_ids": tid.numpy().copy(), "logprobs": lp.numpy().copy()}, ora, d2t, k)
    # new hidden states in the SAME host buffer: the next call must see them (nothing of the old ones may be cached)
    for seed in (14, 15):
        h2 = inputs.hidden_states_bf16(M, d, seed)
        h_host.copy_(torch.from_numpy(h2.view(np.int16).copy()))
        vt.vt_draft_head_host(h_host, Wd, d2td, k, tid, lp, ws)
        parity.check_head({"target_ids": tid.numpy().copy(), "logprobs": lp.numpy().copy()},
                          oracle.draft_head(h2, W, d2t, k, want_logits=True), d2t, k)
