"""vt_coverage_static: the coverage count for callers that cannot allocate device memory.

Some users of this library run where a cudaMalloc is off the table - a plugin inside an inference engine
that owns all device memory, or a process that reserved its whole pool at start-up - so they have no
scratch buffer to hand to vt_coverage.  The static variant keeps its bitmap and counters in an array built
into the library.  This file checks, through the C boundary, that it returns exactly what vt_coverage
returns (counts are integers: bit-exact), twice in a row with different kept sets, so that a bitmap or a
counter left over from the first call would show up in the second.  It is named to be collected last.
"""
import numpy as np
import pytest
import torch

from paper_2603_05210_b200 import inputs

pytestmark = pytest.mark.gpu


def test_static_coverage_matches_workspace_coverage_on_two_calls_in_a_row():
    import paper_2603_05210_b200 as vt
    vt.lib()
    assert torch.cuda.is_available()
    V = inputs.V_LLAMA3
    tokens = inputs.zipf_token_stream(V, 1.1, 300_003, seed=77)
    order, _ = inputs.frequency_ranking(tokens, V)
    tok = torch.from_numpy(tokens).cuda()
    ws = torch.empty(vt.vt_coverage_workspace_bytes(V), dtype=torch.uint8, device="cuda")
    # first call: a large kept set; second call: a smaller, disjoint one - stale bits would inflate its count
    first = torch.from_numpy(np.ascontiguousarray(order[:13264])).cuda()
    second = torch.from_numpy(np.ascontiguousarray(order[20000:24380])).cuda()
    for keep in (first, second):
        want = vt.vt_coverage(tok, keep, V, ws)
        got = vt.vt_coverage_static(tok, keep, V)
        assert got == want, (got, want)
        assert 0 < got[0] < tokens.size
    # and once more with the first set: the array is reusable in either order
    assert vt.vt_coverage_static(tok, first, V) == vt.vt_coverage(tok, first, V, ws)
    # nothing is allocated: the device's free memory is the same before and after a call (the first calls above
    # already loaded the module and looked the array's address up)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    got = vt.vt_coverage_static(tok, second, V)
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, (free_before, free_after)
    assert vt.vt_last_launch_count() == 2            # bitmap + count; not added to the previous call's launches
    assert got == vt.vt_coverage(tok, second, V, ws)
    # a stream that starts off a 16-byte boundary and has a ragged tail (the scalar head / tail path)
    odd = tok[1:300_000 - 2]
    assert odd.data_ptr() % 16 != 0 and odd.numel() % 4 != 0
    assert vt.vt_coverage_static(odd, first, V) == vt.vt_coverage(odd, first, V, ws)
    # the largest vocabulary the built-in bitmap holds, with ids at the top of it
    Vmax = 262144
    rng = np.random.default_rng(5)
    big_tok = torch.from_numpy(np.concatenate([rng.integers(0, Vmax, 50_001), [Vmax - 1, Vmax - 2, Vmax, -1]]).astype(np.int32)).cuda()
    big_keep = torch.from_numpy(np.concatenate([rng.permutation(Vmax - 64)[:5000], np.arange(Vmax - 64, Vmax)]).astype(np.int32)).cuda()
    ws_big = torch.empty(vt.vt_coverage_workspace_bytes(Vmax), dtype=torch.uint8, device="cuda")
    assert vt.vt_coverage_static(big_tok, big_keep, Vmax) == vt.vt_coverage(big_tok, big_keep, Vmax, ws_big)
    # sizes beyond the built-in bitmap are refused before anything is launched
    with pytest.raises(vt.VtError) as e:
        vt.vt_coverage_static(tok, first, 262144 + 1)
    assert e.value.status == vt.VT_ERR_SHAPE
