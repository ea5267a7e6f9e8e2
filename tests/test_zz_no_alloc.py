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
    # sizes beyond the built-in bitmap are refused before anything is launched
    with pytest.raises(vt.VtError) as e:
        vt.vt_coverage_static(tok, first, 262144 + 1)
    assert e.value.status == vt.VT_ERR_SHAPE
