"""The failure path of the bounded device-side waits, driven without any fault: a probe kernel waits on an
mbarrier transaction nobody will complete, with a limit of two milliseconds, gives up, sets the workspace's
status bit and returns.  The library must report VT_ERR_TIMEOUT once, clear the word, and - after
vt_workspace_init - run a normal head call on the same workspace that matches the oracle."""
import numpy as np
import pytest
import torch

from paper_2603_05210_b200 import inputs
from tests import parity
from tests.gpu_util import dev_bf16, dev_i32, run_head

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_workspace_recovers(oracle):
    import paper_2603_05210_b200 as vt
    vt.lib()
    M, d, Vt, k = 8, 512, 3000, 8
    ws = vt.new_workspace(vt.vt_workspace_bytes(M, k))
    assert vt.vt_last_status(ws) == vt.VT_OK
    vt.vt_test_timeout_probe(ws, limit_us=2000)
    assert vt.vt_last_launch_count() == 1
    assert vt.vt_last_status(ws) == vt.VT_ERR_TIMEOUT
    assert vt.vt_last_status(ws) == vt.VT_OK, "reading the status clears it"
    # a second probe on another stream position: the context is intact and the bit is set again
    vt.vt_test_timeout_probe(ws, limit_us=500)
    assert vt.vt_last_status(ws) == vt.VT_ERR_TIMEOUT
    # arrival counters may be mid-count after a real time-out: dirty them, then recover as the header prescribes
    ws[:512].fill_(0x11)
    vt.vt_workspace_init(ws)
    c = inputs.make_case("after-timeout", d=d, V_trim=Vt, M=M, k=k, seed=31, V_full=9000, n_tokens=50_000)
    W_trim = oracle.compact(c.W_full, c.keep_ids)
    for path in (vt.VT_PATH_AUTO, vt.VT_PATH_GEMV, vt.VT_PATH_MMA):
        got = run_head(vt, c.h, dev_bf16(W_trim), c.d2t, k, path, workspace=ws)
        parity.check_head(got, oracle.draft_head(c.h, W_trim, c.d2t, k, want_logits=True), c.d2t, k)
    # argument checks of the probe itself
    for bad in (0, 1_000_001):
        with pytest.raises(vt.VtError) as e:
            vt.vt_test_timeout_probe(ws, limit_us=bad)
        assert e.value.status == vt.VT_ERR_SHAPE
