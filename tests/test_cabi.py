"""Host-side checks of the C boundary that need no GPU: the library loads, exports every symbol that
include/vt.h declares, sizes its workspaces sensibly and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def vt():
    from paper_2603_05210_b200.build import build
    build()
    import paper_2603_05210_b200 as vt
    vt.lib()
    return vt


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "vt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vt_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(vt):
    names = declared_symbols()
    assert len(names) >= 16 and "vt_draft_head" in names and "vt_compact_head" in names and "vt_coverage" in names
    cd = ctypes.CDLL(vt.LIB_PATH)
    for n in names:
        assert hasattr(cd, n), f"libvt.so lacks {n}"
    # and the binding knows each of them
    assert set(names) <= set(vt.SYMBOLS), set(names) - set(vt.SYMBOLS)


def test_status_texts_are_distinct(vt):
    texts = [vt.lib().vt_strerror(i) for i in range(11)]
    assert len(set(texts)) == 11 and texts[0] == b"ok"
    assert vt.lib().vt_strerror(99) == b"unknown status"


def test_workspace_sizes(vt):
    assert vt.vt_workspace_bytes(0, 8) == 0 and vt.vt_workspace_bytes(8, 0) == 0
    assert vt.vt_workspace_bytes(8, vt.VT_MAX_K + 1) == 0
    a, b = vt.vt_workspace_bytes(8, 8), vt.vt_workspace_bytes(16, 8)
    assert a % 256 == 0 and b > a > 256
    assert vt.vt_host_workspace_bytes(8, 4096, 8) >= a + 8 * 4096 * 2 + 2 * 8 * 8 * 4
    assert vt.vt_coverage_workspace_bytes(128256) >= 256 + 128256 // 8
    assert vt.vt_coverage_workspace_bytes(0) == 0


FAKE = 0x10000        # a non-NULL, 256-byte aligned address that is never dereferenced on the host


def head(vt, **kw):
    a = dict(h=FAKE, W=FAKE, d2t=FAKE, M=8, d=4096, Vt=32000, k=8, tid=FAKE, lp=FAKE, did=None, lse=None,
             ws=FAKE, ws_bytes=1 << 30, stream=None)
    a.update(kw)
    return vt.lib().vt_draft_head(a["h"], a["W"], a["d2t"], a["M"], a["d"], a["Vt"], a["k"], a["tid"], a["lp"],
                                  a["did"], a["lse"], a["ws"], a["ws_bytes"], a["stream"])


def test_draft_head_rejects_bad_arguments_before_any_launch(vt):
    assert head(vt, h=None) == vt.VT_ERR_NULL
    assert head(vt, W=None) == vt.VT_ERR_NULL
    assert head(vt, d2t=None) == vt.VT_ERR_NULL
    assert head(vt, tid=None) == vt.VT_ERR_NULL
    assert head(vt, lp=None) == vt.VT_ERR_NULL
    for bad in (dict(d=0), dict(d=4100), dict(M=0), dict(Vt=0), dict(k=0), dict(k=9, Vt=8), dict(k=vt.VT_MAX_K + 1)):
        assert head(vt, **bad) == vt.VT_ERR_SHAPE, bad
    assert head(vt, h=FAKE + 8) == vt.VT_ERR_ALIGN
    assert head(vt, W=FAKE + 2) == vt.VT_ERR_ALIGN
    assert head(vt, tid=FAKE + 2) == vt.VT_ERR_ALIGN
    assert head(vt, ws=None) == vt.VT_ERR_WORKSPACE
    assert head(vt, ws=FAKE + 16) == vt.VT_ERR_WORKSPACE
    assert head(vt, ws_bytes=vt.vt_workspace_bytes(8, 8) - 1) == vt.VT_ERR_WORKSPACE


def test_other_entry_points_reject_bad_arguments(vt):
    L = vt.lib()
    assert L.vt_compact_head(None, 100, 64, FAKE, 10, FAKE, None) == vt.VT_ERR_NULL
    assert L.vt_compact_head(FAKE, 100, 60, FAKE, 10, FAKE, None) == vt.VT_ERR_SHAPE
    assert L.vt_compact_head(FAKE, 100, 64, FAKE, 101, FAKE, None) == vt.VT_ERR_SHAPE
    assert L.vt_compact_head(FAKE + 4, 100, 64, FAKE, 10, FAKE, None) == vt.VT_ERR_ALIGN
    assert L.vt_coverage(FAKE, 0, FAKE, 10, 100, None, None, FAKE, 1 << 20, None) == vt.VT_ERR_EMPTY
    assert L.vt_coverage(FAKE, -1, FAKE, 10, 100, None, None, FAKE, 1 << 20, None) == vt.VT_ERR_SHAPE
    assert L.vt_coverage(FAKE, 5, None, 10, 100, None, None, FAKE, 1 << 20, None) == vt.VT_ERR_NULL
    assert L.vt_coverage(FAKE, 5, FAKE, 10, 100, None, None, FAKE, 16, None) == vt.VT_ERR_WORKSPACE
    assert L.vt_validate_keep_ids(None, 10, 100, FAKE, 1 << 20, None) == vt.VT_ERR_NULL
    assert L.vt_validate_keep_ids(FAKE, 10, 100, None, 0, None) == vt.VT_ERR_WORKSPACE
    assert L.vt_remap(None, FAKE, 5, 10, FAKE, None) == vt.VT_ERR_NULL
    assert L.vt_remap(FAKE, FAKE, -1, 10, FAKE, None) == vt.VT_ERR_SHAPE
    assert L.vt_debug_logits(FAKE, FAKE, 1, 64, 10, None, FAKE, 1 << 20, None, 0) == vt.VT_ERR_NULL
    assert L.vt_workspace_init(None, 1024, None) == vt.VT_ERR_WORKSPACE
    assert L.vt_select_vocab(FAKE, 10, 100, 64, 1e4, 0.5, 0.9, 1, 100, None, None, FAKE, None, None, None, None, FAKE, 1 << 24, None) == vt.VT_ERR_NULL
    assert L.vt_select_vocab(FAKE, 10, 100, 64, 1e4, 0.5, 0.9, 0, 100, FAKE, None, FAKE, None, None, None, None, FAKE, 1 << 24, None) == vt.VT_ERR_SHAPE
    assert L.vt_select_vocab(FAKE, 10, 100, 64, 1e4, 0.5, 0.9, 1, 100, FAKE, None, FAKE, None, None, None, None, FAKE, 64, None) == vt.VT_ERR_WORKSPACE
    assert vt.vt_select_workspace_bytes(128256) >= 128256 * 28 and vt.vt_select_workspace_bytes(0) == 0
    assert L.vt_last_status(None, None) == vt.VT_ERR_WORKSPACE
    assert L.vt_draft_head_host(None, FAKE, FAKE, 1, 64, 10, 1, FAKE, FAKE, FAKE, 1 << 20, None) == vt.VT_ERR_NULL
    assert L.vt_draft_head_path(FAKE, FAKE, FAKE, 1, 64, 10, 1, FAKE, FAKE, None, None, FAKE, 1 << 20, None, 7) \
        in (vt.VT_ERR_SHAPE, vt.VT_ERR_CUDA)


def test_binding_refuses_cpu_tensors(vt):
    import torch
    with pytest.raises(ValueError):
        vt.vt_draft_head(torch.zeros(1, 8, dtype=torch.bfloat16), torch.zeros(4, 8, dtype=torch.bfloat16),
                         torch.zeros(4, dtype=torch.int32), 1)
