"""B200-native draft-model LM head over a trimmed vocabulary (see ``include/vt.h``).

``paper_2603_05210_b200.inputs`` holds the seeded input generators; everything else is the
binding of the CUDA library and is resolved lazily, so importing the generators does not load it.
"""
from __future__ import annotations

import importlib

_BINDING_NAMES = {
    "VtError", "lib", "LIB_PATH", "SYMBOLS", "new_workspace",
    "vt_workspace_bytes", "vt_host_workspace_bytes", "vt_coverage_workspace_bytes", "vt_workspace_init",
    "vt_compact_head", "vt_validate_keep_ids", "vt_draft_head", "vt_draft_head_host", "vt_last_status",
    "vt_coverage", "vt_coverage_enqueue", "vt_coverage_result", "vt_coverage_static", "vt_select_vocab", "vt_select_workspace_bytes", "vt_debug_logits", "vt_fuse_features", "vt_tree_select", "vt_remap", "vt_vocab_maps", "vt_last_launch_count",
    "VT_OK", "VT_ERR_NULL", "VT_ERR_SHAPE", "VT_ERR_ALIGN", "VT_ERR_RANGE", "VT_ERR_DUP", "VT_ERR_EMPTY",
    "VT_ERR_WORKSPACE", "VT_ERR_TIMEOUT", "VT_ERR_CUDA", "VT_ERR_UNSUPPORTED", "VT_MAX_K",
    "VT_PATH_AUTO", "VT_PATH_GEMV", "VT_PATH_MMA", "VT_PATH_MMA_SMALL", "VT_HEAD_STATIC_WEIGHTS", "VT_HEAD_D2T_OFFSETS",
    "vt_test_timeout_probe", "vt_test_late_copy",
}


def __getattr__(name):
    if name in _BINDING_NAMES:
        return getattr(importlib.import_module(".binding", __name__), name)
    if name in ("inputs", "binding", "build"):
        return importlib.import_module("." + name, __name__)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
