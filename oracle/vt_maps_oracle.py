"""CPU oracle for the two index buffers of an EAGLE-3 style draft (Section 1: the draft-to-target and the
target-to-draft map that tie the draft vocabulary to the model's weights).  TEST INFRASTRUCTURE ONLY.

Plain Python loops over the definition; it shares no code with the CUDA path.

  draft -> target, offset form    d2t_offset[i] = keep_ids[i] - i      so that   target id = i + d2t_offset[i]
  target -> draft, membership     t2d[v] = 1 if v is one of keep_ids else 0
  remap through offsets           target_ids[t] = draft_ids[t] + d2t_offset[draft_ids[t]]
"""
from __future__ import annotations

import numpy as np


def d2t_offsets(keep_ids: np.ndarray) -> np.ndarray:
    out = np.zeros(len(keep_ids), dtype=np.int32)
    for i, v in enumerate(keep_ids):
        out[i] = int(v) - i
    return out


def t2d_mask(keep_ids: np.ndarray, V_full: int) -> np.ndarray:
    out = np.zeros(V_full, dtype=np.uint8)
    for v in keep_ids:
        if 0 <= int(v) < V_full:
            out[int(v)] = 1
    return out


def remap_offsets(draft_ids: np.ndarray, offsets: np.ndarray) -> np.ndarray:
    flat = np.asarray(draft_ids).ravel()
    out = np.empty(flat.shape, dtype=np.int32)
    for t, i in enumerate(flat):
        out[t] = int(i) + int(offsets[int(i)])
    return out.reshape(np.asarray(draft_ids).shape)
