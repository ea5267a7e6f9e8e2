"""CPU oracle for the cross-row candidate selection of a draft tree step.  TEST INFRASTRUCTURE ONLY.

The paper's draft step (Section 1) proposes candidate tokens; tree-style drafts expand several rows at once and keep
the globally best continuations.  The paper gives no formula for that step, so this oracle fixes the plain reading:

  score[m, j] = parent[m] + logprobs[m, j]            one fp32 addition (the precision the selection is decided in)
  the T largest scores over all M * k pairs, in descending order; equal scores by ascending flat index m * k + j

and returns, for each selected pair, its row m, its slot j, its token target_ids[m, j] and its score.
Pure Python / numpy; it shares no code with the CUDA path.
"""
from __future__ import annotations

import numpy as np


def tree_select(logprobs: np.ndarray, target_ids: np.ndarray, parent: np.ndarray, T: int) -> dict:
    lp = np.asarray(logprobs, dtype=np.float32)
    M, k = lp.shape
    score = (np.asarray(parent, dtype=np.float32)[:, None] + lp).astype(np.float32)     # IEEE single addition
    flat = score.ravel()
    order = sorted(range(M * k), key=lambda e: (-float(flat[e]), e))[:T]
    order = np.asarray(order, dtype=np.int64)
    return {"rows": (order // k).astype(np.int32), "slots": (order % k).astype(np.int32),
            "tokens": np.asarray(target_ids).ravel()[order].astype(np.int32), "scores": flat[order].astype(np.float32)}
