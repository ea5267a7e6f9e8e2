"""Comparison rules between the CUDA head and the CPU oracle (test-side only).

Tolerances (the bar these tests hold the kernels to):
  * target ids, draft ids, coverage counts: bit-exact;
  * logits: |gpu - oracle| <= 2e-3 * max(1, |oracle|);
  * log-probs and lse: |gpu - oracle| <= 1e-3;
  * top-k ids equal the oracle's except where the oracle's own logits are closer than 1e-3:
    the GPU accumulates in fp32, the oracle in fp64, so candidates within 1e-3 of the k-th logit
    may swap in or out and neighbours closer than 1e-3 may swap places.  Logits that are equal
    bit-for-bit in the oracle must come out in ascending draft-index order.
"""
from __future__ import annotations

import numpy as np

LOGIT_RTOL = 2e-3
LOGPROB_ATOL = 1e-3
TIE_GAP = 1e-3


def check_logits(gpu_logits: np.ndarray, oracle_logits: np.ndarray):
    err = np.abs(gpu_logits.astype(np.float64) - oracle_logits)
    bound = LOGIT_RTOL * np.maximum(1.0, np.abs(oracle_logits))
    bad = err > bound
    assert not bad.any(), (f"{int(bad.sum())} logits out of tolerance; worst |d|={err.max():.3e} at "
                           f"{np.unravel_index(np.argmax(err - bound), err.shape)}")
    return float(err.max())


def check_head(gpu: dict, ora: dict, d2t: np.ndarray, k: int):
    """gpu: target_ids, logprobs, optional draft_ids, lse (numpy).  ora: oracle.draft_head(..., want_logits=True)."""
    x = ora["logits"]
    M, Vt = x.shape
    tid = gpu["target_ids"]
    lp = gpu["logprobs"].astype(np.float64)
    did = gpu.get("draft_ids")
    assert tid.shape == (M, k) and lp.shape == (M, k)
    if did is None:
        # recover draft ids through d2t (a bijection onto the kept ids in every workload here)
        inv = {int(t): i for i, t in enumerate(d2t)}
        assert len(inv) == len(d2t), "cannot invert d2t with repeated entries; ask for draft_ids"
        did = np.array([[inv[int(t)] for t in row] for row in tid], dtype=np.int32)
    assert np.array_equal(tid, d2t[did]), "target_ids != d2t[draft_ids]"
    if gpu.get("lse") is not None:
        assert np.max(np.abs(gpu["lse"].astype(np.float64) - ora["lse"])) <= LOGPROB_ATOL
    n_soft = 0
    for m in range(M):
        g, o = did[m], ora["draft_ids"][m]
        assert len(set(g.tolist())) == k, f"row {m}: repeated ids {g}"
        assert g.min() >= 0 and g.max() < Vt
        xg = x[m, g]
        # (iii) every returned id carries the oracle's log-prob for that id
        assert np.max(np.abs(lp[m] - (xg - ora["lse"][m]))) <= LOGPROB_ATOL, f"row {m}: log-prob mismatch"
        if np.array_equal(g, o):
            continue
        n_soft += 1
        kth = x[m, o[k - 1]]
        # (i) membership: anything the GPU holds that the oracle does not must sit within the tie gap of the
        # k-th logit, and anything it dropped likewise
        extra = [i for i in g if i not in set(o.tolist())]
        missing = [i for i in o if i not in set(g.tolist())]
        for i in extra:
            assert x[m, i] >= kth - TIE_GAP, f"row {m}: id {i} (x={x[m, i]}) is not near the k-th logit {kth}"
        for i in missing:
            assert x[m, i] <= kth + TIE_GAP, f"row {m}: dropped id {i} (x={x[m, i]}) clearly beats the k-th {kth}"
        # (ii) order: descending up to the gap; bit-equal oracle logits in ascending index order
        for j in range(k - 1):
            assert xg[j] >= xg[j + 1] - TIE_GAP, f"row {m}: positions {j},{j + 1} out of order"
    return n_soft


def check_exact_tie_order(did: np.ndarray, x: np.ndarray):
    """Among returned ids whose oracle logits are bit-equal, indices must ascend."""
    for m in range(did.shape[0]):
        xg = x[m, did[m]]
        for j in range(did.shape[1] - 1):
            if xg[j] == xg[j + 1]:
                assert did[m, j] < did[m, j + 1], f"row {m}: tie at {j} not in index order"
