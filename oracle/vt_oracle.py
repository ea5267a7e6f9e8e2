"""ctypes loader for the C oracle.  TEST INFRASTRUCTURE ONLY (see ``vt_oracle.c``)."""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vt_oracle.c")
_LIB = os.path.join(_HERE, "libvt_oracle.so")
_lib = None

_i64 = ctypes.c_int64
_p = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile ``vt_oracle.c`` with gcc (no fast-math, no contraction) if the library is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared",
                               "-fPIC", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        # VT_ORACLE_LIB points the loader at another build of the same source: the mutation test uses it to
        # check that the pins notice a planted mistake
        lib = ctypes.CDLL(os.environ.get("VT_ORACLE_LIB") or build())
        lib.vto_bf16_to_f64.restype = ctypes.c_double
        lib.vto_bf16_to_f64.argtypes = [ctypes.c_uint16]
        lib.vto_num_threads.restype = ctypes.c_int
        lib.vto_compact.restype = None
        lib.vto_compact.argtypes = [_p, _i64, _i64, _p, _i64, _p]
        lib.vto_logits.restype = None
        lib.vto_logits.argtypes = [_p, _p, _i64, _i64, _i64, _p]
        lib.vto_log_softmax.restype = None
        lib.vto_log_softmax.argtypes = [_p, _i64, _i64, _p, _p]
        lib.vto_topk.restype = ctypes.c_int
        lib.vto_topk.argtypes = [_p, _i64, _i64, _i64, _p]
        lib.vto_remap.restype = None
        lib.vto_remap.argtypes = [_p, _i64, _p, _p]
        lib.vto_coverage.restype = ctypes.c_int
        lib.vto_coverage.argtypes = [_p, _i64, _p, _i64, _i64, _p]
        lib.vto_draft_head.restype = ctypes.c_int
        lib.vto_draft_head.argtypes = [_p, _p, _p, _i64, _i64, _i64, _i64, _p, _p, _p, _p, _p]
        _lib = lib
    return _lib


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a, a.ctypes.data_as(_p)


def num_threads() -> int:
    return int(_load().vto_num_threads())


def bf16_to_f64(bits: int) -> float:
    return float(_load().vto_bf16_to_f64(int(bits) & 0xFFFF))


def compact(W_full: np.ndarray, keep_ids: np.ndarray) -> np.ndarray:
    W_full, pw = _c(W_full, np.uint16)
    keep_ids, pk = _c(keep_ids, np.int32)
    V, d = W_full.shape
    out = np.empty((len(keep_ids), d), dtype=np.uint16)
    _load().vto_compact(pw, V, d, pk, len(keep_ids), out.ctypes.data_as(_p))
    return out


def logits(h: np.ndarray, W: np.ndarray) -> np.ndarray:
    h, ph = _c(h, np.uint16)
    W, pw = _c(W, np.uint16)
    M, d = h.shape
    Vt, d2 = W.shape
    assert d == d2
    x = np.empty((M, Vt), dtype=np.float64)
    _load().vto_logits(ph, pw, M, d, Vt, x.ctypes.data_as(_p))
    return x


def log_softmax(x: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    x, px = _c(x, np.float64)
    M, Vt = x.shape
    lp = np.empty_like(x)
    lse = np.empty(M, dtype=np.float64)
    _load().vto_log_softmax(px, M, Vt, lp.ctypes.data_as(_p), lse.ctypes.data_as(_p))
    return lp, lse


def topk(x: np.ndarray, k: int) -> np.ndarray:
    x, px = _c(x, np.float64)
    M, Vt = x.shape
    idx = np.empty((M, k), dtype=np.int32)
    rc = _load().vto_topk(px, M, Vt, k, idx.ctypes.data_as(_p))
    if rc:
        raise ValueError(f"vto_topk failed with {rc} (k={k}, V_trim={Vt})")
    return idx


def remap(draft_idx: np.ndarray, d2t: np.ndarray) -> np.ndarray:
    draft_idx, pi = _c(draft_idx, np.int32)
    d2t, pd = _c(d2t, np.int32)
    out = np.empty_like(draft_idx)
    _load().vto_remap(pi, draft_idx.size, pd, out.ctypes.data_as(_p))
    return out


def coverage(token_ids: np.ndarray, keep_ids: np.ndarray, V_full: int) -> tuple[int, float]:
    """Eq. 2 on a token stream: (covered occurrences, covered / N)."""
    token_ids, pt = _c(token_ids, np.int32)
    keep_ids, pk = _c(keep_ids, np.int32)
    if token_ids.size == 0:
        raise ValueError("coverage of an empty stream is 0/0")
    c = ctypes.c_uint64(0)
    rc = _load().vto_coverage(pt, token_ids.size, pk, keep_ids.size, V_full, ctypes.byref(c))
    if rc:
        raise MemoryError("vto_coverage")
    return int(c.value), float(c.value) / float(token_ids.size)


def draft_head(h: np.ndarray, W_trim: np.ndarray, d2t: np.ndarray, k: int, want_logits: bool = False) -> dict:
    """Full call.  Returns target_ids/draft_ids [M,k] int32, logprobs [M,k], lse [M], optionally logits [M,Vt]."""
    h, ph = _c(h, np.uint16)
    W_trim, pw = _c(W_trim, np.uint16)
    d2t, pd = _c(d2t, np.int32)
    M, d = h.shape
    Vt = W_trim.shape[0]
    assert W_trim.shape[1] == d and d2t.size == Vt
    tid = np.empty((M, k), dtype=np.int32)
    did = np.empty((M, k), dtype=np.int32)
    lp = np.empty((M, k), dtype=np.float64)
    lse = np.empty(M, dtype=np.float64)
    x = np.empty((M, Vt), dtype=np.float64) if want_logits else None
    rc = _load().vto_draft_head(ph, pw, pd, M, d, Vt, k, tid.ctypes.data_as(_p), lp.ctypes.data_as(_p),
                                did.ctypes.data_as(_p), lse.ctypes.data_as(_p),
                                x.ctypes.data_as(_p) if want_logits else None)
    if rc:
        raise ValueError(f"vto_draft_head failed with {rc}")
    out = {"target_ids": tid, "draft_ids": did, "logprobs": lp, "lse": lse}
    if want_logits:
        out["logits"] = x
    return out
