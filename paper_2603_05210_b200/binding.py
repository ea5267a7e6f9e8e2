"""Python binding of ``libvt.so``: argument marshalling only.

Each function has the name of the C entry point it calls (``include/vt.h``) and passes torch
tensors' device pointers and the current CUDA stream through ctypes.  PyTorch provides device
memory and streams; every step of the head runs inside the library's kernels.  There is no
fallback: if the library cannot be loaded the call raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvt.so")

VT_OK = 0
VT_ERR_NULL, VT_ERR_SHAPE, VT_ERR_ALIGN, VT_ERR_RANGE, VT_ERR_DUP = 1, 2, 3, 4, 5
VT_ERR_EMPTY, VT_ERR_WORKSPACE, VT_ERR_TIMEOUT, VT_ERR_CUDA, VT_ERR_UNSUPPORTED = 6, 7, 8, 9, 10
VT_MAX_K = 64
VT_PATH_AUTO, VT_PATH_GEMV, VT_PATH_MMA, VT_PATH_MMA_SMALL = 0, 1, 2, 3
VT_HEAD_STATIC_WEIGHTS, VT_HEAD_D2T_OFFSETS = 0x100, 0x200

# every symbol include/vt.h declares: name -> (restype, argtypes)
_p, _i, _i64, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
SYMBOLS = {
    "vt_strerror": (ctypes.c_char_p, [_i]),
    "vt_last_cuda_error": (_i, []),
    "vt_compact_head": (_i, [_p, _i, _i, _p, _i, _p, _p]),
    "vt_coverage_workspace_bytes": (_sz, [_i]),
    "vt_validate_keep_ids": (_i, [_p, _i, _i, _p, _sz, _p]),
    "vt_workspace_bytes": (_sz, [_i, _i]),
    "vt_workspace_init": (_i, [_p, _sz, _p]),
    "vt_draft_head": (_i, [_p, _p, _p, _i, _i, _i, _i, _p, _p, _p, _p, _p, _sz, _p]),
    "vt_draft_head_path": (_i, [_p, _p, _p, _i, _i, _i, _i, _p, _p, _p, _p, _p, _sz, _p, _i]),
    "vt_host_workspace_bytes": (_sz, [_i, _i, _i]),
    "vt_draft_head_host": (_i, [_p, _p, _p, _i, _i, _i, _i, _p, _p, _p, _sz, _p]),
    "vt_last_status": (_i, [_p, _p]),
    "vt_coverage": (_i, [_p, _i64, _p, _i, _i, _p, _p, _p, _sz, _p]),
    "vt_coverage_enqueue": (_i, [_p, _i64, _p, _i, _i, _p, _sz, _p]),
    "vt_coverage_result": (_i, [_p, _i64, _p, _p, _p]),
    "vt_select_workspace_bytes": (_sz, [_i]),
    "vt_select_vocab": (_i, [_p, _i64, _i, _i, ctypes.c_double, ctypes.c_double, ctypes.c_double, _i, _i, _p, _p, _p, _p, _p,
                            _p, _p, _p, _sz, _p]),
    "vt_coverage_static": (_i, [_p, _i64, _p, _i, _i, _p, _p, _p]),
    "vt_debug_logits": (_i, [_p, _p, _i, _i, _i, _p, _p, _sz, _p, _i]),
    "vt_fuse_features": (_i, [_p, _p, _i, _i, _i, _p, _p, _sz, _p]),
    "vt_tree_select": (_i, [_p, _p, _p, _i, _i, _i, _p, _p, _p, _p, _p]),
    "vt_remap": (_i, [_p, _p, _i64, _i, _p, _p]),
    "vt_vocab_maps": (_i, [_p, _i, _i, _p, _p, _p]),
    "vt_last_launch_count": (_i, []),
    "vt_test_timeout_probe": (_i, [_p, _i, _p]),
    "vt_test_late_copy": (_i, [_p, _p, _sz, _i, _p]),
}

_lib = None


class VtError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = int(status)
        text = lib().vt_strerror(self.status).decode()
        extra = f" (CUDA error {lib().vt_last_cuda_error()})" if self.status == VT_ERR_CUDA else ""
        super().__init__(f"{what}: status {self.status}: {text}{extra}")


def lib() -> ctypes.CDLL:
    """Load ``libvt.so`` from the package directory, building it with nvcc first if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            from .build import build
            build()
        cd = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(cd, name)     # AttributeError if the library lacks a declared symbol
            fn.restype, fn.argtypes = res, args
        _lib = cd
    return _lib


def _check(status: int, what: str):
    if status != VT_OK:
        raise VtError(status, what)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t):
    return None if t is None else t.data_ptr()


def _bf16(t: torch.Tensor, name: str) -> torch.Tensor:
    if t.dtype not in (torch.bfloat16, torch.int16, torch.uint16):
        raise TypeError(f"{name}: expected bf16 data (torch.bfloat16 or a 16-bit integer view), got {t.dtype}")
    if not t.is_cuda or not t.is_contiguous() or t.dim() != 2:
        raise ValueError(f"{name}: expected a contiguous 2-D CUDA tensor")
    return t


def _i32(t: torch.Tensor, name: str) -> torch.Tensor:
    if t.dtype != torch.int32 or not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name}: expected a contiguous int32 CUDA tensor")
    return t


def vt_workspace_bytes(M: int, k: int) -> int:
    return int(lib().vt_workspace_bytes(M, k))


def vt_host_workspace_bytes(M: int, d: int, k: int) -> int:
    return int(lib().vt_host_workspace_bytes(M, d, k))


def vt_coverage_workspace_bytes(V_full: int) -> int:
    return int(lib().vt_coverage_workspace_bytes(V_full))


def vt_workspace_init(workspace: torch.Tensor) -> torch.Tensor:
    _check(lib().vt_workspace_init(workspace.data_ptr(), workspace.numel(), _stream()), "vt_workspace_init")
    return workspace


def new_workspace(nbytes: int, device=None) -> torch.Tensor:
    """A zero-initialised byte buffer of the caller's (torch's caching allocator is 512-byte aligned)."""
    ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device or "cuda")
    return vt_workspace_init(ws)


def vt_compact_head(W_full: torch.Tensor, keep_ids: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    W_full = _bf16(W_full, "W_full")
    keep_ids = _i32(keep_ids, "keep_ids")
    V, d = W_full.shape
    Vt = keep_ids.numel()
    if out is None:
        out = torch.empty((Vt, d), dtype=W_full.dtype, device=W_full.device)
    _check(lib().vt_compact_head(W_full.data_ptr(), V, d, keep_ids.data_ptr(), Vt, out.data_ptr(), _stream()),
           "vt_compact_head")
    return out


def vt_validate_keep_ids(keep_ids: torch.Tensor, V_full: int, workspace: torch.Tensor | None = None) -> int:
    """Returns the status (VT_OK, VT_ERR_RANGE or VT_ERR_DUP) instead of raising for those two."""
    keep_ids = _i32(keep_ids, "keep_ids")
    if workspace is None:
        workspace = torch.empty(vt_coverage_workspace_bytes(V_full), dtype=torch.uint8, device=keep_ids.device)
    st = lib().vt_validate_keep_ids(keep_ids.data_ptr(), keep_ids.numel(), V_full, workspace.data_ptr(),
                                    workspace.numel(), _stream())
    if st not in (VT_OK, VT_ERR_RANGE, VT_ERR_DUP):
        raise VtError(st, "vt_validate_keep_ids")
    return st


def vt_draft_head(h: torch.Tensor, W_trim: torch.Tensor, d2t: torch.Tensor, k: int, *,
                  workspace: torch.Tensor | None = None, path: int = VT_PATH_AUTO,
                  target_ids: torch.Tensor | None = None, logprobs: torch.Tensor | None = None,
                  draft_ids: torch.Tensor | None = None, lse: torch.Tensor | None = None,
                  static_weights: bool = False, d2t_offsets: bool = False):
    """(target_ids [M,k] int32, logprobs [M,k] float32); pass ``draft_ids`` / ``lse`` tensors to receive those too.

    ``static_weights`` sets VT_HEAD_STATIC_WEIGHTS, ``d2t_offsets`` sets VT_HEAD_D2T_OFFSETS (see ``include/vt.h``)."""
    h = _bf16(h, "h")
    W_trim = _bf16(W_trim, "W_trim")
    d2t = _i32(d2t, "d2t")
    M, d = h.shape
    Vt, d2 = W_trim.shape
    if d2 != d or d2t.numel() != Vt:
        raise ValueError("h, W_trim and d2t disagree on d or V_trim")
    if workspace is None:
        workspace = new_workspace(vt_workspace_bytes(M, min(max(k, 1), VT_MAX_K)), h.device)
    if target_ids is None:
        target_ids = torch.empty((M, k), dtype=torch.int32, device=h.device)
    if logprobs is None:
        logprobs = torch.empty((M, k), dtype=torch.float32, device=h.device)
    _check(lib().vt_draft_head_path(h.data_ptr(), W_trim.data_ptr(), d2t.data_ptr(), M, d, Vt, k,
                                    target_ids.data_ptr(), logprobs.data_ptr(), _ptr(draft_ids), _ptr(lse),
                                    workspace.data_ptr(), workspace.numel(), _stream(),
                                    path | (VT_HEAD_STATIC_WEIGHTS if static_weights else 0)
                                    | (VT_HEAD_D2T_OFFSETS if d2t_offsets else 0)), "vt_draft_head")
    return target_ids, logprobs


def vt_draft_head_host(h_host: torch.Tensor, W_trim: torch.Tensor, d2t: torch.Tensor, k: int,
                       target_ids_host: torch.Tensor, logprobs_host: torch.Tensor, workspace: torch.Tensor):
    """Host-buffer form: ``h_host`` and both outputs are CPU tensors (pinned for speed); synchronises."""
    M, d = h_host.shape
    Vt = W_trim.shape[0]
    if h_host.is_cuda or target_ids_host.is_cuda or logprobs_host.is_cuda:
        raise ValueError("vt_draft_head_host takes host tensors for h and the outputs")
    _check(lib().vt_draft_head_host(h_host.data_ptr(), W_trim.data_ptr(), d2t.data_ptr(), M, d, Vt, k,
                                    target_ids_host.data_ptr(), logprobs_host.data_ptr(),
                                    workspace.data_ptr(), workspace.numel(), _stream()), "vt_draft_head_host")
    return target_ids_host, logprobs_host


def vt_last_status(workspace: torch.Tensor) -> int:
    return int(lib().vt_last_status(workspace.data_ptr(), _stream()))


def vt_coverage(token_ids: torch.Tensor, keep_ids: torch.Tensor, V_full: int,
                workspace: torch.Tensor | None = None) -> tuple[int, float]:
    token_ids = _i32(token_ids, "token_ids")
    keep_ids = _i32(keep_ids, "keep_ids")
    if workspace is None:
        workspace = torch.empty(vt_coverage_workspace_bytes(V_full), dtype=torch.uint8, device=keep_ids.device)
    covered = ctypes.c_uint64(0)
    frac = ctypes.c_double(0.0)
    _check(lib().vt_coverage(token_ids.data_ptr() if token_ids.numel() else None, token_ids.numel(),
                             keep_ids.data_ptr(), keep_ids.numel(), V_full,
                             ctypes.addressof(covered), ctypes.addressof(frac),
                             workspace.data_ptr(), workspace.numel(), _stream()), "vt_coverage")
    return int(covered.value), float(frac.value)


def vt_coverage_enqueue(token_ids: torch.Tensor, keep_ids: torch.Tensor, V_full: int, workspace: torch.Tensor) -> None:
    token_ids = _i32(token_ids, "token_ids")
    keep_ids = _i32(keep_ids, "keep_ids")
    _check(lib().vt_coverage_enqueue(token_ids.data_ptr() if token_ids.numel() else None, token_ids.numel(),
                                     keep_ids.data_ptr(), keep_ids.numel(), V_full,
                                     workspace.data_ptr(), workspace.numel(), _stream()), "vt_coverage_enqueue")


def vt_coverage_result(workspace: torch.Tensor, N: int) -> tuple[int, float]:
    covered = ctypes.c_uint64(0)
    frac = ctypes.c_double(0.0)
    _check(lib().vt_coverage_result(workspace.data_ptr(), int(N), ctypes.addressof(covered), ctypes.addressof(frac),
                                    _stream()), "vt_coverage_result")
    return int(covered.value), float(frac.value)


def vt_select_workspace_bytes(V_full: int) -> int:
    return int(lib().vt_select_workspace_bytes(V_full))


def vt_select_vocab(token_ids: torch.Tensor, V_full: int, d: int, F_fixed: float, alpha: float, c_min: float,
                    k_min: int, k_max: int, *, want_cum: bool = False, workspace: torch.Tensor | None = None) -> dict:
    """k* and the frequency ranking (Eq. 1-5).  Returns k_star, C, R, U (at k*), ranked_ids [V_full] and, if asked, cum_counts."""
    token_ids = _i32(token_ids, "token_ids")
    dev = token_ids.device
    ranked = torch.empty(V_full, dtype=torch.int32, device=dev)
    cum = torch.empty(V_full, dtype=torch.int64, device=dev) if want_cum else None
    if workspace is None:
        workspace = torch.empty(vt_select_workspace_bytes(V_full), dtype=torch.uint8, device=dev)
    k_star = ctypes.c_int(0)
    C, R, U, uq = ctypes.c_double(0), ctypes.c_double(0), ctypes.c_double(0), ctypes.c_double(0)
    _check(lib().vt_select_vocab(token_ids.data_ptr() if token_ids.numel() else None, token_ids.numel(), V_full, d,
                                 float(F_fixed), float(alpha), float(c_min), k_min, k_max, ranked.data_ptr(), _ptr(cum),
                                 ctypes.addressof(k_star), ctypes.addressof(C), ctypes.addressof(R), ctypes.addressof(U),
                                 ctypes.addressof(uq), workspace.data_ptr(), workspace.numel(), _stream()), "vt_select_vocab")
    out = {"k_star": int(k_star.value), "C": float(C.value), "R": float(R.value), "U": float(U.value),
           "unique": float(uq.value), "ranked_ids": ranked}
    if want_cum:
        out["cum_counts"] = cum
    return out


def vt_coverage_static(token_ids: torch.Tensor, keep_ids: torch.Tensor, V_full: int) -> tuple[int, float]:
    """``vt_coverage`` without a workspace: the library's built-in scratch is used and nothing is allocated
    here or in the library (for callers that may not allocate; V_full <= 262,144; calls must not overlap)."""
    token_ids = _i32(token_ids, "token_ids")
    keep_ids = _i32(keep_ids, "keep_ids")
    covered = ctypes.c_uint64(0)
    frac = ctypes.c_double(0.0)
    _check(lib().vt_coverage_static(token_ids.data_ptr() if token_ids.numel() else None, token_ids.numel(),
                                    keep_ids.data_ptr(), keep_ids.numel(), V_full,
                                    ctypes.addressof(covered), ctypes.addressof(frac), _stream()),
           "vt_coverage_static")
    return int(covered.value), float(frac.value)


def vt_debug_logits(h: torch.Tensor, W_trim: torch.Tensor, path: int = VT_PATH_AUTO) -> torch.Tensor:
    h = _bf16(h, "h")
    W_trim = _bf16(W_trim, "W_trim")
    M, d = h.shape
    Vt = W_trim.shape[0]
    logits = torch.empty((M, Vt), dtype=torch.float32, device=h.device)
    ws = new_workspace(vt_workspace_bytes(M, 2), h.device)
    _check(lib().vt_debug_logits(h.data_ptr(), W_trim.data_ptr(), M, d, Vt, logits.data_ptr(), ws.data_ptr(),
                                 ws.numel(), _stream(), path), "vt_debug_logits")
    return logits


def vt_fuse_features(h3: torch.Tensor, W_fuse: torch.Tensor, *, out: torch.Tensor | None = None,
                     workspace: torch.Tensor | None = None) -> torch.Tensor:
    """fused [M, d_out] bf16 = h3 [M, d_in] x W_fuse[d_out, d_in]^T, fp32 accumulation, one rounding to bf16."""
    h3 = _bf16(h3, "h3")
    W_fuse = _bf16(W_fuse, "W_fuse")
    M, d_in = h3.shape
    d_out, d2 = W_fuse.shape
    if d2 != d_in:
        raise ValueError("h3 and W_fuse disagree on d_in")
    if out is None:
        out = torch.empty((M, d_out), dtype=h3.dtype, device=h3.device)
    if workspace is None:
        workspace = new_workspace(vt_workspace_bytes(M, 1), h3.device)
    _check(lib().vt_fuse_features(h3.data_ptr(), W_fuse.data_ptr(), M, d_in, d_out, out.data_ptr(), workspace.data_ptr(),
                                  workspace.numel(), _stream()), "vt_fuse_features")
    return out


def vt_tree_select(logprobs: torch.Tensor, target_ids: torch.Tensor, parent_scores: torch.Tensor, T: int):
    """The T best (row, slot) pairs by parent score + log-prob: (rows, slots, tokens, scores), each [T]."""
    M, k = logprobs.shape
    if logprobs.dtype != torch.float32 or parent_scores.dtype != torch.float32 or not logprobs.is_contiguous():
        raise ValueError("logprobs and parent_scores must be contiguous float32 CUDA tensors")
    target_ids = _i32(target_ids, "target_ids")
    dev = logprobs.device
    rows = torch.empty(T, dtype=torch.int32, device=dev)
    slots = torch.empty(T, dtype=torch.int32, device=dev)
    tokens = torch.empty(T, dtype=torch.int32, device=dev)
    scores = torch.empty(T, dtype=torch.float32, device=dev)
    _check(lib().vt_tree_select(logprobs.data_ptr(), target_ids.data_ptr(), parent_scores.data_ptr(), M, k, T,
                                rows.data_ptr(), slots.data_ptr(), tokens.data_ptr(), scores.data_ptr(), _stream()),
           "vt_tree_select")
    return rows, slots, tokens, scores


def vt_remap(draft_ids: torch.Tensor, d2t: torch.Tensor) -> torch.Tensor:
    draft_ids = _i32(draft_ids, "draft_ids")
    d2t = _i32(d2t, "d2t")
    out = torch.empty_like(draft_ids)
    _check(lib().vt_remap(draft_ids.data_ptr(), d2t.data_ptr(), draft_ids.numel(), d2t.numel(), out.data_ptr(),
                          _stream()), "vt_remap")
    return out


def vt_vocab_maps(keep_ids: torch.Tensor, V_full: int) -> tuple[torch.Tensor, torch.Tensor]:
    """(d2t offsets [V_trim] int32, t2d membership mask [V_full] uint8) in the form EAGLE-3 checkpoints store."""
    keep_ids = _i32(keep_ids, "keep_ids")
    off = torch.empty_like(keep_ids)
    mask = torch.empty(V_full, dtype=torch.uint8, device=keep_ids.device)
    _check(lib().vt_vocab_maps(keep_ids.data_ptr(), keep_ids.numel(), V_full, off.data_ptr(), mask.data_ptr(), _stream()),
           "vt_vocab_maps")
    return off, mask


def vt_last_launch_count() -> int:
    return int(lib().vt_last_launch_count())


def vt_test_timeout_probe(workspace: torch.Tensor, limit_us: int) -> None:
    _check(lib().vt_test_timeout_probe(workspace.data_ptr(), int(limit_us), _stream()), "vt_test_timeout_probe")


def vt_test_late_copy(dst: torch.Tensor, src: torch.Tensor, delay_us: int) -> None:
    n = src.numel() * src.element_size()
    if dst.numel() * dst.element_size() != n:
        raise ValueError("dst and src differ in size")
    _check(lib().vt_test_late_copy(dst.data_ptr(), src.data_ptr(), n, int(delay_us), _stream()), "vt_test_late_copy")
