"""Helpers for the GPU parity tests: host arrays -> device tensors, guarded output buffers."""
from __future__ import annotations

import numpy as np
import torch

CANARY = 0x5A


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def dev_i32(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


class Guarded:
    """An output tensor carved out of a byte buffer with canary bytes on both sides."""
    PAD = 256

    def __init__(self, shape, dtype):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.buf = torch.full((n + 2 * self.PAD,), CANARY, dtype=torch.uint8, device="cuda")
        self.t = self.buf[self.PAD:self.PAD + n].view(dtype).view(*shape)
        self.n = n

    def intact(self) -> bool:
        b = self.buf.cpu().numpy()
        return bool((b[:self.PAD] == CANARY).all() and (b[self.PAD + self.n:] == CANARY).all())


def run_head(vt, case_h, W_trim_dev, d2t, k, path, workspace=None):
    """Runs vt_draft_head on device tensors and returns numpy outputs plus the guard check."""
    M = case_h.shape[0]
    h = dev_bf16(case_h)
    d2t_dev = dev_i32(d2t)
    tid, lp = Guarded((M, k), torch.int32), Guarded((M, k), torch.float32)
    did, lse = Guarded((M, k), torch.int32), Guarded((M,), torch.float32)
    ws = workspace if workspace is not None else vt.new_workspace(vt.vt_workspace_bytes(M, k))
    vt.vt_draft_head(h, W_trim_dev, d2t_dev, k, workspace=ws, path=path, target_ids=tid.t, logprobs=lp.t,
                     draft_ids=did.t, lse=lse.t)
    assert vt.vt_last_status(ws) == vt.VT_OK
    torch.cuda.synchronize()
    assert tid.intact() and lp.intact() and did.intact() and lse.intact(), "write outside an output buffer"
    return {"target_ids": tid.t.cpu().numpy(), "logprobs": lp.t.cpu().numpy(),
            "draft_ids": did.t.cpu().numpy(), "lse": lse.t.cpu().numpy()}
