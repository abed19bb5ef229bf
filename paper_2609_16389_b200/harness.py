"""Device-memory plumbing around the C-ABI calls (PyTorch for memory and streams only)."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from . import synth


def _to_device(buf: np.ndarray, device) -> torch.Tensor:
    """Host buffer -> device tensor of raw bytes with 256-byte aligned storage."""
    t = torch.from_numpy(buf.view(np.uint8).reshape(-1))
    return t.to(device, non_blocking=False)


def desc_of(p: synth.Problem, flags: int = 0, device: int = -1, flags2: int = 0) -> B.Desc:
    return B.make_desc(p.M, p.N, p.K, p.ab_dtype, p.c_dtype, p.a_layout, p.b_layout, p.c_layout,
                       p.lda, p.ldb, p.ldc, device=device, flags=flags, flags2=flags2)


class DeviceProblem:
    """A synth.Problem resident on the GPU, with a plan; ``run`` enqueues one GEMM."""

    def __init__(self, p: synth.Problem, flags: int = 0, device="cuda:0", flags2: int = 0):
        self.p = p
        self.device = torch.device(device)
        self.dA = _to_device(p.A, self.device)
        self.dB = _to_device(p.B, self.device)
        self.dC = _to_device(p.C, self.device)
        self.plan = B.Plan(desc_of(p, flags, self.device.index or 0, flags2))

    def run(self, stream: int | None = None, alpha=None, beta=None):
        s = torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream
        self.plan.run(self.dA.data_ptr(), self.dB.data_ptr(), self.dC.data_ptr(),
                      self.p.alpha if alpha is None else alpha,
                      self.p.beta if beta is None else beta, s)

    def reset_c(self):
        self.dC.copy_(torch.from_numpy(self.p.C.view(np.uint8).reshape(-1)))

    def result_buffer(self) -> np.ndarray:
        """The C buffer (flat, storage dtype) copied back to the host."""
        torch.cuda.synchronize(self.device)
        raw = self.dC.cpu().numpy()
        return raw.view(synth.storage_np_dtype(self.p.c_dtype))

    def close(self):
        self.plan.close()


def gemm_host(p: synth.Problem, flags: int = 0, device="cuda:0", flags2: int = 0):
    """Host buffers in, host C buffer out: upload, one GEMM, check the plan, download."""
    dp = DeviceProblem(p, flags, device, flags2)
    try:
        dp.run()
        torch.cuda.synchronize(dp.device)
        dp.plan.check()
        return dp.result_buffer(), dp.plan.info()
    finally:
        dp.close()
