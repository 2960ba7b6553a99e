"""Buffer management around one plan: PyTorch supplies device memory and the stream, the C ABI
does all the arithmetic."""
from __future__ import annotations

import numpy as np
import torch

from .binding import ASI_OK, Batch, Plan


def _stream_handle(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


class LayerRunner:
    """Device buffers of one layer (two factor buffers that alternate as previous/new, core, dW,
    workspaces) and the calls that fill them."""

    def __init__(self, kind, dims, ranks, cout, k=1, stride=1, pad=0, groups=1, bf16=False,
                 device="cuda:0", generic_only=False, flags=0):
        if not torch.cuda.is_available():
            raise RuntimeError("the ASI path needs a CUDA device; there is no CPU fallback")
        self.plan = Plan(kind, dims, ranks, cout, k, stride, pad, groups, bf16,
                         generic_only=generic_only, flags=flags)
        self.dims, self.ranks, self.bf16 = tuple(dims), tuple(ranks), bf16
        self.device = torch.device(device)
        info = self.plan.info
        f32 = dict(dtype=torch.float32, device=self.device)
        self.U = [torch.zeros(info.u_elems, **f32), torch.zeros(info.u_elems, **f32)]
        self.cur = 0                       # index of the buffer holding the latest factors
        self.core = torch.zeros(info.core_elems, **f32)
        self.dW = torch.zeros(info.dw_elems, **f32)
        self.ws_c = torch.zeros(info.compress_ws_bytes, dtype=torch.uint8, device=self.device)
        self.ws_w = torch.zeros(info.wgrad_ws_bytes, dtype=torch.uint8, device=self.device)
        self.in_dtype = torch.bfloat16 if bf16 else torch.float32

    # -- host <-> device helpers ---------------------------------------------------------
    def to_device(self, x: np.ndarray) -> torch.Tensor:
        t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(self.device)
        return t.to(self.in_dtype).contiguous()

    def set_factors(self, U_list):
        flat = np.concatenate([np.ascontiguousarray(u, dtype=np.float32).ravel() for u in U_list])
        self.U[self.cur].copy_(torch.from_numpy(flat))

    def factors(self, which=None):
        buf = self.U[self.cur if which is None else which].cpu().numpy()
        out, off = [], 0
        for d, r in zip(self.dims, self.ranks):
            out.append(buf[off:off + d * r].reshape(d, r).copy())
            off += d * r
        return out

    def core_np(self):
        return self.core.cpu().numpy().reshape(self.ranks).copy()

    def dW_np(self, shape):
        return self.dW.cpu().numpy().reshape(shape).copy()

    # -- the path ------------------------------------------------------------------------
    def compress(self, act: torch.Tensor, stream=None):
        prev, new = self.U[self.cur], self.U[1 - self.cur]
        self.plan.compress(act.data_ptr(), prev.data_ptr(), new.data_ptr(), self.core.data_ptr(),
                           self.ws_c.data_ptr(), self.ws_c.numel(), _stream_handle(stream))
        self.cur = 1 - self.cur

    def init_factors(self, act: torch.Tensor, omega: torch.Tensor, stream=None):
        new = self.U[1 - self.cur]
        self.plan.init_factors(act.data_ptr(), omega.data_ptr(), new.data_ptr(), self.core.data_ptr(),
                               self.ws_c.data_ptr(), self.ws_c.numel(), _stream_handle(stream))
        self.cur = 1 - self.cur

    def init_factors_seeded(self, act: torch.Tensor, seed: int, stream=None):
        """Cold start with the library's counter-based Gaussian test matrices (allocates its scratch once)."""
        need = self.plan.init_seeded_ws_bytes()
        if getattr(self, "ws_seed", None) is None or self.ws_seed.numel() < need:
            self.ws_seed = torch.empty(need, dtype=torch.uint8, device=self.core.device)
        new = self.U[1 - self.cur]
        self.plan.init_factors_seeded(act.data_ptr(), seed, new.data_ptr(), self.core.data_ptr(),
                                      self.ws_seed.data_ptr(), self.ws_seed.numel(), _stream_handle(stream))
        self.cur = 1 - self.cur

    def wgrad(self, dY: torch.Tensor, stream=None):
        self.plan.wgrad(self.core.data_ptr(), self.U[self.cur].data_ptr(), dY.data_ptr(),
                        self.dW.data_ptr(), self.ws_w.data_ptr(), self.ws_w.numel(),
                        _stream_handle(stream))

    def device_status(self, stream=None):
        return self.plan.poll_status(self.ws_c.data_ptr(), _stream_handle(stream))

    def ok(self):
        return self.device_status() == ASI_OK


class StepRunner:
    """The layers of one training step behind the batched entry points: one asi_compress_batched call
    for the forward pass, one asi_wgrad_batched call for the backward pass."""

    def __init__(self, runners):
        self.runners = list(runners)
        self.batch = Batch([r.plan for r in self.runners])

    def compress(self, acts, stream=None):
        rs = self.runners
        self.batch.compress([a.data_ptr() for a in acts], [r.U[r.cur].data_ptr() for r in rs],
                            [r.U[1 - r.cur].data_ptr() for r in rs], [r.core.data_ptr() for r in rs],
                            [r.ws_c.data_ptr() for r in rs], [r.ws_c.numel() for r in rs], _stream_handle(stream))
        for r in rs:
            r.cur = 1 - r.cur

    def wgrad(self, dys, stream=None):
        rs = self.runners
        self.batch.wgrad([r.core.data_ptr() for r in rs], [r.U[r.cur].data_ptr() for r in rs],
                         [d.data_ptr() for d in dys], [r.dW.data_ptr() for r in rs],
                         [r.ws_w.data_ptr() for r in rs], [r.ws_w.numel() for r in rs], _stream_handle(stream))
