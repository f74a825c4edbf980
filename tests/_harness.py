"""Helpers for the GPU parity tests: move seeded host inputs to the device, call the C ABI through
the binding, bring results back as float64 numpy.  The oracle side is called by the tests themselves."""
from __future__ import annotations

import numpy as np
import torch

from paper_2605_01255_b200 import binding as B
from paper_2605_01255_b200 import inputs as I

TOL = {"f32": 1e-5, "bf16": 2e-2}          # the stated parity tolerances (relative Frobenius error)
TOL_DERIVED = {"f32": 2e-6, "bf16": 4e-3}  # what the arithmetic should deliver (one rounding per output)


def to_device(a: np.ndarray, dtype: str) -> torch.Tensor:
    """Host float32 values (already representable in `dtype`) -> CUDA tensor of that dtype."""
    if dtype == "bf16":
        bits = I.f32_to_bf16_bits(a)
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def to_host(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def raw_bits(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.view(torch.int32).cpu().numpy().view(np.uint32)


class GpuLinear:
    """One compressed linear layer's buffers on the device."""

    def __init__(self, m, d_in, d_out, r, seed, dtype):
        self.desc = B.make_desc(m, d_in, d_out, r, seed, dtype)
        self.dtype = dtype
        self.tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
        self.m, self.d_in, self.d_out, self.r = m, d_in, d_out, r
        self.ws_fwd = B.alloc_workspace(self.desc, B.ACX_OP_FWD)
        self.ws_bwd = B.alloc_workspace(self.desc, B.ACX_OP_BWD)
        self.ws_rec = B.alloc_workspace(self.desc, B.ACX_OP_RECONSTRUCT)

    def empty(self, rows, cols, dt=None):
        """An output buffer full of NaN canaries: whatever a call leaves unwritten shows up in the comparison."""
        return torch.full((rows, cols), float("nan"), dtype=dt or self.tdt, device="cuda")

    def fwd(self, X, W, want_xs=True):
        Y, XS = self.empty(self.m, self.d_out), (self.empty(self.m, self.r) if want_xs else None)
        B.acx_linear_fwd(self.desc, X, W, Y, XS, self.ws_fwd)
        return Y, XS

    def bwd(self, G, W, XS, want_dx=True, want_a=True):
        dX = self.empty(self.m, self.d_in) if want_dx else None
        A = self.empty(self.d_out, self.r, torch.float32) if want_a else None
        B.acx_linear_bwd(self.desc, G, W, XS, dX, A, self.ws_bwd)
        return dX, A

    def reconstruct(self, A, dW=None, beta=0.0):
        if dW is None:
            dW = self.empty(self.d_out, self.d_in, torch.float32)
        B.acx_reconstruct(self.desc, A, dW, beta, self.ws_rec)
        return dW

    def sketch(self):
        S = self.empty(self.d_in, self.r)
        B.acx_sketch_materialize(self.desc, S)
        return S

    def check_status(self):
        st = B.acx_last_device_status()
        assert st == B.ACX_OK, B.status_string(st)
