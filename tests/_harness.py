"""Helpers for the GPU parity tests: move seeded host inputs to the device, call the C ABI through
the binding, bring results back as float64 numpy.  The oracle side is called by the tests themselves."""
from __future__ import annotations

import numpy as np
import torch

from paper_2605_01255_b200 import binding as B
from paper_2605_01255_b200 import inputs as I

TOL = {"f32": 1e-5, "bf16": 2e-2}          # the stated parity tolerances (relative Frobenius error)
TOL_DERIVED = {"f32": 2e-6, "bf16": 4e-3}  # what the arithmetic should deliver (one rounding per output)

# Element-wise bounds beside the Frobenius ratios (a norm alone leaves room for a few arbitrarily wrong elements, such
# as one bad tile corner): max over the elements of |gpu - oracle| / (|oracle| + rms(oracle)).
#   "bf16": an output rounded once to bfloat16 from an fp32 accumulator: 2^-9 of its own magnitude plus the accumulation
#           error (a few 1e-6 of the rms); 2^-7 leaves a factor of four.
#   "acc":  an fp32 output of the fp32 path (Y, XS, dX, A, dW there): one chain of fused multiply-adds rounded to
#           nearest, about sqrt(K) * 2^-24 of the rms with a tail of a few sigma.
#   "factor": the gradient factor A of the bf16 path, stage-wise: exact bf16 products summed in the tensor core's fp32
#           accumulator, which adds each group of 16 tokens to the running sum with a truncated (not nearest) rounding:
#           up to 2^-23 of the running sum per add and of one sign, so the error grows linearly with the chain,
#           about (2/3) * n * 2^-24 of the final magnitude for n adds.  The token ranges of the tested sizes are at
#           most 8192 tokens (n = 512): 2e-5 of the rms expected, measured 2.1e-5 at worst; 5e-5 leaves a factor of 2.
#   "dw":   the rebuilt gradient of the bf16 path: A enters as two bfloat16 terms (2^-17 of each |A_ij|), summed over r
#           terms of random sign, then one fp32 chain of length 2r.
#   "e2e":  A and dW computed from the GPU's own stored factor against the oracle's unrounded one: every XS element
#           carries its bfloat16 storage rounding (sigma 2^-9/sqrt(3) of the rms after the token sum, 5-sigma tail).
ELEM_TOL = {"bf16": 2.0 ** -7, "acc": 1e-5, "factor": 5e-5, "dw": 4e-5, "e2e": 2.0 ** -6}


def elementwise_err(got: np.ndarray, want: np.ndarray, per_row: bool = False) -> float:
    """max |got - want| / (|want| + rms(want)); NaN or inf anywhere in `got` gives inf.  per_row: the rms of the element's
    own row (for matrices whose rows differ in scale by orders of magnitude, like the heavy-tailed inputs)."""
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    if got.size == 0:
        return 0.0
    if not np.isfinite(got).all():
        return float("inf")
    if per_row:
        rms = np.sqrt(np.mean(want * want, axis=-1, keepdims=True))
        rms = np.where(rms > 0, rms, np.inf)   # an all-zero row must be reproduced exactly
        bad = (rms == np.inf) & (got != 0)
        return float("inf") if bad.any() else float(np.max(np.abs(got - want) / (np.abs(want) + rms)))
    rms = float(np.sqrt(np.mean(want * want)))
    if rms == 0.0:
        return 0.0 if not got.any() else float("inf")
    return float(np.max(np.abs(got - want) / (np.abs(want) + rms)))


def assert_parity(name: str, got: np.ndarray, want: np.ndarray, kind: str, frob_tol: float, context=None) -> float:
    """Both checks on one output: the relative Frobenius error and the element-wise bound of `kind`."""
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    den = float(np.linalg.norm(want))
    frob = float(np.linalg.norm(got - want)) / den if den > 0 else float(np.linalg.norm(got - want))
    elem = elementwise_err(got, want)
    assert frob <= frob_tol, (name, "frobenius", frob, frob_tol, context)
    assert elem <= ELEM_TOL[kind], (name, "element-wise", elem, ELEM_TOL[kind], context)
    return elem


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
