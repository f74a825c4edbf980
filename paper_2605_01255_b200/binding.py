"""ctypes binding to libacx.so: same names as the C ABI (include/acx.h), argument marshalling only.

torch supplies device memory and streams; every arithmetic step runs in the library's kernels.  If
the library has not been built the import of a symbol raises: there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libacx.so")

ACX_OK = 0
ACX_ERR_INVALID_ARG, ACX_ERR_UNSUPPORTED_SHAPE, ACX_ERR_ALIGNMENT = 1, 2, 3
ACX_ERR_WORKSPACE, ACX_ERR_CUDA, ACX_ERR_TIMEOUT = 4, 5, 6
ACX_ERR_SCRATCH_LIMIT = 7
ACX_BUILTIN_SCRATCH_BYTES = 16 << 20
ACX_F32, ACX_BF16 = 0, 1
ACX_OP_FWD, ACX_OP_BWD, ACX_OP_RECONSTRUCT, ACX_OP_BWD_BUILTIN_SCRATCH, ACX_OP_RSVD, ACX_OP_BIAS_GRAD = 0, 1, 2, 3, 4, 5
ACX_OP_BWD_BIAS = 6

EXPORTS = (
    "acx_workspace_bytes", "acx_linear_fwd", "acx_linear_bwd", "acx_reconstruct",
    "acx_sketch_materialize", "acx_last_device_status", "acx_kernel_launches", "acx_status_string", "acx_version",
    "acx_linear_bwd_factor_builtin_scratch", "acx_reconstruct_adamw", "acx_debug_expired_wait",
    "acx_debug_force_gemm_mode", "acx_linear_fwd_v", "acx_reconstruct_v", "acx_lowrank_adamw", "acx_rsvd_factor", "acx_linear_fwd_bias", "acx_bias_grad", "acx_linear_bwd_bias",
)


class AcxError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s" % (where, status_string(status)))


class acx_adamw_params(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("step", ctypes.c_int32), ("lr", ctypes.c_float), ("beta1", ctypes.c_float),
                ("beta2", ctypes.c_float), ("eps", ctypes.c_float), ("weight_decay", ctypes.c_float)]


class acx_desc(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("sketch_kind", ctypes.c_uint32),
        ("tokens", ctypes.c_int64), ("d_in", ctypes.c_int64), ("d_out", ctypes.c_int64),
        ("r", ctypes.c_int32), ("io_dtype", ctypes.c_int32), ("seed", ctypes.c_uint64),
    ]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if libacx.so is missing (build it with paper_2605_01255_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libacx.so is not built (%s); run `python -m paper_2605_01255_b200.build`. "
                               "There is no CPU or PyTorch fallback." % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, dp = ctypes.c_void_p, ctypes.c_size_t, ctypes.POINTER(acx_desc)
        L.acx_workspace_bytes.restype, L.acx_workspace_bytes.argtypes = sz, [dp, ctypes.c_int]
        L.acx_linear_fwd.restype, L.acx_linear_fwd.argtypes = ctypes.c_int, [dp, vp, vp, vp, vp, vp, sz, vp]
        L.acx_linear_bwd.restype, L.acx_linear_bwd.argtypes = ctypes.c_int, [dp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.acx_linear_bwd_factor_builtin_scratch.restype = ctypes.c_int
        L.acx_linear_bwd_factor_builtin_scratch.argtypes = [dp, vp, vp, vp, vp]
        L.acx_reconstruct.restype, L.acx_reconstruct.argtypes = ctypes.c_int, [dp, vp, vp, ctypes.c_float, vp, sz, vp]
        L.acx_linear_fwd_v.restype, L.acx_linear_fwd_v.argtypes = ctypes.c_int, [dp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.acx_reconstruct_v.restype, L.acx_reconstruct_v.argtypes = ctypes.c_int, [dp, vp, vp, vp, ctypes.c_float, vp, sz, vp]
        L.acx_reconstruct_adamw.restype = ctypes.c_int
        L.acx_reconstruct_adamw.argtypes = [dp, vp, vp, vp, vp, vp, ctypes.POINTER(acx_adamw_params), vp, sz, vp]
        L.acx_lowrank_adamw.restype = ctypes.c_int
        L.acx_lowrank_adamw.argtypes = [dp, vp, vp, vp, vp, vp, ctypes.POINTER(acx_adamw_params), vp, sz, vp]
        L.acx_rsvd_factor.restype, L.acx_rsvd_factor.argtypes = ctypes.c_int, [dp, vp, vp, vp, vp, sz, vp]
        L.acx_linear_fwd_bias.restype, L.acx_linear_fwd_bias.argtypes = ctypes.c_int, [dp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.acx_bias_grad.restype, L.acx_bias_grad.argtypes = ctypes.c_int, [dp, vp, vp, vp, sz, vp]
        L.acx_linear_bwd_bias.restype, L.acx_linear_bwd_bias.argtypes = ctypes.c_int, [dp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.acx_sketch_materialize.restype, L.acx_sketch_materialize.argtypes = ctypes.c_int, [dp, vp, vp]
        L.acx_last_device_status.restype, L.acx_last_device_status.argtypes = ctypes.c_int, [vp]
        L.acx_debug_expired_wait.restype, L.acx_debug_expired_wait.argtypes = ctypes.c_int, [ctypes.c_uint64, vp]
        L.acx_debug_force_gemm_mode.restype, L.acx_debug_force_gemm_mode.argtypes = ctypes.c_int, [ctypes.c_int]
        L.acx_status_string.restype, L.acx_status_string.argtypes = ctypes.c_char_p, [ctypes.c_int]
        L.acx_version.restype, L.acx_version.argtypes = ctypes.c_int, []
        L.acx_kernel_launches.restype, L.acx_kernel_launches.argtypes = ctypes.c_ulonglong, []
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().acx_status_string(int(status)).decode()


def acx_version() -> int:
    return lib().acx_version()


def acx_kernel_launches() -> int:
    return int(lib().acx_kernel_launches())


def make_desc(tokens: int, d_in: int, d_out: int, r: int, seed: int, dtype) -> acx_desc:
    """dtype: torch.float32 / torch.bfloat16 or "f32" / "bf16"."""
    code = {torch.float32: ACX_F32, torch.bfloat16: ACX_BF16, "f32": ACX_F32, "bf16": ACX_BF16}[dtype]
    return acx_desc(ctypes.sizeof(acx_desc), 0, tokens, d_in, d_out, r, code, seed & 0xFFFFFFFFFFFFFFFF)


def io_torch_dtype(desc: acx_desc):
    return torch.bfloat16 if desc.io_dtype == ACX_BF16 else torch.float32


def _ptr(t: Optional[torch.Tensor], shape: Tuple[int, ...], dtype, name: str):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous() or t.dtype != dtype or tuple(t.shape) != tuple(shape):
        raise ValueError("%s must be a contiguous CUDA tensor of shape %s and dtype %s (got %s %s on %s)"
                         % (name, tuple(shape), dtype, tuple(t.shape), t.dtype, t.device))
    return ctypes.c_void_p(t.data_ptr())


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)  # the handle without building a Stream object


def _stream(stream) -> ctypes.c_void_p:
    if stream is not None:
        return ctypes.c_void_p(stream.cuda_stream)
    if _raw_stream is not None:
        return ctypes.c_void_p(_raw_stream(torch.cuda.current_device()))
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, where: str):
    if status != ACX_OK:
        raise AcxError(status, where)


def acx_workspace_bytes(desc: acx_desc, op: int) -> int:
    return int(lib().acx_workspace_bytes(ctypes.byref(desc), op))


def alloc_workspace(desc: acx_desc, op: int, device="cuda") -> Optional[torch.Tensor]:
    n = acx_workspace_bytes(desc, op)
    return torch.empty(n, dtype=torch.uint8, device=device) if n else None


def _ws(ws: Optional[torch.Tensor]):
    if ws is None:
        return None, 0
    if not ws.is_cuda or not ws.is_contiguous():
        raise ValueError("workspace must be a contiguous CUDA tensor")
    return ctypes.c_void_p(ws.data_ptr()), ws.numel() * ws.element_size()


def acx_linear_fwd(desc: acx_desc, X, W, Y, XS, ws=None, stream=None) -> None:
    dt = io_torch_dtype(desc)
    wp, wn = _ws(ws)
    _check(lib().acx_linear_fwd(ctypes.byref(desc), _ptr(X, (desc.tokens, desc.d_in), dt, "X"),
                                _ptr(W, (desc.d_out, desc.d_in), dt, "W"),
                                _ptr(Y, (desc.tokens, desc.d_out), dt, "Y"),
                                _ptr(XS, (desc.tokens, desc.r), dt, "XS"), wp, wn, _stream(stream)), "acx_linear_fwd")


def acx_linear_fwd_v(desc: acx_desc, X, W, Vt, Y, XV, ws=None, stream=None) -> None:
    """Y = X W^T and XV = X V for a second factor given in memory as Vt (r x d_in)."""
    dt = io_torch_dtype(desc)
    wp, wn = _ws(ws)
    _check(lib().acx_linear_fwd_v(ctypes.byref(desc), _ptr(X, (desc.tokens, desc.d_in), dt, "X"),
                                  _ptr(W, (desc.d_out, desc.d_in), dt, "W"),
                                  _ptr(Vt, (desc.r, desc.d_in), dt, "Vt"),
                                  _ptr(Y, (desc.tokens, desc.d_out), dt, "Y"),
                                  _ptr(XV, (desc.tokens, desc.r), dt, "XV"), wp, wn, _stream(stream)), "acx_linear_fwd_v")


def acx_linear_bwd(desc: acx_desc, G_out, W, XS, dX, dW_A, ws=None, stream=None) -> None:
    dt = io_torch_dtype(desc)
    wp, wn = _ws(ws)
    _check(lib().acx_linear_bwd(ctypes.byref(desc), _ptr(G_out, (desc.tokens, desc.d_out), dt, "G_out"),
                                _ptr(W, (desc.d_out, desc.d_in), dt, "W"),
                                _ptr(XS, (desc.tokens, desc.r), dt, "XS"),
                                _ptr(dX, (desc.tokens, desc.d_in), dt, "dX"),
                                _ptr(dW_A, (desc.d_out, desc.r), torch.float32, "dW_A"), wp, wn, _stream(stream)),
           "acx_linear_bwd")


def acx_linear_bwd_factor_builtin_scratch(desc: acx_desc, G_out, XS, dW_A, stream=None) -> None:
    """dW_A = G_out^T XS (bf16 inputs) with the split-K partial sums kept in the scratch array that is
    built into the library, for callers that cannot allocate a workspace.  Calls on one device share that
    array: keep them ordered on the GPU.  Raises AcxError(ACX_ERR_SCRATCH_LIMIT) if the shape needs more
    than ACX_BUILTIN_SCRATCH_BYTES."""
    _check(lib().acx_linear_bwd_factor_builtin_scratch(
        ctypes.byref(desc), _ptr(G_out, (desc.tokens, desc.d_out), torch.bfloat16, "G_out"),
        _ptr(XS, (desc.tokens, desc.r), torch.bfloat16, "XS"),
        _ptr(dW_A, (desc.d_out, desc.r), torch.float32, "dW_A"), _stream(stream)),
        "acx_linear_bwd_factor_builtin_scratch")


def acx_reconstruct(desc: acx_desc, dW_A, dW, beta: float = 0.0, ws=None, stream=None) -> None:
    wp, wn = _ws(ws)
    _check(lib().acx_reconstruct(ctypes.byref(desc), _ptr(dW_A, (desc.d_out, desc.r), torch.float32, "dW_A"),
                                 _ptr(dW, (desc.d_out, desc.d_in), torch.float32, "dW"),
                                 ctypes.c_float(beta), wp, wn, _stream(stream)), "acx_reconstruct")


def acx_reconstruct_v(desc: acx_desc, dW_A, Vt, dW, beta: float = 0.0, ws=None, stream=None) -> None:
    """dW = beta * dW + dW_A Vt for a second factor given in memory as Vt (r x d_in)."""
    wp, wn = _ws(ws)
    _check(lib().acx_reconstruct_v(ctypes.byref(desc), _ptr(dW_A, (desc.d_out, desc.r), torch.float32, "dW_A"),
                                   _ptr(Vt, (desc.r, desc.d_in), io_torch_dtype(desc), "Vt"),
                                   _ptr(dW, (desc.d_out, desc.d_in), torch.float32, "dW"),
                                   ctypes.c_float(beta), wp, wn, _stream(stream)), "acx_reconstruct_v")


def acx_reconstruct_adamw(desc: acx_desc, dW_A, W, m, v, W_lp=None, *, step: int, lr: float, beta1: float = 0.9,
                          beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.0, ws=None, stream=None) -> None:
    """One AdamW step on fp32 master weights W (moments m, v) with the gradient dW_A S^T, which is never written out.
    W_lp (bfloat16, optional) receives the updated weights rounded for the next forward pass."""
    hp = acx_adamw_params(ctypes.sizeof(acx_adamw_params), step, lr, beta1, beta2, eps, weight_decay)
    shape = (desc.d_out, desc.d_in)
    wp, wn = _ws(ws)
    _check(lib().acx_reconstruct_adamw(ctypes.byref(desc), _ptr(dW_A, (desc.d_out, desc.r), torch.float32, "dW_A"),
                                       _ptr(W, shape, torch.float32, "W"), _ptr(m, shape, torch.float32, "m"),
                                       _ptr(v, shape, torch.float32, "v"), _ptr(W_lp, shape, torch.bfloat16, "W_lp"),
                                       ctypes.byref(hp), wp, wn, _stream(stream)), "acx_reconstruct_adamw")


def acx_lowrank_adamw(desc: acx_desc, dW_A, m_A, v_A, W, Vt=None, *, step: int, lr: float, beta1: float = 0.9,
                      beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.0, ws=None, stream=None) -> None:
    """One GaLore-style step: Adam moments m_A, v_A kept for the gradient factor dW_A (d_out x r), the normalised step
    projected back through V^T (Vt, or the seeded sketch when Vt is None) into the fp32 weights W."""
    hp = acx_adamw_params(ctypes.sizeof(acx_adamw_params), step, lr, beta1, beta2, eps, weight_decay)
    fshape = (desc.d_out, desc.r)
    wp, wn = _ws(ws)
    _check(lib().acx_lowrank_adamw(ctypes.byref(desc), _ptr(dW_A, fshape, torch.float32, "dW_A"),
                                   _ptr(m_A, fshape, torch.float32, "m_A"), _ptr(v_A, fshape, torch.float32, "v_A"),
                                   _ptr(Vt, (desc.r, desc.d_in), torch.bfloat16, "Vt"),
                                   _ptr(W, (desc.d_out, desc.d_in), torch.float32, "W"),
                                   ctypes.byref(hp), wp, wn, _stream(stream)), "acx_lowrank_adamw")


def acx_linear_fwd_bias(desc: acx_desc, X, W, bias, Y, XS, ws=None, stream=None) -> None:
    """Y = X W^T + bias (one bias vector of length d_out, bf16) and XS = X S."""
    dt = io_torch_dtype(desc)
    wp, wn = _ws(ws)
    _check(lib().acx_linear_fwd_bias(ctypes.byref(desc), _ptr(X, (desc.tokens, desc.d_in), dt, "X"),
                                     _ptr(W, (desc.d_out, desc.d_in), dt, "W"), _ptr(bias, (desc.d_out,), dt, "bias"),
                                     _ptr(Y, (desc.tokens, desc.d_out), dt, "Y"),
                                     _ptr(XS, (desc.tokens, desc.r), dt, "XS"), wp, wn, _stream(stream)), "acx_linear_fwd_bias")


def acx_bias_grad(desc: acx_desc, G_out, db, ws=None, stream=None) -> None:
    """db = column sums of G_out over the tokens (fp32)."""
    wp, wn = _ws(ws)
    _check(lib().acx_bias_grad(ctypes.byref(desc), _ptr(G_out, (desc.tokens, desc.d_out), io_torch_dtype(desc), "G_out"),
                               _ptr(db, (desc.d_out,), torch.float32, "db"), wp, wn, _stream(stream)), "acx_bias_grad")


def acx_linear_bwd_bias(desc: acx_desc, G_out, W, XS, dX, dW_A, db, ws=None, stream=None) -> None:
    """acx_linear_bwd plus the bias gradient db (column sums of G_out), summed inside the gradient-factor kernel."""
    dt = io_torch_dtype(desc)
    wp, wn = _ws(ws)
    _check(lib().acx_linear_bwd_bias(ctypes.byref(desc), _ptr(G_out, (desc.tokens, desc.d_out), dt, "G_out"),
                                     _ptr(W, (desc.d_out, desc.d_in), dt, "W"), _ptr(XS, (desc.tokens, desc.r), dt, "XS"),
                                     _ptr(dX, (desc.tokens, desc.d_in), dt, "dX"),
                                     _ptr(dW_A, (desc.d_out, desc.r), torch.float32, "dW_A"),
                                     _ptr(db, (desc.d_out,), torch.float32, "db"), wp, wn, _stream(stream)), "acx_linear_bwd_bias")


def acx_rsvd_factor(desc: acx_desc, X, U, Vt, ws=None, stream=None) -> None:
    """Vt = (U^T U)^-1 U^T X (r x d_in): the second factor of the randomized-SVD compressor for the stored sketch U = X S."""
    dt = io_torch_dtype(desc)
    wp, wn = _ws(ws)
    _check(lib().acx_rsvd_factor(ctypes.byref(desc), _ptr(X, (desc.tokens, desc.d_in), dt, "X"),
                                 _ptr(U, (desc.tokens, desc.r), dt, "U"), _ptr(Vt, (desc.r, desc.d_in), dt, "Vt"),
                                 wp, wn, _stream(stream)), "acx_rsvd_factor")


def acx_sketch_materialize(desc: acx_desc, S_out, stream=None) -> None:
    _check(lib().acx_sketch_materialize(ctypes.byref(desc), _ptr(S_out, (desc.d_in, desc.r), io_torch_dtype(desc), "S_out"),
                                        _stream(stream)), "acx_sketch_materialize")


def acx_debug_expired_wait(limit_ns: int, stream=None) -> None:
    """Launches a warp whose bounded wait runs out after limit_ns (test of the time-out reporting path)."""
    _check(lib().acx_debug_expired_wait(int(limit_ns), _stream(stream)), "acx_debug_expired_wait")


def acx_debug_force_gemm_mode(mode: int) -> None:
    """Test/debug: 0 = the cost models pick the tile shape of the forward and dX, 1..4 = force a GEMM mode."""
    _check(lib().acx_debug_force_gemm_mode(int(mode)), "acx_debug_force_gemm_mode")


def acx_last_device_status(stream=None) -> int:
    return int(lib().acx_last_device_status(_stream(stream)))
