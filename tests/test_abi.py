"""CPU checks of the C ABI: the library builds, loads, exports what include/acx.h declares, and
rejects bad arguments before touching the GPU.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

from paper_2605_01255_b200 import binding as B
from paper_2605_01255_b200 import build as acx_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    acx_build.build()
    return B.lib()


def _declared():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            names += re.findall(r"ACX_API\s+[\w\s\*]+?\b(acx_\w+)\s*\(", text)
    return names


def test_every_declared_symbol_is_exported(L):
    names = _declared()
    assert len(names) >= 8
    for n in names:
        assert hasattr(L, n), n
    assert set(B.EXPORTS) <= set(names)


def test_version_and_strings(L):
    assert B.acx_version() == 100
    seen = set()
    for code in range(7):
        s = B.status_string(code)
        assert s and s not in seen
        seen.add(s)
    assert "unknown" in B.status_string(99)


def test_desc_layout_matches_header():
    # 2*u32 + 3*i64 + 2*i32 + u64
    assert ctypes.sizeof(B.acx_desc) == 48
    assert B.acx_desc.seed.offset == 40 and B.acx_desc.r.offset == 32 and B.acx_desc.tokens.offset == 8


def _call_fwd(L, d, x=0x1000, w=0x2000, y=0x3000, xs=0x4000):
    # fake addresses: validation must fail before anything could dereference them
    return L.acx_linear_fwd(ctypes.byref(d), x, w, y, xs, None, 0, None)


def test_argument_validation_happens_on_the_host(L):
    good = dict(tokens=64, d_in=64, d_out=64, r=16, seed=1, dtype="bf16")
    d = B.make_desc(**good)
    d.struct_size = 40
    assert _call_fwd(L, d) == B.ACX_ERR_INVALID_ARG
    d = B.make_desc(**good); d.sketch_kind = 3
    assert _call_fwd(L, d) == B.ACX_ERR_INVALID_ARG
    d = B.make_desc(**good); d.io_dtype = 7
    assert _call_fwd(L, d) == B.ACX_ERR_INVALID_ARG
    assert L.acx_linear_fwd(None, 0x1000, 0x2000, 0x3000, 0x4000, None, 0, None) == B.ACX_ERR_INVALID_ARG
    for bad in (dict(r=8), dict(r=24), dict(r=272), dict(d_in=60), dict(d_out=4), dict(tokens=-1), dict(r=128, d_in=64)):
        d = B.make_desc(**{**good, **bad})
        assert _call_fwd(L, d) == B.ACX_ERR_UNSUPPORTED_SHAPE, bad
        assert B.acx_workspace_bytes(d, B.ACX_OP_BWD) == 0
    # fp32 path: its 64 x 64 output tiles are numbered along one grid dimension (2^31 - 1 of them at most); a token count
    # beyond 65535 row tiles is fine, a tile count that does not fit is refused here, before any launch
    d = B.make_desc(**{**good, "dtype": "f32", "tokens": (1 << 31) - 1, "d_out": 1 << 20})
    assert _call_fwd(L, d) == B.ACX_ERR_UNSUPPORTED_SHAPE
    d = B.make_desc(**{**good, "dtype": "f32", "tokens": 5_000_000})
    assert _call_fwd(L, d, x=0) == B.ACX_ERR_INVALID_ARG      # the shape itself is accepted: the next check fires
    d = B.make_desc(**good)
    assert _call_fwd(L, d, x=0) == B.ACX_ERR_INVALID_ARG
    assert _call_fwd(L, d, y=0x3008) == B.ACX_ERR_ALIGNMENT
    assert L.acx_linear_bwd(ctypes.byref(d), 0x1000, 0x2000, 0x3000, 0x4004, 0x5000, None, 0, None) == B.ACX_ERR_ALIGNMENT
    assert L.acx_linear_bwd(ctypes.byref(d), 0x1000, 0x2000, None, 0x4000, 0x5000, None, 0, None) == B.ACX_ERR_INVALID_ARG
    assert L.acx_reconstruct(ctypes.byref(d), None, 0x1000, 0.0, 0x3000, 1 << 20, None) == B.ACX_ERR_INVALID_ARG
    assert L.acx_reconstruct(ctypes.byref(d), 0x1000, 0x2000, float("nan"), 0x3000, 1 << 20, None) == B.ACX_ERR_INVALID_ARG
    assert L.acx_reconstruct(ctypes.byref(d), 0x1000, 0x2000, 0.0, 0x3004, 1 << 20, None) == B.ACX_ERR_ALIGNMENT
    assert L.acx_sketch_materialize(ctypes.byref(d), 0x1001, None) == B.ACX_ERR_ALIGNMENT


def test_workspace_contract(L):
    big = B.make_desc(16384, 3072, 3072, 128, 0, "bf16")
    need = B.acx_workspace_bytes(big, B.ACX_OP_BWD)
    assert need % 16 == 0
    if need:
        # too small a workspace is refused on the host
        assert L.acx_linear_bwd(ctypes.byref(big), 0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, need - 16, None) == B.ACX_ERR_WORKSPACE
        assert L.acx_linear_bwd(ctypes.byref(big), 0x1000, 0x2000, 0x3000, 0x4000, 0x5000, None, 0, None) == B.ACX_ERR_WORKSPACE
    # reconstruct (bf16): room for the gradient factor split into two bfloat16 terms and for S^T in bfloat16
    need = B.acx_workspace_bytes(big, B.ACX_OP_RECONSTRUCT)
    assert need == 3072 * 128 * 4 + 128 * 3072 * 2
    assert L.acx_reconstruct(ctypes.byref(big), 0x1000, 0x2000, 0.0, 0x3000, need - 16, None) == B.ACX_ERR_WORKSPACE
    assert L.acx_reconstruct(ctypes.byref(big), 0x1000, 0x2000, 0.0, None, 0, None) == B.ACX_ERR_WORKSPACE
    assert B.acx_workspace_bytes(B.make_desc(512, 256, 256, 16, 0, "f32"), B.ACX_OP_RECONSTRUCT) == 0
    assert B.acx_workspace_bytes(big, 99) == 0
    # forward (bf16): room for S^T; a workspace that is given must be large enough (NULL selects in-kernel generation)
    need = B.acx_workspace_bytes(big, B.ACX_OP_FWD)
    assert need == 128 * 3072 * 2
    assert L.acx_linear_fwd(ctypes.byref(big), 0x1000, 0x2000, 0x3000, 0x4000, 0x5000, need - 16, None) == B.ACX_ERR_WORKSPACE
    assert B.acx_workspace_bytes(B.make_desc(512, 256, 256, 16, 0, "f32"), B.ACX_OP_FWD) == 0


def test_binding_rejects_wrong_tensors(L):
    import torch
    d = B.make_desc(8, 64, 64, 16, 0, "f32")
    x = torch.zeros(8, 64)
    with pytest.raises(ValueError):
        B.acx_linear_fwd(d, x, x, x, x)  # CPU tensors are not accepted: there is no host path
