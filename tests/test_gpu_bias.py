"""GPU parity of the affine operator's calls (appendix, "Bias term"): bias added in the forward's epilogue, bias
gradient as the column sum of the output gradient."""
import numpy as np
import pytest
import torch

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import binding as B
from paper_2605_01255_b200 import inputs as I

from _harness import TOL_DERIVED, GpuLinear, raw_bits, to_device, to_host

pytestmark = pytest.mark.gpu

# ragged rows and columns, several tile classes, a d_out whose last 16-column group is half outside
SHAPES = [(777, 264, 136, 48), (2048, 896, 4864, 64), (1031, 72, 1000, 32), (4096, 1024, 1024, 128), (130, 512, 8, 256), (1, 64, 72, 16)]


@pytest.mark.parametrize("m,d_in,d_out,r", SHAPES)
@pytest.mark.parametrize("with_ws", [True, False])
def test_forward_with_bias(m, d_in, d_out, r, with_ws):
    seed = 3 * m + r
    X = I.gaussian((m, d_in), seed + 1, 1.0, "bf16")
    W = I.gaussian((d_out, d_in), seed + 2, 0.02, "bf16")
    b = I.gaussian((d_out,), seed + 3, 0.5, "bf16")
    lin = GpuLinear(m, d_in, d_out, r, seed, "bf16")
    Xd, Wd, bd = to_device(X, "bf16"), to_device(W, "bf16"), to_device(b, "bf16")
    Y, XS = lin.empty(m, d_out), lin.empty(m, r)
    B.acx_linear_fwd_bias(lin.desc, Xd, Wd, bd, Y, XS, lin.ws_fwd if with_ws else None)
    Y_only = lin.empty(m, d_out)
    B.acx_linear_fwd_bias(lin.desc, Xd, Wd, bd, Y_only, None, None)      # the plain GEMM's epilogue
    lin.check_status()
    S = osk.sketch_for_dtype(seed, d_in, r, "bf16")
    Y0, U0 = ol.linear_fwd_bias(X, W, S, b)
    assert ol.rel_frobenius(to_host(Y), Y0) <= TOL_DERIVED["bf16"]
    assert ol.rel_frobenius(to_host(XS), U0) <= TOL_DERIVED["bf16"]
    assert np.array_equal(raw_bits(Y), raw_bits(Y_only))
    # the bias enters before the rounding of Y: closer to the oracle than adding it to a rounded Y would be
    Y_plain, XS_plain = lin.fwd(Xd, Wd)
    assert np.array_equal(raw_bits(XS), raw_bits(XS_plain))
    assert np.max(np.abs(to_host(Y) - Y0)) <= np.max(np.abs(Y0)) * 2.0 ** -8


@pytest.mark.parametrize("m,d_out", [(777, 136), (16384, 3072), (4096, 4864), (33, 8), (5000, 1000)])
def test_bias_gradient(m, d_out):
    G = I.gaussian((m, d_out), m + d_out, 1.0, "bf16")
    desc = B.make_desc(m, 64, d_out, 16, 0, "bf16")
    Gd = to_device(G, "bf16")
    ws = B.alloc_workspace(desc, B.ACX_OP_BIAS_GRAD)
    db = torch.full((d_out,), float("nan"), device="cuda")
    B.acx_bias_grad(desc, Gd, db, ws)
    db2 = torch.full((d_out,), float("nan"), device="cuda")
    B.acx_bias_grad(desc, Gd, db2, ws)
    assert B.acx_last_device_status() == B.ACX_OK
    want = ol.bias_grad(G)
    # fp32 sums of m terms of size one: the error grows like sqrt(m) * 2^-24 against a result of size sqrt(m)
    assert np.linalg.norm(to_host(db) - want) <= 1e-5 * np.linalg.norm(want) + 1e-4
    assert np.array_equal(raw_bits(db), raw_bits(db2))


def test_bias_argument_checks():
    desc = B.make_desc(64, 64, 64, 16, 0, "bf16")
    X = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.AcxError) as e:
        B.acx_linear_fwd_bias(desc, X, X, None, X.clone(), None)
    assert e.value.status == B.ACX_ERR_INVALID_ARG
    with pytest.raises(B.AcxError) as e:
        B.acx_bias_grad(desc, X, torch.zeros(64, device="cuda"), None)
    assert e.value.status == B.ACX_ERR_WORKSPACE
    d0 = B.make_desc(0, 64, 64, 16, 0, "bf16")
    db = torch.full((64,), 7.0, device="cuda")
    B.acx_bias_grad(d0, torch.zeros(0, 64, dtype=torch.bfloat16, device="cuda"), db, None)
    assert torch.count_nonzero(db).item() == 0


# cluster reduction (few row tiles, many tokens per range), workspace reduction (d_out = 8: one tile), ragged everything
BWD_SHAPES = [(16384, 256, 3072, 128), (4096, 896, 4864, 64), (777, 264, 136, 48), (130, 512, 8, 256), (20000, 128, 264, 32),
              (1031, 72, 1000, 32)]


@pytest.mark.parametrize("m,d_in,d_out,r", BWD_SHAPES)
def test_backward_with_fused_bias_gradient(m, d_in, d_out, r):
    seed = 5 * m + r
    W = I.gaussian((d_out, d_in), seed + 2, 0.02, "bf16")
    G = I.gaussian((m, d_out), seed + 3, 1.0, "bf16")
    XSh = I.gaussian((m, r), seed + 4, 1.0, "bf16")
    lin = GpuLinear(m, d_in, d_out, r, seed, "bf16")
    Gd, Wd, XS = to_device(G, "bf16"), to_device(W, "bf16"), to_device(XSh, "bf16")
    dX0, A0 = lin.bwd(Gd, Wd, XS)                                   # the plain backward
    ws = B.alloc_workspace(lin.desc, B.ACX_OP_BWD_BIAS)
    outs = []
    for _ in range(2):
        dX, A = lin.empty(m, d_in), lin.empty(d_out, r, torch.float32)
        db = torch.full((d_out,), float("nan"), device="cuda")
        B.acx_linear_bwd_bias(lin.desc, Gd, Wd, XS, dX, A, db, ws)
        outs.append((dX, A, db))
    lin.check_status()
    dX, A, db = outs[0]
    # dX and A are the plain backward's, bit for bit; db is the oracle's column sum; everything repeats bit for bit
    assert np.array_equal(raw_bits(dX), raw_bits(dX0)) and np.array_equal(raw_bits(A), raw_bits(A0))
    want = ol.bias_grad(G)
    assert np.linalg.norm(to_host(db) - want) <= 1e-5 * np.linalg.norm(want) + 1e-4
    for a, b in zip(outs[0], outs[1]):
        assert np.array_equal(raw_bits(a), raw_bits(b))
    # without dX
    A2, db2 = lin.empty(d_out, r, torch.float32), torch.full((d_out,), float("nan"), device="cuda")
    B.acx_linear_bwd_bias(lin.desc, Gd, None, XS, None, A2, db2, ws)
    assert np.array_equal(raw_bits(A2), raw_bits(A0)) and np.array_equal(raw_bits(db2), raw_bits(db))
    with pytest.raises(B.AcxError) as e:
        B.acx_linear_bwd_bias(lin.desc, Gd, Wd, XS, dX, A, db, None)
    assert e.value.status == B.ACX_ERR_WORKSPACE
