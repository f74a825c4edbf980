"""GPU parity of the explicit-factor calls (Section 4: a stored activation X^ = U V^T with V given in memory,
as a subspace method such as the randomized SVD of Section 5 produces it): acx_linear_fwd_v and
acx_reconstruct_v against the oracle's forward, backward and reconstruct evaluated with that V."""
import numpy as np
import pytest
import torch

from oracle import linear as ol
from paper_2605_01255_b200 import binding as B
from paper_2605_01255_b200 import inputs as I

from _harness import TOL, TOL_DERIVED, GpuLinear, assert_parity, raw_bits, to_device, to_host

pytestmark = pytest.mark.gpu

# (m, d_in, d_out, r): several forward tile classes, ragged rows and columns, r off the 64-column chunk,
# reconstruct slices whose last 64-column chunk is partly or wholly past d_in
SHAPES = [
    (300, 256, 192, 16),
    (777, 520, 264, 48),
    (1500, 1024, 1000, 96),
    (2049, 768, 640, 128),
    (513, 2056, 384, 160),
    (1024, 1000, 1536, 256),
    (1, 64, 8, 64),
]


def _run(m, d_in, d_out, r, dtype, seed):
    X = I.gaussian((m, d_in), seed + 1, 1.0, dtype)
    W = I.gaussian((d_out, d_in), seed + 2, 0.02, dtype)
    G = I.gaussian((m, d_out), seed + 3, 1.0, dtype)
    Vt = I.orthonormal_rows(r, d_in, seed + 4, dtype)
    lin = GpuLinear(m, d_in, d_out, r, seed, dtype)
    Xd, Wd, Gd, Vd = (to_device(a, dtype) for a in (X, W, G, Vt))
    Y, XV = lin.empty(m, d_out), lin.empty(m, r)
    B.acx_linear_fwd_v(lin.desc, Xd, Wd, Vd, Y, XV, lin.ws_fwd)
    dX, A = lin.bwd(Gd, Wd, XV)
    dW = lin.empty(d_out, d_in, torch.float32)
    B.acx_reconstruct_v(lin.desc, A, Vd, dW, 0.0, lin.ws_rec)
    lin.check_status()
    V = Vt.T
    Y0, U0 = ol.linear_fwd(X, W, V)
    XVh, Ah = to_host(XV), to_host(A)
    dX0, A0 = ol.linear_bwd(G, W, XVh)
    tol, ctx = min(TOL[dtype], TOL_DERIVED[dtype]), (m, d_in, d_out, r, dtype)
    out_kind = "bf16" if dtype == "bf16" else "acc"
    assert_parity("Y", to_host(Y), Y0, out_kind, tol, ctx)
    assert_parity("XV", XVh, U0, out_kind, tol, ctx)
    assert_parity("dX", to_host(dX), dX0, out_kind, tol, ctx)
    assert_parity("A", Ah, A0, "factor" if dtype == "bf16" else "acc", tol, ctx)
    assert_parity("dW", to_host(dW), ol.reconstruct(Ah, V), "dw" if dtype == "bf16" else "acc", tol, ctx)
    return lin, (Xd, Wd, Gd, Vd), (Y, XV, A, dW)


@pytest.mark.parametrize("m,d_in,d_out,r", SHAPES)
def test_explicit_v_bf16(m, d_in, d_out, r):
    lin, (Xd, Wd, Gd, Vd), (Y, XV, A, dW) = _run(m, d_in, d_out, r, "bf16", 31 * m + r)
    # accumulation into an existing gradient, and the same bits on a second call
    dW2 = dW.clone()
    B.acx_reconstruct_v(lin.desc, A, Vd, dW2, 1.0, lin.ws_rec)
    assert ol.rel_frobenius(to_host(dW2), 2.0 * to_host(dW)) <= 1e-6
    Y2, XV2 = lin.empty(m, d_out), lin.empty(m, r)
    B.acx_linear_fwd_v(lin.desc, Xd, Wd, Vd, Y2, XV2, lin.ws_fwd)
    assert np.array_equal(raw_bits(Y), raw_bits(Y2)) and np.array_equal(raw_bits(XV), raw_bits(XV2))
    lin.check_status()


@pytest.mark.parametrize("m,d_in,d_out,r", SHAPES[:4])
def test_explicit_v_fp32(m, d_in, d_out, r):
    _run(m, d_in, d_out, r, "f32", 17 * m + r)


def test_explicit_v_is_exact_on_the_row_space():
    """If the rows of X lie in the span of V's columns, X^ = (X V) V^T = X and the rebuilt gradient is the
    uncompressed G^T X (Definition 3.1 with a lossless compressor)."""
    m, d_in, d_out, r = 1024, 512, 384, 64
    Vt = I.orthonormal_rows(r, d_in, 5, "f32")
    C = I.gaussian((m, r), 6, 1.0, "f32")
    X = (C.astype(np.float64) @ Vt.astype(np.float64)).astype(np.float32)
    W = I.gaussian((d_out, d_in), 7, 0.02, "f32")
    G = I.gaussian((m, d_out), 8, 1.0, "f32")
    lin = GpuLinear(m, d_in, d_out, r, 0, "f32")
    Xd, Wd, Gd, Vd = (to_device(a, "f32") for a in (X, W, G, Vt))
    Y, XV = lin.empty(m, d_out), lin.empty(m, r)
    B.acx_linear_fwd_v(lin.desc, Xd, Wd, Vd, Y, XV, lin.ws_fwd)
    _, A = lin.bwd(Gd, Wd, XV)
    dW = lin.empty(d_out, d_in, torch.float32)
    B.acx_reconstruct_v(lin.desc, A, Vd, dW, 0.0, lin.ws_rec)
    lin.check_status()
    assert ol.rel_frobenius(to_host(dW), ol.exact_weight_grad(G, X)) <= 1e-5


def test_explicit_v_rejects_missing_arguments():
    lin = GpuLinear(64, 64, 64, 16, 0, "bf16")
    X, W, Vt = (torch.zeros(s, dtype=torch.bfloat16, device="cuda") for s in ((64, 64), (64, 64), (16, 64)))
    Y, A = lin.empty(64, 64), torch.zeros(64, 16, device="cuda")
    with pytest.raises(B.AcxError) as e:
        B.acx_linear_fwd_v(lin.desc, X, W, Vt, Y, None)
    assert e.value.status == B.ACX_ERR_INVALID_ARG
    with pytest.raises(B.AcxError) as e:
        B.acx_reconstruct_v(lin.desc, A, None, lin.empty(64, 64, torch.float32), 0.0, lin.ws_rec)
    assert e.value.status == B.ACX_ERR_INVALID_ARG
