"""GPU parity on seeded random valid shapes: exercises the tile-shape planners (forward tile classes, dX tile
shapes, factor splits through cluster or workspace, reconstruct slices) away from the round LLaMA sizes."""
import numpy as np
import pytest

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import inputs as I

from _harness import TOL, TOL_DERIVED, GpuLinear, assert_parity, raw_bits, to_device, to_host

pytestmark = pytest.mark.gpu


def _shapes(n, seed):
    g = np.random.Generator(np.random.Philox(seed))
    out = []
    while len(out) < n:
        r = int(g.choice([16, 32, 48, 64, 96, 128, 160, 256]))
        d_in = int(g.integers(max(r, 8) // 8, 160)) * 8
        d_out = int(g.integers(1, 160)) * 8
        m = int(g.choice([1, 7, 64, 129, 255, 300, 777, 1500, 2049, 3333]))
        if r <= d_in:
            out.append((m, d_in, d_out, r))
    return out


@pytest.mark.parametrize("m,d_in,d_out,r", _shapes(24, 2024))
def test_random_shape_bf16(m, d_in, d_out, r):
    seed = m * 7919 + d_in
    X = I.gaussian((m, d_in), seed + 1, 1.0, "bf16")
    W = I.gaussian((d_out, d_in), seed + 2, 0.02, "bf16")
    G = I.gaussian((m, d_out), seed + 3, 1.0, "bf16")
    lin = GpuLinear(m, d_in, d_out, r, seed, "bf16")
    Xd, Wd, Gd = to_device(X, "bf16"), to_device(W, "bf16"), to_device(G, "bf16")
    Y, XS = lin.fwd(Xd, Wd)
    dX, A = lin.bwd(Gd, Wd, XS)
    dW = lin.reconstruct(A)
    lin.check_status()
    S = osk.sketch_for_dtype(seed, d_in, r, "bf16")
    Y0, U0 = ol.linear_fwd(X, W, S)
    XSh = to_host(XS)
    dX0, A0 = ol.linear_bwd(G, W, XSh)
    tol, ctx = min(TOL["bf16"], TOL_DERIVED["bf16"]), (m, d_in, d_out, r)
    assert_parity("Y", to_host(Y), Y0, "bf16", tol, ctx)
    assert_parity("XS", XSh, U0, "bf16", tol, ctx)
    assert_parity("dX", to_host(dX), dX0, "bf16", tol, ctx)
    assert_parity("A", to_host(A), A0, "factor", tol, ctx)
    assert_parity("dW", to_host(dW), ol.reconstruct(to_host(A), S), "dw", tol, ctx)
    # same call again: same bits
    Y2, XS2 = lin.fwd(Xd, Wd)
    dX2, A2 = lin.bwd(Gd, Wd, XS2)
    for a, b in ((Y, Y2), (XS, XS2), (dX, dX2), (A, A2)):
        assert np.array_equal(raw_bits(a), raw_bits(b))


@pytest.mark.parametrize("m,d_in,d_out,r", _shapes(6, 77))
def test_random_shape_fp32(m, d_in, d_out, r):
    seed = m + d_out
    X = I.gaussian((m, d_in), seed + 1, 1.0, "f32")
    W = I.gaussian((d_out, d_in), seed + 2, 0.02, "f32")
    G = I.gaussian((m, d_out), seed + 3, 1.0, "f32")
    lin = GpuLinear(m, d_in, d_out, r, seed, "f32")
    Xd, Wd, Gd = to_device(X, "f32"), to_device(W, "f32"), to_device(G, "f32")
    Y, XS = lin.fwd(Xd, Wd)
    dX, A = lin.bwd(Gd, Wd, XS)
    dW = lin.reconstruct(A)
    lin.check_status()
    S = osk.sketch_for_dtype(seed, d_in, r, "f32")
    Y0, U0 = ol.linear_fwd(X, W, S)
    dX0, A0 = ol.linear_bwd(G, W, to_host(XS))
    tol, ctx = min(TOL["f32"], TOL_DERIVED["f32"]), (m, d_in, d_out, r)
    assert_parity("Y", to_host(Y), Y0, "acc", tol, ctx)
    assert_parity("XS", to_host(XS), U0, "acc", tol, ctx)
    assert_parity("dX", to_host(dX), dX0, "acc", tol, ctx)
    assert_parity("A", to_host(A), A0, "acc", tol, ctx)
    assert_parity("dW", to_host(dW), ol.reconstruct(to_host(A), S), "acc", tol, ctx)


@pytest.mark.parametrize("m,d_in,d_out,r", _shapes(10, 4242))
def test_random_shape_widened_calls(m, d_in, d_out, r):
    """Explicit second factor, bias, bias gradient, randomized-SVD factor and the low-rank optimizer step on the same
    random shapes (one linear layer each), against the oracle."""
    import torch
    from oracle import compressor as oc
    from oracle import optimizer as oo
    from paper_2605_01255_b200 import binding as B

    seed = m * 31 + d_out
    X = I.gaussian((m, d_in), seed + 1, 1.0, "bf16")
    W = I.gaussian((d_out, d_in), seed + 2, 0.02, "bf16")
    G = I.gaussian((m, d_out), seed + 3, 1.0, "bf16")
    b = I.gaussian((d_out,), seed + 4, 0.5, "bf16")
    Vt = I.orthonormal_rows(r, d_in, seed + 5, "bf16")
    lin = GpuLinear(m, d_in, d_out, r, seed, "bf16")
    Xd, Wd, Gd, bd, Vd = (to_device(a, "bf16") for a in (X, W, G, b, Vt))
    tol = TOL_DERIVED["bf16"]
    # explicit V: forward, backward, reconstruct
    Y, XV = lin.empty(m, d_out), lin.empty(m, r)
    B.acx_linear_fwd_v(lin.desc, Xd, Wd, Vd, Y, XV, lin.ws_fwd)
    _, A = lin.bwd(Gd, Wd, XV, want_dx=False)
    dW = lin.empty(d_out, d_in, torch.float32)
    B.acx_reconstruct_v(lin.desc, A, Vd, dW, 0.0, lin.ws_rec)
    Y0, U0 = ol.linear_fwd(X, W, Vt.T)
    assert_parity("Y", to_host(Y), Y0, "bf16", tol)
    assert_parity("XV", to_host(XV), U0, "bf16", tol)
    assert_parity("dW", to_host(dW), ol.reconstruct(to_host(A), Vt.T), "dw", tol)
    # bias in the forward, bias gradient
    Yb, XS = lin.empty(m, d_out), lin.empty(m, r)
    B.acx_linear_fwd_bias(lin.desc, Xd, Wd, bd, Yb, XS, lin.ws_fwd)
    S = osk.sketch_for_dtype(seed, d_in, r, "bf16")
    Yb0, US0 = ol.linear_fwd_bias(X, W, S, b)
    assert_parity("Yb", to_host(Yb), Yb0, "bf16", tol)
    assert_parity("XS", to_host(XS), US0, "bf16", tol)
    db = lin.empty(1, d_out, torch.float32)[0]
    B.acx_bias_grad(lin.desc, Gd, db, B.alloc_workspace(lin.desc, B.ACX_OP_BIAS_GRAD))
    want = ol.bias_grad(G)
    assert np.linalg.norm(to_host(db) - want) <= 1e-5 * np.linalg.norm(want) + 1e-4
    # randomized-SVD second factor of the stored sketch (needs as many tokens as the rank for a meaningful projection)
    if m >= 2 * r:
        Vr = lin.empty(r, d_in)
        B.acx_rsvd_factor(lin.desc, Xd, XS, Vr, B.alloc_workspace(lin.desc, B.ACX_OP_RSVD))
        Uh = to_host(XS)
        V0 = oc.second_factor(X, Uh, 2.0 ** -20)
        assert ol.rel_frobenius(Uh @ to_host(Vr), Uh @ V0) <= 1e-2
    # one low-rank AdamW step with the seeded sketch
    Wm = torch.from_numpy(W.astype(np.float32)).cuda()
    mA, vA = torch.zeros(d_out, r, device="cuda"), torch.zeros(d_out, r, device="cuda")
    _, As = lin.bwd(Gd, Wd, XS, want_dx=False)
    B.acx_lowrank_adamw(lin.desc, As, mA, vA, Wm, step=1, lr=1e-3, weight_decay=0.01, ws=lin.ws_rec)
    W1, m1, v1 = oo.lowrank_adamw_step(to_host(As), S, W.astype(np.float64), 0.0 * to_host(As), 0.0 * to_host(As), 1e-3, 0.9, 0.999,
                                       1e-8, 0.01, 1)
    assert ol.rel_frobenius(to_host(Wm) - W.astype(np.float64), W1 - W.astype(np.float64)) <= 1e-4
    assert ol.rel_frobenius(to_host(mA), m1) <= 2e-6
    lin.check_status()
