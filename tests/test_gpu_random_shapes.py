"""GPU parity on seeded random valid shapes: exercises the tile-shape planners (forward tile classes, dX tile
shapes, factor splits through cluster or workspace, reconstruct slices) away from the round LLaMA sizes."""
import numpy as np
import pytest

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import inputs as I

from _harness import TOL, TOL_DERIVED, GpuLinear, raw_bits, to_device, to_host

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
    errs = {"Y": ol.rel_frobenius(to_host(Y), Y0), "XS": ol.rel_frobenius(XSh, U0), "dX": ol.rel_frobenius(to_host(dX), dX0),
            "A": ol.rel_frobenius(to_host(A), A0), "dW": ol.rel_frobenius(to_host(dW), ol.reconstruct(to_host(A), S))}
    for k, v in errs.items():
        assert v <= TOL["bf16"] and v <= TOL_DERIVED["bf16"], (k, v, errs)
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
    errs = {"Y": ol.rel_frobenius(to_host(Y), Y0), "XS": ol.rel_frobenius(to_host(XS), U0), "dX": ol.rel_frobenius(to_host(dX), dX0),
            "A": ol.rel_frobenius(to_host(A), A0), "dW": ol.rel_frobenius(to_host(dW), ol.reconstruct(to_host(A), S))}
    for k, v in errs.items():
        assert v <= TOL["f32"] and v <= TOL_DERIVED["f32"], (k, v, errs)
