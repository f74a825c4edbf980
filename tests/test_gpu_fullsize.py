"""Parity at the full sizes of the LLaMA-shaped configurations, in the launch configuration the benchmark
times (16384 tokens, bf16): outputs that depend on one token row (Y, XS, dX) are checked on sampled rows,
the gradient factor A completely, dW on sampled rows; plus properties that hold at any size."""
import numpy as np
import pytest

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import inputs as I

from _harness import TOL, TOL_DERIVED, GpuLinear, raw_bits, to_device, to_host

pytestmark = pytest.mark.gpu

CASES = [("llama3b_layer", 0, 128), ("llama3b_layer", 4, 128), ("llama3b_layer", 6, 128), ("llama3b_layer", 0, 256),
         ("llama3b_layer", 6, 32), ("llama1b_layer", 4, 128)]


@pytest.mark.parametrize("name,k,r", CASES)
def test_sampled_rows_at_full_size(name, k, r):
    wl = I.workload(name, r)
    lin = wl.linears[k]
    m = wl.tokens
    seed = I.sketch_seed(0, 0, lin.slot)
    X, W, G = I.make_x(wl, 0, lin), I.make_w(wl, 0, k), I.make_g(wl, 0, k)
    gl = GpuLinear(m, lin.d_in, lin.d_out, r, seed, "bf16")
    Xd, Wd, Gd = to_device(X, "bf16"), to_device(W, "bf16"), to_device(G, "bf16")
    Y, XS = gl.fwd(Xd, Wd)
    dX, A = gl.bwd(Gd, Wd, XS)
    dW = gl.reconstruct(A)
    gl.check_status()

    rows = np.unique(np.concatenate([np.arange(0, 8), np.arange(m - 8, m),
                                     np.random.Generator(np.random.Philox(9)).integers(0, m, 256)]))
    S = osk.sketch_for_dtype(seed, lin.d_in, r, "bf16")
    Y0, U0 = ol.linear_fwd(X[rows], W, S)
    XSh = to_host(XS)
    dX0, _ = ol.linear_bwd(G[rows], W, XSh[rows])   # dX depends on one token row
    _, A0 = ol.linear_bwd(G, W[:, :8], XSh)          # A needs every token (the dX of this call is not used)
    tol, tight = TOL["bf16"], TOL_DERIVED["bf16"]
    errs = {"Y": ol.rel_frobenius(to_host(Y[rows]), Y0), "XS": ol.rel_frobenius(XSh[rows], U0),
            "dX": ol.rel_frobenius(to_host(dX[rows]), dX0), "A": ol.rel_frobenius(to_host(A), A0)}
    orows = np.unique(np.concatenate([np.arange(0, 4), np.arange(lin.d_out - 4, lin.d_out),
                                      np.random.Generator(np.random.Philox(10)).integers(0, lin.d_out, 128)]))
    Ah = to_host(A)
    errs["dW"] = ol.rel_frobenius(to_host(dW[orows]), ol.reconstruct(Ah[orows], S))
    for key, v in errs.items():
        assert v <= tol and v <= tight, (key, v, errs)
    # every row of every output was written: no NaN canaries left
    for t in (Y, XS, dX, A, dW):
        assert bool(t.isfinite().all())
    # properties that hold at any size: Y and dX do not depend on the rank or the seed (Theorem 3.3(a))
    gl2 = GpuLinear(m, lin.d_in, lin.d_out, 16, seed + 1, "bf16")
    Y2, XS2 = gl2.fwd(Xd, Wd)
    dX2, _ = gl2.bwd(Gd, Wd, XS2)
    assert np.array_equal(raw_bits(Y2), raw_bits(Y)) and np.array_equal(raw_bits(dX2), raw_bits(dX))
