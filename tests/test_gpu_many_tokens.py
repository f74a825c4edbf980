"""GPU parity with many more tokens than the benchmark shapes have (hundreds of row tiles per N-tile, token counts that are
not a multiple of anything, token ranges of the gradient factor at their longest) and with feature dimensions far wider than
the benchmark's: every output against the oracle."""
import numpy as np
import pytest

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import binding as B
from paper_2605_01255_b200 import inputs as I

from _harness import ELEM_TOL, TOL, TOL_DERIVED, GpuLinear, assert_parity, elementwise_err, raw_bits, to_device, to_host

pytestmark = pytest.mark.gpu

# The gradient factor sums a token range in the tensor core's fp32 accumulator, 16 tokens per add, each add truncated: the
# error grows with the adds of one range, about (2/3) n 2^-24 of the magnitude (see ELEM_TOL["factor"]).  The library keeps a
# range to at most 65 536 tokens where the split count allows (n = 4096: 1.6e-4); twice that is the bound for a long problem.
LONG_RANGE_FACTOR_TOL = 2 * (2.0 / 3.0) * 4096 * 2.0 ** -24


@pytest.mark.parametrize("m,d_in,d_out,r,long_ranges", [(200003, 128, 264, 32, False), (1000003, 64, 72, 16, True)])
def test_many_tokens(m, d_in, d_out, r, long_ranges):
    seed = 17 + r
    X = I.gaussian((m, d_in), seed + 1, 1.0, "bf16")
    W = I.gaussian((d_out, d_in), seed + 2, 0.02, "bf16")
    G = I.gaussian((m, d_out), seed + 3, 1.0, "bf16")
    lin = GpuLinear(m, d_in, d_out, r, seed, "bf16")
    Xd, Wd, Gd = to_device(X, "bf16"), to_device(W, "bf16"), to_device(G, "bf16")
    Y, XS = lin.fwd(Xd, Wd)
    Y_no, XS_no = lin.empty(m, d_out), lin.empty(m, r)
    B.acx_linear_fwd(lin.desc, Xd, Wd, Y_no, XS_no, None)      # the sketch generated inside the GEMM
    dX, A = lin.bwd(Gd, Wd, XS)
    dW = lin.reconstruct(A)
    lin.check_status()
    assert np.array_equal(raw_bits(Y), raw_bits(Y_no)) and np.array_equal(raw_bits(XS), raw_bits(XS_no))
    S = osk.sketch_for_dtype(seed, d_in, r, "bf16")
    Y0, U0 = ol.linear_fwd(X, W, S)
    XSh = to_host(XS)
    dX0, A0 = ol.linear_bwd(G, W, XSh)
    tol, ctx = min(TOL["bf16"], TOL_DERIVED["bf16"]), (m, d_in, d_out, r)
    assert_parity("Y", to_host(Y), Y0, "bf16", tol, ctx)
    assert_parity("XS", XSh, U0, "bf16", tol, ctx)
    assert_parity("dX", to_host(dX), dX0, "bf16", tol, ctx)
    Ah = to_host(A)
    if long_ranges:
        assert ol.rel_frobenius(Ah, A0) <= LONG_RANGE_FACTOR_TOL, ("A", ol.rel_frobenius(Ah, A0), ctx)
        assert elementwise_err(Ah, A0) <= LONG_RANGE_FACTOR_TOL, ("A", elementwise_err(Ah, A0), ctx)
        assert elementwise_err(Ah, A0) > ELEM_TOL["factor"] / 50       # (and the measured error is of the expected kind, not zero)
    else:
        assert_parity("A", Ah, A0, "factor", tol, ctx)
    assert_parity("dW", to_host(dW), ol.reconstruct(Ah, S), "dw", tol, ctx)
    dX2, A2 = lin.bwd(Gd, Wd, XS)
    assert np.array_equal(raw_bits(dX), raw_bits(dX2)) and np.array_equal(raw_bits(A), raw_bits(A2))


@pytest.mark.parametrize("m,d_in,d_out,r", [(300, 32768, 136, 256), (300, 136, 32768, 32), (2049, 256, 8, 256), (77, 16384, 16384, 128)])
def test_wide_feature_dimensions(m, d_in, d_out, r):
    """512 k-blocks per tile, 129 N-tiles, the widest sketch on the narrowest input that takes it, and a square 16384 layer."""
    seed = 5 + r
    X = I.gaussian((m, d_in), seed + 1, 1.0, "bf16")
    W = I.gaussian((d_out, d_in), seed + 2, 0.02, "bf16")
    G = I.gaussian((m, d_out), seed + 3, 1.0, "bf16")
    lin = GpuLinear(m, d_in, d_out, r, seed, "bf16")
    Xd, Wd, Gd = to_device(X, "bf16"), to_device(W, "bf16"), to_device(G, "bf16")
    Y, XS = lin.fwd(Xd, Wd)
    Y_no, XS_no = lin.empty(m, d_out), lin.empty(m, r)
    B.acx_linear_fwd(lin.desc, Xd, Wd, Y_no, XS_no, None)
    dX, A = lin.bwd(Gd, Wd, XS)
    dW = lin.reconstruct(A)
    lin.check_status()
    assert np.array_equal(raw_bits(Y), raw_bits(Y_no)) and np.array_equal(raw_bits(XS), raw_bits(XS_no))
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
