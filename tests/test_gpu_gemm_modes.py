"""Every tile shape of the forward and dX kernels on the same ragged problems: one CTA per tile of 128 or 256 rows, a pair
of CTAs (tcgen05.mma.cta_group::2) per tile of 256 or 512 rows.  The cost models would pick only one of them per shape, so
the test/debug override acx_debug_force_gemm_mode runs them all; every mode adds the products of a tile in the same order,
so Y, XS and dX must agree bit for bit between the modes, and each is checked against the oracle."""
import numpy as np
import pytest

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import binding as B
from paper_2605_01255_b200 import inputs as I

from _harness import TOL_DERIVED, GpuLinear, assert_parity, raw_bits, to_device, to_host

pytestmark = pytest.mark.gpu

# tokens not a multiple of 128 / 256 / 512, widths that leave partly filled tiles in both directions, every rank class
SHAPES = [(1000, 520, 776, 48), (2500, 1024, 1000, 128), (515, 264, 264, 16), (3333, 896, 1288, 64), (300, 2056, 520, 256),
          (4100, 512, 2048, 32)]


@pytest.fixture(autouse=True)
def _reset_mode():
    yield
    B.acx_debug_force_gemm_mode(0)


@pytest.mark.parametrize("m,d_in,d_out,r", SHAPES)
def test_all_gemm_modes_agree_and_match_the_oracle(m, d_in, d_out, r):
    seed = 13 * m + r
    X = I.gaussian((m, d_in), seed + 1, 1.0, "bf16")
    W = I.gaussian((d_out, d_in), seed + 2, 0.02, "bf16")
    G = I.gaussian((m, d_out), seed + 3, 1.0, "bf16")
    lin = GpuLinear(m, d_in, d_out, r, seed, "bf16")
    Xd, Wd, Gd = to_device(X, "bf16"), to_device(W, "bf16"), to_device(G, "bf16")
    S = osk.sketch_for_dtype(seed, d_in, r, "bf16")
    Y0, U0 = ol.linear_fwd(X, W, S)
    ref = None
    for mode in (1, 2, 3, 4):
        B.acx_debug_force_gemm_mode(mode)
        Y, XS = lin.fwd(Xd, Wd)                                   # sketch read from the workspace
        Y_gen, XS_gen = lin.empty(m, d_out), lin.empty(m, r)
        B.acx_linear_fwd(lin.desc, Xd, Wd, Y_gen, XS_gen, None)   # sketch generated inside the GEMM
        Y_plain, _ = lin.fwd(Xd, Wd, want_xs=False)
        dX, _ = lin.bwd(Gd, Wd, XS, want_a=False)
        lin.check_status()
        ctx = (m, d_in, d_out, r, "mode", mode)
        assert_parity("Y", to_host(Y), Y0, "bf16", TOL_DERIVED["bf16"], ctx)
        assert_parity("XS", to_host(XS), U0, "bf16", TOL_DERIVED["bf16"], ctx)
        dX0, _ = ol.linear_bwd(G, W, np.zeros((m, r)))
        assert_parity("dX", to_host(dX), dX0, "bf16", TOL_DERIVED["bf16"], ctx)
        bits = [raw_bits(t) for t in (Y, XS, dX)]
        for name, a, b in (("Y generated", Y_gen, Y), ("XS generated", XS_gen, XS), ("Y plain", Y_plain, Y)):
            assert np.array_equal(raw_bits(a), raw_bits(b)), (name, ctx)
        if ref is None:
            ref = bits
        else:
            for name, a, b in zip(("Y", "XS", "dX"), bits, ref):
                assert np.array_equal(a, b), (name, "differs from mode 1", ctx)
    with pytest.raises(B.AcxError):
        B.acx_debug_force_gemm_mode(9)
