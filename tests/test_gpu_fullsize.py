"""Parity at the full sizes of the LLaMA-shaped configurations, in the launch configuration the benchmark
times (16384 tokens, bf16): outputs that depend on one token row (Y, XS, dX) are checked on sampled rows that
cover every 128-row block of the problem (so both halves of every 256-row tile and the last row are seen), the
gradient factor A completely, dW on sampled rows covering every 128-row block of d_out; plus properties that
hold at any size.  Both forward variants run: with the sketch written out once into the workspace and with the
sketch generated inside the GEMM (no workspace); their bits must agree."""
import numpy as np
import pytest

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import binding as B
from paper_2605_01255_b200 import inputs as I

from _harness import TOL, TOL_DERIVED, GpuLinear, assert_parity, raw_bits, to_device, to_host

pytestmark = pytest.mark.gpu

# (workload, linear index, rank).  The LLaMA-3B layer at every rank of its sweep and all seven linears of the
# LLaMA-1B layer (q, k, v, o share a shape but not their data).
CASES = ([("llama3b_layer", 0, 128), ("llama3b_layer", 3, 128), ("llama3b_layer", 4, 128), ("llama3b_layer", 6, 128),
          ("llama3b_layer", 0, 256), ("llama3b_layer", 4, 256), ("llama3b_layer", 6, 32), ("llama3b_layer", 0, 64),
          ("llama3b_layer", 5, 64), ("llama3b_layer", 6, 64), ("llama3b_layer", 4, 32)] +
         [("llama1b_layer", k, 128) for k in range(7)])


def block_rows(n, block, per_block, seed):
    """Sorted sample of rows of [0, n): `per_block` random rows of every `block`-row block, the first and last 8 rows."""
    g = np.random.Generator(np.random.Philox(seed))
    picks = [np.arange(0, min(8, n)), np.arange(max(0, n - 8), n)]
    for b0 in range(0, n, block):
        picks.append(b0 + g.integers(0, min(block, n - b0), per_block))
    return np.unique(np.concatenate(picks))


def check_linear_at_full_size(wl, k, r, layer=0, seed_base=0, full_a=True, rows_per_block=2, other_rank_check=True):
    lin = wl.linears[k]
    m = wl.tokens
    seed = I.sketch_seed(seed_base, layer, lin.slot)
    X, W, G = I.make_x(wl, layer, lin), I.make_w(wl, layer, k), I.make_g(wl, layer, k)
    gl = GpuLinear(m, lin.d_in, lin.d_out, r, seed, "bf16")
    Xd, Wd, Gd = to_device(X, "bf16"), to_device(W, "bf16"), to_device(G, "bf16")
    Y, XS = gl.fwd(Xd, Wd)
    # the same forward with the sketch generated inside the GEMM: the variant that stores nothing of S anywhere
    Y_gen, XS_gen = gl.empty(m, lin.d_out), gl.empty(m, r)
    B.acx_linear_fwd(gl.desc, Xd, Wd, Y_gen, XS_gen, None)
    dX, A = gl.bwd(Gd, Wd, XS)
    dW = gl.reconstruct(A)
    gl.check_status()
    assert np.array_equal(raw_bits(Y), raw_bits(Y_gen)) and np.array_equal(raw_bits(XS), raw_bits(XS_gen))

    rows = block_rows(m, 128, rows_per_block, 9 + k)
    S = osk.sketch_for_dtype(seed, lin.d_in, r, "bf16")
    Y0, U0 = ol.linear_fwd(X[rows], W, S)
    XSh = to_host(XS)
    dX0, _ = ol.linear_bwd(G[rows], W, XSh[rows])   # dX depends on one token row
    tol, ctx = min(TOL["bf16"], TOL_DERIVED["bf16"]), (wl.name, lin.name, r, layer)
    assert_parity("Y", to_host(Y_gen[rows]), Y0, "bf16", tol, ctx)
    assert_parity("XS", to_host(XS_gen[rows]), U0, "bf16", tol, ctx)
    assert_parity("dX", to_host(dX[rows]), dX0, "bf16", tol, ctx)
    Ah = to_host(A)
    if full_a:
        _, A0 = ol.linear_bwd(G, W[:, :8], XSh)      # A needs every token (the dX of this call is not used)
        assert_parity("A", Ah, A0, "factor", tol, ctx)
    else:                                            # sampled rows of A: a row of A is one column of G against all of XS
        arows = block_rows(lin.d_out, 128, rows_per_block, 11 + k)
        assert_parity("A", Ah[arows], G[:, arows].astype(np.float64).T @ XSh, "factor", tol, ctx)
    orows = block_rows(lin.d_out, 128, 1, 10 + k)
    assert_parity("dW", to_host(dW[orows]), ol.reconstruct(Ah[orows], S), "dw", tol, ctx)
    # every row of every output was written: no NaN canaries left
    for t in (Y, XS, dX, A, dW):
        assert bool(t.isfinite().all())
    if other_rank_check:
        # properties that hold at any size: Y and dX do not depend on the rank or the seed (Theorem 3.3(a))
        gl2 = GpuLinear(m, lin.d_in, lin.d_out, 16, seed + 1, "bf16")
        Y2, XS2 = gl2.fwd(Xd, Wd)
        dX2, _ = gl2.bwd(Gd, Wd, XS2)
        assert np.array_equal(raw_bits(Y2), raw_bits(Y)) and np.array_equal(raw_bits(dX2), raw_bits(dX))


@pytest.mark.parametrize("name,k,r", CASES)
def test_sampled_rows_at_full_size(name, k, r):
    check_linear_at_full_size(I.workload(name, r), k, r)
