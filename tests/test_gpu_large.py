"""More than 2^31 output elements in one call (1 000 003 tokens x 2200 outputs: Y and G_out are 4.4 GB each): row
offsets no longer fit 32 bits and the token count is ragged against every tile size.  Inputs are drawn on the
device (seeded); the oracle checks sampled rows of Y, XS, dX and sampled rows of A over all tokens."""
import numpy as np
import pytest
import torch

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import binding as B

from _harness import TOL_DERIVED, to_host

pytestmark = pytest.mark.gpu


def _rows(t, rows):
    """Sampled rows of a very large tensor as float64, one plain slice copy per row (no index kernels on a tensor
    with more than 2^31 elements)."""
    return np.stack([t[int(i)].float().cpu().numpy().astype(np.float64) for i in rows])


def test_one_million_tokens_offsets_beyond_32_bits():
    m, d_in, d_out, r, seed = 1_000_003, 256, 2200, 32, 17
    assert m * d_out > 2 ** 31
    g = torch.Generator(device="cuda").manual_seed(1234)
    X = torch.randn(m, d_in, device="cuda", generator=g).bfloat16()
    W = (torch.randn(d_out, d_in, device="cuda", generator=g) * 0.02).bfloat16()
    G = torch.randn(m, d_out, device="cuda", generator=g).bfloat16()
    desc = B.make_desc(m, d_in, d_out, r, seed, "bf16")
    Y = torch.full((m, d_out), float("nan"), dtype=torch.bfloat16, device="cuda")
    XS = torch.full((m, r), float("nan"), dtype=torch.bfloat16, device="cuda")
    dX = torch.full((m, d_in), float("nan"), dtype=torch.bfloat16, device="cuda")
    A = torch.full((d_out, r), float("nan"), device="cuda")
    B.acx_linear_fwd(desc, X, W, Y, XS, B.alloc_workspace(desc, B.ACX_OP_FWD))
    B.acx_linear_bwd(desc, G, W, XS, dX, A, B.alloc_workspace(desc, B.ACX_OP_BWD))
    assert B.acx_last_device_status() == B.ACX_OK
    for t in (Y, XS, dX, A):                      # no canary left anywhere
        assert bool(t.isfinite().all())

    rows = np.unique(np.concatenate([np.arange(0, 4), np.arange(m - 4, m), [2 ** 19 - 1, 2 ** 19, 976_128, 976_129],
                                     np.random.Generator(np.random.Philox(3)).integers(0, m, 96)]))
    S = osk.sketch_for_dtype(seed, d_in, r, "bf16")
    Wh = to_host(W)
    XSr = _rows(XS, rows)
    Y0, U0 = ol.linear_fwd(_rows(X, rows), Wh, S)
    dX0, _ = ol.linear_bwd(_rows(G, rows), Wh, XSr)
    tol = TOL_DERIVED["bf16"]
    assert ol.rel_frobenius(_rows(Y, rows), Y0) <= tol
    assert ol.rel_frobenius(XSr, U0) <= tol
    assert ol.rel_frobenius(_rows(dX, rows), dX0) <= tol
    # rows of A (= columns of G_out) over all one million tokens
    cols = np.array([0, 1, 1099, 2198, 2199] + list(np.random.Generator(np.random.Philox(4)).integers(0, d_out, 11)))
    Gc = np.stack([G[:, int(c)].float().cpu().numpy().astype(np.float64) for c in cols])   # strided copies, one per column
    A0 = Gc @ to_host(XS)
    # a token range is one fp32 accumulation chain in the tensor core and its rounding error grows with the chain
    # (1.4e-4 with 8 ranges of 125 000 tokens); the planner keeps ranges to 65 536 tokens (here 32 ranges of 31 000)
    assert ol.rel_frobenius(_rows(A, cols), A0) <= 1e-4
