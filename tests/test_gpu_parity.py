"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import binding as B
from paper_2605_01255_b200 import inputs as I

from _harness import TOL, TOL_DERIVED, GpuLinear, assert_parity, raw_bits, to_device, to_host

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------ sketch: bit-exact
SKETCH_CASES = [(0, 256, 16), (3, 896, 64), (4, 4864, 64), (5, 2048, 128), (6, 8192, 128), (7, 3072, 32),
                (8, 3072, 64), (9, 3072, 128), (10, 3072, 256), (0xFEDCBA9876543210, 8192, 256), (11, 264, 48)]


@pytest.mark.parametrize("seed,d_in,r", SKETCH_CASES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sketch_bits_match_oracle(seed, d_in, r, dtype):
    lin = GpuLinear(8, d_in, 8, r, seed, dtype)
    got = raw_bits(lin.sketch())
    want = osk.sketch(seed, d_in, r)
    if dtype == "bf16":
        want_bits = (osk.round_to_bf16(want).view(np.uint32) >> 16).astype(np.uint16)
    else:
        want_bits = want.view(np.uint32)
    assert got.shape == want_bits.shape
    assert np.array_equal(got, want_bits), "first mismatch at %s" % (np.argwhere(got != want_bits)[:1],)


# ------------------------------------------------------------------ full element-wise parity
def _run_case(m, d_in, d_out, r, seed, dtype, data_seed=0):
    X = I.gaussian((m, d_in), 100 + data_seed, 1.0, dtype)
    W = I.gaussian((d_out, d_in), 200 + data_seed, 0.02, dtype)
    G = I.gaussian((m, d_out), 300 + data_seed, 1.0, dtype)
    lin = GpuLinear(m, d_in, d_out, r, seed, dtype)
    dX_, W_, G_ = to_device(X, dtype), to_device(W, dtype), to_device(G, dtype)
    Y, XS = lin.fwd(dX_, W_)
    dX, A = lin.bwd(G_, W_, XS)
    dW = lin.reconstruct(A)
    lin.check_status()

    S = osk.sketch_for_dtype(seed, d_in, r, dtype)
    Y0, U0 = ol.linear_fwd(X, W, S)
    tol = min(TOL[dtype], TOL_DERIVED[dtype])   # the stated tolerance and the tighter one the arithmetic should deliver
    out_kind = "bf16" if dtype == "bf16" else "acc"
    dw_kind = "dw" if dtype == "bf16" else "acc"
    ctx = (m, d_in, d_out, r, dtype)
    errs = {"Y": assert_parity("Y", to_host(Y), Y0, out_kind, tol, ctx), "XS": assert_parity("XS", to_host(XS), U0, out_kind, tol, ctx)}
    # stage-wise: the backward is checked from the factor the GPU actually stored
    XS_stored = to_host(XS)
    dX0, A0 = ol.linear_bwd(G, W, XS_stored)
    errs["dX"] = assert_parity("dX", to_host(dX), dX0, out_kind, tol, ctx)
    errs["A"] = assert_parity("A", to_host(A), A0, "factor" if dtype == "bf16" else "acc", tol, ctx)
    errs["dW"] = assert_parity("dW", to_host(dW), ol.reconstruct(to_host(A), S), dw_kind, tol, ctx)
    # end to end from the oracle's own factor (adds the storage rounding of XS)
    _, A_e2e = ol.linear_bwd(G, W, U0)
    e2e_kind = "e2e" if dtype == "bf16" else "acc"
    errs["A_e2e"] = assert_parity("A_e2e", to_host(A), A_e2e, e2e_kind, tol, ctx)
    errs["dW_e2e"] = assert_parity("dW_e2e", to_host(dW), ol.reconstruct(A_e2e, S), e2e_kind, tol, ctx)
    return errs


def test_config1_single_linear_fp32():
    _run_case(512, 256, 256, 16, 0, "f32")


@pytest.mark.parametrize("d_in,d_out", [(896, 4864), (4864, 896)])
def test_config2_qwen_mlp_bf16(d_in, d_out):
    _run_case(4096, d_in, d_out, 64, 1, "bf16")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("m,d_in,d_out,r", [(777, 264, 136, 48), (1, 64, 64, 16), (130, 512, 8, 256), (1031, 72, 1000, 32)])
def test_ragged_shapes(m, d_in, d_out, r, dtype):
    _run_case(m, d_in, d_out, r, 5, dtype, data_seed=m)


def test_zero_tokens_is_a_noop_and_zeroes_the_factor():
    for dtype in ("f32", "bf16"):
        lin = GpuLinear(0, 64, 64, 16, 0, dtype)
        W = to_device(I.gaussian((64, 64), 1, 0.02, dtype), dtype)
        X = lin.empty(0, 64)
        Y, XS = lin.fwd(X, W)
        assert Y.shape == (0, 64) and XS.shape == (0, 16)
        A = torch.full((64, 16), 7.0, device="cuda")
        B.acx_linear_bwd(lin.desc, lin.empty(0, 64), W, XS, lin.empty(0, 64), A, lin.ws_bwd)
        lin.check_status()
        assert float(A.abs().max()) == 0.0


def test_reconstruct_accumulates():
    m, d_in, d_out, r = 64, 128, 72, 32
    lin = GpuLinear(m, d_in, d_out, r, 9, "bf16")
    A = I.gaussian((d_out, r), 1, 1.0, "f32")
    prev = I.gaussian((d_out, d_in), 2, 1.0, "f32")
    S = osk.sketch_for_dtype(9, d_in, r, "bf16")
    for beta in (1.0, 0.5):
        dW = to_device(prev, "f32")
        lin.reconstruct(to_device(A, "f32"), dW, beta)
        assert_parity("dW", to_host(dW), ol.reconstruct(A, S, prev, beta), "dw", TOL_DERIVED["bf16"], beta)
    # beta = 0 must not read dW: NaNs in it may not leak
    dW = torch.full((d_out, d_in), float("nan"), device="cuda")
    lin.reconstruct(to_device(A, "f32"), dW, 0.0)
    assert bool(torch.isfinite(dW).all())


def test_input_gradient_ignores_rank_and_seed_and_runs_are_reproducible():
    m, d_in, d_out = 512, 256, 384
    for dtype in ("f32", "bf16"):
        X = to_device(I.gaussian((m, d_in), 1, 1.0, dtype), dtype)
        W = to_device(I.gaussian((d_out, d_in), 2, 0.02, dtype), dtype)
        G = to_device(I.gaussian((m, d_out), 3, 1.0, dtype), dtype)
        outs = []
        for r, seed in ((16, 0), (64, 1), (64, 1)):
            lin = GpuLinear(m, d_in, d_out, r, seed, dtype)
            Y, XS = lin.fwd(X, W)
            dX, A = lin.bwd(G, W, XS)
            outs.append((raw_bits(Y), raw_bits(XS), raw_bits(dX), raw_bits(A)))
        # Theorem 3.3(a): dX (and Y) do not depend on the compression at all
        assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][2], outs[1][2])
        # same arguments twice: every output bit for bit
        for a, b in zip(outs[1], outs[2]):
            assert np.array_equal(a, b)


def test_optional_outputs():
    m, d_in, d_out, r = 256, 128, 128, 16
    lin = GpuLinear(m, d_in, d_out, r, 2, "bf16")
    X = to_device(I.gaussian((m, d_in), 1, 1.0, "bf16"), "bf16")
    W = to_device(I.gaussian((d_out, d_in), 2, 0.02, "bf16"), "bf16")
    G = to_device(I.gaussian((m, d_out), 3, 1.0, "bf16"), "bf16")
    _, XS = lin.fwd(X, W)
    dX, A = lin.bwd(G, W, XS)
    dX_only, none_a = lin.bwd(G, W, XS, want_a=False)
    none_dx, A_only = lin.bwd(G, W, XS, want_dx=False)
    assert none_a is None and none_dx is None
    assert np.array_equal(raw_bits(dX), raw_bits(dX_only)) and np.array_equal(raw_bits(A), raw_bits(A_only))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("m,d_in,d_out,r", [(600, 264, 1000, 48), (2048, 896, 4864, 64), (130, 512, 8, 256)])
def test_forward_without_the_factor_gives_the_same_output(m, d_in, d_out, r, dtype):
    """Linears that share an input store its factor once: with XS = NULL only Y is computed, and it is the same Y."""
    X = I.gaussian((m, d_in), 11, 1.0, dtype)
    W = I.gaussian((d_out, d_in), 12, 0.02, dtype)
    lin = GpuLinear(m, d_in, d_out, r, 3, dtype)
    Xd, Wd = to_device(X, dtype), to_device(W, dtype)
    Y_full, _ = lin.fwd(Xd, Wd)
    Y_only, none = lin.fwd(Xd, Wd, want_xs=False)
    lin.check_status()
    assert none is None
    assert np.array_equal(raw_bits(Y_full), raw_bits(Y_only))
    Y0, _ = ol.linear_fwd(X, W, np.zeros((d_in, r)))
    assert_parity("Y", to_host(Y_only), Y0, "bf16" if dtype == "bf16" else "acc", TOL_DERIVED[dtype])


# the last row: a last N-tile that is cut down to the W columns that exist (3072: 120 of 248; 736: 8, the narrowest; 968: rounding
# brings it back to the full height; 976: exactly full)
@pytest.mark.parametrize("m,d_in,d_out,r", [(600, 264, 1000, 48), (2048, 896, 4864, 64), (130, 512, 8, 256), (4096, 1024, 1024, 128),
                                           (300, 128, 3072, 128), (1100, 320, 736, 48), (1100, 320, 968, 48), (1100, 320, 976, 48)])
def test_forward_with_and_without_workspace_gives_the_same_bits(m, d_in, d_out, r):
    """With a workspace S^T is written out once and read back by the GEMM; without one every thread block
    regenerates its slices of S.  Same sketch values, same products: Y and XS agree bit for bit, and both are
    checked against the oracle."""
    X = I.gaussian((m, d_in), 21, 1.0, "bf16")
    W = I.gaussian((d_out, d_in), 22, 0.02, "bf16")
    lin = GpuLinear(m, d_in, d_out, r, 9, "bf16")
    assert lin.ws_fwd is not None and lin.ws_fwd.numel() >= r * d_in * 2
    Xd, Wd = to_device(X, "bf16"), to_device(W, "bf16")
    Y_ws, XS_ws = lin.fwd(Xd, Wd)
    Y_no, XS_no = lin.empty(m, d_out), lin.empty(m, r)
    B.acx_linear_fwd(lin.desc, Xd, Wd, Y_no, XS_no, None)
    lin.check_status()
    assert np.array_equal(raw_bits(Y_ws), raw_bits(Y_no)) and np.array_equal(raw_bits(XS_ws), raw_bits(XS_no))
    S = osk.sketch_for_dtype(9, d_in, r, "bf16")
    Y0, U0 = ol.linear_fwd(X, W, S)
    assert_parity("XS", to_host(XS_no), U0, "bf16", TOL_DERIVED["bf16"])
    assert_parity("Y", to_host(Y_no), Y0, "bf16", TOL_DERIVED["bf16"])
    with pytest.raises(B.AcxError) as e:  # a workspace that is given must be large enough
        B.acx_linear_fwd(lin.desc, Xd, Wd, Y_no, XS_no, lin.ws_fwd[:64])
    assert e.value.status == B.ACX_ERR_WORKSPACE


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """Every device-side wait of the library is bounded; one that expires sets the status word and the kernel returns."""
    assert B.acx_last_device_status() == B.ACX_OK
    B.acx_debug_expired_wait(2_000_000)            # 2 ms on a barrier nobody signals
    assert B.acx_last_device_status() == B.ACX_ERR_TIMEOUT
    assert B.acx_last_device_status() == B.ACX_OK  # reported once, then cleared
    _run_case(130, 264, 136, 48, 5, "bf16", data_seed=3)   # the context still computes correctly
    with pytest.raises(B.AcxError):
        B.acx_debug_expired_wait(0)
