"""Statistical properties of the method measured through the CUDA path (Theorem 3.2(a): the weight gradient of a linear
operator stays unbiased under an unbiased compressor; Theorem 3.4's compression term for the Gaussian sketch):
the mean over seeds of the rebuilt gradient converges to the exact G^T X at the 1/sqrt(trials) rate, and its mean
squared error matches the closed form ((d_in + 1) / r) ||G^T X||_F^2 of the oracle's pins."""
import numpy as np
import pytest
import torch

from oracle import linear as ol
from paper_2605_01255_b200 import binding as B
from paper_2605_01255_b200 import inputs as I

from _harness import to_device, to_host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_rebuilt_gradient_is_unbiased_with_the_predicted_variance(dtype):
    m, d_in, d_out, r, trials = 256, 128, 64, 32, 256
    X = I.gaussian((m, d_in), 1, 1.0, dtype)
    W = I.gaussian((d_out, d_in), 2, 0.02, dtype)
    G = I.gaussian((m, d_out), 3, 1.0, dtype)
    Xd, Wd, Gd = (to_device(a, dtype) for a in (X, W, G))
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    exact = ol.exact_weight_grad(G, X)
    acc = torch.zeros(d_out, d_in, device="cuda")        # sum over seeds, accumulated by the library (beta = 1)
    sq_err, means = 0.0, {}
    Y, XS = torch.empty(m, d_out, dtype=tdt, device="cuda"), torch.empty(m, r, dtype=tdt, device="cuda")
    dX, A = torch.empty(m, d_in, dtype=tdt, device="cuda"), torch.empty(d_out, r, device="cuda")
    one = torch.empty(d_out, d_in, device="cuda")
    for seed in range(trials):
        desc = B.make_desc(m, d_in, d_out, r, 1000 + seed, dtype)
        ws = {op: B.alloc_workspace(desc, op) for op in (B.ACX_OP_FWD, B.ACX_OP_BWD, B.ACX_OP_RECONSTRUCT)}
        B.acx_linear_fwd(desc, Xd, Wd, Y, XS, ws[B.ACX_OP_FWD])
        B.acx_linear_bwd(desc, Gd, Wd, XS, dX, A, ws[B.ACX_OP_BWD])
        B.acx_reconstruct(desc, A, one, 0.0, ws[B.ACX_OP_RECONSTRUCT])
        B.acx_reconstruct(desc, A, acc, 1.0, ws[B.ACX_OP_RECONSTRUCT])
        sq_err += float(np.sum((to_host(one) - exact) ** 2))
        if seed + 1 in (16, 64, 256):
            means[seed + 1] = ol.rel_frobenius(to_host(acc) / (seed + 1), exact)
    assert B.acx_last_device_status() == B.ACX_OK
    # one draw is far off (relative error about sqrt((d_in + 1) / r) = 2), the mean closes in like 1 / sqrt(trials)
    predicted = np.sqrt((d_in + 1) / r)
    for n, err in means.items():
        assert 0.6 * predicted / np.sqrt(n) <= err <= 1.5 * predicted / np.sqrt(n), (n, err)
    assert means[256] < 0.35 * means[16]
    # mean squared error of one draw: ((d_in + 1) / r) ||G^T X||_F^2 for S with iid N(0, 1/r) entries
    mse = sq_err / trials
    want = (d_in + 1) / r * float(np.sum(exact ** 2))
    assert abs(mse / want - 1.0) < 0.1


def test_per_sample_sketches_through_per_sample_calls():
    """The variance analysis takes the compression randomness independent across samples.  The ABI has one seed per
    call, so a batch with per-sample sketches is one call per sample (its own seed) and the full gradient is the sum
    over samples of A_b S_b^T, accumulated by acx_reconstruct with beta = 1.  Checked against the oracle's sum."""
    samples, seq, d_in, d_out, r = 6, 512, 256, 192, 32
    dtype = "bf16"
    W = I.gaussian((d_out, d_in), 2, 0.02, dtype)
    Wd = to_device(W, dtype)
    dW = torch.zeros(d_out, d_in, device="cuda")
    want = np.zeros((d_out, d_in))
    exact = np.zeros((d_out, d_in))
    for b in range(samples):
        X = I.gaussian((seq, d_in), 10 + b, 1.0, dtype)
        G = I.gaussian((seq, d_out), 50 + b, 1.0, dtype)
        desc = B.make_desc(seq, d_in, d_out, r, 7000 + b, dtype)          # a fresh sketch for every sample
        ws = {op: B.alloc_workspace(desc, op) for op in (B.ACX_OP_FWD, B.ACX_OP_BWD, B.ACX_OP_RECONSTRUCT)}
        Y = torch.empty(seq, d_out, dtype=torch.bfloat16, device="cuda")
        XS = torch.empty(seq, r, dtype=torch.bfloat16, device="cuda")
        dX = torch.empty(seq, d_in, dtype=torch.bfloat16, device="cuda")
        A = torch.empty(d_out, r, device="cuda")
        B.acx_linear_fwd(desc, to_device(X, dtype), Wd, Y, XS, ws[B.ACX_OP_FWD])
        B.acx_linear_bwd(desc, to_device(G, dtype), Wd, XS, dX, A, ws[B.ACX_OP_BWD])
        B.acx_reconstruct(desc, A, dW, 1.0, ws[B.ACX_OP_RECONSTRUCT])     # dW += A_b S_b^T
        from oracle import sketch as osk
        S = osk.sketch_for_dtype(7000 + b, d_in, r, dtype)
        want += ol.reconstruct(to_host(A), S)
        exact += ol.exact_weight_grad(G, X)
    assert B.acx_last_device_status() == B.ACX_OK
    assert ol.rel_frobenius(to_host(dW), want) <= 1e-5
    # with independent sketches the squared errors of the samples add: sum_b ((d_in + 1) / r) ||G_b^T X_b||_F^2, which for
    # these independent synthetic samples is ((d_in + 1) / r) times the squared norm of the summed gradient as well
    one = np.sqrt((d_in + 1) / r)
    err = ol.rel_frobenius(to_host(dW), exact)
    assert 0.85 * one <= err <= 1.15 * one
