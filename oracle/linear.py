"""Oracle for the compressed linear operator, float64 numpy.  TEST INFRASTRUCTURE.

Notation follows the paper: X (m x d_in) is the layer input, W (d_out x d_in)
the weight, G = dL/dZ (m x d_out) the incoming gradient, and the stored
activation is the factor pair U (m x k), V (d_in x k) with X_hat = U V^T
(Definition 3.1; Section 4).  For the random-projection compressor the pair is
U = X S, V = S with a sketch S (d_in x r), E[S S^T] = I, so X_hat = X S S^T.

Every function is the defining formula written out with one library matmul per
product; nothing is blocked, fused or reordered.  Inputs are promoted to
float64, so callers pass the already-rounded fp32/bf16 values the GPU sees.
"""
from __future__ import annotations

import numpy as np


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def linear_fwd(X, W, S):
    """Forward of Definition 3.1 for a linear operator.

    Z = X W^T is computed exactly from X; the activation is kept only as the
    factor U = X S (the other factor, V = S, is implied by the seed).
    Returns (Y, U).
    """
    X, W, S = _f64(X), _f64(W), _f64(S)
    return X @ W.T, X @ S


def linear_bwd(G, W, U):
    """Backward of the compressed linear operator (Definition 3.1, Section 4).

    dX = G W is the exact input gradient (Theorem 3.3(a): it needs neither X
    nor X_hat).  The weight gradient G^T X_hat = (G^T U) V^T is returned as its
    left factor A = G^T U (d_out x k); the right factor is V.
    Returns (dX, A).
    """
    G, W, U = _f64(G), _f64(W), _f64(U)
    return G @ W, G.T @ U


def reconstruct(A, V, dW_prev=None, beta=0.0):
    """Optimizer strategy (i) of Section 4: rebuild the full gradient A V^T.

    With beta != 0 the result is added to beta * dW_prev (gradient accumulation).
    """
    dW = _f64(A) @ _f64(V).T
    if beta != 0.0:
        dW = dW + beta * _f64(dW_prev)
    return dW


def exact_weight_grad(G, X):
    """G_W = G^T X, the uncompressed weight gradient of a linear operator (Definition 3.1)."""
    return _f64(G).T @ _f64(X)


def reconstruct_activation(U, V):
    """X_hat = U V^T (Definition 3.1)."""
    return _f64(U) @ _f64(V).T


def activation_error(X, U, V):
    """Delta X = X_hat - X (Definition 3.1)."""
    return reconstruct_activation(U, V) - _f64(X)


def rel_frobenius(got, want):
    """||got - want||_F / ||want||_F, the parity measure of the test-suite."""
    got, want = _f64(got), _f64(want)
    den = np.linalg.norm(want)
    num = np.linalg.norm(got - want)
    return num / den if den > 0 else num


def linear_fwd_bias(X, W, S, b):
    """Forward of the affine operator Z = X W^T + B (appendix, "Bias term") with B = 1 b^T, one bias vector
    added to every token's row.  Returns (Z, U) like linear_fwd."""
    Y, U = linear_fwd(X, W, S)
    return Y + _f64(b)[None, :], U


def bias_grad(G):
    """Gradient of the bias vector: G_B = dL/dZ for the bias matrix B (appendix, "Bias term"), summed over the
    rows that share the vector b.  It does not involve X, so compression leaves it exact."""
    return _f64(G).sum(axis=0)
