"""Oracle for the randomized-SVD activation compressor, float64 numpy.  TEST INFRASTRUCTURE.

Section 5 (set-up) names the randomized SVD of Halko, Martinsson and Tropp (SIAM Review 2011) as the paper's
low-error compressor next to the random projection.  Its steps for an activation X (m x d) and a test matrix
Omega (d x k):

    Y = X Omega                      range finder, Algorithm 4.1 (no power iterations)
    Q = orthonormal basis of Y       m x k
    B = Q^T X                        k x d, first step of Algorithm 5.1
    X_hat = Q B                      the orthogonal projection of X on the range of Y

Algorithm 5.1 goes on to an SVD of B, which re-expresses the same X_hat (all k components are kept), so the
factor pair of Section 4 can be read off here already: U = Q, V^T = B.

The same X_hat has a second factorisation that needs no orthogonalisation: with U = Y itself,
V^T = (Y^T Y)^-1 Y^T X (the least-squares coefficients of X on the columns of Y), because Q Q^T = Y (Y^T Y)^-1 Y^T.
`sketch_projection_factors` writes that out; an optional ridge (relative to the largest diagonal entry of Y^T Y)
keeps the k x k solve defined when Y is rank deficient.
"""
from __future__ import annotations

import numpy as np


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def rsvd_factors(X, Omega):
    """(Q, B) with X_hat = Q B: range finder and projection of the randomized SVD (Algorithms 4.1 and 5.1)."""
    X, Omega = _f64(X), _f64(Omega)
    Y = X @ Omega
    Q, _ = np.linalg.qr(Y)
    return Q, Q.T @ X


def sketch_projection_factors(X, Omega, ridge_rel=0.0):
    """(U, Vt) with U = X Omega and Vt = (U^T U + ridge I)^-1 U^T X, ridge = ridge_rel * max diag(U^T U)."""
    X, Omega = _f64(X), _f64(Omega)
    U = X @ Omega
    G = U.T @ U
    G = G + ridge_rel * np.max(np.diag(G)) * np.eye(G.shape[0])
    return U, np.linalg.solve(G, U.T @ X)


def second_factor(X, U, ridge_rel=0.0):
    """Vt = (U^T U + ridge I)^-1 U^T X for a given first factor U (what is computed from a stored, rounded U)."""
    X, U = _f64(X), _f64(U)
    G = U.T @ U
    G = G + ridge_rel * np.max(np.diag(G)) * np.eye(G.shape[0])
    return np.linalg.solve(G, U.T @ X)
