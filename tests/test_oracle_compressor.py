"""Pins of the randomized-SVD compressor oracle: what Halko, Martinsson and Tropp (2011) and linear algebra fix."""
import numpy as np

from oracle import compressor as oc
from oracle import linear as ol


def _rand(shape, seed):
    return np.random.Generator(np.random.Philox(seed)).standard_normal(shape)


def _decaying(m, d, seed, power=1.0):
    u, _ = np.linalg.qr(_rand((m, d), seed))
    v, _ = np.linalg.qr(_rand((d, d), seed + 1))
    s = 1.0 / np.arange(1, d + 1) ** power
    return (u * s) @ v.T, s


def test_exact_on_inputs_of_rank_at_most_k():
    X = _rand((60, 5), 1) @ _rand((5, 24), 2)          # rank 5
    Om = _rand((24, 8), 3)
    Q, B = oc.rsvd_factors(X, Om)
    assert np.allclose(Q.T @ Q, np.eye(8), atol=1e-12)
    assert ol.rel_frobenius(Q @ B, X) < 1e-10


def test_both_factorisations_give_the_same_projection():
    X, Om = _rand((50, 20), 4), _rand((20, 6), 5)
    Q, B = oc.rsvd_factors(X, Om)
    U, Vt = oc.sketch_projection_factors(X, Om)
    assert np.allclose(U, X @ Om)
    assert np.allclose(U @ Vt, Q @ B, atol=1e-10)
    # orthogonal projection on range(Y): residual orthogonal to Y, and projecting twice changes nothing
    Xh = U @ Vt
    assert np.allclose((X @ Om).T @ (X - Xh), 0, atol=1e-9)
    U2, Vt2 = oc.sketch_projection_factors(Xh, Om)
    assert np.allclose(U2 @ Vt2, Xh, atol=1e-9)
    # second_factor recomputes Vt from a given U
    assert np.allclose(oc.second_factor(X, U), Vt, atol=1e-10)


def test_never_worse_than_the_random_projection_and_never_better_than_the_truncated_svd():
    X, s = _decaying(80, 32, 6)
    k = 8
    best = np.sqrt(np.sum(s[k:] ** 2))                  # Eckart-Young: no rank-k matrix is closer
    for seed in range(5):
        Om = _rand((32, k), 10 + seed) / np.sqrt(k)
        Q, B = oc.rsvd_factors(X, Om)
        err = np.linalg.norm(X - Q @ B)
        assert err >= best * (1 - 1e-12)
        # X Om Om^T lies in the range of Y = X Om, and the projection is the closest point of that range
        assert err <= np.linalg.norm(X - X @ Om @ Om.T) * (1 + 1e-12)


def test_expected_error_obeys_the_bound_of_theorem_10_5():
    # E ||X - Q Q^T X||_F <= (1 + k/(p-1))^(1/2) (sum_{j>k} sigma_j^2)^(1/2) for target rank k and oversampling p >= 2
    X, s = _decaying(100, 40, 7, power=1.5)
    k, p = 6, 4
    errs = []
    for seed in range(60):
        Q, B = oc.rsvd_factors(X, _rand((40, k + p), 100 + seed))
        errs.append(np.linalg.norm(X - Q @ B))
    bound = np.sqrt(1 + k / (p - 1)) * np.sqrt(np.sum(s[k:] ** 2))
    assert np.mean(errs) <= bound
    assert np.mean(errs) >= np.sqrt(np.sum(s[k + p:] ** 2))   # and cannot beat the best rank-(k+p) approximation


def test_small_ridge_changes_little_and_rescues_rank_deficient_sketches():
    X, Om = _rand((64, 24), 8), _rand((24, 8), 9)
    U, Vt = oc.sketch_projection_factors(X, Om)
    _, Vr = oc.sketch_projection_factors(X, Om, ridge_rel=2.0 ** -20)
    assert ol.rel_frobenius(U @ Vr, U @ Vt) < 1e-4
    Xlow = _rand((64, 3), 10) @ _rand((3, 24), 11)      # rank 3 < k = 8: Y^T Y is singular
    U, Vr = oc.sketch_projection_factors(Xlow, Om, ridge_rel=2.0 ** -20)
    assert np.all(np.isfinite(Vr))
    assert ol.rel_frobenius(U @ Vr, Xlow) < 1e-4
