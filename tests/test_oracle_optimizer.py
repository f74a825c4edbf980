"""Pins of the AdamW oracle: closed forms of special cases and an independent library implementation."""
import numpy as np
import torch

from oracle import optimizer as oo


def _rand(shape, seed):
    return np.random.Generator(np.random.Philox(seed)).standard_normal(shape)


def test_first_step_is_a_signed_step_of_size_lr():
    # t = 1, m = v = 0: m_hat = g, v_hat = g^2, so the Adam part is g / (|g| + eps)
    W, g = _rand((5, 7), 1), _rand((5, 7), 2)
    lr, eps, wd = 1e-3, 1e-8, 0.1
    W1, m1, v1 = oo.adamw_step(W, 0 * W, 0 * W, g, lr, 0.9, 0.999, eps, wd, 1)
    assert np.allclose(m1, 0.1 * g, rtol=1e-14) and np.allclose(v1, 0.001 * g * g, rtol=1e-12)
    assert np.allclose(W1, W - lr * (g / (np.abs(g) + eps) + wd * W), rtol=1e-12, atol=1e-15)


def test_zero_gradient_only_decays():
    W, m, v = _rand((4, 4), 3), _rand((4, 4), 4), np.abs(_rand((4, 4), 5))
    W1, m1, v1 = oo.adamw_step(W, m, v, 0 * W, 1e-2, 0.9, 0.99, 1e-8, 0.0, 3)
    assert np.allclose(m1, 0.9 * m) and np.allclose(v1, 0.99 * v)
    # weight decay is decoupled: with lr * wd it shrinks W whatever the moments are
    W2, _, _ = oo.adamw_step(W, 0 * m, 0 * v + 1.0, 0 * W, 1e-2, 0.9, 0.99, 1e-8, 0.5, 3)
    assert np.allclose(W2, W * (1 - 1e-2 * 0.5))


def test_matches_torch_adamw_over_several_steps():
    W0 = _rand((6, 9), 6)
    grads = [_rand((6, 9), 10 + i) for i in range(5)]
    lr, b1, b2, eps, wd = 3e-3, 0.8, 0.95, 1e-6, 0.05
    p = torch.nn.Parameter(torch.tensor(W0, dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
    W, m, v = W0, 0 * W0, 0 * W0
    for t, g in enumerate(grads, start=1):
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        W, m, v = oo.adamw_step(W, m, v, g, lr, b1, b2, eps, wd, t)
        assert np.allclose(W, p.detach().numpy(), rtol=1e-12, atol=1e-14), t
    st = opt.state[p]
    assert np.allclose(m, st["exp_avg"].numpy(), rtol=1e-12) and np.allclose(v, st["exp_avg_sq"].numpy(), rtol=1e-12)


def test_reconstruct_adamw_uses_the_factored_gradient():
    A, V = _rand((6, 3), 20), _rand((8, 3), 21)
    W, m, v = _rand((6, 8), 22), _rand((6, 8), 23), np.abs(_rand((6, 8), 24))
    got = oo.reconstruct_adamw(A, V, W, m, v, 1e-3, 0.9, 0.999, 1e-8, 0.01, 4)
    want = oo.adamw_step(W, m, v, A @ V.T, 1e-3, 0.9, 0.999, 1e-8, 0.01, 4)
    for a, b in zip(got, want):
        assert np.array_equal(a, b)
    # a transposed or dropped factor would change the gradient
    assert not np.allclose(got[1], oo.adamw_step(W, m, v, (V @ A.T).T[:, ::-1], 1e-3, 0.9, 0.999, 1e-8, 0.01, 4)[1])


def test_lowrank_first_step_projects_a_signed_step_back():
    # t = 1 with zero moments: N = A / (|A| + eps), so the step is lr * sign(A) V^T (Section 4, strategy (ii))
    A, V, W = _rand((6, 3), 30), _rand((8, 3), 31), _rand((6, 8), 32)
    lr, eps, wd = 2e-3, 1e-8, 0.1
    W1, m1, v1 = oo.lowrank_adamw_step(A, V, W, 0 * A, 0 * A, lr, 0.9, 0.999, eps, wd, 1)
    assert m1.shape == A.shape and v1.shape == A.shape
    assert np.allclose(m1, 0.1 * A, rtol=1e-14) and np.allclose(v1, 0.001 * A * A, rtol=1e-12)
    assert np.allclose(W1, W * (1 - lr * wd) - lr * (A / (np.abs(A) + eps)) @ V.T, rtol=1e-12, atol=1e-15)
    # the step lies in the row space of V^T: a direction orthogonal to the columns of V is untouched (up to decay)
    q, _ = np.linalg.qr(np.concatenate([V, _rand((8, 5), 33)], axis=1))
    z = q[:, 3:]
    assert np.allclose(W1 @ z, (W * (1 - lr * wd)) @ z, atol=1e-14)


def test_lowrank_with_coordinate_columns_is_adamw_on_those_columns():
    # V = the first k columns of the identity: the projected gradient is the gradient of W[:, :k], and the update is
    # plain AdamW there; the other columns only see the decoupled weight decay.  Checked against torch over 4 steps.
    d_out, d_in, k = 5, 9, 4
    V = np.eye(d_in)[:, :k]
    W0 = _rand((d_out, d_in), 40)
    lr, b1, b2, eps, wd = 3e-3, 0.85, 0.97, 1e-7, 0.02
    p = torch.nn.Parameter(torch.tensor(W0[:, :k].copy(), dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
    W, m, v = W0, np.zeros((d_out, k)), np.zeros((d_out, k))
    for t in range(1, 5):
        A = _rand((d_out, k), 50 + t)
        p.grad = torch.tensor(A, dtype=torch.float64)
        opt.step()
        W, m, v = oo.lowrank_adamw_step(A, V, W, m, v, lr, b1, b2, eps, wd, t)
        assert np.allclose(W[:, :k], p.detach().numpy(), rtol=1e-12, atol=1e-14), t
        assert np.allclose(W[:, k:], W0[:, k:] * (1 - lr * wd) ** t, rtol=1e-12), t
    assert np.allclose(m, opt.state[p]["exp_avg"].numpy(), rtol=1e-12)
    assert np.allclose(v, opt.state[p]["exp_avg_sq"].numpy(), rtol=1e-12)


def test_lowrank_differs_from_the_full_update_and_from_a_transposed_factor():
    # the normalisation happens in the factor space: it is not AdamW on the rebuilt gradient (strategy (i))
    A, V = _rand((6, 3), 60), np.linalg.qr(_rand((8, 3), 61))[0]
    W = _rand((6, 8), 62)
    lo, _, _ = oo.lowrank_adamw_step(A, V, W, 0 * A, 0 * A, 1e-2, 0.9, 0.999, 1e-8, 0.0, 1)
    full, _, _ = oo.reconstruct_adamw(A, V, W, 0 * W, 0 * W, 1e-2, 0.9, 0.999, 1e-8, 0.0, 1)
    assert not np.allclose(lo, full, atol=1e-4)
    # second moments enter through their square root: a dropped sqrt changes the second step
    W2, m2, v2 = oo.lowrank_adamw_step(2 * A, V, lo, 0.1 * A, 0.001 * A * A, 1e-2, 0.9, 0.999, 1e-8, 0.0, 2)
    m_hat = (0.9 * 0.1 * A + 0.1 * 2 * A) / (1 - 0.81)
    v_hat = (0.999 * 0.001 * A * A + 0.001 * 4 * A * A) / (1 - 0.999 ** 2)
    assert np.allclose(W2, lo - 1e-2 * (m_hat / (np.sqrt(v_hat) + 1e-8)) @ V.T, rtol=1e-12, atol=1e-15)
