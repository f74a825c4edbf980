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
