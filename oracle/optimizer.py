"""Oracle for the optimizer step on a reconstructed gradient, float64 numpy.  TEST INFRASTRUCTURE.

Section 4 of the paper, optimizer strategy (i): the full gradient is rebuilt from the factor pair,
G_W_hat = A V^T, and handed to a standard update; the experiments use AdamW (Section 5, set-up).  AdamW is the
decoupled-weight-decay Adam of Loshchilov & Hutter (ICLR 2019, Algorithm 2), written out step by step:

    m <- beta1 m + (1 - beta1) g            v <- beta2 v + (1 - beta2) g^2
    m_hat = m / (1 - beta1^t)               v_hat = v / (1 - beta2^t)
    W <- W - lr * ( m_hat / (sqrt(v_hat) + eps) + weight_decay * W )

with t >= 1 the number of the step.  Nothing is fused or reordered.
"""
from __future__ import annotations

import numpy as np


def adamw_step(W, m, v, g, lr, beta1, beta2, eps, weight_decay, t):
    """One AdamW step on float64 copies; returns (W_new, m_new, v_new)."""
    W, m, v, g = (np.asarray(a, dtype=np.float64) for a in (W, m, v, g))
    m_new = beta1 * m + (1.0 - beta1) * g
    v_new = beta2 * v + (1.0 - beta2) * g * g
    m_hat = m_new / (1.0 - beta1 ** t)
    v_hat = v_new / (1.0 - beta2 ** t)
    W_new = W - lr * (m_hat / (np.sqrt(v_hat) + eps) + weight_decay * W)
    return W_new, m_new, v_new


def reconstruct_adamw(A, V, W, m, v, lr, beta1, beta2, eps, weight_decay, t):
    """Strategy (i): g = A V^T (the reconstructed weight gradient), then one AdamW step with it."""
    g = np.asarray(A, dtype=np.float64) @ np.asarray(V, dtype=np.float64).T
    return adamw_step(W, m, v, g, lr, beta1, beta2, eps, weight_decay, t)


def lowrank_adamw_step(A, V, W, mA, vA, lr, beta1, beta2, eps, weight_decay, t):
    """Strategy (ii) of Section 4: a GaLore-style update with the optimizer states kept in the factor space.

    The left gradient factor A = G^T U (d_out x k) is the weight gradient projected on the columns of V, so it plays
    the part of GaLore's projected gradient R_t (Zhao et al., ICML 2024, Algorithm 2, with the projection on the right
    and scale alpha = 1): Adam's moments are kept for A (d_out x k each instead of d_out x d_in), the normalised step
    N is formed there and projected back through V^T; weight decay is decoupled as in AdamW.

        mA <- beta1 mA + (1 - beta1) A          vA <- beta2 vA + (1 - beta2) A^2
        N = (mA / (1 - beta1^t)) / (sqrt(vA / (1 - beta2^t)) + eps)
        W <- W - lr * (N V^T + weight_decay * W)

    Returns (W_new, mA_new, vA_new).
    """
    A, V, W, mA, vA = (np.asarray(a, dtype=np.float64) for a in (A, V, W, mA, vA))
    mA_new = beta1 * mA + (1.0 - beta1) * A
    vA_new = beta2 * vA + (1.0 - beta2) * A * A
    N = (mA_new / (1.0 - beta1 ** t)) / (np.sqrt(vA_new / (1.0 - beta2 ** t)) + eps)
    W_new = W - lr * (N @ V.T + weight_decay * W)
    return W_new, mA_new, vA_new
