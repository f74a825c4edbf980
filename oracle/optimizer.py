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
