"""Sketch seeds across training steps (Theorem 3.2(a): the gradient estimate is unbiased in expectation over the
compression randomness).  With a fresh seed per step the mean over steps of the rebuilt gradient approaches G^T X at
the Monte-Carlo rate; with one fixed seed it stays at the projection G^T X S S^T however many steps are averaged.
Oracle and seed bookkeeping only (CPU)."""
import numpy as np

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import inputs as I

M, D_IN, D_OUT, R = 96, 64, 24, 16


def _mean_rebuilt_gradient(steps, fresh):
    X = I.gaussian((M, D_IN), 1, 1.0, "f32")
    G = I.gaussian((M, D_OUT), 2, 1.0, "f32")
    W = np.zeros((D_OUT, D_IN))
    acc = np.zeros((D_OUT, D_IN))
    for step in range(steps):
        seed = I.sketch_seed(11, 3, 2, step if fresh else 0)
        S = osk.sketch_for_dtype(seed, D_IN, R, "f32")
        _, U = ol.linear_fwd(X, W, S)
        _, A = ol.linear_bwd(G, W, U)
        acc += ol.reconstruct(A, S)
    return acc / steps, ol.exact_weight_grad(G, X)


def test_fresh_seeds_average_to_the_exact_gradient_and_a_fixed_seed_does_not():
    errs = {}
    for steps in (16, 256):
        mean, exact = _mean_rebuilt_gradient(steps, fresh=True)
        errs[steps] = ol.rel_frobenius(mean, exact)
    # closed-form rate: sqrt((d_in + 1) / (r * steps))
    for steps, e in errs.items():
        want = np.sqrt((D_IN + 1) / (R * steps))
        assert 0.6 * want <= e <= 1.5 * want, (steps, e, want)
    assert errs[256] < 0.4 * errs[16]                      # 1/sqrt(steps): a factor of 4 expected
    fixed16, exact = _mean_rebuilt_gradient(16, fresh=False)
    fixed256, _ = _mean_rebuilt_gradient(256, fresh=False)
    assert np.array_equal(fixed16, fixed256) or ol.rel_frobenius(fixed16, fixed256) < 1e-12   # averaging changes nothing
    assert ol.rel_frobenius(fixed256, exact) > 5 * errs[256]


def test_step_seeds_are_distinct_and_step_zero_is_the_plain_seed():
    seen = set()
    for step in range(4):
        for layer in range(28):
            for slot in range(4):
                seen.add(I.sketch_seed(7, layer, slot, step))
    assert len(seen) == 4 * 28 * 4
    assert I.sketch_seed(7, 5, 2) == I.sketch_seed(7, 5, 2, 0) == 7 + 16 * 5 + 2
