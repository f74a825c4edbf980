"""GPU parity of the layer-stack harness against the oracle, on a small stack with the heavy-tailed,
low-rank input recipe of the 28-layer configuration."""
import gc

import numpy as np
import pytest
import torch

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import inputs as I
from paper_2605_01255_b200 import stack as S

from _harness import TOL, TOL_DERIVED, assert_parity, to_device, to_host

pytestmark = pytest.mark.gpu


def _small_workload():
    lins = (I.Linear("q", 256, 256, 0), I.Linear("k", 256, 256, 0), I.Linear("v", 256, 256, 0), I.Linear("o", 256, 256, 1),
            I.Linear("gate", 256, 640, 2), I.Linear("up", 256, 640, 2), I.Linear("down", 640, 256, 3))
    return I.Workload("small_stack", 600, lins, 32, "bf16", "heavy_lowrank", 3)


def test_small_stack_matches_the_oracle_layer_by_layer():
    wl = _small_workload()
    m, L, r = wl.tokens, wl.layers, wl.r
    Wh = {(l, k): I.make_w(wl, l, k) for l in range(L) for k in range(len(wl.linears))}
    Xh = {(l, lin.slot): I.make_x(wl, l, lin) for l in range(L) for lin in wl.linears}
    Gh = {(l, k): I.make_g(wl, l, k) for l in range(L) for k in range(len(wl.linears))}
    W = {key: to_device(v, "bf16") for key, v in Wh.items()}
    st = S.CompressedStack(wl, W, seed_base=77)

    # forward over all layers: only XS survives
    Ys = {}
    for l in range(L):
        outs = st.forward_layer(l, lambda s: to_device(Xh[(l, s)], "bf16"), keep_y=True)
        for k, y in enumerate(outs):
            Ys[(l, k)] = y
    # backward, last layer first, with reconstruction of every dW
    dXs, dWs = {}, {}
    for l in reversed(range(L)):
        dW = {k: torch.empty(lin.d_out, lin.d_in, dtype=torch.float32, device="cuda") for k, lin in enumerate(wl.linears)}
        outs = st.backward_layer(l, lambda k: to_device(Gh[(l, k)], "bf16"), keep_dx=True, dW=dW)
        for k, dx in enumerate(outs):
            dXs[(l, k)], dWs[(l, k)] = dx, dW[k]
    st.check_status()

    tol, tight = TOL["bf16"], TOL_DERIVED["bf16"]
    for l in range(L):
        for k, lin in enumerate(wl.linears):
            Sm = osk.sketch_for_dtype(I.sketch_seed(77, l, lin.slot), lin.d_in, r, "bf16")
            Y0, U0 = ol.linear_fwd(Xh[(l, lin.slot)], Wh[(l, k)], Sm)
            XS = to_host(st.XS[(l, lin.slot)])
            dX0, A0 = ol.linear_bwd(Gh[(l, k)], Wh[(l, k)], XS)
            ctx, t = (l, lin.name), min(tol, tight)
            assert_parity("Y", to_host(Ys[(l, k)]), Y0, "bf16", t, ctx)
            assert_parity("XS", XS, U0, "bf16", t, ctx)
            assert_parity("dX", to_host(dXs[(l, k)]), dX0, "bf16", t, ctx)
            assert_parity("A", to_host(st.A[(l, k)]), A0, "factor", t, ctx)
            assert_parity("dW", to_host(dWs[(l, k)]), ol.reconstruct(to_host(st.A[(l, k)]), Sm), "dw", t, ctx)
    # linears that share an input share the stored factor and the sketch
    rep = S.report(wl)
    assert rep.stored_bytes_compressed == sum(t.numel() * t.element_size() for t in st.XS.values())


def test_stored_activation_memory_is_what_the_report_says():
    """Peak device memory of a compressed forward grows by the stored XS only (Y and X buffers are reused)."""
    wl = _small_workload()
    W = {(l, k): to_device(I.make_w(wl, 0, k), "bf16") for l in range(wl.layers) for k in range(len(wl.linears))}
    X = {s: to_device(I.make_x(wl, 0, next(l for l in wl.linears if l.slot == s)), "bf16") for s in S.slots_of(wl)}
    gc.collect()                      # tensors of earlier tests that only a reference cycle keeps alive go now, not mid-measurement
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    st = S.CompressedStack(wl, W)
    for l in range(wl.layers):
        st.forward_layer(l, lambda s: X[s])
    st.check_status()
    rep = S.report(wl)
    held = torch.cuda.memory_allocated() - before
    scratch = st._Y.numel() * 2 + st._dX.numel() * 2 + st._ws.numel() + rep.factor_bytes
    # allocator granularity: every tensor is rounded up to 512 bytes
    n_tensors = len(st.XS) + len(st.A) + 3
    assert rep.stored_bytes_compressed + scratch <= held <= rep.stored_bytes_compressed + scratch + 512 * n_tensors


def test_stack_backward_with_lowrank_optimizer_states():
    """Optimizer strategy (ii) of Section 4 through the stack harness: two steps on one layer, the moments of every
    linear kept for its gradient factor, against the oracle."""
    from oracle import optimizer as oo

    wl = I.Workload("one_layer", 600, _small_workload().linears, 32, "bf16", "heavy_lowrank", 1)
    m, r = wl.tokens, wl.r
    Wh = {(0, k): I.make_w(wl, 0, k) for k in range(len(wl.linears))}
    Xh = {lin.slot: I.make_x(wl, 0, lin) for lin in wl.linears}
    W = {key: to_device(v, "bf16") for key, v in Wh.items()}
    st = S.CompressedStack(wl, W, seed_base=5)
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.05)
    state = {k: (torch.from_numpy(Wh[(0, k)].astype(np.float32)).cuda(), torch.zeros(lin.d_out, r, device="cuda"),
                 torch.zeros(lin.d_out, r, device="cuda")) for k, lin in enumerate(wl.linears)}
    ref = {k: (Wh[(0, k)].astype(np.float64), np.zeros((lin.d_out, r)), np.zeros((lin.d_out, r))) for k, lin in enumerate(wl.linears)}
    for step in (1, 2):
        Gh = {k: I.gaussian((m, lin.d_out), 100 * step + k, 1.0, "bf16") for k, lin in enumerate(wl.linears)}
        st.forward_layer(0, lambda s: to_device(Xh[s], "bf16"))
        st.backward_layer(0, lambda k: to_device(Gh[k], "bf16"), lowrank=state, step=step, **hp)
        st.check_status()
        for k, lin in enumerate(wl.linears):
            Sm = osk.sketch_for_dtype(I.sketch_seed(5, 0, lin.slot), lin.d_in, r, "bf16")
            Wp = ref[k][0]
            ref[k] = oo.lowrank_adamw_step(to_host(st.A[(0, k)]), Sm, *ref[k], hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                                           hp["weight_decay"], step)
            assert ol.rel_frobenius(to_host(state[k][1]), ref[k][1]) <= 2e-6
            assert ol.rel_frobenius(to_host(state[k][0]) - Wp, ref[k][0] - Wp) <= 1e-4
            ref[k] = (to_host(state[k][0]), to_host(state[k][1]), to_host(state[k][2]))   # carry the GPU state on
