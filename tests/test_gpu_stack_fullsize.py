"""The 28-layer LLaMA-3B-shaped stack at full size (16384 tokens, heavy-tailed low-rank inputs, r = 128) through
the stack harness, in the order the benchmark runs it: forward over all layers keeping only XS, then the backward
from the last layer with reconstruction.  Layers 0, 13 and 27 are checked with the gradient factor A of all seven
linears compared in full and the token-row outputs (Y, XS, dX) and dW on rows sampled from every 128-row block;
layers 5, 20 and 24 on sampled rows of every output (at least 256 rows each).  The other layers run on the inputs
of the nearest checked layer (their outputs are not looked at), so that the host generates six layers of inputs,
not twenty-eight."""
import numpy as np
import pytest
import torch

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import inputs as I
from paper_2605_01255_b200 import stack as S

from _harness import TOL, TOL_DERIVED, assert_parity, to_device, to_host
from test_gpu_fullsize import block_rows

pytestmark = pytest.mark.gpu

FULL_LAYERS, SAMPLED_LAYERS = (0, 13, 27), (5, 20, 24)
SEED_BASE = 4040


def test_stack28_heavy_tailed_at_full_size():
    wl = I.workload("llama3b_stack28")
    m, r, L = wl.tokens, wl.r, wl.layers
    checked = sorted(FULL_LAYERS + SAMPLED_LAYERS)
    source = {l: min(checked, key=lambda c: (abs(c - l), c)) for l in range(L)}   # whose inputs an unchecked layer reuses
    n_lin = len(wl.linears)
    slots = sorted(S.slots_of(wl))
    tol = min(TOL["bf16"], TOL_DERIVED["bf16"])

    Wd = {(c, k): to_device(I.make_w(wl, c, k), "bf16") for c in checked for k in range(n_lin)}
    st = S.CompressedStack(wl, {(l, k): Wd[(source[l], k)] for l in range(L) for k in range(n_lin)}, seed_base=SEED_BASE)
    Xd = {}

    def x_dev(c):
        if c not in Xd:
            Xd.clear()   # one layer's inputs on the device at a time
            Xd[c] = {s: to_device(I.make_x(wl, c, next(lin for lin in wl.linears if lin.slot == s)), "bf16") for s in slots}
        return Xd[c]

    # ---- forward over all layers: only XS survives; Y and XS of the checked layers are compared right away
    for l in range(L):
        xs = x_dev(source[l])
        outs = st.forward_layer(l, lambda s: xs[s], keep_y=(l in checked))
        if l not in checked:
            continue
        st.check_status()
        for k, lin in enumerate(wl.linears):
            rows = block_rows(m, 128, 2, 100 * l + k)
            Xh = to_host(xs[lin.slot][rows])   # the bf16 values the kernel read, exactly
            Sm = osk.sketch_for_dtype(I.sketch_seed(SEED_BASE, l, lin.slot), lin.d_in, r, "bf16")
            Y0, U0 = ol.linear_fwd(Xh, to_host(Wd[(l, k)]), Sm)
            ctx = ("layer", l, lin.name)
            assert_parity("Y", to_host(outs[k][rows]), Y0, "bf16", tol, ctx)
            assert_parity("XS", to_host(st.XS[(l, lin.slot)][rows]), U0, "bf16", tol, ctx)
            assert bool(outs[k].isfinite().all())
        del outs

    # ---- backward, last layer first, with reconstruction
    dW = {k: torch.empty(lin.d_out, lin.d_in, dtype=torch.float32, device="cuda") for k, lin in enumerate(wl.linears)}
    Gd_cache = {}

    def g_dev(c):
        if c not in Gd_cache:
            Gd_cache.clear()
            Gd_cache[c] = [to_device(I.make_g(wl, c, k), "bf16") for k in range(n_lin)]
        return Gd_cache[c]

    for l in reversed(range(L)):
        gs = g_dev(source[l])
        if l in checked:
            for t in dW.values():
                t.fill_(float("nan"))
        outs = st.backward_layer(l, lambda k: gs[k], keep_dx=(l in checked), dW=dW)
        if l not in checked:
            continue
        st.check_status()
        for k, lin in enumerate(wl.linears):
            ctx = ("layer", l, lin.name)
            Wh = to_host(Wd[(l, k)])
            XSh = to_host(st.XS[(l, lin.slot)])
            rows = block_rows(m, 128, 2, 200 * l + k)
            Gh_rows = to_host(gs[k][rows])
            dX0, _ = ol.linear_bwd(Gh_rows, Wh, XSh[rows])
            assert_parity("dX", to_host(outs[k][rows]), dX0, "bf16", tol, ctx)
            Ah = to_host(st.A[(l, k)])
            if l in FULL_LAYERS:
                A0 = to_host(gs[k]).T @ XSh
                assert_parity("A", Ah, A0, "factor", tol, ctx)
            else:
                arows = block_rows(lin.d_out, 128, 2, 300 * l + k)
                A0 = to_host(gs[k][:, arows]).T @ XSh
                assert_parity("A", Ah[arows], A0, "factor", tol, ctx)
            Sm = osk.sketch_for_dtype(I.sketch_seed(SEED_BASE, l, lin.slot), lin.d_in, r, "bf16")
            orows = block_rows(lin.d_out, 128, 2, 400 * l + k)
            assert_parity("dW", to_host(dW[k][orows]), ol.reconstruct(Ah[orows], Sm), "dw", tol, ctx)
            assert bool(outs[k].isfinite().all()) and bool(dW[k].isfinite().all())
        del outs
    # the stored activations of the whole stack are the XS buffers and nothing else
    rep = S.report(wl)
    assert rep.stored_bytes_compressed == sum(t.numel() * t.element_size() for t in st.XS.values())
