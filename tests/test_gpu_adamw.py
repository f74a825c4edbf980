"""GPU parity of the fused reconstruct + AdamW call against the oracle (optimizer strategy (i) of Section 4)."""
import numpy as np
import pytest
import torch

from oracle import linear as ol
from oracle import optimizer as oo
from oracle import sketch as osk
from paper_2605_01255_b200 import binding as B
from paper_2605_01255_b200 import inputs as I

from _harness import to_device, to_host

pytestmark = pytest.mark.gpu

HP = dict(lr=2e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
# g is formed from A split into two bf16 terms (relative error 2^-17 = 7.6e-6 per element) with fp32 accumulation, the
# update in fp32: the moments and the step W_new - W inherit a few 1e-6 to 1e-5 of relative error; with these
# hyper-parameters the step is a sizeable fraction of W, so W itself carries about the same.
TOL_MOMENT, TOL_W, TOL_DELTA = 2e-5, 2e-5, 1e-3


@pytest.mark.parametrize("d_out,d_in,r", [(264, 520, 48), (1000, 72, 32), (8, 512, 256), (3072, 3072, 128), (1024, 8192, 128)])
def test_two_adamw_steps_match_the_oracle(d_out, d_in, r):
    seed = 5
    desc = B.make_desc(128, d_in, d_out, r, seed, "bf16")
    S = osk.sketch_for_dtype(seed, d_in, r, "bf16")
    W = I.gaussian((d_out, d_in), 1, 0.02, "f32").astype(np.float64)
    m = 0.01 * I.gaussian((d_out, d_in), 2, 1.0, "f32").astype(np.float64)
    v = 1e-4 * np.abs(I.gaussian((d_out, d_in), 3, 1.0, "f32")).astype(np.float64)
    Wd, md, vd = (torch.from_numpy(a.astype(np.float32)).cuda() for a in (W, m, v))
    W_lp = torch.full((d_out, d_in), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = B.alloc_workspace(desc, B.ACX_OP_RECONSTRUCT)
    for step in (1, 2):
        A = I.gaussian((d_out, r), 10 + step, 1.0, "f32")
        W0 = to_host(Wd)
        B.acx_reconstruct_adamw(desc, to_device(A, "f32"), Wd, md, vd, W_lp if step == 1 else None, step=step, ws=ws, **HP)
        assert B.acx_last_device_status() == B.ACX_OK
        W1, m1, v1 = oo.reconstruct_adamw(A, S, W0, m, v, HP["lr"], HP["beta1"], HP["beta2"], HP["eps"], HP["weight_decay"], step)
        gW, gm, gv = to_host(Wd), to_host(md), to_host(vd)
        assert ol.rel_frobenius(gm, m1) <= TOL_MOMENT and ol.rel_frobenius(gv, v1) <= TOL_MOMENT
        assert ol.rel_frobenius(gW, W1) <= TOL_W
        assert ol.rel_frobenius(gW - W0, W1 - W0) <= TOL_DELTA
        if step == 1:  # the low-precision copy is the new W rounded to bfloat16, ties to even
            want = osk.round_to_bf16(gW.astype(np.float32))
            assert np.array_equal(W_lp.float().cpu().numpy(), want)
        m, v = gm, gv   # carry the GPU's own state into the next step, like a training loop


def test_adamw_argument_checks():
    desc = B.make_desc(128, 64, 64, 16, 0, "bf16")
    t = torch.zeros(64, 64, device="cuda")
    A = torch.zeros(64, 16, device="cuda")
    ws = B.alloc_workspace(desc, B.ACX_OP_RECONSTRUCT)
    with pytest.raises(B.AcxError) as e:
        B.acx_reconstruct_adamw(desc, A, t, t.clone(), t.clone(), step=0, lr=1e-3, ws=ws)
    assert e.value.status == B.ACX_ERR_INVALID_ARG
    with pytest.raises(B.AcxError) as e:
        B.acx_reconstruct_adamw(desc, A, t, t.clone(), t.clone(), step=1, lr=1e-3, ws=None)
    assert e.value.status == B.ACX_ERR_WORKSPACE
    d32 = B.make_desc(128, 64, 64, 16, 0, "f32")
    with pytest.raises(B.AcxError) as e:
        B.acx_reconstruct_adamw(d32, A, t, t.clone(), t.clone(), step=1, lr=1e-3, ws=ws)
    assert e.value.status == B.ACX_ERR_INVALID_ARG
