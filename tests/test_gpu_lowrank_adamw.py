"""GPU parity of the low-rank-state optimizer call against the oracle (optimizer strategy (ii) of Section 4)."""
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
# The moments and the normalised step are formed in fp32 with IEEE operations (a few 1e-7).  The step then goes through
# the reconstruct kernel as two bf16 terms (2^-17 = 7.6e-6 per element) times V^T in bf16 with fp32 accumulation, so the
# update W_new - W carries about 1e-5; it is about a tenth of W here, which leaves W itself within a few 1e-6.
TOL_MOMENT, TOL_W, TOL_DELTA = 2e-6, 5e-6, 5e-5


def _steps(desc, V, Vd, d_out, d_in, r):
    W = I.gaussian((d_out, d_in), 1, 0.02, "f32").astype(np.float64)
    m = 0.01 * I.gaussian((d_out, r), 2, 1.0, "f32").astype(np.float64)
    v = 1e-4 * np.abs(I.gaussian((d_out, r), 3, 1.0, "f32")).astype(np.float64)
    Wd, md, vd = (torch.from_numpy(a.astype(np.float32)).cuda() for a in (W, m, v))
    ws = B.alloc_workspace(desc, B.ACX_OP_RECONSTRUCT)
    for step in (1, 2):
        A = I.gaussian((d_out, r), 10 + step, 1.0, "f32")
        W0, m0, v0 = to_host(Wd), to_host(md), to_host(vd)
        B.acx_lowrank_adamw(desc, to_device(A, "f32"), md, vd, Wd, Vd, step=step, ws=ws, **HP)
        assert B.acx_last_device_status() == B.ACX_OK
        W1, m1, v1 = oo.lowrank_adamw_step(A, V, W0, m0, v0, HP["lr"], HP["beta1"], HP["beta2"], HP["eps"], HP["weight_decay"], step)
        gW = to_host(Wd)
        assert ol.rel_frobenius(to_host(md), m1) <= TOL_MOMENT and ol.rel_frobenius(to_host(vd), v1) <= TOL_MOMENT
        assert ol.rel_frobenius(gW, W1) <= TOL_W
        assert ol.rel_frobenius(gW - W0, W1 - W0) <= TOL_DELTA


@pytest.mark.parametrize("d_out,d_in,r", [(264, 520, 48), (1000, 72, 32), (8, 512, 256), (3072, 3072, 128), (1024, 8192, 128)])
def test_two_lowrank_steps_with_the_seeded_sketch(d_out, d_in, r):
    seed = 7
    desc = B.make_desc(128, d_in, d_out, r, seed, "bf16")
    _steps(desc, osk.sketch_for_dtype(seed, d_in, r, "bf16"), None, d_out, d_in, r)


@pytest.mark.parametrize("d_out,d_in,r", [(264, 520, 48), (2048, 1000, 96)])
def test_two_lowrank_steps_with_an_explicit_basis(d_out, d_in, r):
    desc = B.make_desc(128, d_in, d_out, r, 0, "bf16")
    Vt = I.orthonormal_rows(r, d_in, 4, "bf16")
    _steps(desc, Vt.T, to_device(Vt, "bf16"), d_out, d_in, r)


def test_lowrank_adamw_argument_checks():
    desc = B.make_desc(128, 64, 64, 16, 0, "bf16")
    W = torch.zeros(64, 64, device="cuda")
    A = torch.zeros(64, 16, device="cuda")
    ws = B.alloc_workspace(desc, B.ACX_OP_RECONSTRUCT)
    with pytest.raises(B.AcxError) as e:
        B.acx_lowrank_adamw(desc, A, A.clone(), A.clone(), W, step=0, lr=1e-3, ws=ws)
    assert e.value.status == B.ACX_ERR_INVALID_ARG
    with pytest.raises(B.AcxError) as e:
        B.acx_lowrank_adamw(desc, A, A.clone(), A.clone(), W, step=1, lr=1e-3, ws=None)
    assert e.value.status == B.ACX_ERR_WORKSPACE
    d32 = B.make_desc(128, 64, 64, 16, 0, "f32")
    with pytest.raises(B.AcxError) as e:
        B.acx_lowrank_adamw(d32, A, A.clone(), A.clone(), W, step=1, lr=1e-3, ws=ws)
    assert e.value.status == B.ACX_ERR_INVALID_ARG
