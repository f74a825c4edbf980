"""Calls on different CUDA streams: the library keeps no scratch of its own for these calls (each gets the caller's
workspace), so two linear layers stepped at the same time on two streams give the bits they give one after the other."""
import numpy as np
import pytest
import torch

from paper_2605_01255_b200 import binding as B

from _harness import raw_bits

pytestmark = pytest.mark.gpu


def _layer(m, d_in, d_out, r, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    desc = B.make_desc(m, d_in, d_out, r, seed, "bf16")
    t = dict(desc=desc,
             X=torch.randn(m, d_in, device="cuda", generator=g).bfloat16(),
             W=(torch.randn(d_out, d_in, device="cuda", generator=g) * 0.02).bfloat16(),
             G=torch.randn(m, d_out, device="cuda", generator=g).bfloat16(),
             ws_f=B.alloc_workspace(desc, B.ACX_OP_FWD), ws_b=B.alloc_workspace(desc, B.ACX_OP_BWD),
             ws_r=B.alloc_workspace(desc, B.ACX_OP_RECONSTRUCT))
    return t


def _outputs(t):
    d = t["desc"]
    nan = float("nan")
    return dict(Y=torch.full((d.tokens, d.d_out), nan, device="cuda", dtype=torch.bfloat16),
                XS=torch.full((d.tokens, d.r), nan, device="cuda", dtype=torch.bfloat16),
                dX=torch.full((d.tokens, d.d_in), nan, device="cuda", dtype=torch.bfloat16),
                A=torch.full((d.d_out, d.r), nan, device="cuda"), dW=torch.full((d.d_out, d.d_in), nan, device="cuda"))


def _step(t, o, stream, with_ws):
    d = t["desc"]
    B.acx_linear_fwd(d, t["X"], t["W"], o["Y"], o["XS"], t["ws_f"] if with_ws else None, stream=stream)
    B.acx_linear_bwd(d, t["G"], t["W"], o["XS"], o["dX"], o["A"], t["ws_b"], stream=stream)
    B.acx_reconstruct(d, o["A"], o["dW"], 0.0, t["ws_r"], stream=stream)


@pytest.mark.parametrize("with_ws", [True, False])
def test_two_streams_give_the_serial_bits(with_ws):
    layers = [_layer(4096, 1024, 1536, 128, 3), _layer(3000, 776, 520, 48, 4)]
    serial = []
    for t in layers:
        o = _outputs(t)
        _step(t, o, None, with_ws)
        serial.append(o)
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for rep in range(3):
        both = [_outputs(t) for t in layers]
        torch.cuda.synchronize()
        for k in range(4):                                   # interleave the calls of the two layers
            for t, o, s in zip(layers, both, streams):
                _step(t, o, s, with_ws)
        torch.cuda.synchronize()
        assert B.acx_last_device_status() == B.ACX_OK
        for o, o0 in zip(both, serial):
            for name in o:
                assert np.array_equal(raw_bits(o[name]), raw_bits(o0[name])), (name, rep)
