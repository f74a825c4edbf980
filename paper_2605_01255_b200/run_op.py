"""Run one call of the library a few times on random inputs: the command to profile a single kernel.

    python -m paper_2605_01255_b200.run_op {fwd,fwd_nows,fwd_plain,fwd_v,dx,factor,reconstruct,reconstruct_v,adamw,lowrank_adamw,rsvd,factor_bias} tokens,d_in,d_out,r [launches] [f32|bf16]

`fwd_nows` is the forward without a workspace (the sketch generated inside the GEMM), `fwd_plain` the forward of a linear
whose input's factor another linear stores (XS = NULL); `dx` and `factor` are acx_linear_bwd with the other output left out.  Prints "ok" after checking the
device status word.  Inputs come from torch.randn on the device (values do not matter for a profile).
"""
from __future__ import annotations

import sys

import torch

from . import binding as B


def main(argv) -> int:
    if len(argv) < 2:
        print(__doc__)
        return 2
    op = argv[0]
    m, d_in, d_out, r = (int(x) for x in argv[1].split(","))
    launches = int(argv[2]) if len(argv) > 2 else 3
    dtype = argv[3] if len(argv) > 3 else "bf16"
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    d = B.make_desc(m, d_in, d_out, r, 0, dtype)
    dev = "cuda"
    X = torch.randn(m, d_in, device=dev).to(tdt)
    W = (torch.randn(d_out, d_in, device=dev) * 0.02).to(tdt)
    G = torch.randn(m, d_out, device=dev).to(tdt)
    XS = torch.randn(m, r, device=dev).to(tdt)
    Y = torch.empty(m, d_out, device=dev, dtype=tdt)
    dX = torch.empty(m, d_in, device=dev, dtype=tdt)
    A = torch.randn(d_out, r, device=dev)
    Vt = (torch.randn(r, d_in, device=dev) * d_in ** -0.5).to(tdt) if op.endswith("_v") or op == "rsvd" else None
    ws_v = B.alloc_workspace(d, B.ACX_OP_RSVD) if op == "rsvd" else None
    dW = torch.empty(d_out, d_in, device=dev)
    mom = torch.zeros(d_out, d_in, device=dev) if op == "adamw" else None
    var = torch.zeros(d_out, d_in, device=dev) if op == "adamw" else None
    W_lp = torch.empty(d_out, d_in, device=dev, dtype=torch.bfloat16) if op == "adamw" else None
    mA, vA = torch.zeros(d_out, r, device=dev), torch.zeros(d_out, r, device=dev)
    db = torch.empty(d_out, device=dev) if op == "factor_bias" else None
    ws_bb = B.alloc_workspace(d, B.ACX_OP_BWD_BIAS) if op == "factor_bias" else None
    ws_f = B.alloc_workspace(d, B.ACX_OP_FWD)
    ws_b = B.alloc_workspace(d, B.ACX_OP_BWD)
    ws_r = B.alloc_workspace(d, B.ACX_OP_RECONSTRUCT)
    for _ in range(launches):
        if op == "fwd":
            B.acx_linear_fwd(d, X, W, Y, XS, ws_f)
        elif op == "fwd_nows":
            B.acx_linear_fwd(d, X, W, Y, XS)
        elif op == "fwd_plain":
            B.acx_linear_fwd(d, X, W, Y, None)
        elif op == "fwd_v":
            B.acx_linear_fwd_v(d, X, W, Vt, Y, XS)
        elif op == "reconstruct_v":
            B.acx_reconstruct_v(d, A, Vt, dW, 0.0, ws_r)
        elif op == "dx":
            B.acx_linear_bwd(d, G, W, XS, dX, None, ws_b)
        elif op == "factor":
            B.acx_linear_bwd(d, G, W, XS, None, A, ws_b)
        elif op == "reconstruct":
            B.acx_reconstruct(d, A, dW, 0.0, ws_r)
        elif op == "factor_bias":
            B.acx_linear_bwd_bias(d, G, None, XS, None, A, db, ws_bb)
        elif op == "rsvd":
            B.acx_rsvd_factor(d, X, XS, Vt, ws_v)
        elif op == "lowrank_adamw":
            B.acx_lowrank_adamw(d, A, mA, vA, dW, step=2, lr=1e-3, weight_decay=0.01, ws=ws_r)
        elif op == "adamw":
            B.acx_reconstruct_adamw(d, A, dW, mom, var, W_lp, step=2, lr=1e-3, weight_decay=0.01, ws=ws_r)
        else:
            raise SystemExit("unknown op %r" % op)
    torch.cuda.synchronize()
    st = B.acx_last_device_status()
    if st != B.ACX_OK:
        raise SystemExit(B.status_string(st))
    print("ok")
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv[1:]))
