"""The workspace-free gradient factor: acx_linear_bwd_factor_builtin_scratch against acx_linear_bwd.

Some users of the library cannot hand it a workspace: their memory pool already owns the GPU, or they
run inside a callback that may not re-enter the allocator.  For them the library carries a 16 MiB
scratch array of its own.  This file checks, through the C ABI, that the factor computed in that
array equals the one computed in a caller's workspace, on two calls in a row that use different
amounts of the array (so stale contents of the first call lie under the second), and that a shape
whose partial sums do not fit is refused before anything is launched.

It is named to be collected last, so a run that stops at the first failure has run everything else.
"""
import ctypes
import gc

import numpy as np
import pytest
import torch

from paper_2605_01255_b200 import binding as B
from paper_2605_01255_b200 import inputs as I

from oracle import linear as ol

from _harness import TOL_DERIVED, GpuLinear, assert_parity, to_device, to_host

pytestmark = pytest.mark.gpu


def _factor_both_ways(m, d_out, r, seed):
    Gh, XSh = I.gaussian((m, d_out), 40 + seed, 1.0, "bf16"), I.gaussian((m, r), 50 + seed, 1.0, "bf16")
    G, XS = to_device(Gh, "bf16"), to_device(XSh, "bf16")
    W = torch.zeros(d_out, 256, dtype=torch.bfloat16, device="cuda")
    lin = GpuLinear(m, 256, d_out, r, seed, "bf16")
    _, A_ws = lin.bwd(G, W, XS, want_dx=False)
    A_builtin = torch.full((d_out, r), float("nan"), dtype=torch.float32, device="cuda")
    gc.collect()   # tensors of earlier tests or calls that only await collection must not be freed in mid-measurement
    torch.cuda.synchronize()
    allocated = torch.cuda.memory_allocated()
    B.acx_linear_bwd_factor_builtin_scratch(lin.desc, G, XS, A_builtin)
    assert torch.cuda.memory_allocated() == allocated
    lin.check_status()
    # and against the CPU oracle's factor of the same inputs (Section 4: A = G^T U)
    _, A0 = ol.linear_bwd(Gh, np.zeros((d_out, 8)), XSh)
    assert_parity("A (built-in scratch)", to_host(A_builtin), A0, "factor", TOL_DERIVED["bf16"], (m, d_out, r))
    return lin, A_ws, A_builtin


def test_builtin_scratch_factor_matches_workspace_factor_twice_in_a_row():
    # first a shape that splits the tokens many ways (large part of the array), then a smaller one
    for m, d_out, r, seed in ((8192, 512, 128, 1), (3000, 264, 48, 2)):
        lin, A_ws, A_builtin = _factor_both_ways(m, d_out, r, seed)
        assert B.acx_workspace_bytes(lin.desc, B.ACX_OP_BWD_BUILTIN_SCRATCH) > 0, "case must exercise the scratch"
        want, got = to_host(A_ws), to_host(A_builtin)
        assert np.isfinite(got).all()
        err = np.linalg.norm(got - want) / np.linalg.norm(want)
        assert err <= TOL_DERIVED["bf16"], err


def test_builtin_scratch_limit_and_dtype_are_checked_before_launch():
    m, d_out, r = 16384, 9472, 256
    desc = B.make_desc(m, 256, d_out, r, 0, "bf16")
    if B.acx_workspace_bytes(desc, B.ACX_OP_BWD_BUILTIN_SCRATCH) <= B.ACX_BUILTIN_SCRATCH_BYTES:
        pytest.skip("this GPU's split plan fits the built-in scratch")
    G = torch.zeros(m, d_out, dtype=torch.bfloat16, device="cuda")
    XS = torch.zeros(m, r, dtype=torch.bfloat16, device="cuda")
    A = torch.full((d_out, r), 3.0, dtype=torch.float32, device="cuda")
    launches = B.acx_kernel_launches()
    with pytest.raises(B.AcxError) as e:
        B.acx_linear_bwd_factor_builtin_scratch(desc, G, XS, A)
    assert e.value.status == B.ACX_ERR_SCRATCH_LIMIT
    assert B.acx_kernel_launches() == launches and float(A.min()) == 3.0
    # fp32 descriptors are not served by this entry point
    desc32 = B.make_desc(64, 64, 64, 16, 0, "f32")
    rc = B.lib().acx_linear_bwd_factor_builtin_scratch(ctypes.byref(desc32), G.data_ptr(), XS.data_ptr(),
                                                       A.data_ptr(), None)
    assert rc == B.ACX_ERR_INVALID_ARG
