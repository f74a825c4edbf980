"""Layer-stack harness: the compressed linear operator applied to every linear of a stack of decoder layers.

Forward pass: each linear computes Y = X W^T and the factor XS through ``acx_linear_fwd``; of the layer
input only XS is kept (one per distinct input: q/k/v share one, gate/up share one), which is the memory
saving of Definition 3.1.  Backward pass, last layer first: ``acx_linear_bwd`` gives dX and the gradient
factor A = G^T XS per linear, and ``acx_reconstruct`` rebuilds dW when asked (optimizer strategy (i) of
Section 4).  Everything numeric happens in libacx; this module only owns buffers and call order.

The nonlinear operators between the linears are not part of this library, so the layer inputs X and the
output gradients G are supplied by the caller (synthetic in the tests and the benchmark).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Dict, List, Optional, Tuple

import torch

from . import binding as B
from . import inputs as I


@dataclass
class StackReport:
    layers: int
    tokens: int
    stored_bytes_compressed: int    # sum of the XS kept for the backward pass
    stored_bytes_uncompressed: int  # what keeping X itself would take
    factor_bytes: int               # sum of the gradient factors A (fp32)
    dense_grad_bytes: int           # what dense fp32 weight gradients would take

    @property
    def saved_bytes(self) -> int:
        return self.stored_bytes_uncompressed - self.stored_bytes_compressed


def slots_of(wl: I.Workload) -> Dict[int, int]:
    """slot -> width of the distinct layer inputs of a workload."""
    return {lin.slot: lin.d_in for lin in wl.linears}


def report(wl: I.Workload, tokens: Optional[int] = None, layers: Optional[int] = None) -> StackReport:
    m, L = tokens or wl.tokens, layers or wl.layers
    e = 2 if wl.dtype == "bf16" else 4
    slots = slots_of(wl)
    return StackReport(
        layers=L, tokens=m,
        stored_bytes_compressed=L * len(slots) * m * wl.r * e,
        stored_bytes_uncompressed=L * sum(m * d * e for d in slots.values()),
        factor_bytes=L * sum(lin.d_out * wl.r * 4 for lin in wl.linears),
        dense_grad_bytes=L * sum(lin.d_out * lin.d_in * 4 for lin in wl.linears))


class CompressedStack:
    """Buffers and call order for `layers` decoder layers of `wl.linears`.

    weights[(layer, k)] are device tensors (d_out x d_in) supplied by the caller; several layers may
    share one tensor.  XS is kept per (layer, slot); Y and dX go to scratch buffers that are reused by
    every layer, so the only activation memory that grows with depth is the stored XS.
    """

    def __init__(self, wl: I.Workload, weights: Dict[Tuple[int, int], torch.Tensor], tokens: Optional[int] = None,
                 layers: Optional[int] = None, seed_base: int = 0, device="cuda"):
        self.wl, self.m, self.L = wl, tokens or wl.tokens, layers or wl.layers
        self.dtype = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
        self.dev = torch.device(device)
        self.weights = weights
        self.seed_base = seed_base
        self.desc = {}
        for l in range(self.L):
            for k, lin in enumerate(wl.linears):
                self.desc[(l, k)] = self._desc(l, k, 0)
        slots = slots_of(wl)
        self.XS = {(l, s): torch.empty(self.m, wl.r, dtype=self.dtype, device=self.dev) for l in range(self.L) for s in slots}
        self.A = {(l, k): torch.empty(lin.d_out, wl.r, dtype=torch.float32, device=self.dev)
                  for l in range(self.L) for k, lin in enumerate(wl.linears)}
        widest_out = max(lin.d_out for lin in wl.linears)
        widest_in = max(lin.d_in for lin in wl.linears)
        self._Y = torch.empty(self.m * widest_out, dtype=self.dtype, device=self.dev)
        self._dX = torch.empty(self.m * widest_in, dtype=self.dtype, device=self.dev)
        ws_b = max(B.acx_workspace_bytes(d, B.ACX_OP_BWD) for d in self.desc.values())
        ws_r = max(B.acx_workspace_bytes(d, B.ACX_OP_RECONSTRUCT) for d in self.desc.values())
        ws_f = max(B.acx_workspace_bytes(d, B.ACX_OP_FWD) for d in self.desc.values())
        self._ws = torch.empty(max(ws_f, ws_b, ws_r, 16), dtype=torch.uint8, device=self.dev)

    def _desc(self, l: int, k: int, sketch_step: int):
        """Descriptor of linear k of layer l with the sketch seed of training step `sketch_step`."""
        if sketch_step == 0 and (l, k) in self.desc:
            return self.desc[(l, k)]
        lin = self.wl.linears[k]
        return B.make_desc(self.m, lin.d_in, lin.d_out, self.wl.r, I.sketch_seed(self.seed_base, l, lin.slot, sketch_step), self.wl.dtype)

    def _view(self, flat: torch.Tensor, rows: int, cols: int) -> torch.Tensor:
        return flat[: rows * cols].view(rows, cols)

    def forward_layer(self, l: int, x_of_slot: Callable[[int], torch.Tensor], keep_y: bool = False,
                      sketch_step: int = 0) -> List[Optional[torch.Tensor]]:
        """Runs the linears of layer l; x_of_slot(slot) returns that layer's input (tokens x width).

        sketch_step: number of the training step.  With optimizer strategy (i) (the full gradient rebuilt every step)
        pass the step counter, the same in forward_layer and backward_layer of one step: every step then draws fresh
        sketches, which is what makes the rebuilt gradients unbiased over the run (Theorem 3.2(a) takes the
        expectation over the compression randomness; a sketch that never changes would project every step's gradient
        on the same r-dimensional subspace).  Leave it 0 with strategy (ii) (`lowrank`), whose moments live in the
        factor space and need the second factor to stay fixed."""
        outs: List[Optional[torch.Tensor]] = []
        stored = set()  # the factor of an input is written by the first linear that reads it, the others skip it
        for k, lin in enumerate(self.wl.linears):
            Y = torch.empty(self.m, lin.d_out, dtype=self.dtype, device=self.dev) if keep_y else self._view(self._Y, self.m, lin.d_out)
            XS = None if lin.slot in stored else self.XS[(l, lin.slot)]
            stored.add(lin.slot)
            B.acx_linear_fwd(self._desc(l, k, sketch_step), x_of_slot(lin.slot), self.weights[(l, k)], Y, XS, self._ws)
            outs.append(Y if keep_y else None)
        return outs

    def backward_layer(self, l: int, g_of_linear: Callable[[int], torch.Tensor], keep_dx: bool = False,
                       dW: Optional[Dict[int, torch.Tensor]] = None, beta: float = 0.0,
                       lowrank: Optional[Dict[int, Tuple[torch.Tensor, torch.Tensor, torch.Tensor]]] = None,
                       step: int = 1, sketch_step: int = 0, **hyper) -> List[Optional[torch.Tensor]]:
        """Runs the backward of layer l; g_of_linear(k) returns dL/dY of linear k.  If dW is given
        (k -> d_out x d_in fp32) the full gradient is rebuilt into it as beta * dW + A S^T (optimizer strategy (i) of
        Section 4).  If lowrank is given (k -> (fp32 weights, m_A, v_A)) the GaLore-style step of strategy (ii) is applied
        to those weights instead, with `step` and the AdamW hyper-parameters in `hyper` (lr=..., weight_decay=..., ...).
        sketch_step: the value given to forward_layer for this step (0 with `lowrank`, which needs a fixed sketch)."""
        if lowrank is not None and sketch_step != 0:
            raise ValueError("low-rank optimizer states need the same sketch in every step: leave sketch_step at 0")
        outs: List[Optional[torch.Tensor]] = []
        for k, lin in enumerate(self.wl.linears):
            dX = torch.empty(self.m, lin.d_in, dtype=self.dtype, device=self.dev) if keep_dx else self._view(self._dX, self.m, lin.d_in)
            desc = self._desc(l, k, sketch_step)
            B.acx_linear_bwd(desc, g_of_linear(k), self.weights[(l, k)], self.XS[(l, lin.slot)], dX,
                             self.A[(l, k)], self._ws)
            if dW is not None and k in dW:
                B.acx_reconstruct(desc, self.A[(l, k)], dW[k], beta, self._ws)
            if lowrank is not None and k in lowrank:
                Wm, mA, vA = lowrank[k]
                B.acx_lowrank_adamw(self.desc[(l, k)], self.A[(l, k)], mA, vA, Wm, step=step, ws=self._ws, **hyper)
            outs.append(dX if keep_dx else None)
        return outs

    def check_status(self) -> None:
        st = B.acx_last_device_status()
        if st != B.ACX_OK:
            raise B.AcxError(st, "CompressedStack")
