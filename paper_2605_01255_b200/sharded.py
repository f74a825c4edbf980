"""Host logic of token-sharded data parallelism for the compressed linear step (not used by the default benchmark,
which runs independent replicas).

Every rank holds the same weights and the same sketch seeds and processes its own shard of the tokens.  Forward and
dX are row-wise in the tokens, so they need no exchange.  The gradient factor is a sum over tokens,
A = sum over ranks of G_r^T (X_r S) (Section 4: the weight gradient in factored form), and S depends only on the seed,
so the one collective of a step is a sum of the factors A (d_out x r each) instead of the d_out x d_in gradients:
at LLaMA3-3B shapes with r = 128, 16.3 MB per decoder layer instead of 453 MB.  The factors of all linears travel in
one flat fp32 bucket, one all-reduce per call.  Works on any torch.distributed backend (NCCL on GPUs; gloo in the CPU
tests); the reduction order is the backend's, so bitwise reproducibility across world sizes is not claimed.
"""
from __future__ import annotations

from typing import Optional, Sequence, Tuple

import torch
import torch.distributed as dist


def token_shard(tokens: int, rank: int, world: int) -> Tuple[int, int]:
    """(first token, number of tokens) of a rank: contiguous shards whose sizes differ by at most one."""
    if not (0 <= rank < world):
        raise ValueError("rank %d outside world of %d" % (rank, world))
    base, extra = divmod(tokens, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def factor_bucket_bytes(factors: Sequence[torch.Tensor]) -> int:
    return sum(a.numel() * 4 for a in factors)


def allreduce_factors(factors: Sequence[torch.Tensor], group=None, bucket: Optional[torch.Tensor] = None) -> None:
    """Sums the gradient factors (fp32, any shapes) over the ranks, in place, with one all-reduce.

    `bucket` may be a preallocated flat fp32 tensor of at least the total size (it is overwritten)."""
    if not factors:
        return
    for a in factors:
        if a.dtype != torch.float32:
            raise ValueError("gradient factors are fp32")
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return
    total = sum(a.numel() for a in factors)
    flat = bucket[:total] if bucket is not None else torch.empty(total, dtype=torch.float32, device=factors[0].device)
    if flat.numel() < total or flat.dtype != torch.float32:
        raise ValueError("bucket too small or not fp32")
    off = 0
    for a in factors:
        flat[off:off + a.numel()].copy_(a.reshape(-1))
        off += a.numel()
    dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
    off = 0
    for a in factors:
        a.copy_(flat[off:off + a.numel()].view_as(a))
        off += a.numel()


class ShardedStep:
    """Call order of one token-sharded training step over a stack of layers.  The compute is injected:

        fwd_layer(l)            forward of every linear of layer l on this rank's token shard (XS kept)
        bwd_layer(l)            dX and the LOCAL gradient factors of layer l
        factors_of_layer(l)     the fp32 factor tensors of layer l (summed in place over the ranks)
        reconstruct_layer(l)    whatever consumes the summed factors (rebuild dW, or an optimizer step)

    The factors of one layer travel as one bucket; the reduction of layer l is started right after its factors
    exist and is only waited for after the backward of layer l-1 has been queued, so on a GPU it overlaps that
    layer's dX and factor kernels (`comm_stream`: a side stream for the collective; None runs it in line, as the
    CPU tests do).  `bucket` is a flat fp32 tensor large enough for the largest layer.
    """

    def __init__(self, n_layers: int, fwd_layer, bwd_layer, factors_of_layer, reconstruct_layer, group=None,
                 bucket: Optional[torch.Tensor] = None, comm_stream=None, on_reduce=None):
        self.n_layers = n_layers
        self.fwd_layer, self.bwd_layer = fwd_layer, bwd_layer
        self.factors_of_layer, self.reconstruct_layer = factors_of_layer, reconstruct_layer
        self.group, self.bucket, self.comm_stream = group, bucket, comm_stream
        self.on_reduce = on_reduce            # on_reduce(l, "begin" | "end"): timing hooks, called on the stream that reduces
        self.reduced_bytes = 0

    def _reduce(self, l: int):
        """Starts the all-reduce of layer l's factors; returns what _finish needs to wait for it."""
        factors = list(self.factors_of_layer(l))
        self.reduced_bytes += factor_bucket_bytes(factors)
        if self.comm_stream is None:
            if self.on_reduce:
                self.on_reduce(l, "begin")
            allreduce_factors(factors, self.group, self.bucket)
            if self.on_reduce:
                self.on_reduce(l, "end")
            return None
        main = torch.cuda.current_stream()
        ready = torch.cuda.Event()
        ready.record(main)
        with torch.cuda.stream(self.comm_stream):
            self.comm_stream.wait_event(ready)
            if self.on_reduce:
                self.on_reduce(l, "begin")
            allreduce_factors(factors, self.group, self.bucket)
            if self.on_reduce:
                self.on_reduce(l, "end")
            done = torch.cuda.Event()
            done.record(self.comm_stream)
        return done

    def _finish(self, done) -> None:
        if done is not None:
            torch.cuda.current_stream().wait_event(done)

    def run(self) -> None:
        for l in range(self.n_layers):
            self.fwd_layer(l)
        pending = None
        for l in reversed(range(self.n_layers)):
            self.bwd_layer(l)
            done = self._reduce(l)
            if pending is not None:   # the layer above: its sum had the time of this layer's backward to arrive
                self._finish(pending[1])
                self.reconstruct_layer(pending[0])
            pending = (l, done)
        if pending is not None:
            self._finish(pending[1])
            self.reconstruct_layer(pending[0])
