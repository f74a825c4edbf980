"""Host logic of token-sharded data parallelism for the compressed linear step (not used by the default benchmark,
which runs independent replicas).

Every rank holds the same weights and the same sketch seeds and processes its own shard of the tokens.  Forward and
dX are row-wise in the tokens, so they need no exchange.  The gradient factor is a sum over tokens,
A = sum over ranks of G_r^T (X_r S) (Section 4: the weight gradient in factored form), and S depends only on the seed,
so the one collective of a step is a sum of the factors A (d_out x r each) instead of the d_out x d_in gradients:
at LLaMA3-3B shapes with r = 128, 11.5 MB per decoder layer instead of 453 MB.  The factors of all linears travel in
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
