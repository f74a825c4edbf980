"""Host logic of the multi-GPU benchmark: independent replicas, one process per GPU.

The compressed linear step has no exchange between GPUs (one GPU, no sharding): N ranks run N replicas
of the same step on their own batches.  The only communication is the barrier around the timed region
and the reduction of the timing: the step time of the job is the maximum over ranks, and the job's
throughput is the tokens of all ranks divided by it.  Works on any torch.distributed backend (NCCL on
GPUs; gloo in the CPU tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def world_info():
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def barrier(device=None) -> None:
    """Device work done, every rank here, device work done: the bracket around a timed region."""
    on_gpu = device is not None and torch.device(device).type == "cuda"
    if on_gpu:
        torch.cuda.synchronize()
    if world_info()[1] > 1:
        dist.barrier()
    if on_gpu:
        torch.cuda.synchronize()


def max_over_ranks(x: float, device=None) -> float:
    if world_info()[1] == 1:
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(tokens_per_rank: int, ms_local: float, device=None):
    """(tokens/s of the whole job, ms of the slowest rank) for replicas that each process tokens_per_rank."""
    ms = max_over_ranks(ms_local, device)
    return world_info()[1] * tokens_per_rank / (ms * 1e-3), ms
