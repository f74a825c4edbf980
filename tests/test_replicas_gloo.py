"""The N > 1 path of the benchmark on CPU: two gloo ranks, replicas only (no data-path collective)."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_01255_b200 import replicas as R


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert R.world_info() == (rank, world)
        R.barrier()
        ms_local = 10.0 + 5.0 * rank          # rank 1 is the slow one
        value, ms = R.job_throughput(16384, ms_local)
        out.put((rank, value, ms))
        R.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_sum_of_tokens():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, ms in got:
        assert ms == 15.0                                   # the maximum over ranks, on every rank
        assert abs(value - 2 * 16384 / 15e-3) < 1e-6        # tokens of all ranks / slowest time


def test_single_process_needs_no_process_group():
    assert R.world_info() == (0, 1)
    R.barrier()
    assert R.job_throughput(100, 2.0) == (100 / 2e-3, 2.0)
