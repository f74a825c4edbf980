"""Token-sharded data parallelism on CPU: two gloo ranks, the factors of their shards summed by one all-reduce equal
the factors of the whole batch (Section 4: the gradient factor is a sum over tokens, the sketch depends on the seed only)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import linear as ol
from oracle import sketch as osk
from paper_2605_01255_b200 import inputs as I
from paper_2605_01255_b200 import sharded as S

M, D_IN, R = 301, 64, 16      # an odd token count: shards of 151 and 150
D_OUTS = (24, 40)             # two linears that read the same input
SEED = 7


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _inputs():
    X = I.gaussian((M, D_IN), 1, 1.0, "f32")
    Gs = [I.gaussian((M, d), 2 + k, 1.0, "f32") for k, d in enumerate(D_OUTS)]
    return X, Gs


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        X, Gs = _inputs()
        t0, n = S.token_shard(M, rank, world)
        sketch = osk.sketch_for_dtype(SEED, D_IN, R, "f32")          # same seed on every rank: same S
        U = X[t0:t0 + n].astype(np.float64) @ sketch
        factors = [torch.from_numpy((G[t0:t0 + n].astype(np.float64).T @ U).astype(np.float32)) for G in Gs]
        bucket = torch.empty(S.factor_bucket_bytes(factors) // 4, dtype=torch.float32)
        S.allreduce_factors(factors, bucket=bucket)
        out.put((rank, n, [a.numpy().copy() for a in factors]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_sum_of_shard_factors_is_the_factor_of_the_batch():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted((o for o in (out.get(timeout=180) for _ in procs)), key=lambda o: o[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [151, 150]
    X, Gs = _inputs()
    sketch = osk.sketch_for_dtype(SEED, D_IN, R, "f32")
    _, U = ol.linear_fwd(X, np.zeros((8, D_IN)), sketch)
    for k, G in enumerate(Gs):
        _, A = ol.linear_bwd(G, np.zeros((G.shape[1], D_IN)), U)
        for rank in range(2):
            assert got[rank][2][k].shape == A.shape
            assert ol.rel_frobenius(got[rank][2][k], A) < 1e-6      # fp32 factors, fp32 sum
        assert np.array_equal(got[0][2][k], got[1][2][k])           # both ranks hold the same sum


def test_token_shards_cover_the_batch_once():
    for tokens, world in ((16384, 8), (301, 2), (5, 8), (0, 3)):
        spans = [S.token_shard(tokens, r, world) for r in range(world)]
        assert spans[0][0] == 0 and sum(n for _, n in spans) == tokens
        for (a, n), (b, _) in zip(spans, spans[1:]):
            assert a + n == b
        assert max(n for _, n in spans) - min(n for _, n in spans) <= 1
    with pytest.raises(ValueError):
        S.token_shard(10, 2, 2)


def test_single_process_is_a_noop():
    a = torch.ones(3, 4)
    S.allreduce_factors([a])
    assert torch.equal(a, torch.ones(3, 4))
    with pytest.raises(ValueError):
        S.allreduce_factors([a.double()])


# ---- the whole sharded step (forward, backward, one bucket per layer, reconstruct) with the compute injected
N_LAYERS = 2


def _step_inputs():
    """Per layer: X (M x D_IN), one G and one W per linear; the same on every rank (each takes its token shard)."""
    data = []
    for l in range(N_LAYERS):
        X = I.gaussian((M, D_IN), 10 + l, 1.0, "f32")
        Gs = [I.gaussian((M, d), 20 + 4 * l + k, 1.0, "f32") for k, d in enumerate(D_OUTS)]
        data.append((X, Gs))
    return data


def _step_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        data = _step_inputs()
        t0, n = S.token_shard(M, rank, world)
        sketches = [osk.sketch_for_dtype(SEED + l, D_IN, R, "f32") for l in range(N_LAYERS)]   # same seeds on every rank
        U, A, dW, log = {}, {}, {}, []

        def fwd_layer(l):
            log.append(("fwd", l))
            U[l] = data[l][0][t0:t0 + n].astype(np.float64) @ sketches[l]

        def bwd_layer(l):
            log.append(("bwd", l))
            A[l] = [torch.from_numpy((G[t0:t0 + n].astype(np.float64).T @ U[l]).astype(np.float32)) for G in data[l][1]]

        def reconstruct_layer(l):
            log.append(("rec", l))
            dW[l] = [a.numpy().astype(np.float64) @ sketches[l].T for a in A[l]]

        bucket = torch.empty(sum(d * R for d in D_OUTS), dtype=torch.float32)
        step = S.ShardedStep(N_LAYERS, fwd_layer, bwd_layer, lambda l: A[l], reconstruct_layer, bucket=bucket,
                             on_reduce=lambda l, what: log.append((what, l)))
        step.run()
        out.put((rank, log, {l: [w.copy() for w in dW[l]] for l in dW}, step.reduced_bytes))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_sharded_step_rebuilds_the_gradient_of_the_whole_batch():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_step_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted((o for o in (out.get(timeout=180) for _ in procs)), key=lambda o: o[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # order: forwards in layer order; the reduction of a layer starts right after its backward and its
    # reconstruction comes after the backward of the layer below has been queued
    want_log = [("fwd", 0), ("fwd", 1), ("bwd", 1), ("begin", 1), ("end", 1), ("bwd", 0), ("begin", 0), ("end", 0),
                ("rec", 1), ("rec", 0)]
    data = _step_inputs()
    for rank, log, dW, nbytes in got:
        assert log == want_log
        assert nbytes == N_LAYERS * sum(d * R for d in D_OUTS) * 4      # one bucket of factors per layer, nothing else
        for l, (X, Gs) in enumerate(data):
            sketch = osk.sketch_for_dtype(SEED + l, D_IN, R, "f32")
            _, Ufull = ol.linear_fwd(X, np.zeros((8, D_IN)), sketch)
            for k, G in enumerate(Gs):
                _, Afull = ol.linear_bwd(G, np.zeros((G.shape[1], D_IN)), Ufull)
                assert ol.rel_frobenius(dW[l][k], ol.reconstruct(Afull, sketch)) < 1e-6
