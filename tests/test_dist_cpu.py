"""The N-sharded data-parallel EM step on two CPU ranks (gloo): each rank's statistics over its own rows, one
all-reduce (sum) of (N_k, S1, S2, loglik), replicated parameter update.  The per-rank compute stands in for
gmm_em_step with the float64 oracle; what is tested is the sharding and exchange logic bench.py uses for N > 1 GPUs.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import gmm_oracle as orc
from paper_2606_10896_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n_per_rank, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        spec = synth.CONFIGS[1].with_n(n_per_rank)
        X = synth.sample_host(spec, stream=rank)                       # every rank draws its own shard
        pi, mu, var = synth.init_params(X, spec)
        params = [torch.from_numpy(a) for a in (pi, mu, var)]
        for p in params:                                               # rank 0's initial parameters for everybody
            dist.broadcast(p, 0)
        pi, mu, var = (p.numpy() for p in params)
        N_global = n_per_rank * world
        trace = []
        for _ in range(3):
            Nk, S1, S2, L = orc.em_step(X, pi, mu, var, nthreads=1)
            bufs = [torch.from_numpy(Nk), torch.from_numpy(S1), torch.from_numpy(S2), torch.tensor([L], dtype=torch.float64)]
            for b in bufs:
                dist.all_reduce(b)
            trace.append(float(bufs[3][0]))
            pi, mu, var = orc.finalize_moments(N_global, bufs[0].numpy(), bufs[1].numpy(), bufs[2].numpy(),
                                               spec.var_floor, mu, var)
            pi, mu, var = pi.astype(np.float32), mu.astype(np.float32), var.astype(np.float32)
        q.put((rank, pi, mu, var, trace))
    finally:
        dist.destroy_process_group()


def test_two_rank_sharded_em_equals_single_process():
    world, n_per_rank = 2, 1500
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, n_per_rank, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = [q.get(timeout=180) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    results.sort(key=lambda r: r[0])
    # replicas agree bit for bit
    for a, b in zip(results[0][1:4], results[1][1:4]):
        assert np.array_equal(a, b)
    assert results[0][4] == results[1][4]
    # and equal the single-process run over the concatenated shards
    spec = synth.CONFIGS[1].with_n(n_per_rank)
    X = np.concatenate([synth.sample_host(spec, stream=r) for r in range(world)])
    pi, mu, var = synth.init_params(synth.sample_host(spec, stream=0), spec)
    trace = []
    for _ in range(3):
        Nk, S1, S2, L = orc.em_step(X, pi, mu, var, nthreads=1)
        trace.append(L)
        pi, mu, var = orc.finalize_moments(len(X), Nk, S1, S2, spec.var_floor, mu, var)
        pi, mu, var = pi.astype(np.float32), mu.astype(np.float32), var.astype(np.float32)
    np.testing.assert_allclose(results[0][4], trace, rtol=1e-12)
    np.testing.assert_allclose(results[0][1], pi, rtol=1e-6)
    np.testing.assert_allclose(results[0][2], mu, rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(results[0][3], var, rtol=1e-5)
