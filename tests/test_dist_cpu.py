"""The N-sharded data-parallel EM step on two CPU ranks (gloo), through the shipped code: ShardedEM packs every rank's
(N_k, S1, S2, loglik) into one float64 buffer, reduces it with one all-reduce (or an ordered all-gather) and applies
the replicated parameter update -- the lines bench.py runs for N > 1 GPUs.  Only the per-rank compute is injected
here: the float64 oracle stands in for gmm_em_step / gmm_finalize, which need a GPU.
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
from paper_2606_10896_b200.sharded import ShardedEM, pack_size


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _oracle_step(X, pi, mu, var):
    return orc.em_step(X, pi, mu, var, nthreads=1)


def _oracle_finalize(N, Nk, S1, S2, var_floor, pi, mu, var):
    p, m, v = orc.finalize_moments(N, Nk.numpy(), S1.numpy(), S2.numpy(), var_floor, mu, var)
    pi[...] = p.astype(np.float32)
    mu[...] = m.astype(np.float32)
    var[...] = v.astype(np.float32)


def _worker(rank, world, port, n_per_rank, ordered, q):
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
        em = ShardedEM(em_step=_oracle_step, finalize=_oracle_finalize, ordered=ordered)
        assert em.world() == world
        trace = em.fit(X, pi, mu, var, n_per_rank * world, 3, spec.var_floor)
        assert em._buf.numel() == pack_size(spec.K, spec.D)            # one buffer, one collective per iteration
        q.put((rank, pi, mu, var, trace.tolist()))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("ordered", [False, True])
def test_two_rank_sharded_em_equals_single_process(ordered):
    world, n_per_rank = 2, 1500
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, n_per_rank, ordered, q)) for r in range(world)]
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


def test_sharded_em_without_a_process_group_is_the_plain_iteration():
    spec = synth.CONFIGS[1].with_n(800)
    X = synth.sample_host(spec)
    pi, mu, var = synth.init_params(X, spec)
    em = ShardedEM(em_step=_oracle_step, finalize=_oracle_finalize)
    p, m, v = pi.copy(), mu.copy(), var.copy()
    L = em.step(X, p, m, v, len(X), spec.var_floor)
    Nk, S1, S2, Lr = orc.em_step(X, pi, mu, var, nthreads=1)
    pr, mr, vr = orc.finalize_moments(len(X), Nk, S1, S2, spec.var_floor, mu, var)
    assert L == Lr
    np.testing.assert_array_equal(m, mr.astype(np.float32))
    np.testing.assert_array_equal(v, vr.astype(np.float32))
    np.testing.assert_array_equal(p, pr.astype(np.float32))
