"""The EM iteration sharded over the points (one process per GPU): every rank takes gmm_em_step over its own rows, the
sufficient statistics and the log-likelihood travel in ONE packed float64 buffer of K (2 D + 1) + 1 values through one
all-reduce (sum), and the parameter update is replicated on every rank.

The statistics are additive over points (Algorithm 1 adds per-tile statistics into one set of O(K D) buffers; the
paper's Limitations section sketches the same for chunks of a data set that exceeds one device), so nothing else has to
cross between ranks, and 1 MB (K = 1024, D = 128) to 50 MB (K = 4096, D = 768) per iteration against hundreds of
milliseconds of compute needs no fused collective.

`torch.distributed` does the exchange (NCCL on GPUs, gloo on CPU).  The per-rank compute and the update are the
library's gmm_em_step / gmm_finalize unless other callables are passed in (the CPU tests pass the oracle's, so that
the packing, the reduction and the update call below are the lines that run in production).
"""
from __future__ import annotations

from typing import Callable, Optional

import numpy as np
import torch
import torch.distributed as dist


def pack_size(K: int, D: int) -> int:
    return K * (2 * D + 1) + 1


class ShardedEM:
    """One EM iteration over points sharded across the ranks of a process group.

    ctx        a flashgmm.Context on this rank's device (not needed when em_step and finalize are given)
    group      the torch.distributed process group (None: the default group; with no initialised group or a world of one
               the exchange is skipped)
    em_step    callable (X, pi, mu, var) -> (Nk [K], S1 [K, D], S2 [K, D], loglik) over this rank's rows
    finalize   callable (N_global, Nk, S1, S2, var_floor, pi, mu, var) updating pi, mu, var in place
    ordered    sum the ranks' buffers in rank order after an all-gather instead of an all-reduce: the result then does
               not depend on the reduction algorithm the backend picks (costs world x the bytes)
    """

    def __init__(self, ctx=None, group=None, em_step: Optional[Callable] = None, finalize: Optional[Callable] = None,
                 ordered: bool = False):
        if (em_step is None or finalize is None) and ctx is None:
            raise ValueError("pass a flashgmm.Context, or both em_step and finalize")
        self.ctx = ctx
        self.group = group
        self.em_step = em_step or (lambda X, pi, mu, var: ctx.gmm_em_step(X, pi, mu, var))
        self.finalize = finalize or (lambda N, Nk, S1, S2, fl, pi, mu, var: ctx.gmm_finalize(N, Nk, S1, S2, fl, pi, mu, var))
        self.ordered = ordered
        self._buf = None

    def world(self) -> int:
        if not (dist.is_available() and dist.is_initialized()):
            return 1
        return dist.get_world_size(self.group)

    def _buffer(self, K: int, D: int, device) -> torch.Tensor:
        n = pack_size(K, D)
        if self._buf is None or self._buf.numel() != n or self._buf.device != torch.device(device):
            self._buf = torch.empty(n, dtype=torch.float64, device=device)
        return self._buf

    def reduce(self, Nk, S1, S2, loglik: float):
        """(Nk, S1, S2, loglik) summed over the ranks.  The inputs may be torch tensors or numpy arrays; the outputs are
        views of one packed float64 tensor on the inputs' device."""
        Nk_t, S1_t, S2_t = (torch.as_tensor(a) for a in (Nk, S1, S2))
        K, D = S1_t.shape
        buf = self._buffer(K, D, Nk_t.device)
        KD = K * D
        buf[:K].copy_(Nk_t)
        buf[K:K + KD].copy_(S1_t.reshape(-1))
        buf[K + KD:K + 2 * KD].copy_(S2_t.reshape(-1))
        buf[K + 2 * KD] = float(loglik)
        world = self.world()
        if world > 1:
            if self.ordered:
                parts = [torch.empty_like(buf) for _ in range(world)]
                dist.all_gather(parts, buf, group=self.group)
                buf.copy_(parts[0])
                for p in parts[1:]:
                    buf.add_(p)
            else:
                dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=self.group)
        return buf[:K], buf[K:K + KD].view(K, D), buf[K + KD:K + 2 * KD].view(K, D), float(buf[K + 2 * KD].item())

    def step(self, X, pi, mu, var, N_global: int, var_floor: float) -> float:
        """One EM iteration: pi, mu, var are updated in place on every rank; returns the global log-likelihood under the
        parameters that entered the step."""
        Nk, S1, S2, L = self.em_step(X, pi, mu, var)
        Nk, S1, S2, L = self.reduce(Nk, S1, S2, L)
        self.finalize(int(N_global), Nk, S1, S2, float(var_floor), pi, mu, var)
        return L

    def fit(self, X, pi, mu, var, N_global: int, iters: int, var_floor: float = 1e-6, tol: float = 0.0):
        """`iters` iterations (the loop of gmm_fit); returns the trace of global log-likelihoods."""
        trace = []
        for t in range(int(iters)):
            trace.append(self.step(X, pi, mu, var, N_global, var_floor))
            if tol > 0.0 and t > 0 and abs(trace[t] - trace[t - 1]) <= tol * abs(trace[t]):
                break
        return np.asarray(trace, np.float64)
