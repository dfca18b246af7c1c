"""Seeded synthetic inputs shaped like the paper's workloads (Table 1: K=1024, D=128, N=10K..100M; the IVF
datasets' shapes of Section 4.4 with K up to 4096).

This module is the one piece shared by the CUDA path's tests/benchmark and the CPU oracle's tests.  It holds none of
the method's arithmetic: it only draws points from a known diagonal mixture, picks initial parameters, and picks
subsample rows.  The public benchmark datasets the paper uses (SIFT1M, Deep10M, GloVe-100) are not reproduced; these
draws stand in for them.

Recipe (all seeded):
  * mixture: means ~ N(0, mean_std^2) per dimension, per-dimension std ~ U[std_lo, std_hi], weights ~ Dirichlet(1)
    (K exponential draws, normalised); with ``normalize`` the means are scaled to unit L2 norm;
  * a point: component c by inverse CDF of the weights, x = mu_c + std_c * z with z ~ N(0, 1), rounded once to
    float32; with ``normalize`` each point is then divided by its L2 norm;
  * initial parameters: means = the first K points or K distinct seeded rows, variances = the global per-dimension
    population variance (float64 accumulate), weights uniform.

Host draws use numpy's PCG64; device draws use torch's CUDA generator in fixed-size chunks (so a 51 GB X never
needs host memory).  The two streams differ; a test or benchmark uses one of them for both the GPU path and the
oracle, and the oracle always receives rows copied from the array the GPU saw.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class MixtureSpec:
    name: str
    N: int
    D: int
    K: int
    mean_std: float
    std_lo: float
    std_hi: float
    normalize: bool
    init: str          # "first" (first K points) or "random" (K distinct seeded rows)
    iters: int
    seed: int
    var_floor: float = 1e-6

    def with_n(self, n: int) -> "MixtureSpec":
        return replace(self, N=int(n))


CONFIGS = {
    1: MixtureSpec("tiny", 10_000, 16, 8, 5.0, 0.5, 2.0, False, "first", 10, 1),
    2: MixtureSpec("paper-100K", 100_000, 128, 1024, 3.0, 0.5, 1.5, False, "random", 30, 2),
    3: MixtureSpec("paper-1M", 1_000_000, 128, 1024, 3.0, 0.5, 1.5, False, "random", 30, 3),
    4: MixtureSpec("paper-100M", 100_000_000, 128, 1024, 3.0, 0.5, 1.5, False, "random", 30, 4),
    5: MixtureSpec("ivf-10M", 10_000_000, 768, 4096, 1.0, 0.02, 0.08, True, "random", 20, 5),
}


def true_params(spec: MixtureSpec):
    """(weights [K], means [K, D], stds [K, D]) of the generating mixture, float64."""
    rng = np.random.Generator(np.random.PCG64(spec.seed))
    means = rng.normal(0.0, spec.mean_std, size=(spec.K, spec.D))
    if spec.normalize:
        means /= np.linalg.norm(means, axis=1, keepdims=True)
    stds = rng.uniform(spec.std_lo, spec.std_hi, size=(spec.K, spec.D))
    w = rng.exponential(1.0, size=spec.K)
    w /= w.sum()
    return w, means, stds


def sample_host(spec: MixtureSpec, n: int | None = None, stream: int = 0) -> np.ndarray:
    """n (default spec.N) points as float32 [n, D], drawn on the host."""
    n = spec.N if n is None else int(n)
    w, means, stds = true_params(spec)
    rng = np.random.Generator(np.random.PCG64([spec.seed, 7919 + stream]))
    comp = np.searchsorted(np.cumsum(w), rng.random(n), side="right").clip(0, spec.K - 1)
    X = np.empty((n, spec.D), np.float32)
    step = max(1, (1 << 24) // spec.D)
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        c = comp[lo:hi]
        x = means[c] + stds[c] * rng.standard_normal((hi - lo, spec.D))
        if spec.normalize:
            x /= np.linalg.norm(x, axis=1, keepdims=True)
        X[lo:hi] = x.astype(np.float32)
    return X


def sample_device(spec: MixtureSpec, device, n: int | None = None, chunk_rows: int = 1 << 20, stream: int = 0):
    """n (default spec.N) points as a float32 torch tensor [n, D] generated on ``device`` in chunks.

    ``stream`` selects an independent draw from the same mixture (one per rank in a sharded run)."""
    import torch

    n = spec.N if n is None else int(n)
    w, means, stds = true_params(spec)
    gen = torch.Generator(device=device)
    gen.manual_seed(spec.seed * 1_000_003 + 17 + 7919 * stream)
    cdf = torch.tensor(np.cumsum(w), dtype=torch.float64, device=device)
    means_d = torch.tensor(means, dtype=torch.float32, device=device)
    stds_d = torch.tensor(stds, dtype=torch.float32, device=device)
    X = torch.empty((n, spec.D), dtype=torch.float32, device=device)
    for lo in range(0, n, chunk_rows):
        hi = min(n, lo + chunk_rows)
        u = torch.rand(hi - lo, dtype=torch.float64, device=device, generator=gen)
        c = torch.searchsorted(cdf, u, right=True).clamp_(0, spec.K - 1)
        z = torch.randn((hi - lo, spec.D), dtype=torch.float32, device=device, generator=gen)
        x = torch.addcmul(means_d[c], stds_d[c], z)
        if spec.normalize:
            x = x / x.norm(dim=1, keepdim=True)
        X[lo:hi] = x
        del u, c, z, x
    return X


def distinct_rows(N: int, n: int, seed: int) -> np.ndarray:
    """n distinct row indices in [0, N), seeded, in draw order (partial Fisher-Yates on a sparse permutation)."""
    if n > N:
        raise ValueError("cannot draw more distinct rows than there are rows")
    rng = np.random.Generator(np.random.PCG64([seed, 104729]))
    swapped: dict[int, int] = {}
    out = np.empty(n, np.int64)
    for j in range(n):
        r = j + int(rng.integers(0, N - j))
        vj = swapped.get(j, j)
        vr = swapped.get(r, r)
        out[j] = vr
        swapped[r] = vj
    return out


def subsample_rows(N: int, n: int, seed: int) -> np.ndarray:
    """n distinct seeded row indices, sorted ascending (the rows an oracle check gathers)."""
    return np.sort(distinct_rows(N, min(n, N), seed ^ 0x5BD1E995))


def global_variance(X) -> np.ndarray:
    """Per-dimension population variance of X (numpy array or torch tensor), accumulated in float64 -> [D]."""
    if isinstance(X, np.ndarray):
        step = max(1, (1 << 24) // X.shape[1])
        s1 = np.zeros(X.shape[1])
        s2 = np.zeros(X.shape[1])
        for lo in range(0, X.shape[0], step):
            x = X[lo:lo + step].astype(np.float64)
            s1 += x.sum(0)
            s2 += (x * x).sum(0)
        m = s1 / X.shape[0]
        return s2 / X.shape[0] - m * m
    import torch

    s1 = torch.zeros(X.shape[1], dtype=torch.float64, device=X.device)
    s2 = torch.zeros_like(s1)
    step = max(1, (1 << 24) // X.shape[1])
    for lo in range(0, X.shape[0], step):
        x = X[lo:lo + step].double()
        s1 += x.sum(0)
        s2 += (x * x).sum(0)
    m = s1 / X.shape[0]
    return (s2 / X.shape[0] - m * m).cpu().numpy()


def init_params(X, spec: MixtureSpec):
    """Initial (pi [K], mu [K, D], var [K, D]) as float32 numpy arrays, per the config's init rule."""
    K, D = spec.K, spec.D
    N = X.shape[0]
    rows = np.arange(K) if spec.init == "first" else distinct_rows(N, K, spec.seed)
    if isinstance(X, np.ndarray):
        mu = X[rows].astype(np.float32)
    else:
        import torch

        mu = X[torch.as_tensor(rows, device=X.device)].cpu().numpy().astype(np.float32)
    gv = global_variance(X)
    var = np.broadcast_to(gv.astype(np.float32), (K, D)).copy()
    pi = np.full(K, 1.0 / K, np.float32)
    return pi, mu, var
