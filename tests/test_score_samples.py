"""Per-point log-density log p(x_i) under the mixture (Section 2; the per-point log-sum-exp of Section 3.2), the quantity
a kernel density estimate evaluates (Discussion, Section 6): parity of gmm_score_samples with the oracle.

The oracle side is oracle.gmm_oracle.responsibilities()[1], which tests/test_oracle_pins.py pins against brute-force
linear-space densities, a library log-sum-exp over univariate normal log-pdfs and scikit-learn's score_samples.

Tolerance, per point: 1e-5 |log p| + 1e-4.  The kernel forms direct-difference logits in fp32 (float64 beyond D = 128)
whose rounding is about 1e-7 of the summed magnitudes (a few hundred at D = 128), and the output is fp32.
"""
import numpy as np
import pytest

from oracle import gmm_oracle


def _case(seed, N, D, K, spread=2.0):
    rng = np.random.Generator(np.random.PCG64(seed))
    mu = rng.normal(0, spread, (K, D)).astype(np.float32)
    var = (rng.uniform(0.4, 1.6, (K, D)) ** 2).astype(np.float32)
    pi = rng.dirichlet(np.ones(K)).astype(np.float32)
    lab = rng.integers(0, K, N)
    X = (mu[lab] + 1.3 * np.sqrt(var[lab]) * rng.standard_normal((N, D))).astype(np.float32)
    return X, pi, mu, var


@pytest.mark.gpu
@pytest.mark.parametrize("N,D,K", [(1, 3, 1), (1000, 16, 8), (5000, 128, 1024), (3001, 130, 70), (700, 768, 64),
                                   ((1 << 20) + 1000, 8, 4)])
def test_gpu_score_samples_match_oracle(N, D, K):
    import torch
    from paper_2606_10896_b200 import flashgmm as fg

    X, pi, mu, var = _case(N % 1000 + D + K, N, D, K)
    if K > 4:
        pi = pi.copy()
        pi[1] = 0.0                        # a component of weight zero contributes nothing
        pi /= pi.sum()
    lz = gmm_oracle.responsibilities(X, pi, mu, var)[1]
    t = lambda v: torch.as_tensor(np.ascontiguousarray(v), device="cuda:0")
    with fg.Context(0) as ctx:
        logp, total = ctx.gmm_score_samples(t(X), t(pi), t(mu), t(var))
        logp2, total2 = ctx.gmm_score_samples(t(X), t(pi), t(mu), t(var))
        assert torch.equal(logp, logp2) and total == total2
        ll_step = ctx.gmm_em_step(t(X), t(pi), t(mu), t(var))[3]
    got = logp.cpu().numpy().astype(np.float64)
    assert got.shape == (N,) and np.isfinite(got).all()
    excess = np.abs(got - lz) - (1e-5 * np.abs(lz) + 1e-4)
    assert excess.max() <= 0, f"point {int(np.argmax(excess))}: {got[np.argmax(excess)]} vs {lz[np.argmax(excess)]}"
    assert abs(total - lz.sum()) <= 1e-5 * abs(lz.sum()) + 1e-6
    assert abs(total - ll_step) <= 1e-5 * abs(ll_step) + 1e-6


@pytest.mark.gpu
@pytest.mark.parametrize("N,D,K,forced", [(9_000 + 13, 200, 130, True), (7_001, 131, 70, True), (12_000, 768, 4096, False)])
def test_gpu_score_samples_by_screening_on_wide_data(monkeypatch, N, D, K, forced):
    """Wide data (D > 128) with sparse posteriors: one tensor sweep screens the (point, component) pairs and the few that can
    matter are evaluated exactly (the EM step's screening route without its statistics).  Clustered data with a component
    collapsed onto a point and a zero-weight component; pieces of 4096 points; at the two small shapes the route is forced
    (its automatic limit is zero there), at K = 4096 it is the automatic choice."""
    import torch
    from paper_2606_10896_b200 import flashgmm as fg

    monkeypatch.setenv("GMM_WIDE_PIECE", "4096")
    if forced:
        monkeypatch.setenv("GMM_WIDE_PROBE_LIMIT", "8")
    rng = np.random.default_rng(N + K)
    centres = (rng.normal(size=(K, D)) * 0.3).astype(np.float32)
    w = rng.uniform(0.5, 1.5, K)
    w /= w.sum()
    z = rng.choice(K, size=N, p=w)
    sig = rng.uniform(0.7, 1.3, size=(K, D)) * 0.3
    X = (centres[z] + rng.normal(size=(N, D)) * sig[z]).astype(np.float32)
    mu = (centres + 0.015 * rng.normal(size=(K, D))).astype(np.float32)
    var = (sig ** 2 * rng.uniform(0.8, 1.25, size=(K, D))).astype(np.float32)
    pi = w.astype(np.float32)
    mu[0], var[0] = X[7], 1e-6
    pi[3] = 0.0
    pi = (pi / pi.sum()).astype(np.float32)
    lz = gmm_oracle.responsibilities(X, pi, mu, var)[1]
    t = lambda v: torch.as_tensor(np.ascontiguousarray(v), device="cuda:0")
    with fg.Context(0) as ctx:
        logp, total = ctx.gmm_score_samples(t(X), t(pi), t(mu), t(var))
        assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
        logp2, total2 = ctx.gmm_score_samples(t(X), t(pi), t(mu), t(var))
        assert torch.equal(logp, logp2) and total == total2
        ctx.gmm_set_path(fg.GMM_PATH_FP32)
        logp3, total3 = ctx.gmm_score_samples(t(X), t(pi), t(mu), t(var))
        assert ctx.gmm_last_path() == fg.GMM_PATH_FP32
    got = logp.cpu().numpy().astype(np.float64)
    assert got.shape == (N,) and np.isfinite(got).all()
    excess = np.abs(got - lz) - (1e-5 * np.abs(lz) + 1e-4)
    assert excess.max() <= 0, f"point {int(np.argmax(excess))}: {got[np.argmax(excess)]} vs {lz[np.argmax(excess)]}"
    assert abs(total - lz.sum()) <= 1e-5 * abs(lz.sum()) + 1e-6
    assert np.abs(logp3.cpu().numpy() - got).max() <= 2e-5 * np.abs(lz).max() + 2e-4 and abs(total3 - total) <= 1e-5 * abs(total)


@pytest.mark.gpu
def test_gpu_score_samples_rejects_bad_parameters():
    import torch
    from paper_2606_10896_b200 import flashgmm as fg

    X, pi, mu, var = _case(3, 100, 4, 3)
    var = var.copy()
    var[1, 2] = 0.0
    t = lambda v: torch.as_tensor(np.ascontiguousarray(v), device="cuda:0")
    with fg.Context(0) as ctx:
        with pytest.raises(fg.GmmError):
            ctx.gmm_score_samples(t(X), t(pi), t(mu), t(var))
