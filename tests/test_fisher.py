"""Fisher-vector encoding under a diagonal Gaussian mixture (the per-group use of the fused pattern that the paper's
Discussion, Section 6, names): pins of the CPU oracle, and parity of the CUDA path.

The oracle (oracle/fisher.py) writes the definition out point by point over materialised responsibilities.  It is pinned
by what the definition fixes independently of it: the numerically differentiated mean log-likelihood (the Fisher vector
is its gradient in the means and standard deviations, coordinate-wise scaled by sigma / sqrt(pi) and
sigma / sqrt(2 pi)), the closed form for one component, the vanishing gradient at a maximum-likelihood fit, and a
hand-computed two-point case.  The GPU path goes through the per-group sufficient statistics (N_k, S1, S2) instead, so
it shares no formula with the oracle.

Tolerance of the GPU comparison: the statistics carry the EM step's relative error of about 1e-6 of the data scale per
component; a Fisher coordinate divides differences of them by T sigma sqrt(pi), so the bound used is
2e-5 * (1 + max|G|) absolute, for mixtures with pi_k >= 1e-3 / K and sigma within a factor 30 of the data scale.
"""
import numpy as np
import pytest

from oracle import gmm_oracle
from oracle.fisher import fisher_vector, fisher_vectors, mean_log_likelihood


def _mixture(seed, K, D, spread=2.0):
    rng = np.random.Generator(np.random.PCG64(seed))
    mu = rng.normal(0, spread, (K, D)).astype(np.float32)
    var = rng.uniform(0.4, 1.6, (K, D)).astype(np.float32) ** 2
    pi = rng.dirichlet(np.ones(K) * 3.0).astype(np.float32)
    return pi, mu, var


def _sample(seed, T, pi, mu, var):
    rng = np.random.Generator(np.random.PCG64(seed))
    K, D = mu.shape
    lab = rng.choice(K, size=T, p=np.asarray(pi, np.float64) / np.asarray(pi, np.float64).sum())
    return (mu[lab] + np.sqrt(var[lab]) * rng.standard_normal((T, D))).astype(np.float32)


def test_one_component_closed_form():
    rng = np.random.Generator(np.random.PCG64(5))
    X = rng.normal(1.0, 2.0, (400, 3)).astype(np.float32)
    mu = np.array([[0.5, 1.5, -1.0]], np.float32)
    var = np.array([[1.5, 4.0, 0.7]], np.float32)
    G = fisher_vector(X, np.ones(1, np.float32), mu, var)
    z = (X.astype(np.float64) - mu.astype(np.float64)) / np.sqrt(var.astype(np.float64))
    np.testing.assert_allclose(G[0, 0], z.mean(0), rtol=1e-12)
    np.testing.assert_allclose(G[1, 0], ((z * z).mean(0) - 1.0) / np.sqrt(2.0), rtol=1e-12)


def test_one_component_at_its_own_moments_gives_zero():
    rng = np.random.Generator(np.random.PCG64(6))
    X = rng.normal(-2.0, 0.5, (256, 4)).astype(np.float32)
    X64 = X.astype(np.float64)
    # float32 parameters: the sample moments rounded, so zero up to that rounding
    mu = X64.mean(0, keepdims=True).astype(np.float32)
    var = X64.var(0, keepdims=True).astype(np.float32)
    G = fisher_vector(X, np.ones(1, np.float32), mu, var)
    assert np.abs(G).max() < 1e-6


def test_is_the_scaled_gradient_of_the_mean_log_likelihood():
    # central differences in float64 on every coordinate of a small mixture
    pi, mu, var = _mixture(7, 3, 2)
    X = _sample(8, 50, pi, mu, var)
    G = fisher_vector(X, pi, mu, var)
    pi64, mu64, sd = pi.astype(np.float64), mu.astype(np.float64), np.sqrt(var.astype(np.float64))
    h = 1e-5
    for k in range(3):
        for d in range(2):
            mp, mm = mu64.copy(), mu64.copy()
            mp[k, d] += h
            mm[k, d] -= h
            dmu = (mean_log_likelihood(X, pi64, mp, sd ** 2) - mean_log_likelihood(X, pi64, mm, sd ** 2)) / (2 * h)
            sp, sm = sd.copy(), sd.copy()
            sp[k, d] += h
            sm[k, d] -= h
            dsd = (mean_log_likelihood(X, pi64, mu64, sp ** 2) - mean_log_likelihood(X, pi64, mu64, sm ** 2)) / (2 * h)
            assert G[0, k, d] == pytest.approx(sd[k, d] / np.sqrt(pi64[k]) * dmu, rel=1e-6, abs=1e-9)
            assert G[1, k, d] == pytest.approx(sd[k, d] / np.sqrt(2 * pi64[k]) * dsd, rel=1e-6, abs=1e-9)


def test_two_points_two_components_by_hand():
    # x = -1 and x = +1, components N(-1, 1) and N(+1, 1), equal weights: r(x = -1) = (1, e^-2) / (1 + e^-2)
    X = np.array([[-1.0], [1.0]], np.float32)
    pi = np.array([0.5, 0.5], np.float32)
    mu = np.array([[-1.0], [1.0]], np.float32)
    var = np.ones((2, 1), np.float32)
    a = 1.0 / (1.0 + np.exp(-2.0))          # responsibility of the own component
    b = 1.0 - a
    G = fisher_vector(X, pi, mu, var)
    # component 0: point -1 has z = 0, point +1 has z = 2 and weight b
    assert G[0, 0, 0] == pytest.approx(b * 2.0 / (2 * np.sqrt(0.5)), rel=1e-12)
    assert G[0, 1, 0] == pytest.approx(-b * 2.0 / (2 * np.sqrt(0.5)), rel=1e-12)
    assert G[1, 0, 0] == pytest.approx((a * (0 - 1) + b * (4 - 1)) / (2 * np.sqrt(1.0)), rel=1e-12)
    assert G[1, 1, 0] == pytest.approx(G[1, 0, 0], rel=1e-12)


def test_vanishes_at_a_converged_fit_of_the_group_itself():
    # at a stationary point of EM on the group the gradient in (mu, sigma) is zero (Eq. 2-3 are its roots)
    pi, mu, var = _mixture(9, 3, 2, spread=4.0)
    X = _sample(10, 600, pi, mu, var)
    p, m, v = pi.astype(np.float64), mu.astype(np.float64), var.astype(np.float64)
    for _ in range(300):
        p, m, v, _ = gmm_oracle.em_iteration(X, p, m, v)[:4]
    G = fisher_vector(X, p, m, v)
    assert np.abs(G).max() < 1e-6


def test_zero_weight_component_and_empty_group_give_zeros_and_groups_are_independent():
    pi, mu, var = _mixture(11, 4, 3)
    pi = pi.copy()
    pi[2] = 0.0
    pi /= pi.sum()
    X = _sample(12, 90, np.where(pi > 0, pi, 0), mu, var)
    G = fisher_vectors(X, [0, 40, 40, 90], pi, mu, var)
    assert G.shape == (3, 2, 4, 3)
    assert np.all(G[:, :, 2, :] == 0.0) and np.all(G[1] == 0.0)
    np.testing.assert_array_equal(G[0], fisher_vector(X[:40], pi, mu, var))
    np.testing.assert_array_equal(G[2], fisher_vector(X[40:], pi, mu, var))
    # the groups' vectors, weighted by their sizes, add up to the vector of their union
    np.testing.assert_allclose((40 * G[0] + 50 * G[2]) / 90, fisher_vector(X, pi, mu, var), atol=1e-13)


# ------------------------------------------------------------------------------------------------------------------
# GPU parity
# ------------------------------------------------------------------------------------------------------------------

def _gpu_case(seed, K, D, sizes):
    """A mixture, and groups drawn from a perturbed copy of it (so that the vectors are not all close to zero)."""
    pi, mu, var = _mixture(seed, K, D)
    rng = np.random.Generator(np.random.PCG64(seed + 1000))
    parts = []
    for g, T in enumerate(sizes):
        shift = (0.3 * rng.standard_normal((K, D))).astype(np.float32)
        widen = np.float32(rng.uniform(0.7, 1.4)) ** 2
        parts.append(_sample(seed + 2000 + g, T, pi, mu + shift, var * widen))
    X = np.concatenate(parts) if parts else np.zeros((0, D), np.float32)
    offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    return X, offsets, pi, mu, var


def _run_gpu(X, offsets, pi, mu, var, path=None, repeat=True):
    import torch
    from paper_2606_10896_b200 import flashgmm as fg

    t = lambda v: torch.as_tensor(np.ascontiguousarray(v), device="cuda:0")
    with fg.Context(0) as ctx:
        if path is not None:
            ctx.gmm_set_path(path)
        Xd, pid, mud, vard = t(X), t(pi), t(mu), t(var)
        fv, ll = ctx.gmm_fisher_vectors(Xd, offsets, pid, mud, vard)
        if repeat:
            # (the tensor path may pick its filter for ill-conditioned components from the previous call's count: the
            # second and third calls run the same kernels)
            fv, ll = ctx.gmm_fisher_vectors(Xd, offsets, pid, mud, vard)
            fv2, ll2 = ctx.gmm_fisher_vectors(Xd, offsets, pid, mud, vard)
            assert torch.equal(fv, fv2) and ll == ll2, "not deterministic"
        used = ctx.gmm_last_path()
    return fv.cpu().numpy().astype(np.float64), ll, used


def _check_against_oracle(X, offsets, pi, mu, var, path=None):
    G_ref = fisher_vectors(X, offsets, pi, mu, var)
    lo, hi = int(offsets[0]), int(offsets[-1])
    ll_ref = float(gmm_oracle.responsibilities(X[lo:hi], pi, mu, var)[1].sum()) if hi > lo else 0.0
    G_gpu, ll, used = _run_gpu(X, offsets, pi, mu, var, path)
    assert G_gpu.shape == G_ref.shape and np.isfinite(G_gpu).all()
    tol = 2e-5 * (1.0 + np.abs(G_ref).max())
    err = np.abs(G_gpu - G_ref).max()
    assert err <= tol, f"max |dG| = {err:.3e} > {tol:.3e}"
    assert abs(ll - ll_ref) <= 1e-5 * abs(ll_ref) + 1e-9
    return G_gpu, used


@pytest.mark.gpu
@pytest.mark.parametrize("K,D,sizes", [
    (1, 3, [5, 1, 40]),
    (8, 16, [1000, 0, 1, 63, 129]),
    (64, 64, [2000, 3001, 500, 64]),
    (70, 130, [900, 1500]),
    (256, 128, [3000, 20000, 7001]),
    (1024, 128, [30000, 12000]),
])
def test_gpu_fisher_vectors_match_oracle(K, D, sizes):
    X, offsets, pi, mu, var = _gpu_case(K + D, K, D, sizes)
    G, _ = _check_against_oracle(X, offsets, pi, mu, var)
    for g, T in enumerate(sizes):
        if T == 0:
            assert np.all(G[g] == 0.0)


@pytest.mark.gpu
def test_gpu_fisher_vectors_on_either_path_and_with_a_zero_weight_component():
    from paper_2606_10896_b200 import flashgmm as fg

    X, offsets, pi, mu, var = _gpu_case(77, 128, 64, [4000, 2500])
    pi = pi.copy()
    pi[5] = 0.0
    pi /= pi.sum()
    for path in (fg.GMM_PATH_TENSOR, fg.GMM_PATH_FP32):
        G, used = _check_against_oracle(X, offsets, pi, mu, var, path)
        assert used == path
        assert np.all(G[:, :, 5, :] == 0.0)


@pytest.mark.gpu
def test_gpu_fisher_vectors_groups_inside_a_larger_array_and_bad_offsets():
    import torch
    from paper_2606_10896_b200 import flashgmm as fg

    X, offsets, pi, mu, var = _gpu_case(31, 32, 24, [700, 300, 500])
    # groups that leave rows out at both ends and between them
    sub = np.array([100, 650, 650, 1400], np.int64)
    G_ref = fisher_vectors(X, sub, pi, mu, var)
    G_gpu, _, _ = _run_gpu(X, sub, pi, mu, var)
    assert np.abs(G_gpu - G_ref).max() <= 2e-5 * (1.0 + np.abs(G_ref).max())
    t = lambda v: torch.as_tensor(np.ascontiguousarray(v), device="cuda:0")
    with fg.Context(0) as ctx:
        for bad in ([0, 800, 700], [-1, 10], [0, len(X) + 1]):
            with pytest.raises(fg.GmmError):
                ctx.gmm_fisher_vectors(t(X), np.array(bad, np.int64), t(pi), t(mu), t(var))
