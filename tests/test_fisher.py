"""Fisher-vector encoding under a diagonal Gaussian mixture (the per-group use of the fused pattern that the paper's
Discussion, Section 6, names): pins of the CPU oracle, and parity of the CUDA path.

The oracle (oracle/fisher.py) writes the definition out point by point over materialised responsibilities.  It is pinned
by what the definition fixes independently of it: the numerically differentiated mean log-likelihood (the Fisher vector
is its gradient in the means and standard deviations, coordinate-wise scaled by sigma / sqrt(pi) and
sigma / sqrt(2 pi)), the closed form for one component, the vanishing gradient at a maximum-likelihood fit, and a
hand-computed two-point case.  The GPU path goes through the per-group sufficient statistics (N_k, S1, S2) instead, so
it shares no formula with the oracle.

Tolerance of the GPU comparison, per coordinate (k, d) of a group of T points, with A_k = N_k / (T sqrt(pi_k)), the
group's share N_k / T of component k over the square root of the component's weight (about sqrt(pi_k) <= 1 for a group
that resembles the mixture, up to 1 / sqrt(pi_k) for a group that sits on one light component):

    f x [ 2e-5 (1 + max|G|)  +  A_k (0.5 e + 4e-5 (1 + mu_kd^2 / var_kd)) ]

The bracket is a worst-case bound.  First term: rounding of the statistics for ordinary coordinates.  Last term: a
coordinate is a difference of the raw moments N_k, S1, S2, which the tile kernels deliver to about 4e-6 relative (tensor
path; 2e-7 on the FP32 path), and the difference cancels by (1 + mu^2 / var).  Middle term: an error e (in bits) of a
logit moves a contested responsibility by up to r (1 - r) ln 2 e <= 0.17 e, coherently over points that share a region,
and enters a coordinate times |z| or |z^2 - 1| (taken as 3).  On the tensor path e = 8 x 1.5e-4 sqrt(N / K) bits, the
kernel's own error bound for the components it does not recompute exactly (N = all points of the call); on the FP32
path e = 2e-4 bits (fp32 rounding of logits of a few hundred bits).

The factor f brings the bound down to about ten times the error measured in each regime (largest |dG| / bracket over
this file's cases, B200):
    groups drawn from the mixture (every test but the one below), either path:   0.013 measured,  f = 0.1
    a group that sits on one light component next to a close copy of it (the bound's worst case: every responsibility
    of the group contested, A_k near 1 / (2 sqrt(pi_k)) = 50):
        tensor path   0.084 (K = 256, D = 64) and 0.31 (K = 1024, D = 128) measured,   f = 1
        FP32 path     0.0013 and 0.0040 measured,                                     f = 0.04
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


def _tolerance(G_ref, X, offsets, pi, mu, var, tensor_path, contested=False):
    """The per-coordinate bound of this file's header."""
    f = (1.0 if tensor_path else 0.04) if contested else 0.1
    n_all = int(sum(int(offsets[g + 1]) - int(offsets[g]) for g in range(len(offsets) - 1)))
    e_bits = 8 * 1.5e-4 * np.sqrt(max(n_all, 1) / len(pi)) if tensor_path else 2e-4
    tol = np.full(G_ref.shape, 2e-5 * (1.0 + np.abs(G_ref).max()))
    pi64 = np.asarray(pi, np.float64)
    ratio = 1.0 + np.asarray(mu, np.float64) ** 2 / np.asarray(var, np.float64)          # [K, D]
    for g in range(len(offsets) - 1):
        lo, hi = int(offsets[g]), int(offsets[g + 1])
        if hi == lo:
            continue
        Nk = gmm_oracle.em_step(X[lo:hi], pi, mu, var)[0]
        A = np.where(pi64 > 0, Nk / ((hi - lo) * np.sqrt(np.where(pi64 > 0, pi64, 1.0))), 0.0)
        tol[g] += (A[:, None] * (0.5 * e_bits + 4e-5 * ratio))[None]
    return f * tol


def _check_against_oracle(X, offsets, pi, mu, var, path=None, contested=False):
    G_ref = fisher_vectors(X, offsets, pi, mu, var)
    lo, hi = int(offsets[0]), int(offsets[-1])
    ll_ref = float(gmm_oracle.responsibilities(X[lo:hi], pi, mu, var)[1].sum()) if hi > lo else 0.0
    G_gpu, ll, used = _run_gpu(X, offsets, pi, mu, var, path)
    assert G_gpu.shape == G_ref.shape and np.isfinite(G_gpu).all()
    from paper_2606_10896_b200 import flashgmm as fg
    tol = _tolerance(G_ref, X, offsets, pi, mu, var, used == fg.GMM_PATH_TENSOR, contested)
    excess = np.abs(G_gpu - G_ref) - tol
    worst = np.unravel_index(np.argmax(excess), excess.shape)
    assert excess.max() <= 0, f"|dG| = {np.abs(G_gpu - G_ref)[worst]:.3e} > {tol[worst]:.3e} at (group, part, k, d) = {worst}"
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
    (1024, 256, [6000, 9000]),          # wide data on the tensor path
    (600, 520, [5000, 300, 0]),
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
    G_gpu, _, used = _run_gpu(X, sub, pi, mu, var)
    assert np.all(np.abs(G_gpu - G_ref) <= _tolerance(G_ref, X, sub, pi, mu, var, used == fg.GMM_PATH_TENSOR))
    t = lambda v: torch.as_tensor(np.ascontiguousarray(v), device="cuda:0")
    with fg.Context(0) as ctx:
        for bad in ([0, 800, 700], [-1, 10], [0, len(X) + 1]):
            with pytest.raises(fg.GmmError):
                ctx.gmm_fisher_vectors(t(X), np.array(bad, np.int64), t(pi), t(mu), t(var))


@pytest.mark.gpu
@pytest.mark.parametrize("K,D,T", [(256, 64, 2000), (1024, 128, 6000)])
def test_gpu_fisher_vectors_of_a_group_that_sits_on_one_light_component(K, D, T):
    # every point from the lightest component and a close copy of it: contested responsibilities, N_k / T about 1/2 at
    # pi_k of 1e-4, the largest amplification of statistic errors a group can have; beside two ordinary groups
    from paper_2606_10896_b200 import flashgmm as fg

    pi, mu, var = _mixture(K + D, K, D)
    k0 = int(np.argmin(pi))
    k1 = (k0 + 1) % K
    mu, var = mu.copy(), var.copy()
    mu[k1] = mu[k0] + 0.5 * np.sqrt(var[k0])
    var[k1] = var[k0]
    own = np.zeros(K)
    own[k0] = 1.0
    parts = [_sample(50, T, pi, mu, var * np.float32(1.2)), _sample(99, T, own, mu + 0.2, var), _sample(51, T // 2, pi, mu, var)]
    X = np.concatenate(parts)
    offsets = np.array([0, T, 2 * T, 2 * T + T // 2], np.int64)
    for path in (fg.GMM_PATH_TENSOR, fg.GMM_PATH_FP32):
        _check_against_oracle(X, offsets, pi, mu, var, path, contested=True)


@pytest.mark.gpu
def test_gpu_fisher_vectors_many_small_groups_beside_a_large_one():
    # one call that mixes both routes of the tensor path: 60 groups of 0 .. 3000 points share launches (several groups
    # per launch, sorted by size), the group of 60,000 points is accumulated on its own
    from paper_2606_10896_b200 import flashgmm as fg

    rng = np.random.Generator(np.random.PCG64(2024))
    sizes = [int(v) for v in rng.integers(1, 3000, 60)]
    sizes[7] = 0
    sizes[20] = 60000
    sizes[41] = 64
    sizes[42] = 65
    X, offsets, pi, mu, var = _gpu_case(5, 128, 32, sizes)
    G, used = _check_against_oracle(X, offsets, pi, mu, var)
    assert used == fg.GMM_PATH_TENSOR
    assert np.all(G[7] == 0.0)
