"""Pins of the float64 CPU oracle against what the paper and the mathematics fix (Section 2, Eq. 1-3, Algorithm 1):
closed forms, brute force on tiny inputs, invariants, symmetries and independent library routines (scipy's normal
log-pdf and log-sum-exp, scikit-learn's diagonal Gaussian mixture).  None of these re-types the oracle's own
formula; each would fail for a dropped term, a wrong sign, a transposed operand or a wrong index somewhere in it.
"""
import math
from pathlib import Path

import numpy as np
import pytest
from scipy.special import logsumexp
from scipy.stats import multivariate_normal, norm

from oracle import gmm_oracle as orc

GOLDEN = Path(__file__).parent / "golden"


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def _random_problem(seed, N, D, K, spread=3.0):
    r = _rng(seed)
    mu = r.normal(0, spread, (K, D))
    var = r.uniform(0.3, 2.0, (K, D))
    pi = r.dirichlet(np.ones(K))
    comp = r.integers(0, K, N)
    X = (mu[comp] + np.sqrt(var[comp]) * r.standard_normal((N, D))).astype(np.float32)
    return X, pi, mu, var


def _library_responsibilities(X, pi, mu, var):
    """R and logZ from scipy primitives only (univariate normal log-pdf summed over d, library log-sum-exp)."""
    X = X.astype(np.float64)
    ell = np.log(pi)[None, :] + norm.logpdf(X[:, None, :], mu[None], np.sqrt(var)[None]).sum(-1)
    lz = logsumexp(ell, axis=1)
    return np.exp(ell - lz[:, None]), lz


def test_two_point_closed_form_golden():
    vals = {}
    for line in (GOLDEN / "two_point_two_component.txt").read_text().splitlines():
        if line and not line.startswith("#"):
            k, v = line.split()
            vals[k] = float(v)
    X = np.array([[-1.0], [1.0]], np.float32)
    pi, mu, var = np.array([0.5, 0.5]), np.array([[-1.0], [1.0]]), np.ones((2, 1))
    R, lz = orc.responsibilities(X, pi, mu, var)
    assert R[1, 1] == pytest.approx(vals["a"], abs=1e-15)
    assert R[0, 0] == pytest.approx(vals["a"], abs=1e-15)
    Nk, S1, S2, L = orc.em_step(X, pi, mu, var)
    assert L == pytest.approx(vals["loglik"], abs=1e-14)
    np.testing.assert_allclose(Nk, [1, 1], atol=1e-15)
    np.testing.assert_allclose(S1[:, 0], [-vals["tanh1"], vals["tanh1"]], atol=1e-15)
    np.testing.assert_allclose(S2[:, 0], [1, 1], atol=1e-15)
    pn, mn, vn, L2, _, _ = orc.em_iteration(X, pi, mu, var)
    np.testing.assert_allclose(pn, [0.5, 0.5], atol=1e-15)
    np.testing.assert_allclose(mn[:, 0], [-vals["tanh1"], vals["tanh1"]], atol=1e-15)
    np.testing.assert_allclose(vn[:, 0], [vals["sech2_1"]] * 2, atol=1e-15)
    assert L2 == L
    # the fixture's numbers are themselves the stated closed forms
    assert vals["tanh1"] == pytest.approx(math.tanh(1.0), abs=1e-16)
    assert vals["sech2_1"] == pytest.approx(1 - math.tanh(1.0) ** 2, abs=1e-16)


@pytest.mark.parametrize("N,D", [(1, 1), (57, 3), (1000, 16)])
def test_k1_closed_forms(N, D):
    r = _rng(10 + N)
    X = (r.normal(2.0, 3.0, (N, D)) * r.uniform(0.5, 2, D)).astype(np.float32)
    Xd = X.astype(np.float64)
    mu0, var0 = r.normal(0, 1, (1, D)), r.uniform(0.5, 2, (1, D))
    Nk, S1, S2, L = orc.em_step(X, [1.0], mu0, var0)
    assert Nk[0] == pytest.approx(N, rel=1e-14)
    np.testing.assert_allclose(S1[0], Xd.sum(0), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(S2[0], (Xd * Xd).sum(0), rtol=1e-12)
    L_ref = norm.logpdf(Xd, mu0, np.sqrt(var0)).sum()
    assert L == pytest.approx(L_ref, rel=1e-12)
    pn, mn, vn, _, _, _ = orc.em_iteration(X, [1.0], mu0, var0)
    assert pn[0] == pytest.approx(1.0, abs=1e-14)
    np.testing.assert_allclose(mn[0], Xd.mean(0), rtol=1e-12, atol=1e-12)
    if N > 1:
        np.testing.assert_allclose(vn[0], Xd.var(0), rtol=1e-10)
        # after the update the log-likelihood of a single Gaussian is -(N/2) sum_d (1 + log 2 pi var_d)
        _, _, _, L1 = orc.em_step(X, pn, mn, vn)
        assert L1 == pytest.approx(-0.5 * N * np.sum(1 + np.log(2 * np.pi * Xd.var(0))), rel=1e-12)


@pytest.mark.parametrize("N,D,K", [(8, 2, 3), (5, 1, 2), (7, 2, 1)])
def test_brute_force_tiny(N, D, K):
    X, pi, mu, var = _random_problem(3, N, D, K, spread=1.5)
    R, lz = orc.responsibilities(X, pi, mu, var)
    Rb, p = orc.brute_force(X, pi, mu, var)
    np.testing.assert_allclose(R, Rb, rtol=1e-11, atol=1e-300)
    np.testing.assert_allclose(lz, np.log(p), rtol=1e-12)
    ell = orc.log_joint(X, pi, mu, var)
    np.testing.assert_allclose(np.exp(ell).sum(1), p, rtol=1e-12)


def test_against_scipy_primitives_nonsquare():
    # K != D and every parameter distinct: a transposed or mis-indexed operand cannot survive this
    X, pi, mu, var = _random_problem(4, 203, 5, 7)
    R, lz = orc.responsibilities(X, pi, mu, var)
    Rl, lzl = _library_responsibilities(X, pi, mu, var)
    np.testing.assert_allclose(R, Rl, rtol=1e-10, atol=1e-300)
    np.testing.assert_allclose(lz, lzl, rtol=1e-13)
    Nk, S1, S2, L = orc.em_step(X, pi, mu, var)
    Xd = X.astype(np.float64)
    np.testing.assert_allclose(Nk, Rl.sum(0), rtol=1e-11)
    np.testing.assert_allclose(S1, Rl.T @ Xd, rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(S2, Rl.T @ (Xd * Xd), rtol=1e-10)
    assert L == pytest.approx(lzl.sum(), rel=1e-13)


def test_responsibilities_sum_to_one_and_bounds():
    X, pi, mu, var = _random_problem(5, 500, 16, 8, spread=5.0)
    R, _ = orc.responsibilities(X, pi, mu, var)
    np.testing.assert_allclose(R.sum(1), 1.0, atol=1e-14)
    assert (R >= 0).all() and (R <= 1).all()


@pytest.mark.parametrize("threads", [1, 3, 8])
def test_conservation_laws(threads):
    X, pi, mu, var = _random_problem(6, 4001, 9, 13)
    Nk, S1, S2, L = orc.em_step(X, pi, mu, var, nthreads=threads)
    Xd = X.astype(np.float64)
    assert Nk.sum() == pytest.approx(len(X), rel=1e-12)
    np.testing.assert_allclose(S1.sum(0), Xd.sum(0), rtol=1e-10, atol=1e-9)
    np.testing.assert_allclose(S2.sum(0), (Xd * Xd).sum(0), rtol=1e-11)
    pn, _, _, _, _, _ = orc.em_iteration(X, pi, mu, var, nthreads=threads)
    assert pn.sum() == pytest.approx(1.0, abs=1e-12)


def test_thread_count_does_not_change_results_beyond_rounding():
    X, pi, mu, var = _random_problem(7, 3000, 6, 5)
    a = orc.em_step(X, pi, mu, var, nthreads=1)
    b = orc.em_step(X, pi, mu, var, nthreads=7)
    for u, v in zip(a[:3], b[:3]):
        np.testing.assert_allclose(u, v, rtol=1e-12, atol=1e-12)
    assert a[3] == pytest.approx(b[3], rel=1e-13)


def test_additivity_over_chunks():
    X, pi, mu, var = _random_problem(8, 2500, 6, 5)
    full = orc.em_step(X, pi, mu, var)
    parts = [orc.em_step(X[lo:lo + 700], pi, mu, var) for lo in range(0, len(X), 700)]
    for j in range(3):
        np.testing.assert_allclose(full[j], sum(p[j] for p in parts), rtol=1e-11, atol=1e-11)
    assert full[3] == pytest.approx(sum(p[3] for p in parts), rel=1e-13)


def test_centred_variance_equals_moment_form():
    X, pi, mu, var = _random_problem(9, 1500, 7, 6)
    pn, mn, vn, L, Nk, S1 = orc.em_iteration(X, pi, mu, var)
    Nk2, S12, S2, L2 = orc.em_step(X, pi, mu, var)
    np.testing.assert_allclose(Nk, Nk2, rtol=1e-14)
    pm, mm, vm = orc.finalize_moments(len(X), Nk2, S12, S2, 0.0, mu, var)
    np.testing.assert_allclose(pn, pm, rtol=1e-14)
    np.testing.assert_allclose(mn, mm, rtol=1e-14)
    np.testing.assert_allclose(vn, vm, rtol=1e-10)


def test_em_iteration_matches_library_weighted_moments():
    X, pi, mu, var = _random_problem(11, 800, 4, 6)
    Rl, _ = _library_responsibilities(X, pi, mu, var)
    Xd = X.astype(np.float64)
    pn, mn, vn, _, _, _ = orc.em_iteration(X, pi, mu, var)
    for k in range(len(pi)):
        m = np.average(Xd, axis=0, weights=Rl[:, k])
        v = np.average((Xd - m) ** 2, axis=0, weights=Rl[:, k])
        np.testing.assert_allclose(mn[k], m, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(vn[k], v, rtol=1e-10)
        assert pn[k] == pytest.approx(Rl[:, k].mean(), rel=1e-11)


def test_loglik_trace_is_nondecreasing_and_is_under_entering_params():
    from paper_2606_10896_b200 import synth

    spec = synth.CONFIGS[1].with_n(3000)
    X = synth.sample_host(spec)
    pi, mu, var = synth.init_params(X, spec)
    out = orc.fit(X, pi, mu, var, 12, var_floor=0.0, keep_params=True)
    tr = out["trace"]
    assert len(tr) == 12
    assert (np.diff(tr) >= -1e-9 * np.abs(tr[1:])).all()
    assert tr[-1] > tr[0]
    for t in (0, 5, 11):
        p, m, v = out["params"][t]
        assert orc.em_step(X, p, m, v)[3] == pytest.approx(tr[t], rel=1e-14)
    np.testing.assert_array_equal(out["params"][12][1], out["mu"])


def test_fit_tolerance_stops_early():
    X, pi, mu, var = _random_problem(12, 600, 2, 2, spread=6.0)
    out = orc.fit(X, pi, mu, var, 200, tol=1e-9)
    assert 2 <= out["iters_done"] < 200
    tr = out["trace"]
    assert abs(tr[-1] - tr[-2]) <= 1e-9 * abs(tr[-1])


def test_permutation_symmetry():
    X, pi, mu, var = _random_problem(13, 400, 5, 6)
    r = _rng(99)
    pp, pk = r.permutation(len(X)), r.permutation(len(pi))
    a = orc.em_step(X, pi, mu, var, nthreads=1)
    b = orc.em_step(X[pp], pi[pk], mu[pk], var[pk], nthreads=1)
    np.testing.assert_allclose(a[0][pk], b[0], rtol=1e-11)
    np.testing.assert_allclose(a[1][pk], b[1], rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(a[2][pk], b[2], rtol=1e-10)
    assert a[3] == pytest.approx(b[3], rel=1e-13)


def test_identical_components_share_equally():
    r = _rng(14)
    X = r.normal(0, 2, (300, 4)).astype(np.float32)
    K = 5
    mu = np.tile(r.normal(0, 1, (1, 4)), (K, 1))
    var = np.tile(r.uniform(0.5, 2, (1, 4)), (K, 1))
    pi = np.full(K, 1 / K)
    R, _ = orc.responsibilities(X, pi, mu, var)
    np.testing.assert_allclose(R, 1 / K, rtol=1e-13)
    pn, mn, vn, _, _, _ = orc.em_iteration(X, pi, mu, var)
    Xd = X.astype(np.float64)
    np.testing.assert_allclose(mn, np.tile(Xd.mean(0), (K, 1)), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(vn, np.tile(Xd.var(0), (K, 1)), rtol=1e-10)


def test_translation_and_scaling():
    X, pi, mu, var = _random_problem(15, 500, 3, 4)
    # use values exactly representable after the transform so float32 storage adds no error
    X = np.round(X * 64) / 64
    X = X.astype(np.float32)
    c = np.array([2.0, -4.0, 0.5])
    a = orc.em_step(X, pi, mu, var)
    b = orc.em_step((X + c).astype(np.float32), pi, mu + c, var)
    np.testing.assert_allclose(a[0], b[0], rtol=1e-10)
    assert a[3] == pytest.approx(b[3], rel=1e-12)
    np.testing.assert_allclose(b[1], a[1] + c[None] * a[0][:, None], rtol=1e-9, atol=1e-9)
    s = 4.0
    d = orc.em_step((X * s).astype(np.float32), pi, mu * s, var * s * s)
    np.testing.assert_allclose(a[0], d[0], rtol=1e-10)
    assert d[3] == pytest.approx(a[3] - len(X) * X.shape[1] * math.log(s), rel=1e-12)


def test_hard_assignment_limit_gives_per_cluster_moments():
    r = _rng(16)
    centres = np.array([[-1000.0, 0.0], [1000.0, 0.0], [0.0, 2000.0]])
    lab = r.integers(0, 3, 900)
    X = (centres[lab] + r.standard_normal((900, 2))).astype(np.float32)
    pn, mn, vn, _, Nk, _ = orc.em_iteration(X, np.full(3, 1 / 3), centres, np.ones((3, 2)))
    Xd = X.astype(np.float64)
    for k in range(3):
        sel = Xd[lab == k]
        assert Nk[k] == pytest.approx(len(sel), rel=1e-13)
        np.testing.assert_allclose(mn[k], sel.mean(0), rtol=1e-12)
        np.testing.assert_allclose(vn[k], sel.var(0), rtol=1e-9)


def test_isotropic_reduction_matches_paper_density_and_eq3():
    X, pi, mu, _ = _random_problem(17, 300, 6, 4)
    s2 = np.array([0.7, 1.3, 2.1, 0.4])
    var = np.repeat(s2[:, None], 6, axis=1)
    ell = orc.log_joint(X, pi, mu, var)
    Xd = X.astype(np.float64)
    for k in range(4):      # the paper's N(x | mu_k, sigma_k^2 I) from a library routine
        ref = np.log(pi[k]) + multivariate_normal(mu[k], s2[k] * np.eye(6)).logpdf(Xd)
        np.testing.assert_allclose(ell[:, k], ref, rtol=1e-12)
    Rl, _ = _library_responsibilities(X, pi, mu, var)
    pn, mn, vn, _, Nk, _ = orc.em_iteration(X, pi, mu, var)
    for k in range(4):      # Eq. 3: (1 / (D N_k)) sum_i r_ik ||x_i - mu_k||^2 with the updated mean
        eq3 = (Rl[:, k] * ((Xd - mn[k]) ** 2).sum(1)).sum() / (6 * Nk[k])
        assert vn[k].mean() == pytest.approx(eq3, rel=1e-10)


def test_against_sklearn_diag_mixture():
    from sklearn.mixture import GaussianMixture

    X, pi, mu, var = _random_problem(18, 700, 5, 6)
    Xd = X.astype(np.float64)
    gm = GaussianMixture(n_components=6, covariance_type="diag", reg_covar=0.0)
    gm.weights_, gm.means_, gm.covariances_ = pi, mu, var
    gm.precisions_cholesky_ = 1.0 / np.sqrt(var)
    R, lz = orc.responsibilities(X, pi, mu, var)
    np.testing.assert_allclose(lz, gm.score_samples(Xd), rtol=1e-12)
    np.testing.assert_allclose(R, gm.predict_proba(Xd), rtol=1e-9, atol=1e-300)
    one = GaussianMixture(n_components=6, covariance_type="diag", reg_covar=0.0, max_iter=1, tol=0.0,
                          weights_init=pi, means_init=mu, precisions_init=1.0 / var)
    import warnings

    with warnings.catch_warnings():
        warnings.simplefilter("ignore")
        one.fit(Xd)
    pn, mn, vn, _, _, _ = orc.em_iteration(X, pi, mu, var)
    np.testing.assert_allclose(pn, one.weights_, rtol=1e-9)
    np.testing.assert_allclose(mn, one.means_, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(vn, one.covariances_, rtol=1e-8)


def test_variance_floor_and_empty_component_rule():
    r = _rng(19)
    X = np.concatenate([np.zeros((50, 2)), r.normal(10, 1, (50, 2))]).astype(np.float32)
    mu = np.array([[0.0, 0.0], [10.0, 10.0], [1e4, 1e4]])
    var = np.ones((3, 2))
    pi = np.array([0.5, 0.5, 0.0])
    pn, mn, vn, L, Nk, _ = orc.em_iteration(X, pi, mu, var, var_floor=1e-3)
    assert np.isfinite(L)
    assert Nk[2] == 0.0 and pn[2] == 0.0
    np.testing.assert_array_equal(mn[2], mu[2])          # frozen
    np.testing.assert_array_equal(vn[2], var[2])
    np.testing.assert_allclose(vn[0], 1e-3)              # 50 identical points -> variance 0 -> floored
    assert not np.isnan(pn).any() and not np.isnan(mn).any() and not np.isnan(vn).any()
    _, _, vm = orc.finalize_moments(len(X), *orc.em_step(X, pi, mu, var)[:3], 1e-3, mu, var)
    np.testing.assert_allclose(vm[0], 1e-3)


def test_topm_against_sorting_the_brute_force_row():
    X, pi, mu, var = _random_problem(20, 64, 2, 6, spread=1.0)
    Rb, _ = orc.brute_force(X, pi, mu, var)
    for m in (1, 2, 4, 6):
        idx, resp, nxt = orc.topm(X, pi, mu, var, m)
        order = np.argsort(-Rb, axis=1, kind="stable")
        np.testing.assert_array_equal(idx, order[:, :m])
        np.testing.assert_allclose(resp, np.take_along_axis(Rb, order[:, :m], 1), rtol=1e-11)
        if m < 6:
            np.testing.assert_allclose(nxt, np.take_along_axis(Rb, order[:, m:m + 1], 1)[:, 0], rtol=1e-11)
        else:
            assert (nxt == 0).all()


def test_topm_ties_go_to_smaller_index():
    X = np.zeros((3, 2), np.float32)
    mu = np.zeros((4, 2))
    idx, resp, _ = orc.topm(X, np.full(4, 0.25), mu, np.ones((4, 2)), 2)
    np.testing.assert_array_equal(idx, [[0, 1]] * 3)
    np.testing.assert_allclose(resp, 0.25)


def test_isotropic_iteration_is_eq3_as_printed():
    """The isotropic oracle against the paper's Eq. 1-3 evaluated from library responsibilities, and against the mean
    over d of the diagonal update (the two must coincide when the old variances are isotropic)."""
    X, pi, mu, _ = _random_problem(21, 500, 5, 4)
    s2 = np.array([0.8, 1.4, 0.5, 2.0])
    var = np.repeat(s2[:, None], 5, axis=1)
    Xd = X.astype(np.float64)
    Rl, lzl = _library_responsibilities(X, pi, mu, var)
    pn, mn, vn, L = orc.em_iteration_isotropic(X, pi, mu, var)
    assert L == pytest.approx(lzl.sum(), rel=1e-13)
    for k in range(4):
        Nk = Rl[:, k].sum()
        m = (Rl[:, k, None] * Xd).sum(0) / Nk                                   # Eq. 2
        v = (Rl[:, k] * ((Xd - m) ** 2).sum(1)).sum() / (5 * Nk)                # Eq. 3
        assert pn[k] == pytest.approx(Nk / len(X), rel=1e-11)
        np.testing.assert_allclose(mn[k], m, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(vn[k], v, rtol=1e-10)                        # every d carries the same value
    _, md, vd, _, _, _ = orc.em_iteration(X, pi, mu, var)
    np.testing.assert_allclose(mn, md, rtol=1e-13)
    np.testing.assert_allclose(vn[:, 0], vd.mean(1), rtol=1e-10)
