"""GPU parity: the CUDA path, called through the C ABI, against the float64 CPU oracle on the same seeded inputs.

Tolerances and the two comparison modes (teacher-forced / free-running) are defined in tests/parity_util.py.
Every test here runs for each kernel path that supports the shape (FP32 CUDA-core path: any shape; tensor-core
path: see include/flashgmm.h).
"""
import numpy as np
import pytest
import torch

from oracle import gmm_oracle as orc
from paper_2606_10896_b200 import synth
from tests.parity_util import assert_params_close, assert_stats_close, assert_topm_matches, data_scale, oracle_resp_at

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module")
def fg():
    from paper_2606_10896_b200 import flashgmm

    return flashgmm


@pytest.fixture()
def ctx(fg):
    c = fg.Context(0)
    yield c
    c.close()


def _t(a, dtype=torch.float32):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=dtype, device=DEV).contiguous()


def _paths(fg, D, K):
    """The FP32 path always; the tensor-core path wherever GMM_PATH_AUTO would pick it."""
    paths = [fg.GMM_PATH_FP32]
    if fg.tensor_path_supports(D, K) and fg.gmm_auto_path(D, K) == fg.GMM_PATH_TENSOR:
        paths.append(fg.GMM_PATH_TENSOR)
    return paths


def _gpu_step(ctx, X_d, pi, mu, var):
    Nk, S1, S2, L = ctx.gmm_em_step(X_d, _t(pi), _t(mu), _t(var))
    return Nk.cpu().numpy(), S1.cpu().numpy(), S2.cpu().numpy(), L


def _check_topm(X, pi, mu, var, m, idx_g, resp_g, what):
    """The GPU's top-m rows against the oracle's under the tie rule of tests/parity_util.py; resp_g = None checks the
    indices alone."""
    idx_g = np.asarray(idx_g)
    idx_r, resp_r, next_r = orc.topm(X, pi, mu, var, m)
    r_at_g = oracle_resp_at(orc, X, pi, mu, var, idx_g)
    assert idx_g.min() >= 0 and idx_g.max() < len(pi), f"{what}: index out of range"
    assert_topm_matches(idx_g, resp_g, idx_r, resp_r, next_r, r_at_g, what=what, check_values=resp_g is not None)


def _teacher_forced(fg, ctx, X, spec, iters, paths=None):
    N, D = X.shape
    s = data_scale(X)
    pi0, mu0, var0 = synth.init_params(X, spec)
    ref = orc.fit(X, pi0, mu0, var0, iters, var_floor=spec.var_floor, keep_params=True)
    X_d = _t(X)
    for path in (paths or _paths(fg, D, spec.K)):
        ctx.gmm_set_path(path)
        for t in range(iters):
            p_t, m_t, v_t = ref["params"][t]
            # the GPU holds float32 parameters: step both sides from the same float32 values
            p32, m32, v32 = p_t.astype(np.float32), m_t.astype(np.float32), v_t.astype(np.float32)
            Nk_r, S1_r, S2_r, L_r = orc.em_step(X, p32, m32, v32)
            pr, mr, vr, _, _, _ = orc.em_iteration(X, p32, m32, v32, var_floor=spec.var_floor)
            Nk_g, S1_g, S2_g, L_g = _gpu_step(ctx, X_d, p32, m32, v32)
            what = f"path {path} iteration {t}"
            assert abs(L_g - L_r) <= 1e-5 * abs(L_r), f"{what}: loglik {L_g} vs {L_r}"
            assert abs(Nk_g.sum() - N) <= 1e-6 * N * 10, f"{what}: sum N_k = {Nk_g.sum()} vs N = {N}"
            assert_stats_close(N, s, (Nk_g, S1_g, S2_g), (Nk_r, S1_r, S2_r), what)
            pi_d, mu_d, var_d = _t(p32), _t(m32), _t(v32)
            ctx.gmm_finalize(N, _t(Nk_g, torch.float64), _t(S1_g, torch.float64), _t(S2_g, torch.float64),
                             spec.var_floor, pi_d, mu_d, var_d)
            assert_params_close(N, s, (pi_d.cpu().numpy(), mu_d.cpu().numpy(), var_d.cpu().numpy()), (pr, mr, vr),
                                Nk_r, what)
        assert ctx.gmm_last_path() == path


def test_config1_teacher_forced_10_iterations(fg, ctx):
    spec = synth.CONFIGS[1]
    _teacher_forced(fg, ctx, synth.sample_host(spec), spec, spec.iters)


def test_config1_free_running_fit(fg, ctx):
    spec = synth.CONFIGS[1]
    X = synth.sample_host(spec)
    pi0, mu0, var0 = synth.init_params(X, spec)
    ref = orc.fit(X, pi0, mu0, var0, spec.iters, var_floor=spec.var_floor)
    for path in _paths(fg, spec.D, spec.K):
        ctx.gmm_set_path(path)
        pi, mu, var = _t(pi0), _t(mu0), _t(var0)
        trace, done = ctx.gmm_fit(_t(X), pi, mu, var, spec.iters, spec.var_floor)
        assert done == spec.iters
        np.testing.assert_allclose(trace, ref["trace"], rtol=1e-4)
        assert (np.diff(trace) >= -1e-6 * np.abs(trace[1:])).all()
        s = data_scale(X)
        Nk = orc.em_step(X, ref["pi"], ref["mu"], ref["var"])[0]
        # after 10 free-running iterations the parameters have not drifted apart
        assert np.abs(mu.cpu().numpy() - ref["mu"])[Nk >= 1].max() <= 1e-3 * s


def test_config2_cut_teacher_forced(fg, ctx):
    # K=1024, D=128 with N=3000: 47 point tiles of 64 with a ragged tail of 56
    spec = synth.CONFIGS[2].with_n(3000)
    _teacher_forced(fg, ctx, synth.sample_host(spec), spec, 3)


@pytest.mark.parametrize("filt", ["plain", "tight"])
def test_tensor_ill_conditioned_mode_with_either_filter(fg, filt, monkeypatch):
    # The tile kernel has two filters for the pairs of flagged components (the host picks one per launch from the number of
    # points per component); either must give the right statistics on any input.  N = 3000 < 3 K: from the second
    # iteration on most components are flagged.
    monkeypatch.setenv("GMM_TC_FILTER", filt)
    spec = synth.CONFIGS[2].with_n(3000)
    with fg.Context(0) as c:
        _teacher_forced(fg, c, synth.sample_host(spec), spec, 4, paths=[fg.GMM_PATH_TENSOR])


@pytest.mark.parametrize("order", ["0", "1", "2"])
def test_tensor_ill_conditioned_mode_under_both_issue_orders(fg, order, monkeypatch):
    # From the second iteration on, N=3000 < 3K leaves most components collapsed onto single points at the variance
    # floor: the tensor path runs its exact-recomputation protocol.  Three point tiles per group of CTAs, so the
    # interleaved order issues E(2) between M(0) and M(1).  Every MMA issue order (pairs, interleaved, dynamic) must give
    # the same, correct statistics.
    monkeypatch.setenv("GMM_TC_ORDER", order)
    spec = synth.CONFIGS[2].with_n(3000)
    with fg.Context(0) as c:
        _teacher_forced(fg, c, synth.sample_host(spec), spec, 3, paths=[fg.GMM_PATH_TENSOR])


def test_tensor_path_with_groups_of_more_than_8_ctas(fg, ctx):
    """K = 2048: a group of 16 CTAs covers the components of a tile, so the (max, sum) pairs and, in the ill-conditioned
    mode, the lower bounds are collected in several rounds.  Teacher-forced over 3 iterations on N = 4000 points: from the
    second iteration on most components have collapsed and the exact-recomputation protocol runs."""
    import dataclasses

    spec = dataclasses.replace(synth.CONFIGS[2].with_n(4000), K=2048)
    X = synth.sample_host(spec)
    _teacher_forced(fg, ctx, X, spec, 3, paths=[fg.GMM_PATH_TENSOR])


def test_tensor_path_accumulates_over_pieces(fg, monkeypatch):
    # The tensor path converts X to its fp16 planes and launches the tile kernel once per piece of points (2^19 by
    # default).  With pieces of 1024 points a 3000-point problem takes three launches, the last one ragged (952 points,
    # 14 tiles + a tail of 56): statistics and log-likelihood must still be those of one pass over all points.
    monkeypatch.setenv("GMM_TC_PIECE", "1024")
    spec = synth.CONFIGS[2].with_n(3000)
    with fg.Context(0) as c:
        _teacher_forced(fg, c, synth.sample_host(spec), spec, 2, paths=[fg.GMM_PATH_TENSOR])


def test_bounded_wait_runs_out_and_the_gpu_stays_usable(fg, monkeypatch):
    # Every device-side wait of the tensor path is bounded.  A test hook makes one CTA of the first group keep its
    # exchange slot of the first tile empty (a flag that nothing sets); with the limit shortened to 100 ms its peers'
    # waits run out, every role of those CTAs leaves through the abort path, the kernel ends by itself and the call
    # returns GMM_ETIMEOUT.  Nothing faults or hangs: a fresh context then computes the same step correctly.
    spec = synth.CONFIGS[2].with_n(3000)
    X = synth.sample_host(spec)
    pi0, mu0, var0 = synth.init_params(X, spec)
    p32, m32, v32 = pi0.astype(np.float32), mu0.astype(np.float32), var0.astype(np.float32)
    monkeypatch.setenv("GMM_TC_TEST_SILENT_RANK", "3")
    monkeypatch.setenv("GMM_TC_TEST_WAIT_MS", "100")
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        with pytest.raises(fg.GmmError) as err:
            _gpu_step(c, _t(X), p32, m32, v32)
        assert err.value.code == fg.GMM_ETIMEOUT
    monkeypatch.delenv("GMM_TC_TEST_SILENT_RANK")
    monkeypatch.delenv("GMM_TC_TEST_WAIT_MS")
    ref = orc.em_step(X, p32, m32, v32)
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        got = _gpu_step(c, _t(X), p32, m32, v32)
        assert abs(got[3] - ref[3]) <= 1e-5 * abs(ref[3])
        assert_stats_close(len(X), data_scale(X), got[:3], ref[:3], "after a timed-out call")


def test_config2_free_running_30_iterations(fg, ctx):
    """Config 2 as specified (N = 100,000, D = 128, K = 1024, 30 iterations): both sides iterate freely from the same
    initial parameters; the log-likelihood traces agree to 1e-4 relative at every iteration."""
    spec = synth.CONFIGS[2]
    X = synth.sample_host(spec)
    pi0, mu0, var0 = synth.init_params(X, spec)
    ref = orc.fit(X, pi0, mu0, var0, spec.iters, var_floor=spec.var_floor)
    for path in _paths(fg, spec.D, spec.K):
        ctx.gmm_set_path(path)
        pi, mu, var = _t(pi0), _t(mu0), _t(var0)
        trace, done = ctx.gmm_fit(_t(X), pi, mu, var, spec.iters, spec.var_floor)
        assert done == spec.iters
        np.testing.assert_allclose(trace, ref["trace"], rtol=1e-4, err_msg=f"path {path}")


@pytest.mark.parametrize("N,D,K", [(1, 1, 1), (127, 16, 8), (129, 96, 129), (64, 100, 1), (1000, 3, 65),
                                    (257, 128, 128), (333, 130, 70), (500, 100, 200), (300, 30, 64), (700, 9, 1000),
                                    (1500, 128, 4096), (900, 64, 2048), (700, 100, 1500)])
def test_odd_shapes_one_step(fg, ctx, N, D, K):
    rng = np.random.Generator(np.random.PCG64(N * 1000 + D * 10 + K))
    mu = rng.normal(0, 2, (K, D))
    var = rng.uniform(0.3, 2.0, (K, D))
    pi = rng.dirichlet(np.ones(K))
    X = (mu[rng.integers(0, K, N)] + rng.standard_normal((N, D))).astype(np.float32)
    s = max(data_scale(X), 1.0)
    p32, m32, v32 = pi.astype(np.float32), mu.astype(np.float32), var.astype(np.float32)
    ref = orc.em_step(X, p32, m32, v32)
    for path in _paths(fg, D, K):
        ctx.gmm_set_path(path)
        got = _gpu_step(ctx, _t(X), p32, m32, v32)
        assert abs(got[3] - ref[3]) <= 1e-5 * abs(ref[3]) + 1e-6
        assert_stats_close(N, s, got[:3], ref[:3], f"path {path} shape {(N, D, K)}")


def test_x_pointer_that_is_only_4_byte_aligned(fg, ctx):
    # Both paths use 16-byte loads of X when they can; a view that starts one float into an allocation must take the scalar
    # loads and give the same statistics.
    N, D, K = 333, 96, 129
    rng = np.random.Generator(np.random.PCG64(7))
    mu = rng.normal(0, 2, (K, D))
    var = rng.uniform(0.3, 2.0, (K, D))
    pi = rng.dirichlet(np.ones(K))
    X = (mu[rng.integers(0, K, N)] + rng.standard_normal((N, D))).astype(np.float32)
    s = max(data_scale(X), 1.0)
    p32, m32, v32 = pi.astype(np.float32), mu.astype(np.float32), var.astype(np.float32)
    ref = orc.em_step(X, p32, m32, v32)
    buf = torch.empty(N * D + 1, dtype=torch.float32, device=DEV)
    X_d = buf[1:].view(N, D)
    X_d.copy_(torch.from_numpy(X))
    assert X_d.data_ptr() % 16 == 4
    for path in _paths(fg, D, K):
        ctx.gmm_set_path(path)
        got = _gpu_step(ctx, X_d, p32, m32, v32)
        assert abs(got[3] - ref[3]) <= 1e-5 * abs(ref[3]) + 1e-6
        assert_stats_close(N, s, got[:3], ref[:3], f"path {path}, X misaligned")


@pytest.mark.parametrize("N,D,K", [(1, 1, 1), (127, 16, 8), (64, 100, 1), (333, 60, 33)])
def test_forced_tensor_path_on_small_mixtures(fg, ctx, N, D, K):
    """Shapes AUTO sends to the FP32 path still run on the tensor path when forced (mostly padding, so no speed
    claim); the expanded quadratic form is held to three times the parity tolerance here."""
    rng = np.random.Generator(np.random.PCG64(N * 1000 + D * 10 + K))
    mu = rng.normal(0, 2, (K, D))
    var = rng.uniform(0.3, 2.0, (K, D))
    pi = rng.dirichlet(np.ones(K))
    X = (mu[rng.integers(0, K, N)] + rng.standard_normal((N, D))).astype(np.float32)
    s = max(data_scale(X), 1.0)
    p32, m32, v32 = pi.astype(np.float32), mu.astype(np.float32), var.astype(np.float32)
    ref = orc.em_step(X, p32, m32, v32)
    ctx.gmm_set_path(fg.GMM_PATH_TENSOR)
    got = _gpu_step(ctx, _t(X), p32, m32, v32)
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
    assert abs(got[3] - ref[3]) <= 3e-5 * abs(ref[3]) + 1e-6
    assert_stats_close(N, 3 * s, got[:3], ref[:3], f"forced tensor shape {(N, D, K)}")


def test_auto_path_choice(fg, ctx):
    assert fg.gmm_auto_path(128, 1024) == fg.GMM_PATH_TENSOR
    assert fg.gmm_auto_path(16, 8) == fg.GMM_PATH_FP32
    # D > 128: the two-sweep tensor path (up to D = 1024), for which AUTO also looks at the points per component
    assert fg.gmm_auto_path(768, 4096) == fg.GMM_PATH_TENSOR and fg.tensor_path_supports(768, 4096)
    assert fg.gmm_auto_path(1025, 64) == fg.GMM_PATH_FP32 and not fg.tensor_path_supports(1025, 64)
    assert fg.gmm_auto_path(128, 4096) == fg.GMM_PATH_TENSOR and fg.gmm_auto_path(128, 4097) == fg.GMM_PATH_FP32
    X = _t(np.random.default_rng(0).normal(size=(500, 16)).astype(np.float32))
    pi, mu, var = _t(np.full(8, 1 / 8)), _t(np.random.default_rng(1).normal(size=(8, 16))), _t(np.ones((8, 16)))
    ctx.gmm_em_step(X, pi, mu, var)
    assert ctx.gmm_last_path() == fg.GMM_PATH_FP32
    K = 128
    pi, mu, var = _t(np.full(K, 1 / K)), _t(np.random.default_rng(1).normal(size=(K, 16))), _t(np.ones((K, 16)))
    ctx.gmm_em_step(X, pi, mu, var)
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR


def test_runs_are_bit_identical(fg, ctx):
    spec = synth.CONFIGS[2].with_n(5000)
    X = synth.sample_host(spec)
    pi, mu, var = synth.init_params(X, spec)
    X_d = _t(X)
    for path in _paths(fg, spec.D, spec.K):
        ctx.gmm_set_path(path)
        a = _gpu_step(ctx, X_d, pi, mu, var)
        b = _gpu_step(ctx, X_d, pi, mu, var)
        for u, v in zip(a[:3], b[:3]):
            assert np.array_equal(u, v)
        assert a[3] == b[3]


def test_zero_weight_and_far_components(fg, ctx):
    rng = np.random.Generator(np.random.PCG64(5))
    X = np.concatenate([rng.normal(0, 1, (200, 4)), rng.normal(8, 1, (200, 4))]).astype(np.float32)
    mu = np.array([[0.0] * 4, [8.0] * 4, [1e3] * 4, [4.0] * 4], np.float32)
    var = np.ones((4, 4), np.float32)
    pi = np.array([0.5, 0.5, 0.0, 0.0], np.float32)
    ref = orc.em_step(X, pi, mu, var)
    for path in _paths(fg, 4, 4):
        ctx.gmm_set_path(path)
        Nk, S1, S2, L = _gpu_step(ctx, _t(X), pi, mu, var)
        assert np.isfinite(L) and abs(L - ref[3]) <= 1e-5 * abs(ref[3])
        assert Nk[2] == 0.0 and Nk[3] == 0.0
        assert not np.isnan(S1).any() and not np.isnan(S2).any()
        # finalize keeps the empty components' mean and variance
        pi_d, mu_d, var_d = _t(pi), _t(mu), _t(var)
        ctx.gmm_finalize(len(X), _t(Nk, torch.float64), _t(S1, torch.float64), _t(S2, torch.float64), 1e-6, pi_d,
                         mu_d, var_d)
        assert np.array_equal(mu_d.cpu().numpy()[2:], mu[2:]) and np.array_equal(var_d.cpu().numpy()[2:], var[2:])
        assert pi_d.cpu().numpy()[2] == 0.0


def test_variance_floor_is_applied(fg, ctx):
    X = np.concatenate([np.zeros((50, 2)), np.full((50, 2), 10.0)]).astype(np.float32)
    mu = np.array([[0.0, 0.0], [10.0, 10.0]], np.float32)
    var = np.ones((2, 2), np.float32)
    pi = np.array([0.5, 0.5], np.float32)
    pi_d, mu_d, var_d = _t(pi), _t(mu), _t(var)
    trace, _ = ctx.gmm_fit(_t(X), pi_d, mu_d, var_d, 2, 1e-3)
    np.testing.assert_allclose(var_d.cpu().numpy(), 1e-3, rtol=1e-6)
    ref = orc.fit(X, pi, mu, var, 2, var_floor=1e-3)
    np.testing.assert_allclose(trace, ref["trace"], rtol=1e-5)


def test_invalid_arguments_and_parameters(fg, ctx):
    X = _t(np.zeros((10, 4), np.float32))
    pi, mu, var = _t(np.full(2, 0.5)), _t(np.zeros((2, 4))), _t(np.ones((2, 4)))
    with pytest.raises(fg.GmmError) as e:
        ctx.gmm_assign_topm(X, pi, mu, var, 3)
    assert e.value.code == fg.GMM_EINVAL
    with pytest.raises(fg.GmmError) as e:
        ctx.gmm_fit(X, pi, mu, var, 0)
    assert e.value.code == fg.GMM_EINVAL
    bad = var.clone()
    bad[1, 2] = 0.0
    with pytest.raises(fg.GmmError) as e:
        ctx.gmm_em_step(X, pi, mu, bad)
    assert e.value.code == fg.GMM_ENUMERIC
    negpi = _t(np.array([1.5, -0.5]))
    with pytest.raises(fg.GmmError) as e:
        ctx.gmm_em_step(X, negpi, mu, var)
    assert e.value.code == fg.GMM_ENUMERIC
    # the context is still usable afterwards
    ctx.gmm_em_step(X, pi, mu, var)
    # misaligned pointer
    buf = torch.zeros(10 * 4 * 4 + 8, dtype=torch.uint8, device=DEV)
    rc = fg.lib.gmm_em_step(ctx._h, buf.data_ptr() + 1, 10, 4, 2, pi.data_ptr(), mu.data_ptr(), var.data_ptr(),
                            torch.zeros(2, dtype=torch.float64, device=DEV).data_ptr(),
                            torch.zeros(8, dtype=torch.float64, device=DEV).data_ptr(),
                            torch.zeros(8, dtype=torch.float64, device=DEV).data_ptr(),
                            __import__("ctypes").byref(__import__("ctypes").c_double()))
    assert rc == fg.GMM_EALIGN


def test_host_streaming_matches_device_call(fg, ctx):
    spec = synth.CONFIGS[2].with_n(4000)
    X = synth.sample_host(spec)
    pi, mu, var = synth.init_params(X, spec)
    for path in _paths(fg, spec.D, spec.K):
        ctx.gmm_set_path(path)
        a = _gpu_step(ctx, _t(X), pi, mu, var)
        b = ctx.gmm_em_step_host(X, pi, mu, var)
        for u, v in zip(a[:3], b[:3]):
            assert np.array_equal(u, v)
        assert a[3] == b[3]


def test_host_streaming_multiple_chunks_is_additive(fg, ctx):
    # D=2048 makes a staging chunk hold 16384 rows, so 40000 rows take three chunks
    rng = np.random.Generator(np.random.PCG64(77))
    N, D, K = 40_000, 2048, 4
    mu = rng.normal(0, 1, (K, D)).astype(np.float32)
    var = rng.uniform(0.5, 1.5, (K, D)).astype(np.float32)
    pi = np.full(K, 1 / K, np.float32)
    X = (mu[rng.integers(0, K, N)] + rng.standard_normal((N, D), dtype=np.float32)).astype(np.float32)
    ctx.gmm_set_path(fg.GMM_PATH_FP32)
    a = _gpu_step(ctx, _t(X), pi, mu, var)
    b = ctx.gmm_em_step_host(X, pi, mu, var)
    for u, v in zip(a[:3], b[:3]):
        # float32 per-CTA partials are grouped differently when the points arrive in chunks
        np.testing.assert_allclose(u, v, rtol=1e-5, atol=1e-5 * np.abs(v).max())
    assert b[3] == pytest.approx(a[3], rel=1e-9)


@pytest.mark.parametrize("cfg,n,m", [(1, 2000, 1), (1, 2000, 2), (1, 1999, 4), (1, 500, 8), (2, 1500, 2), (2, 1200, 4)])
def test_topm_against_oracle(fg, ctx, cfg, n, m):
    spec = synth.CONFIGS[cfg].with_n(n)
    X = synth.sample_host(spec)
    pi0, mu0, var0 = synth.init_params(X, spec)
    fit = orc.fit(X, pi0, mu0, var0, 3, var_floor=spec.var_floor)
    p32, m32, v32 = (fit[k].astype(np.float32) for k in ("pi", "mu", "var"))
    idx_g, resp_g = ctx.gmm_assign_topm(_t(X), _t(p32), _t(m32), _t(v32), m)
    torch.cuda.synchronize()
    _check_topm(X, p32, m32, v32, m, idx_g.cpu().numpy(), resp_g.cpu().numpy(), f"cfg {cfg} m {m}")


def _random_mixture(rng, N, D, K, spread=2.0):
    X = (rng.normal(size=(N, D)) * spread).astype(np.float32)
    mu = (X[rng.choice(N, K, replace=K > N)] + 0.1 * rng.normal(size=(K, D))).astype(np.float32)
    var = rng.uniform(0.5, 2.0, size=(K, D)).astype(np.float32)
    pi = rng.dirichlet(np.ones(K)).astype(np.float32)
    return X, pi, mu, var


def _topm_tensor_vs_oracle(fg, ctx, X, pi, mu, var, m, what, expect_path=None):
    ctx.gmm_set_path(fg.GMM_PATH_TENSOR)
    idx_g, resp_g = ctx.gmm_assign_topm(_t(X), _t(pi), _t(mu), _t(var), m)
    torch.cuda.synchronize()
    assert ctx.gmm_last_path() == (expect_path or fg.GMM_PATH_TENSOR)
    _check_topm(X, pi, mu, var, m, idx_g.cpu().numpy(), resp_g.cpu().numpy(), what)


@pytest.mark.parametrize("N,D,K,m", [(1500, 128, 1024, 4), (777, 30, 100, 2), (2000, 100, 200, 8), (300, 9, 1000, 1),
                                     (4097, 64, 640, 3), (129, 128, 64, 4), (1000, 128, 1024, 1),
                                     (1500, 128, 4096, 4), (1100, 96, 2048, 2)])
def test_topm_tensor_path_against_oracle(fg, ctx, N, D, K, m):
    """Tensor-core selection + exact refinement (Sections 4.2-4.3): several tiles of 128 points with a ragged tail, odd
    numbers of 128-component chunks, dimensions that do not fill the 64-column atoms, and K beyond what the E+M tile
    kernel takes (the paper's IVF sizes go up to K = 4096)."""
    X, pi, mu, var = _random_mixture(np.random.default_rng(N + D + K), N, D, K)
    _topm_tensor_vs_oracle(fg, ctx, X, pi, mu, var, m, f"tensor top-m N={N} D={D} K={K} m={m}")


@pytest.mark.parametrize("N,D,K,m,path", [(3000, 128, 1024, 1, "tensor"), (2500, 64, 200, 4, "tensor"), (1100, 96, 4096, 1, "tensor"),
                                          (2000, 100, 300, 8, "tensor"), (2000, 16, 8, 2, "fp32"), (900, 130, 70, 1, "fp32")])
def test_topm_indices_only(fg, ctx, N, D, K, m, path):
    """gmm_assign_topm without a responsibility array (the hard assignment of Section 4.2 for m = 1): the indices must be
    those the oracle ranks first; the values used for the comparison are the oracle's own responsibilities at the GPU's
    indices.  Also at the initial parameters of config 2, where posteriors are broad."""
    cases = [_random_mixture(np.random.default_rng(N + D + K + m), N, D, K)]
    if K == 1024:
        spec = synth.CONFIGS[2].with_n(N)
        Xc = synth.sample_host(spec)
        cases.append((Xc,) + tuple(synth.init_params(Xc, spec)))
    for X, pi, mu, var in cases:
        ctx.gmm_set_path(fg.GMM_PATH_TENSOR if path == "tensor" else fg.GMM_PATH_FP32)
        idx_g, none = ctx.gmm_assign_topm(_t(X), _t(pi), _t(mu), _t(var), m, indices_only=True)
        torch.cuda.synchronize()
        assert none is None
        idx_g = idx_g.cpu().numpy()
        _check_topm(X, pi, mu, var, m, idx_g, None, f"indices only N={N} D={D} K={K} m={m}")
        # and the same indices as the call that also returns the values, except where those tie
        idx_f, resp_f = ctx.gmm_assign_topm(_t(X), _t(pi), _t(mu), _t(var), m)
        torch.cuda.synchronize()
        differ = (idx_f.cpu().numpy() != idx_g).any(axis=1)
        assert differ.mean() <= 0.01


def test_topm_tensor_path_after_em_iterations(fg, ctx):
    spec = synth.CONFIGS[2].with_n(3000)
    X = synth.sample_host(spec)
    pi0, mu0, var0 = synth.init_params(X, spec)
    for iters in (0, 3):            # broad posteriors at the initial parameters, sharp ones (and collapsed components) later
        fit = orc.fit(X, pi0, mu0, var0, iters, var_floor=spec.var_floor) if iters else {"pi": pi0, "mu": mu0, "var": var0}
        p32, m32, v32 = (np.asarray(fit[k], np.float32) for k in ("pi", "mu", "var"))
        _topm_tensor_vs_oracle(fg, ctx, X, p32, m32, v32, 4, f"config 2 after {iters} iterations")


def test_topm_tensor_path_degenerate_parameters(fg, ctx):
    rng = np.random.default_rng(11)
    N, D, K = 3000, 128, 256
    X = rng.normal(size=(N, D)).astype(np.float32)
    mu = X[:K].copy()
    pi = np.full(K, 1 / K, np.float32)
    var = np.ones((K, D), np.float32)
    # a few components collapsed onto their point at the variance floor: evaluated exactly for every point
    v = var.copy(); v[:5] = 1e-6
    _topm_tensor_vs_oracle(fg, ctx, X, pi, mu, v, 4, "5 collapsed components")
    v = var.copy(); v[:40] = 1e-6
    v[40:60, ::7] = 1e-4            # narrow in some dimensions only: the cheap test must look at those
    _topm_tensor_vs_oracle(fg, ctx, X, pi, mu, v, 4, "60 ill-conditioned components")
    # more of them than the tensor-core kernels take (256): the FP32 kernels run (decided on the device)
    X5, pi5, mu5, var5 = _random_mixture(np.random.default_rng(12), 2000, 64, 512, spread=1.0)
    var5[:300] = 1e-6
    _topm_tensor_vs_oracle(fg, ctx, X5, pi5, mu5, var5, 2, "300 collapsed components")
    # zero weights; exactly equal components (ties go to the smaller index); posteriors spread over hundreds of components
    p2 = pi.copy(); p2[::2] = 0; p2 /= p2.sum()
    _topm_tensor_vs_oracle(fg, ctx, X, p2, mu, var, 4, "zero weights")
    m2 = mu.copy(); m2[10:20] = m2[10]
    _topm_tensor_vs_oracle(fg, ctx, X, pi, m2, var, 8, "identical components")
    _topm_tensor_vs_oracle(fg, ctx, X, pi, (mu * 0.01).astype(np.float32), var * 100, 4, "diffuse posteriors")
    # all components identical: every point ties K ways
    Xz = np.zeros((200, D), np.float32)
    idx, resp = ctx.gmm_assign_topm(_t(Xz), _t(pi), _t(np.zeros((K, D))), _t(var), 3)
    torch.cuda.synchronize()
    assert np.array_equal(idx.cpu().numpy(), np.tile([0, 1, 2], (200, 1)))
    np.testing.assert_allclose(resp.cpu().numpy(), 1 / K, rtol=1e-5)


def test_topm_tensor_path_over_several_pieces(fg, ctx, monkeypatch):
    """Pieces of 1024 points (instead of 2^19): the candidate records and the planes of Y are reused piece after piece."""
    monkeypatch.setenv("GMM_TC_PIECE", "1024")
    c2 = fg.Context(0)
    try:
        X, pi, mu, var = _random_mixture(np.random.default_rng(5), 2500, 64, 256)
        _topm_tensor_vs_oracle(fg, c2, X, pi, mu, var, 2, "three pieces")
    finally:
        c2.close()


def test_topm_exact_ties_go_to_the_smaller_index(fg, ctx):
    X = _t(np.zeros((70, 4), np.float32))
    K = 6
    idx, resp = ctx.gmm_assign_topm(X, _t(np.full(K, 1 / K)), _t(np.zeros((K, 4))), _t(np.ones((K, 4))), 3)
    torch.cuda.synchronize()
    assert np.array_equal(idx.cpu().numpy(), np.tile([0, 1, 2], (70, 1)))
    np.testing.assert_allclose(resp.cpu().numpy(), 1 / K, rtol=1e-5)


def test_data_far_from_the_origin(fg, ctx):
    """All points and means sit 300 standard deviations from the origin.  Both paths form their products, and accumulate
    their sums, about a per-dimension centre of the means and shift the statistics back in float64, so the offset costs
    no precision: the updated parameters (whose variance is the cancelling difference S2 / N_k - mu^2, here 1 against
    90,000) must meet the ordinary tolerances, and so must the raw statistics relative to their own size."""
    rng = np.random.default_rng(21)
    N, D, K = 4000, 64, 96
    X, pi, mu, var = _random_mixture(rng, N, D, K, spread=1.5)
    X = (X + 300.0).astype(np.float32)
    mu = (mu + 300.0).astype(np.float32)
    s = data_scale(X)
    ref = orc.em_step(X, pi, mu, var)
    pr, mr, vr, _, _, _ = orc.em_iteration(X, pi, mu, var, var_floor=1e-6)
    for path in _paths(fg, D, K):
        ctx.gmm_set_path(path)
        got = _gpu_step(ctx, _t(X), pi, mu, var)
        what = f"path {path}, data far from the origin"
        assert abs(got[3] - ref[3]) <= 1e-5 * abs(ref[3]), path
        assert_stats_close(N, s, got[:3], ref[:3], what)
        pi_d, mu_d, var_d = _t(pi), _t(mu), _t(var)
        ctx.gmm_finalize(N, _t(got[0], torch.float64), _t(got[1], torch.float64), _t(got[2], torch.float64), 1e-6,
                         pi_d, mu_d, var_d)
        assert_params_close(N, s, (pi_d.cpu().numpy(), mu_d.cpu().numpy(), var_d.cpu().numpy()), (pr, mr, vr), ref[0], what)
        idx_g, resp_g = ctx.gmm_assign_topm(_t(X), _t(pi), _t(mu), _t(var), 3)
        torch.cuda.synchronize()
        _check_topm(X, pi, mu, var, 3, idx_g.cpu().numpy(), resp_g.cpu().numpy(), f"path {path}, far from the origin")


def test_errors_of_asynchronous_calls_surface_at_the_next_synchronising_call(fg, ctx):
    """gmm_assign_topm returns with its work in flight, so what its kernels find wrong (here var <= 0) cannot come back
    as its return value: the device-side status word keeps it until gmm_sync_status, or the next call that synchronises,
    reports it; the report clears it."""
    rng = np.random.default_rng(5)
    for D, K in ((16, 8), (64, 128)):                   # FP32 kernels; tensor-core assignment
        X, pi, mu, var = _random_mixture(rng, 500, D, K)
        bad = var.copy()
        bad[K // 2, 3] = 0.0
        with fg.Context(0) as c:
            c.gmm_assign_topm(_t(X), _t(pi), _t(mu), _t(bad), 2)                # asynchronous: no error yet
            with pytest.raises(fg.GmmError) as e:
                c.gmm_sync_status()
            assert e.value.code == fg.GMM_ENUMERIC
            c.gmm_sync_status()                                                 # reported once, then clean
            c.gmm_assign_topm(_t(X), _t(pi), _t(mu), _t(bad), 2)
            with pytest.raises(fg.GmmError) as e:                               # ... or at the next synchronising call
                c.gmm_em_step(_t(X), _t(pi), _t(mu), _t(var))
            assert e.value.code == fg.GMM_ENUMERIC
            Nk = c.gmm_em_step(_t(X), _t(pi), _t(mu), _t(var))[0]              # and the context stays usable
            assert abs(float(Nk.sum()) - 500) < 1e-3


def test_non_finite_data_is_reported_and_fit_keeps_the_last_good_parameters(fg, ctx):
    rng = np.random.default_rng(6)
    X, pi, mu, var = _random_mixture(rng, 3000, 32, 16)
    for poison in (np.nan, np.inf):
        Xb = X.copy()
        Xb[1234, 5] = poison
        for path in _paths(fg, 32, 16) + [fg.GMM_PATH_TENSOR]:
            ctx.gmm_set_path(path)
            with pytest.raises(fg.GmmError) as e:
                ctx.gmm_em_step(_t(Xb), _t(pi), _t(mu), _t(var))
            assert e.value.code == fg.GMM_ENUMERIC
            pi_d, mu_d, var_d = _t(pi), _t(mu), _t(var)
            with pytest.raises(fg.GmmError) as e:
                ctx.gmm_fit(_t(Xb), pi_d, mu_d, var_d, 3)
            assert e.value.code == fg.GMM_ENUMERIC
            # the failed iteration's update was not applied
            assert np.array_equal(mu_d.cpu().numpy(), mu) and np.array_equal(var_d.cpu().numpy(), var)
            assert np.array_equal(pi_d.cpu().numpy(), pi)
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    ctx.gmm_em_step(_t(X), _t(pi), _t(mu), _t(var))


def test_fit_stops_on_the_relative_change_of_the_log_likelihood(fg, ctx):
    """tol > 0 (the paper's "sufficiently small change", Section 2): the same stopping iteration as the oracle's loop."""
    spec = synth.CONFIGS[1]
    X = synth.sample_host(spec)
    pi0, mu0, var0 = synth.init_params(X, spec)
    tol = 2e-4
    ref = orc.fit(X, pi0, mu0, var0, 40, var_floor=spec.var_floor)["trace"]
    stop = next((t + 1 for t in range(1, len(ref)) if abs(ref[t] - ref[t - 1]) <= tol * abs(ref[t])), len(ref))
    assert 2 <= stop < 40
    for path in _paths(fg, spec.D, spec.K):
        ctx.gmm_set_path(path)
        trace, done = ctx.gmm_fit(_t(X), _t(pi0), _t(mu0), _t(var0), 40, spec.var_floor, tol=tol)
        assert done == stop and len(trace) == stop
        np.testing.assert_allclose(trace, ref[:stop], rtol=1e-4)


def test_update_counts_report_floored_variances_and_empty_components(fg, ctx):
    rng = np.random.default_rng(8)
    N, D, K = 2000, 8, 5
    X = rng.normal(size=(N, D)).astype(np.float32)
    X[:, 0] = 2.0                                        # a constant dimension: every live component's variance there is 0
    pi = np.array([0.5, 0.5, 0.0, 0.0, 0.0], np.float32)            # three components get no weight at all
    mu = rng.normal(size=(K, D)).astype(np.float32)
    var = np.ones((K, D), np.float32)
    Nk, S1, S2, _ = ctx.gmm_em_step(_t(X), _t(pi), _t(mu), _t(var))
    pi_d, mu_d, var_d = _t(pi), _t(mu), _t(var)
    ctx.gmm_finalize(N, Nk, S1, S2, 1e-3, pi_d, mu_d, var_d)
    assert ctx.gmm_update_counts() == (2, 3)
    ctx.gmm_finalize_isotropic(N, Nk, S1, S2, 1e-3, pi_d, mu_d, var_d)
    assert ctx.gmm_update_counts() == (0, 3)
    pi_d, mu_d, var_d = _t(pi), _t(mu), _t(var)
    ctx.gmm_fit(_t(X), pi_d, mu_d, var_d, 2, 1e-3)
    assert ctx.gmm_update_counts() == (2, 3)


def test_scratch_allocation_failure_is_reported_as_enomem(fg):
    """All but 256 MB of the free device memory is taken before the first call that needs the 600 MB of scratch."""
    free_b, _ = torch.cuda.mem_get_info()
    hog = torch.empty(max(0, free_b - (256 << 20)), dtype=torch.uint8, device=DEV)
    try:
        X = _t(np.zeros((100, 128), np.float32))
        K = 1024
        with fg.Context(0) as c:
            with pytest.raises(fg.GmmError) as e:
                c.gmm_em_step(X, _t(np.full(K, 1 / K)), _t(np.zeros((K, 128))), _t(np.ones((K, 128))))
            assert e.value.code == fg.GMM_ENOMEM
    finally:
        del hog
        torch.cuda.empty_cache()


@pytest.mark.parametrize("N,D,K", [(3000, 3, 1), (7001, 3, 5), (2000, 8, 2)])
def test_forced_tensor_path_small_dimension_far_from_the_origin(fg, ctx, N, D, K):
    """Few dimensions, few components, data 50 units from the origin: log2 Z of a point is small while the error estimate
    of the expanded form is not negligible, and the log-likelihood sums that error instead of averaging it out; the limit
    above which components are recomputed exactly is therefore capped by the dimension."""
    rng = np.random.default_rng(N + D + K)
    X = (rng.normal(size=(N, D)) * 0.7 + 50.0).astype(np.float32)
    mu = (X[rng.integers(0, N, K)] + 0.1 * rng.normal(size=(K, D))).astype(np.float32)
    var = rng.uniform(0.3, 2.0, size=(K, D)).astype(np.float32)
    pi = rng.dirichlet(np.ones(K)).astype(np.float32)
    ref = orc.em_step(X, pi, mu, var)
    ctx.gmm_set_path(fg.GMM_PATH_TENSOR)
    for _ in range(2):                      # the second call may run the other filter
        got = _gpu_step(ctx, _t(X), pi, mu, var)
        assert abs(got[3] - ref[3]) <= 1e-5 * abs(ref[3])
        assert_stats_close(N, data_scale(X), got[:3], ref[:3], f"forced tensor path N={N} D={D} K={K}")


def test_scratch_does_not_grow_with_n(fg, ctx):
    assert fg.gmm_scratch_bytes(128, 1024) == fg.gmm_scratch_bytes(128, 1024)
    spec = synth.CONFIGS[2]
    Xs = synth.sample_device(spec.with_n(2_000), DEV)
    Xl = synth.sample_device(spec.with_n(300_000), DEV)
    pi, mu, var = (_t(a) for a in synth.init_params(Xs, spec.with_n(2_000)))
    ctx.gmm_em_step(Xs, pi, mu, var)
    torch.cuda.synchronize()
    free_small = torch.cuda.mem_get_info()[0]
    ctx.gmm_em_step(Xl, pi, mu, var)
    torch.cuda.synchronize()
    free_large = torch.cuda.mem_get_info()[0]
    assert free_small == free_large, "device memory in use changed with N"


def test_config3_full_size_conservation_and_subsample(fg, ctx):
    """N = 1M, K = 1024, D = 128 in the launch configuration the benchmark times: conservation laws at full N
    (sum_k N_k = N, sum_k S1 = column sums of X, sum_k S2 = column sums of X^2) and one oracle step on a seeded
    50K-row subsample that the GPU re-runs on the same rows."""
    spec = synth.CONFIGS[3]
    X = synth.sample_device(spec, DEV)
    pi0, mu0, var0 = synth.init_params(X, spec)
    N = spec.N
    col1 = X.double().sum(0).cpu().numpy()
    col2 = (X.double() ** 2).sum(0).cpu().numpy()
    rows = synth.subsample_rows(N, 50_000, spec.seed)
    Xsub_d = X[torch.as_tensor(rows, device=DEV)].contiguous()
    Xsub = Xsub_d.cpu().numpy()
    s = data_scale(Xsub)
    ref = orc.em_step(Xsub, pi0, mu0, var0)
    for path in _paths(fg, spec.D, spec.K):
        ctx.gmm_set_path(path)
        Nk, S1, S2, L = _gpu_step(ctx, X, pi0, mu0, var0)
        assert abs(Nk.sum() - N) <= 1e-6 * N
        np.testing.assert_allclose(S1.sum(0), col1, rtol=1e-5, atol=1e-5 * N * s)
        np.testing.assert_allclose(S2.sum(0), col2, rtol=1e-5)
        assert np.isfinite(L)
        got = _gpu_step(ctx, Xsub_d, pi0, mu0, var0)
        assert abs(got[3] - ref[3]) <= 1e-5 * abs(ref[3])
        assert_stats_close(len(rows), s, got[:3], ref[:3], f"path {path} config 3 subsample")
    _full_size_topm_check(fg, ctx, X, spec, pi0, mu0, var0, "config 3, all rows, sampled")


def test_config3_full_oracle_step_after_five_iterations(fg, ctx):
    """Where the tensor path's accuracy knob is loose it must be checked against the oracle itself: the limit above which a
    component's logits are recomputed exactly grows with sqrt(N / K) (4.7e-3 here against 1e-3 on a 50K-row subsample),
    and after a few iterations from the data-row initialisation some components have collapsed onto points and others
    are narrow in a few dimensions.  So: five EM iterations on the GPU (AUTO path), then ONE float64 oracle step over
    all 1M rows at those parameters, compared per component at the ordinary tolerances."""
    spec = synth.CONFIGS[3]
    X = synth.sample_device(spec, DEV)
    pi0, mu0, var0 = synth.init_params(X, spec)
    N = spec.N
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    pi_d, mu_d, var_d = _t(pi0), _t(mu0), _t(var0)
    ctx.gmm_fit(X, pi_d, mu_d, var_d, 5, spec.var_floor)
    p5, m5, v5 = pi_d.cpu().numpy(), mu_d.cpu().numpy(), var_d.cpu().numpy()
    Xh = X.cpu().numpy()
    s = data_scale(Xh[:200_000])
    Nk_r, S1_r, S2_r, L_r = orc.em_step(Xh, p5, m5, v5)
    pr, mr, vr = orc.finalize_moments(N, Nk_r, S1_r, S2_r, spec.var_floor, m5.astype(np.float64), v5.astype(np.float64))
    got = _gpu_step(ctx, X, p5, m5, v5)
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR and ctx.gmm_last_exact_count() > 0
    what = "config 3, all 1M rows, after 5 iterations, AUTO path vs oracle"
    assert abs(got[3] - L_r) <= 1e-5 * abs(L_r), what
    assert_stats_close(N, s, got[:3], (Nk_r, S1_r, S2_r), what)
    assert_params_close(N, s, _params_from(ctx, N, got, spec.var_floor, p5, m5, v5), (pr, mr, vr), Nk_r, what)


def _full_size_topm_check(fg, ctx, X, spec, pi0, mu0, var0, what, n_rows=3000):
    """Top-4 assignment over ALL rows of X, as bench.py --assign-m 4 launches it, under the parameters one EM iteration
    gives; a seeded sample of rows is compared with the oracle's assignment of those rows one by one."""
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    pi, mu, var = _t(pi0), _t(mu0), _t(var0)
    Nk, S1, S2, _ = ctx.gmm_em_step(X, pi, mu, var)
    ctx.gmm_finalize(spec.N, Nk, S1, S2, spec.var_floor, pi, mu, var)
    idx, resp = ctx.gmm_assign_topm(X, pi, mu, var, 4)
    torch.cuda.synchronize()
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
    assert int(idx.min()) >= 0 and int(idx.max()) < spec.K
    rows = synth.subsample_rows(spec.N, n_rows, spec.seed + 17)
    rows_d = torch.as_tensor(rows, device=DEV)
    _check_topm(X[rows_d].cpu().numpy(), pi.cpu().numpy(), mu.cpu().numpy(), var.cpu().numpy(), 4,
                idx[rows_d].cpu().numpy(), resp[rows_d].cpu().numpy(), what)


def _column_sums(X):
    """Column sums of X and X^2 in float64, in chunks (X may be tens of GB)."""
    s1 = torch.zeros(X.shape[1], dtype=torch.float64, device=X.device)
    s2 = torch.zeros_like(s1)
    step = 1 << 22
    for lo in range(0, X.shape[0], step):
        x = X[lo:lo + step].double()
        s1 += x.sum(0)
        s2 += (x * x).sum(0)
    return s1.cpu().numpy(), s2.cpu().numpy()


def test_config4_full_size_conservation_additivity_and_subsample(fg, ctx):
    """N = 100M, K = 1024, D = 128 (51.2 GB of X) in the launch configuration the benchmark times (AUTO path = the
    tensor-core kernel): the conservation laws hold at full N, the statistics of the whole equal the sum over two
    halves (long accumulation chains), device memory in use does not grow with N, and one oracle step on a seeded
    50K-row subsample matches the GPU on the same rows."""
    spec = synth.CONFIGS[4]
    free_b, _ = torch.cuda.mem_get_info()
    if free_b < 60e9:
        pytest.skip("needs 60 GB of free device memory")
    X = synth.sample_device(spec, DEV)
    pi0, mu0, var0 = synth.init_params(X, spec)
    N = spec.N
    col1, col2 = _column_sums(X)
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    torch.cuda.synchronize()
    Nk, S1, S2, L = _gpu_step(ctx, X, pi0, mu0, var0)
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
    free_after = torch.cuda.mem_get_info()[0]
    s = float(np.sqrt(synth.global_variance(X[:1_000_000]).mean()))
    assert abs(Nk.sum() - N) <= 1e-6 * N
    np.testing.assert_allclose(S1.sum(0), col1, rtol=1e-5, atol=1e-5 * N * s)
    np.testing.assert_allclose(S2.sum(0), col2, rtol=1e-5)
    assert np.isfinite(L)
    # additivity over two halves
    h = N // 2
    a = _gpu_step(ctx, X[:h], pi0, mu0, var0)
    b = _gpu_step(ctx, X[h:], pi0, mu0, var0)
    assert torch.cuda.mem_get_info()[0] == free_after, "device memory in use changed with N"
    np.testing.assert_allclose(a[0] + b[0], Nk, rtol=1e-6, atol=1e-6 * N / spec.K)
    np.testing.assert_allclose(a[2] + b[2], S2, rtol=2e-5, atol=1e-5 * N / spec.K)
    assert abs((a[3] + b[3]) - L) <= 1e-9 * abs(L)
    _full_size_topm_check(fg, ctx, X, spec, pi0, mu0, var0, "config 4, all rows, sampled")
    # The regime the benchmark times: parameters after five iterations (collapsed and narrow components; the exact
    # recomputation protocol active with the limit of N = 100M, 4.7e-2, fifty times that of the subsample check below).
    # No oracle run of this size is affordable; the FP32 kernels (no approximation to tune; themselves checked against
    # the oracle) take all 100M rows in six seconds, so the tensor path is compared with them over ALL rows at the
    # ordinary tolerances.
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    pi_d, mu_d, var_d = _t(pi0), _t(mu0), _t(var0)
    ctx.gmm_fit(X, pi_d, mu_d, var_d, 5, spec.var_floor)
    p5, m5, v5 = pi_d.cpu().numpy(), mu_d.cpu().numpy(), var_d.cpu().numpy()
    t_ = _gpu_step(ctx, X, p5, m5, v5)
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR and ctx.gmm_last_exact_count() > 0
    ctx.gmm_set_path(fg.GMM_PATH_FP32)
    f_ = _gpu_step(ctx, X, p5, m5, v5)
    what = "config 4, all 100M rows, after 5 iterations, tensor vs FP32 path"
    assert abs(t_[3] - f_[3]) <= 1e-5 * abs(f_[3]), what
    assert_stats_close(N, s, t_[:3], f_[:3], what)
    assert_params_close(N, s, _params_from(ctx, N, t_, spec.var_floor, p5, m5, v5),
                        _params_from(ctx, N, f_, spec.var_floor, p5, m5, v5), f_[0], what)
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    # oracle on a seeded subsample, GPU re-run on the same rows
    rows = synth.subsample_rows(N, 50_000, spec.seed)
    Xsub_d = X[torch.as_tensor(rows, device=DEV)].contiguous()
    del X
    Xsub = Xsub_d.cpu().numpy()
    ref = orc.em_step(Xsub, pi0, mu0, var0)
    got = _gpu_step(ctx, Xsub_d, pi0, mu0, var0)
    assert abs(got[3] - ref[3]) <= 1e-5 * abs(ref[3])
    assert_stats_close(len(rows), data_scale(Xsub), got[:3], ref[:3], "config 4 subsample")


def _config5_subsample_check(fg, ctx, X, spec, pi0, mu0, var0, idx, resp, p1, m1, v1):
    """Oracle on a seeded 20K-row subsample: one EM step from the initial parameters (the GPU re-runs it on the same
    rows; with 5 points per component AUTO takes the FP32 kernels there) and the top-4 rows of the full-size assignment."""
    rows = synth.subsample_rows(spec.N, 20_000, spec.seed)
    rows_d = torch.as_tensor(rows, device=DEV)
    Xsub_d = X[rows_d].contiguous()
    Xsub = Xsub_d.cpu().numpy()
    ref = orc.em_step(Xsub, pi0, mu0, var0)
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    got = _gpu_step(ctx, Xsub_d, pi0, mu0, var0)
    assert abs(got[3] - ref[3]) <= 1e-5 * abs(ref[3])
    assert_stats_close(len(rows), data_scale(Xsub), got[:3], ref[:3], "config 5 subsample")
    _check_topm(Xsub, p1, m1, v1, 4, idx[rows_d].cpu().numpy(), resp[rows_d].cpu().numpy(), "config 5 top-4 subsample")


def _params_from(ctx, N, stats, var_floor, pi, mu, var):
    pi_d, mu_d, var_d = _t(pi), _t(mu), _t(var)
    ctx.gmm_finalize(N, _t(stats[0], torch.float64), _t(stats[1], torch.float64), _t(stats[2], torch.float64), var_floor,
                     pi_d, mu_d, var_d)
    return pi_d.cpu().numpy(), mu_d.cpu().numpy(), var_d.cpu().numpy()


def test_config5_shape_tensor_path_against_fp32_path_and_oracle_subsample(fg, ctx):
    """The IVF coarse-quantizer shape (D = 768, K = 4096, unit-norm vectors) on 1M device-generated points, the launch
    configuration the benchmark times (AUTO = the two-sweep tensor path).  No oracle run of this size is affordable, so:
    conservation laws at that N; the tensor path against the FP32 kernels (which have no approximation to tune, and are
    themselves checked against the oracle on the subsample below) over the SAME 1M rows at the ordinary tolerances, at
    the initial parameters and at the parameters five EM iterations later (sharp posteriors, a thousand components
    collapsed onto single points, hundreds that hold a few dozen points); the oracle on a seeded 20K-row subsample for
    the step and the top-4 output."""
    spec = synth.CONFIGS[5].with_n(1_000_000)
    X = synth.sample_device(spec, DEV)
    pi0, mu0, var0 = synth.init_params(X, spec)
    N = spec.N
    s = float(np.sqrt(synth.global_variance(X[:200_000]).mean()))
    col1, col2 = _column_sums(X)
    pi, mu, var = pi0, mu0, var0
    for stage in ("initial parameters", "after 5 iterations"):
        ctx.gmm_set_path(fg.GMM_PATH_AUTO)
        t_ = _gpu_step(ctx, X, pi, mu, var)
        assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR, stage
        assert abs(t_[0].sum() - N) <= 1e-5 * N
        np.testing.assert_allclose(t_[2].sum(0), col2, rtol=1e-4)
        np.testing.assert_allclose(t_[1].sum(0), col1, rtol=1e-4, atol=1e-4 * N * 0.04)
        ctx.gmm_set_path(fg.GMM_PATH_FP32)
        f_ = _gpu_step(ctx, X, pi, mu, var)
        what = f"config 5 shape, 1M rows, tensor vs FP32 path, {stage}"
        assert abs(t_[3] - f_[3]) <= 1e-5 * abs(f_[3]), what
        assert_stats_close(N, s, t_[:3], f_[:3], what)
        assert_params_close(N, s, _params_from(ctx, N, t_, spec.var_floor, pi, mu, var),
                            _params_from(ctx, N, f_, spec.var_floor, pi, mu, var), f_[0], what)
        if stage == "initial parameters":
            ctx.gmm_set_path(fg.GMM_PATH_AUTO)
            pi_d, mu_d, var_d = _t(pi0), _t(mu0), _t(var0)
            ctx.gmm_fit(X, pi_d, mu_d, var_d, 5, spec.var_floor)
            pi, mu, var = pi_d.cpu().numpy(), mu_d.cpu().numpy(), var_d.cpu().numpy()
    assert ctx.gmm_last_exact_count() == 0            # (the last step ran on the FP32 path)
    # parameters after one update from the initial ones for the top-m check, as config 5 prescribes after its fit
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    st = _gpu_step(ctx, X, pi0, mu0, var0)
    p1, m1, v1 = _params_from(ctx, N, st, spec.var_floor, pi0, mu0, var0)
    idx, resp = ctx.gmm_assign_topm(X, _t(p1), _t(m1), _t(v1), 4)
    torch.cuda.synchronize()
    _config5_subsample_check(fg, ctx, X, spec, pi0, mu0, var0, idx, resp, p1, m1, v1)


def test_config5_full_size_fit_and_assignment(fg, ctx):
    """Config 5 as stated: N = 10M (30.7 GB of X), 20 EM iterations (gmm_fit, AUTO path), then gmm_assign_topm with m = 4,
    the hard assignment and gmm_score_samples over all N; conservation at full N, a non-decreasing log-likelihood trace, device memory in use independent of N,
    the oracle on a seeded 20K-row subsample for one step and for the top-4 output."""
    spec = synth.CONFIGS[5]
    free_b, _ = torch.cuda.mem_get_info()
    if free_b < 40e9:
        pytest.skip("needs 40 GB of free device memory")
    X = synth.sample_device(spec, DEV)
    pi0, mu0, var0 = synth.init_params(X, spec)
    N = spec.N
    col1, col2 = _column_sums(X)
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    pi_d, mu_d, var_d = _t(pi0), _t(mu0), _t(var0)
    ctx.gmm_em_step(X[:300_000], pi_d, mu_d, var_d)               # allocates the scratch
    torch.cuda.synchronize()
    free_small = torch.cuda.mem_get_info()[0]
    trace, done = ctx.gmm_fit(X, pi_d, mu_d, var_d, spec.iters, spec.var_floor)
    assert done == spec.iters == 20 and ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
    assert torch.cuda.mem_get_info()[0] == free_small, "device memory in use changed with N"
    assert np.all(np.isfinite(trace))
    # (variances pinned at the floor and frozen empty components may break the monotone growth by a hair)
    assert (np.diff(trace) >= -1e-7 * np.abs(trace[1:])).all(), trace
    Nk, S1, S2, L = _gpu_step(ctx, X, pi_d.cpu().numpy(), mu_d.cpu().numpy(), var_d.cpu().numpy())
    assert abs(Nk.sum() - N) <= 1e-5 * N
    np.testing.assert_allclose(S2.sum(0), col2, rtol=1e-4)
    np.testing.assert_allclose(S1.sum(0), col1, rtol=1e-4, atol=1e-4 * N * 0.04)
    assert L >= trace[-1] - 1e-7 * abs(L)
    idx, resp = ctx.gmm_assign_topm(X, pi_d, mu_d, var_d, 4)
    torch.cuda.synchronize()
    assert int(idx.min()) >= 0 and int(idx.max()) < spec.K and ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
    # the hard assignment and the per-point log-densities over all N, by the same screening route: the arg-max is the
    # top-4's first entry wherever the two leading responsibilities are not within the tie width, and the densities add up
    # to the log-likelihood of the step above; both against the oracle on the subsample
    idx1, _ = ctx.gmm_assign_topm(X, pi_d, mu_d, var_d, 1, indices_only=True)
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
    clear = (resp[:, 0] - resp[:, 1]) > 1e-5
    assert bool((idx1[:, 0][clear] == idx[:, 0][clear]).all()) and float(clear.float().mean()) > 0.9
    logp, total = ctx.gmm_score_samples(X, pi_d, mu_d, var_d)
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR and abs(total - L) <= 1e-6 * abs(L)
    p1, m1, v1 = pi_d.cpu().numpy(), mu_d.cpu().numpy(), var_d.cpu().numpy()
    rows = synth.subsample_rows(spec.N, 20_000, spec.seed)
    rows_d = torch.as_tensor(rows, device=DEV)
    Xsub = X[rows_d].contiguous().cpu().numpy()
    lz = orc.responsibilities(Xsub, p1, m1, v1)[1]
    got = logp[rows_d].cpu().numpy().astype(np.float64)
    assert (np.abs(got - lz) <= 1e-5 * np.abs(lz) + 1e-4).all()
    _check_topm(Xsub, p1, m1, v1, 1, idx1[rows_d].cpu().numpy(), None, "config 5 hard assignment subsample")
    _config5_subsample_check(fg, ctx, X, spec, pi0, mu0, var0, idx, resp, p1, m1, v1)


def test_isotropic_update_and_fit_match_the_papers_model(fg, ctx):
    """gmm_finalize_isotropic and gmm_fit with GMM_COV_ISOTROPIC against the isotropic oracle (the paper's Eq. 3)."""
    spec = synth.CONFIGS[2].with_n(6000)
    X = synth.sample_host(spec)
    s = data_scale(X)
    pi0, mu0, var0 = synth.init_params(X, spec)
    var0 = np.full_like(var0, var0.mean())                       # isotropic start: sigma^2 = mean global variance
    pr, mr, vr, L_r = orc.em_iteration_isotropic(X, pi0, mu0, var0, spec.var_floor)
    Nk_r = orc.em_step(X, pi0, mu0, var0)[0]
    for path in _paths(fg, spec.D, spec.K):
        ctx.gmm_set_path(path)
        Nk, S1, S2, L = ctx.gmm_em_step(_t(X), _t(pi0), _t(mu0), _t(var0))
        assert abs(L - L_r) <= 1e-5 * abs(L_r)
        pi_d, mu_d, var_d = _t(pi0), _t(mu0), _t(var0)
        ctx.gmm_finalize_isotropic(len(X), Nk, S1, S2, spec.var_floor, pi_d, mu_d, var_d)
        v = var_d.cpu().numpy()
        assert (v == v[:, :1]).all()
        assert_params_close(len(X), s, (pi_d.cpu().numpy(), mu_d.cpu().numpy(), v), (pr, mr, vr), Nk_r, f"path {path}")
    # gmm_fit with the isotropic update, teacher-forced: one iteration at a time from the oracle's parameters
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    ctx.gmm_set_covariance(fg.GMM_COV_ISOTROPIC)
    p, m, v = pi0.astype(np.float64), mu0.astype(np.float64), var0.astype(np.float64)
    for it in range(3):
        p32, m32, v32 = p.astype(np.float32), m.astype(np.float32), v.astype(np.float32)
        Nk_it = orc.em_step(X, p32, m32, v32)[0]
        p, m, v, L = orc.em_iteration_isotropic(X, p32, m32, v32, spec.var_floor)
        pi_d, mu_d, var_d = _t(p32), _t(m32), _t(v32)
        trace, done = ctx.gmm_fit(_t(X), pi_d, mu_d, var_d, 1, spec.var_floor)
        assert done == 1 and abs(trace[0] - L) <= 1e-5 * abs(L)
        assert_params_close(len(X), s, (pi_d.cpu().numpy(), mu_d.cpu().numpy(), var_d.cpu().numpy()), (p, m, v), Nk_it,
                            f"isotropic fit iteration {it}")
    ctx.gmm_set_covariance(fg.GMM_COV_DIAG)
