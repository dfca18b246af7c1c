"""GPU parity of the tensor-core path for wide data (128 < D <= 1024: the two sweeps of Algorithm 1 on tcgen05) against
the float64 CPU oracle, through the C ABI.  Tolerances: tests/parity_util.py (the same as for every other path).

What the path does with the components it cannot treat through the expanded quadratic form (collapsed ones, and ones
that hold few points) is part of what is tested: they are evaluated exactly by the FP32 kernels as a packed
sub-mixture, and gmm_last_exact_count reports how many there were.
"""
import numpy as np
import pytest
import torch

from oracle import gmm_oracle as orc
from paper_2606_10896_b200 import synth
from tests.parity_util import assert_params_close, assert_stats_close, data_scale

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


def _clustered(rng, N, D, K, sep=0.3, spread=0.3):
    """K clusters of about N / K points each (weights between 0.5 and 1.5 of the mean), parameters near the truth.  Centres
    and noise are of the same size per dimension (sum_d mu^2 / var about D, as for unit-norm embeddings); in hundreds of
    dimensions the clusters are still tens of standard deviations apart."""
    centres = (rng.normal(size=(K, D)) * sep).astype(np.float32)
    w = rng.uniform(0.5, 1.5, K)
    w /= w.sum()
    z = rng.choice(K, size=N, p=w)
    sig = rng.uniform(0.7, 1.3, size=(K, D)) * spread
    X = (centres[z] + rng.normal(size=(N, D)) * sig[z]).astype(np.float32)
    mu = (centres + 0.05 * spread * rng.normal(size=(K, D))).astype(np.float32)
    var = (sig ** 2 * rng.uniform(0.8, 1.25, size=(K, D))).astype(np.float32)
    pi = w.astype(np.float32)
    return X, pi, mu, var


def _step_and_check(fg, ctx, X, pi, mu, var, what, var_floor=1e-6):
    N = len(X)
    s = data_scale(X)
    ref = orc.em_step(X, pi, mu, var)
    pr, mr, vr, _, _, _ = orc.em_iteration(X, pi, mu, var, var_floor=var_floor)
    Nk, S1, S2, L = ctx.gmm_em_step(_t(X), _t(pi), _t(mu), _t(var))
    got = (Nk.cpu().numpy(), S1.cpu().numpy(), S2.cpu().numpy())
    assert abs(L - ref[3]) <= 1e-5 * abs(ref[3]), f"{what}: loglik {L} vs {ref[3]}"
    assert abs(got[0].sum() - N) <= 1e-5 * N, f"{what}: sum N_k = {got[0].sum()}"
    assert_stats_close(N, s, got, ref[:3], what)
    pi_d, mu_d, var_d = _t(pi), _t(mu), _t(var)
    ctx.gmm_finalize(N, Nk, S1, S2, var_floor, pi_d, mu_d, var_d)
    assert_params_close(N, s, (pi_d.cpu().numpy(), mu_d.cpu().numpy(), var_d.cpu().numpy()), (pr, mr, vr), ref[0], what)
    return got


@pytest.mark.parametrize("N,D,K", [(20_000, 200, 130), (16_384 + 77, 768, 128), (30_000, 1024, 64), (25_000, 129, 70),
                                   (40_000, 768, 256), (300, 256, 1)])
def test_wide_tensor_path_one_step_against_oracle(fg, ctx, N, D, K):
    """Ragged last slice of dimensions (200 = 128 + 72, 129), the largest D, a ragged last slice of components (130, 70),
    tiles and batches with a ragged tail, one component."""
    X, pi, mu, var = _clustered(np.random.default_rng(N + D + K), N, D, K)
    assert fg.tensor_path_supports(D, K)
    ctx.gmm_set_path(fg.GMM_PATH_TENSOR)
    _step_and_check(fg, ctx, X, pi, mu, var, f"wide tensor N={N} D={D} K={K}")
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR


def test_wide_path_over_several_pieces_and_bit_identical_runs(fg, monkeypatch):
    """Pieces of 1024 points (instead of 2^17): planes, log Z buffer and partial blocks are reused piece after piece; two
    calls give the same bits."""
    monkeypatch.setenv("GMM_WIDE_PIECE", "1024")
    X, pi, mu, var = _clustered(np.random.default_rng(3), 5000, 384, 40)
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        a = _step_and_check(fg, c, X, pi, mu, var, "five pieces")
        Nk, S1, S2, L = c.gmm_em_step(_t(X), _t(pi), _t(mu), _t(var))
        for u, v in zip(a, (Nk, S1, S2)):
            assert np.array_equal(u, v.cpu().numpy())


def test_wide_path_with_collapsed_and_low_weight_components(fg, ctx):
    """Components collapsed onto a data point at the variance floor (the expanded form cannot represent them), components
    narrow in a few dimensions only, and components of tiny weight: all are evaluated exactly, the rest on the tensor
    cores, and the two must agree on the normaliser."""
    rng = np.random.default_rng(17)
    N, D, K = 30_000, 320, 96
    X, pi, mu, var = _clustered(rng, N, D, K)
    for j in range(6):                       # collapsed onto a point
        mu[j] = X[100 + j]
        var[j] = 1e-6
    var[6:10, ::5] = 1e-5                    # narrow in every fifth dimension
    pi[10:14] = 3e-4                         # about nine points' worth of weight each
    pi = (pi / pi.sum()).astype(np.float32)
    ctx.gmm_set_path(fg.GMM_PATH_TENSOR)
    _step_and_check(fg, ctx, X, pi, mu, var, "collapsed / narrow / light components")
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
    assert 10 <= ctx.gmm_last_exact_count() <= 20
    # zero weights: no NaN, N_k = 0 there
    pi2 = pi.copy()
    pi2[20:30] = 0
    pi2 = (pi2 / pi2.sum()).astype(np.float32)
    got = _step_and_check(fg, ctx, X, pi2, mu, var, "zero weights")
    assert np.all(got[0][20:30] == 0)


def test_wide_auto_path_rule(fg, ctx):
    """AUTO on wide data with K >= 64.  From 128 points per component on: the two tensor sweeps, with a few components
    evaluated exactly (more than half of them: the FP32 kernels).  Below: one tensor sweep that only screens the pairs, every
    component evaluated exactly where it matters - unless a sample of the points marks too many pairs (clusters that
    overlap), in which case the FP32 kernels take the step."""
    rng = np.random.default_rng(5)
    D, K = 256, 64
    assert fg.gmm_auto_path(D, K) == fg.GMM_PATH_TENSOR and fg.gmm_auto_path(D, 32) == fg.GMM_PATH_FP32
    X, pi, mu, var = _clustered(rng, 200 * K, D, K)
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    ctx.gmm_em_step(_t(X), _t(pi), _t(mu), _t(var))
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR and ctx.gmm_last_exact_count() == 0
    _step_and_check(fg, ctx, X[:100 * K], pi, mu, var, "100 points per component, separate clusters")
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR and ctx.gmm_last_exact_count() == K      # (one marked pair per point)
    K2, D2 = 1024, 512
    X2, pi2, mu2, var2 = _clustered(np.random.default_rng(15), 40 * K2, D2, K2)
    with fg.Context(0) as c2:
        _step_and_check(fg, c2, X2, pi2, mu2, var2, "40 points per component: screening sweep + exact pairs")
        assert c2.gmm_last_path() == fg.GMM_PATH_TENSOR and c2.gmm_last_exact_count() == K2
        marked, kept, dense = c2.gmm_last_exact_pairs()
        assert dense == 0 and 40 * K2 <= kept <= marked <= 40 * K2 * 64
    v2 = var.copy()
    v2[:40] = 1e-6
    ctx.gmm_em_step(_t(X), _t(pi), _t(mu), _t(v2))
    assert ctx.gmm_last_path() == fg.GMM_PATH_FP32 and ctx.gmm_last_exact_count() == 0
    Xo, pio, muo, varo = _clustered(np.random.default_rng(6), 50 * K, D, K, sep=0.01)       # clusters on top of each other
    _step_and_check(fg, ctx, Xo, pio, muo, varo, "50 points per component, overlapping clusters")
    assert ctx.gmm_last_path() == fg.GMM_PATH_FP32


@pytest.mark.parametrize("N,D,K", [(9_000 + 13, 200, 130), (6_000, 768, 256), (40_000, 320, 96), (7_000 + 1, 131, 70)])
def test_wide_screen_mode_against_oracle(fg, monkeypatch, N, D, K):
    """GMM_WIDE_MODE=screen: one tensor sweep screens every (point, component) pair, all marked pairs are evaluated exactly
    (no component goes through the second tensor sweep).  With collapsed, narrow, light and zero-weight components; pieces
    of 4096 points; the same bits in a second run."""
    monkeypatch.setenv("GMM_WIDE_MODE", "screen")
    monkeypatch.setenv("GMM_WIDE_SPARSE", "2")           # (at these small K the dense kernels would be cheaper: keep to the pairs)
    monkeypatch.setenv("GMM_WIDE_PIECE", "4096")
    X, pi, mu, var = _clustered(np.random.default_rng(N + D), N, D, K)
    mu[0], var[0] = X[7], 1e-6
    var[1, ::7] = 1e-5
    pi[2] = 2e-4
    pi[3] = 0.0
    pi = (pi / pi.sum()).astype(np.float32)
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        a = _step_and_check(fg, c, X, pi, mu, var, f"screen mode N={N} D={D} K={K}")
        assert c.gmm_last_path() == fg.GMM_PATH_TENSOR and c.gmm_last_exact_count() == K - 1       # (all with a weight)
        marked, kept, dense = c.gmm_last_exact_pairs()
        assert dense == 0 and N <= kept <= marked
        assert a[0][3] == 0.0
        Nk, S1, S2, _ = c.gmm_em_step(_t(X), _t(pi), _t(mu), _t(var))
        for u, v in zip(a, (Nk, S1, S2)):
            assert np.array_equal(u, v.cpu().numpy())
        if D == 131:       # (rows that are not whole 16-byte groups: the pair kernels' scalar loads; also the assignment's)
            _assign_and_check(fg, c, X, pi, mu, var, 3, "assignment by screening, D = 131")
            _assign_and_check(fg, c, X, pi, mu, var, 1, "hard assignment by screening, D = 131", indices_only=True)


@pytest.mark.parametrize("N,D,K", [(3, 129, 64), (31, 136, 65), (129, 1024, 64), (4097, 200, 257), (257, 1020, 129)])
def test_wide_screening_routes_at_odd_sizes(fg, monkeypatch, N, D, K):
    """The screening routes (EM step, top-4 and hard assignment, per-point log-densities) forced at sizes that leave tiles,
    pieces, slices of dimensions and groups of components ragged - three points; fewer points than a tile; the widest rows;
    an odd number of component chunks - with zero-weight components and one collapsed onto a point; all against the
    oracle."""
    from oracle import gmm_oracle
    monkeypatch.setenv("GMM_WIDE_MODE", "screen")
    monkeypatch.setenv("GMM_WIDE_SPARSE", "2")
    monkeypatch.setenv("GMM_WIDE_PIECE", "4096")
    rng = np.random.default_rng(N + D + K)
    X, pi, mu, var = _clustered(rng, max(N, 2 * K), D, K)
    X = X[:N].copy()
    pi[rng.integers(0, K, 3)] = 0.0
    mu[1], var[1] = X[0], 1e-6
    pi = (pi / pi.sum()).astype(np.float32)
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        _step_and_check(fg, c, X, pi, mu, var, f"screening at N={N} D={D} K={K}")
        assert c.gmm_last_path() == fg.GMM_PATH_TENSOR
        _assign_and_check(fg, c, X, pi, mu, var, 4, "top-4 by screening")
        assert c.gmm_last_path() == fg.GMM_PATH_TENSOR
        _assign_and_check(fg, c, X, pi, mu, var, 1, "hard assignment by screening", indices_only=True)
        logp, total = c.gmm_score_samples(_t(X), _t(pi), _t(mu), _t(var))
        assert c.gmm_last_path() == fg.GMM_PATH_TENSOR
        lz = gmm_oracle.responsibilities(X, pi, mu, var)[1]
        got = logp.cpu().numpy().astype(np.float64)
        assert (np.abs(got - lz) <= 1e-5 * np.abs(lz) + 1e-4).all() and abs(total - lz.sum()) <= 1e-5 * abs(lz.sum()) + 1e-6


def test_wide_host_streaming_matches_device_call(fg, monkeypatch):
    """gmm_em_step_host on wide data: the rows arrive in staging buffers of one piece each (here 4096 rows: three chunks), the
    automatic choice of the mode looks at the first chunk's rows, and the step gives the bits of the device call."""
    monkeypatch.setenv("GMM_WIDE_PIECE", "4096")
    monkeypatch.setenv("GMM_WIDE_PROBE_LIMIT", "8")      # (so that the probe's verdict, not the size of K D, decides)
    X, pi, mu, var = _clustered(np.random.default_rng(31), 10_000, 200, 130)
    mu[0], var[0] = X[7], 1e-6
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        a = c.gmm_em_step(_t(X), _t(pi), _t(mu), _t(var))
        assert c.gmm_last_path() == fg.GMM_PATH_TENSOR and c.gmm_last_exact_count() == 130       # "screen"
        b = c.gmm_em_step_host(X, pi, mu, var)
        assert c.gmm_last_path() == fg.GMM_PATH_TENSOR and c.gmm_last_exact_count() == 130
        for u, v in zip(a[:3], b[:3]):
            assert np.array_equal(u.cpu().numpy(), v)
        assert a[3] == b[3]


def test_wide_screen_mode_with_a_first_pass_for_the_threshold(fg, monkeypatch):
    """GMM_WIDE_PRE=1: every tile first sweeps the leading product once for the largest lower bound alone, so that the sweep
    proper marks against a final threshold (the filter then finds little to drop); GMM_WIDE_HI=1 and 0: all three products
    for the components flagged by the rounding estimate, or for every component.  Same results at the ordinary tolerances."""
    monkeypatch.setenv("GMM_WIDE_MODE", "screen")
    monkeypatch.setenv("GMM_WIDE_SPARSE", "2")
    monkeypatch.setenv("GMM_WIDE_PIECE", "4096")
    N, D, K = 9_000 + 13, 200, 130
    X, pi, mu, var = _clustered(np.random.default_rng(N + D), N, D, K)
    mu[0], var[0] = X[7], 1e-6
    var[1, ::7] = 1e-5
    pi[2] = 2e-4
    pi = (pi / pi.sum()).astype(np.float32)
    for pre, hi in (("1", "2"), ("0", "1"), ("1", "1"), ("0", "0")):
        monkeypatch.setenv("GMM_WIDE_PRE", pre)
        monkeypatch.setenv("GMM_WIDE_HI", hi)
        with fg.Context(0) as c:
            c.gmm_set_path(fg.GMM_PATH_TENSOR)
            _step_and_check(fg, c, X, pi, mu, var, f"screen mode, first pass {pre}, leading product {hi}")
            assert c.gmm_last_path() == fg.GMM_PATH_TENSOR and c.gmm_last_exact_count() == K
            marked, kept, dense = c.gmm_last_exact_pairs()
            assert dense == 0 and N <= kept <= marked


def test_wide_screen_mode_more_pairs_than_stored_values(fg, monkeypatch):
    """Clusters on top of each other, every pair marked: more marked pairs in a piece (40,000 x 130) than the buffer of exact
    pair values holds (32 x 2^17), so the statistics kernel evaluates its pairs itself."""
    monkeypatch.setenv("GMM_WIDE_MODE", "screen")
    monkeypatch.setenv("GMM_WIDE_SPARSE", "2")
    N, D, K = 40_000, 200, 130
    X, pi, mu, var = _clustered(np.random.default_rng(77), N, D, K, sep=0.01)
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        _step_and_check(fg, c, X, pi, mu, var, "every pair marked")
        marked, kept, dense = c.gmm_last_exact_pairs()
        assert dense == 0 and marked > 32 * 2 ** 17 and kept > N


def test_wide_screen_mode_free_running_fit(fg, monkeypatch):
    monkeypatch.setenv("GMM_WIDE_MODE", "screen")
    rng = np.random.default_rng(19)
    N, D, K = 12_000, 256, 64
    X, pi, mu, var = _clustered(rng, N, D, K)
    mu0 = X[rng.choice(N, K, replace=False)].copy()
    var0 = np.tile(X.astype(np.float64).var(0).astype(np.float32), (K, 1))
    pi0 = np.full(K, 1 / K, np.float32)
    ref = orc.fit(X, pi0, mu0, var0, 8, var_floor=1e-6)
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        pi_d, mu_d, var_d = _t(pi0), _t(mu0), _t(var0)
        trace, done = c.gmm_fit(_t(X), pi_d, mu_d, var_d, 8, 1e-6)
        assert done == 8 and c.gmm_last_path() == fg.GMM_PATH_TENSOR and c.gmm_last_exact_count() > 0
        np.testing.assert_allclose(trace, ref["trace"], rtol=1e-5)
        Nk = orc.em_step(X, ref["pi"], ref["mu"], ref["var"])[0]
        assert np.abs(mu_d.cpu().numpy() - ref["mu"])[Nk >= 1].max() <= 1e-3 * data_scale(X)


def test_wide_free_running_fit_matches_the_oracle_trace(fg, ctx):
    rng = np.random.default_rng(9)
    N, D, K = 20_000, 256, 64
    X, pi, mu, var = _clustered(rng, N, D, K)
    mu0 = X[rng.choice(N, K, replace=False)].copy()
    var0 = np.tile(X.astype(np.float64).var(0).astype(np.float32), (K, 1))
    pi0 = np.full(K, 1 / K, np.float32)
    ref = orc.fit(X, pi0, mu0, var0, 10, var_floor=1e-6)
    ctx.gmm_set_path(fg.GMM_PATH_TENSOR)
    pi_d, mu_d, var_d = _t(pi0), _t(mu0), _t(var0)
    trace, done = ctx.gmm_fit(_t(X), pi_d, mu_d, var_d, 10, 1e-6)
    assert done == 10 and ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
    np.testing.assert_allclose(trace, ref["trace"], rtol=1e-4)
    s = data_scale(X)
    Nk = orc.em_step(X, ref["pi"], ref["mu"], ref["var"])[0]
    assert np.abs(mu_d.cpu().numpy() - ref["mu"])[Nk >= 1].max() <= 1e-3 * s


def test_wide_path_reports_non_finite_data(fg, ctx):
    X, pi, mu, var = _clustered(np.random.default_rng(2), 3000, 200, 16)
    X[77, 150] = np.nan
    ctx.gmm_set_path(fg.GMM_PATH_TENSOR)
    with pytest.raises(fg.GmmError) as e:
        ctx.gmm_em_step(_t(X), _t(pi), _t(mu), _t(var))
    assert e.value.code == fg.GMM_ENUMERIC
    X[77, 150] = 0.0
    ctx.gmm_em_step(_t(X), _t(pi), _t(mu), _t(var))


def test_wide_data_far_from_the_origin(fg, ctx):
    X, pi, mu, var = _clustered(np.random.default_rng(4), 12_000, 256, 48)
    X = (X + 200.0).astype(np.float32)
    mu = (mu + 200.0).astype(np.float32)
    ctx.gmm_set_path(fg.GMM_PATH_TENSOR)
    _step_and_check(fg, ctx, X, pi, mu, var, "wide, 200 units from the origin")


def _with_listed_components(rng, N, D, K, sep=0.3):
    X, pi, mu, var = _clustered(rng, N, D, K, sep=sep)
    for j in range(5):                       # collapsed onto a point
        mu[j] = X[50 + j]
        var[j] = 1e-6
    pi[8:14] = 2e-4                          # light, broad
    pi = (pi / pi.sum()).astype(np.float32)
    return X, pi, mu, var


@pytest.mark.parametrize("mode", ["0", "1", "2"])
def test_listed_components_pair_by_pair_or_densely(fg, monkeypatch, mode):
    """The components the tensor passes leave out are evaluated exactly either pair by pair (the pairs the first sweep
    could not rule out: GMM_WIDE_SPARSE=2 always, 1 = the default when they are few) or by the FP32 kernels over the whole
    sub-mixture (0); all three match the oracle, and the counters say which route ran."""
    monkeypatch.setenv("GMM_WIDE_SPARSE", mode)
    monkeypatch.setenv("GMM_WIDE_PIECE", "8192")
    X, pi, mu, var = _with_listed_components(np.random.default_rng(31), 20_000, 288, 80)
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        a = _step_and_check(fg, c, X, pi, mu, var, f"listed components, GMM_WIDE_SPARSE={mode}")
        assert c.gmm_last_path() == fg.GMM_PATH_TENSOR and c.gmm_last_exact_count() >= 11
        marked, kept, dense = c.gmm_last_exact_pairs()
        if mode == "0":
            assert (marked, kept, dense) == (0, 0, 0)
        else:
            # every collapsed component keeps its own point, a light one its cluster (about 250 points)
            assert dense == 0 and kept >= 5 + 6 * 100 and marked >= kept and marked < 20 * kept
        Nk, S1, S2, _ = c.gmm_em_step(_t(X), _t(pi), _t(mu), _t(var))
        for u, v in zip(a, (Nk, S1, S2)):
            assert np.array_equal(u, v.cpu().numpy())            # same bits in a second run


def test_many_marked_pairs_go_to_the_dense_kernels(fg, ctx):
    """Clusters that overlap almost completely: every point is a candidate for every light component, more than one pair
    in 64 is marked, and the step hands the sub-mixture of those pieces to the FP32 kernels."""
    X, pi, mu, var = _clustered(np.random.default_rng(37), 24_000, 256, 64, sep=0.01)
    pi[3:9] = 5e-4
    pi = (pi / pi.sum()).astype(np.float32)
    ctx.gmm_set_path(fg.GMM_PATH_TENSOR)
    _step_and_check(fg, ctx, X, pi, mu, var, "overlapping clusters, light components")
    marked, kept, dense = ctx.gmm_last_exact_pairs()
    assert ctx.gmm_last_exact_count() >= 6 and dense == 1 and marked > 24_000 * 6 // 64


# ---- top-m assignment on wide data (paper Sections 4.2-4.3) ---------------------------------------------------------

def _assign_and_check(fg, ctx, X, pi, mu, var, m, what, indices_only=False):
    from tests.parity_util import assert_topm_matches, oracle_resp_at

    idx, resp = ctx.gmm_assign_topm(_t(X), _t(pi), _t(mu), _t(var), m, indices_only=indices_only)
    ctx.gmm_sync_status()
    idx_g = idx.cpu().numpy()
    resp_g = None if resp is None else resp.cpu().numpy()
    idx_r, resp_r, next_r = orc.topm(X, pi, mu, var, m)
    assert idx_g.min() >= 0 and idx_g.max() < len(pi), f"{what}: index out of range"
    for row in idx_g[:: max(1, len(idx_g) // 500)]:
        assert len(set(row.tolist())) == m, f"{what}: repeated component in a row"
    r_at_g = oracle_resp_at(orc, X, pi, mu, var, idx_g)
    assert_topm_matches(idx_g, resp_g, idx_r, resp_r, next_r, r_at_g, what=what, check_values=resp_g is not None)
    return idx_g, resp_g


@pytest.mark.parametrize("m", [1, 2, 4, 8])
def test_wide_assignment_against_oracle(fg, ctx, m):
    """Tiles with a ragged tail, a ragged last slice of dimensions and of components; m + 2 <= 6 and m + 2 = 10 reported
    candidates."""
    X, pi, mu, var = _clustered(np.random.default_rng(100 + m), 9_000 + 77, 200, 130)
    ctx.gmm_set_path(fg.GMM_PATH_TENSOR)
    _assign_and_check(fg, ctx, X, pi, mu, var, m, f"wide assignment m={m}")
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
    if m == 4:
        _assign_and_check(fg, ctx, X, pi, mu, var, m, "wide assignment, indices only", indices_only=True)


def test_wide_assignment_with_listed_components_ties_and_overlap(fg, monkeypatch):
    """(a) Collapsed components own their point; (b) two identical components tie exactly on every point of their cluster
    (the smaller index first); (c) clusters that overlap: many components matter for a point, the rows go to the FP32
    kernels; (d) pieces of 4096 points."""
    monkeypatch.setenv("GMM_WIDE_PIECE", "4096")
    rng = np.random.default_rng(55)
    X, pi, mu, var = _with_listed_components(rng, 12_000, 288, 80)
    mu[40], var[40], pi[40] = mu[41], var[41], pi[41]          # an exact copy: ties
    pi = (pi / pi.sum()).astype(np.float32)
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        idx, resp = _assign_and_check(fg, c, X, pi, mu, var, 4, "wide assignment with listed components")
        assert c.gmm_last_path() == fg.GMM_PATH_TENSOR
        for j in range(5):                                      # the point a collapsed component sits on
            assert idx[50 + j, 0] == j and resp[50 + j, 0] > 0.999
        tied = np.flatnonzero((idx[:, 0] == 40) | (idx[:, 0] == 41))
        assert len(tied) > 50 and np.all(idx[tied, 0] == 40) and np.all(idx[tied, 1] == 41)
        Xo, pio, muo, varo = _clustered(np.random.default_rng(56), 6_000, 256, 64, sep=0.02)
        _assign_and_check(fg, c, Xo, pio, muo, varo, 4, "wide assignment, overlapping clusters")


def test_wide_hard_assignment_by_screening(fg, monkeypatch):
    """m = 1, indices only: every component screened by the leading product, the marked pairs evaluated exactly, the
    largest taken.  (a) separate clusters with collapsed, light and zero-weight components and an exact copy of a component
    (the smaller index wins), pieces of 4096 points; (b) clusters on top of each other: the sample marks too many pairs and
    the call takes the route with six candidates per point (and the FP32 kernels for its uncertain rows); (c) the same
    forced through the screening route, whose pieces then go to the FP32 kernels."""
    monkeypatch.setenv("GMM_WIDE_PIECE", "4096")
    monkeypatch.setenv("GMM_WIDE_PROBE_LIMIT", "8")      # (at this small K D the automatic limit is zero: the other route is cheaper)
    rng = np.random.default_rng(91)
    X, pi, mu, var = _with_listed_components(rng, 12_000 + 5, 288, 80)
    mu[40], var[40], pi[40] = mu[41], var[41], pi[41]          # an exact copy: ties
    pi[20] = 0.0
    pi = (pi / pi.sum()).astype(np.float32)
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        idx, _ = _assign_and_check(fg, c, X, pi, mu, var, 1, "hard assignment by screening", indices_only=True)
        assert c.gmm_last_path() == fg.GMM_PATH_TENSOR
        for j in range(5):                                      # the point a collapsed component sits on
            assert idx[50 + j, 0] == j
        assert np.sum(idx[:, 0] == 40) > 50 and not np.any(idx[:, 0] == 41) and not np.any(idx[:, 0] == 20)
        idx2, _ = c.gmm_assign_topm(_t(X), _t(pi), _t(mu), _t(var), 1, indices_only=True)
        assert np.array_equal(idx, idx2.cpu().numpy())
        for m in (1, 4, 8):                                     # the general top-m by the same route, with responsibilities
            idx4, resp4 = _assign_and_check(fg, c, X, pi, mu, var, m, f"top-{m} by screening")
            assert np.array_equal(idx4[:, 0], idx[:, 0])
            if m > 1:
                tied = np.flatnonzero(idx4[:, 0] == 40)
                assert np.all(idx4[tied, 1] == 41) and np.allclose(resp4[tied, 0], resp4[tied, 1])
        Xo, pio, muo, varo = _clustered(np.random.default_rng(92), 6_000, 256, 64, sep=0.02)
        _assign_and_check(fg, c, Xo, pio, muo, varo, 1, "hard assignment, overlapping clusters", indices_only=True)
    monkeypatch.setenv("GMM_WIDE_MODE", "screen")
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        _assign_and_check(fg, c, Xo, pio, muo, varo, 1, "hard assignment, overlapping clusters, screening forced", indices_only=True)


def test_wide_assignment_path_choice(fg, ctx):
    """AUTO takes the tensor path for K >= 64 (by screening, which does not mind collapsed components; with GMM_WIDE_MODE=sweeps
    the route with six candidates per point, which leaves a mixture with more than half of its components ill-conditioned
    to the FP32 kernels); FP32 when forced."""
    X, pi, mu, var = _clustered(np.random.default_rng(8), 5_000, 256, 64)
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    _assign_and_check(fg, ctx, X, pi, mu, var, 2, "AUTO")
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
    ctx.gmm_set_path(fg.GMM_PATH_FP32)
    _assign_and_check(fg, ctx, X, pi, mu, var, 2, "FP32 forced")
    assert ctx.gmm_last_path() == fg.GMM_PATH_FP32
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    v2 = var.copy()
    v2[:40] = 1e-6
    _assign_and_check(fg, ctx, X, pi, mu, v2, 2, "40 of 64 collapsed")      # (either route, by what the sample of rows marks)


def test_wide_assignment_by_candidates(fg, monkeypatch):
    """GMM_WIDE_MODE=sweeps keeps the assignment on the route that reports six or ten candidates per point from a sweep over
    the evaluated components: the same cases as above, and the mixture that route leaves to the FP32 kernels."""
    monkeypatch.setenv("GMM_WIDE_MODE", "sweeps")
    monkeypatch.setenv("GMM_WIDE_PIECE", "4096")
    rng = np.random.default_rng(55)
    X, pi, mu, var = _with_listed_components(rng, 12_000, 288, 80)
    with fg.Context(0) as c:
        c.gmm_set_path(fg.GMM_PATH_TENSOR)
        for m in (1, 4, 8):
            _assign_and_check(fg, c, X, pi, mu, var, m, f"assignment by candidates m={m}")
            assert c.gmm_last_path() == fg.GMM_PATH_TENSOR
        _assign_and_check(fg, c, X, pi, mu, var, 4, "assignment by candidates, indices only", indices_only=True)
        Xo, pio, muo, varo = _clustered(np.random.default_rng(56), 6_000, 256, 64, sep=0.02)
        _assign_and_check(fg, c, Xo, pio, muo, varo, 4, "assignment by candidates, overlapping clusters")
        Xc, pic, muc, varc = _clustered(np.random.default_rng(8), 5_000, 256, 64)
        varc[:40] = 1e-6
        _assign_and_check(fg, c, Xc, pic, muc, varc, 2, "40 of 64 collapsed")
        assert c.gmm_last_path() == fg.GMM_PATH_FP32


def test_wide_path_at_its_largest_shape(fg, ctx):
    """D = 1024 and K = 4096, the limits of the path, on 560,000 device-generated points (just above the 128 points per
    component from which AUTO takes it).  No oracle step of this size is affordable: the tensor path against the FP32 kernels
    over the same rows at the ordinary tolerances (the FP32 kernels are checked against the oracle at this D in the cases
    above), conservation of the weights, and the top-4 assignment against the oracle on a subsample of 1,500 rows."""
    N, D, K = 560_000, 1024, 4096
    g = torch.Generator(device=DEV)
    g.manual_seed(20260611)
    centres = torch.randn(K, D, device=DEV, generator=g) * 0.3
    z = torch.randint(0, K, (N,), device=DEV, generator=g)
    X = centres[z]
    X += 0.3 * torch.randn(N, D, device=DEV, generator=g)
    X = X.contiguous()
    del z
    pi = np.full(K, 1.0 / K, np.float32)
    mu = (centres + 0.015 * torch.randn(K, D, device=DEV, generator=g)).cpu().numpy()
    var = (0.09 * (0.8 + 0.45 * torch.rand(K, D, device=DEV, generator=g))).cpu().numpy()
    s = float(np.sqrt(X[:50_000].double().var(0).mean().item()))
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    Nk, S1, S2, L = ctx.gmm_em_step(X, _t(pi), _t(mu), _t(var))
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
    t_ = (Nk.cpu().numpy(), S1.cpu().numpy(), S2.cpu().numpy(), L)
    assert abs(t_[0].sum() - N) <= 1e-5 * N
    ctx.gmm_set_path(fg.GMM_PATH_FP32)
    Nk, S1, S2, Lf = ctx.gmm_em_step(X, _t(pi), _t(mu), _t(var))
    f_ = (Nk.cpu().numpy(), S1.cpu().numpy(), S2.cpu().numpy(), Lf)
    what = "D = 1024, K = 4096: tensor vs FP32 path"
    assert abs(t_[3] - f_[3]) <= 1e-5 * abs(f_[3]), what
    assert_stats_close(N, s, t_[:3], f_[:3], what)

    def params(st):
        pi_d, mu_d, var_d = _t(pi), _t(mu), _t(var)
        ctx.gmm_finalize(N, _t(st[0], torch.float64), _t(st[1], torch.float64), _t(st[2], torch.float64), 1e-6, pi_d, mu_d, var_d)
        return pi_d.cpu().numpy(), mu_d.cpu().numpy(), var_d.cpu().numpy()

    assert_params_close(N, s, params(t_), params(f_), f_[0], what)
    ctx.gmm_set_path(fg.GMM_PATH_AUTO)
    idx, resp = ctx.gmm_assign_topm(X, _t(pi), _t(mu), _t(var), 4)
    ctx.gmm_sync_status()
    assert ctx.gmm_last_path() == fg.GMM_PATH_TENSOR
    rows = torch.as_tensor(synth.subsample_rows(N, 1500, 7), device=DEV)
    Xs = X[rows].cpu().numpy()
    from tests.parity_util import assert_topm_matches, oracle_resp_at
    idx_g, resp_g = idx[rows].cpu().numpy(), resp[rows].cpu().numpy()
    idx_r, resp_r, next_r = orc.topm(Xs, pi, mu, var, 4)
    assert_topm_matches(idx_g, resp_g, idx_r, resp_r, next_r, oracle_resp_at(orc, Xs, pi, mu, var, idx_g), what="largest shape, top-4")
