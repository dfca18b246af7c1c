"""gmm_em_step_static -- the entry point for callers that cannot allocate device memory (hosts whose device heap
belongs to another allocator, or that may not block on the driver's allocator) -- checked through the C ABI against
the float64 oracle and against gmm_em_step on the same inputs, twice in a row so that stale contents of the shared
static scratch would show.

Collected last on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import gmm_oracle as orc
from paper_2606_10896_b200 import synth
from tests.parity_util import assert_stats_close, data_scale

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _t(a, dtype=torch.float32):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=dtype, device=DEV).contiguous()


def test_static_scratch_entry_point_matches_em_step_twice_in_a_row():
    from paper_2606_10896_b200 import flashgmm as fg

    # K * D = 16384 with a ragged last tile; the second problem is smaller so it reuses scratch the first one
    # wrote with different contents and a different layout.
    problems = [(70_003, 128, 128, 11), (9_001, 16, 200, 12)]
    with fg.Context(0) as ctx:
        ctx.gmm_set_path(fg.GMM_PATH_FP32)
        for N, D, K, seed in problems:
            rng = np.random.Generator(np.random.PCG64(seed))
            mu = rng.normal(0, 3, (K, D)).astype(np.float32)
            var = rng.uniform(0.3, 2.0, (K, D)).astype(np.float32)
            pi = rng.dirichlet(np.ones(K)).astype(np.float32)
            X = (mu[rng.integers(0, K, N)] + rng.standard_normal((N, D))).astype(np.float32)
            s = data_scale(X)
            X_d, pi_d, mu_d, var_d = _t(X), _t(pi), _t(mu), _t(var)
            Nk_r, S1_r, S2_r, L_r = ctx.gmm_em_step(X_d, pi_d, mu_d, var_d)
            ref = (Nk_r.cpu().numpy(), S1_r.cpu().numpy(), S2_r.cpu().numpy())
            Nk_o, S1_o, S2_o, L_o = orc.em_step(X, pi, mu, var)          # the float64 definition, same fp32 inputs
            out = (torch.full((K,), 7.0, dtype=torch.float64, device=DEV),
                   torch.full((K, D), -3.0, dtype=torch.float64, device=DEV),
                   torch.full((K, D), 5.0, dtype=torch.float64, device=DEV))
            first = None
            for call in range(2):
                L = fg.gmm_em_step_static(X_d, pi_d, mu_d, var_d, out)
                got = tuple(o.cpu().numpy() for o in out)
                assert abs(L - L_r) <= 1e-5 * abs(L_r), (call, L, L_r)
                assert abs(got[0].sum() - N) <= 1e-5 * N
                assert_stats_close(N, s, got, ref, f"static call {call} shape {(N, D, K)}")
                assert abs(L - L_o) <= 1e-5 * abs(L_o), (call, L, L_o)
                assert_stats_close(N, s, got, (Nk_o, S1_o, S2_o), f"static call {call} vs oracle, shape {(N, D, K)}")
                if first is None:
                    first = (L, got)
                else:       # same inputs, same launch configuration: the same bits
                    assert L == first[0]
                    for u, v in zip(got, first[1]):
                        assert np.array_equal(u, v)


def test_static_scratch_entry_point_rejects_oversized_shapes():
    from paper_2606_10896_b200 import flashgmm as fg

    X = _t(np.zeros((10, 64), np.float32))
    K = 1024          # K * D = 65536 > 32768
    out = (torch.zeros(K, dtype=torch.float64, device=DEV), torch.zeros((K, 64), dtype=torch.float64, device=DEV),
           torch.zeros((K, 64), dtype=torch.float64, device=DEV))
    with pytest.raises(fg.GmmError) as e:
        fg.gmm_em_step_static(X, _t(np.full(K, 1 / K)), _t(np.zeros((K, 64))), _t(np.ones((K, 64))), out)
    assert e.value.code == fg.GMM_EUNSUPPORTED
