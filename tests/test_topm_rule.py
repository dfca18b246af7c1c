"""The top-m comparison rule itself (tests/parity_util.py), on hand-made cases: a checker that accepts a wrong answer
would make every GPU top-m test meaningless.  Rule (Sections 4.2-4.3 return the clusters of largest responsibility;
results that differ only where responsibilities tie within 1e-6 are both right): everything is judged by the
oracle's responsibilities at the indices involved, never by the values the implementation under test reports."""
import numpy as np

from oracle import gmm_oracle as orc
from tests.parity_util import oracle_resp_at, topm_disagreements


def _case():
    # one point, K = 4: oracle r = [0.5, 0.3, 0.2 - 5e-7, 5e-7] (descending), m = 2 -> top-2 = {0, 1}, (m+1)-th = 0.2
    R = np.array([[0.5, 0.3, 0.2 - 5e-7, 5e-7]])
    idx_r = np.array([[0, 1]], np.int32)
    resp_r = np.array([[0.5, 0.3]])
    next_r = np.array([0.2 - 5e-7])
    return R, idx_r, resp_r, next_r


def _bad(idx_g, resp_g, R, idx_r, resp_r, next_r, **kw):
    r_at = np.take_along_axis(R, np.asarray(idx_g, np.int64), axis=1)
    return topm_disagreements(np.asarray(idx_g), None if resp_g is None else np.asarray(resp_g), idx_r, resp_r, next_r,
                              r_at, **kw)[0]


def test_identical_answer_passes_and_wrong_values_fail():
    R, idx_r, resp_r, next_r = _case()
    assert _bad([[0, 1]], [[0.5, 0.3]], R, idx_r, resp_r, next_r) == 0
    assert _bad([[0, 1]], [[0.5, 0.31]], R, idx_r, resp_r, next_r) == 1
    assert _bad([[1, 0]], [[0.3, 0.5]], R, idx_r, resp_r, next_r) == 1           # not descending


def test_wrong_index_with_the_right_value_fails_also_for_the_mth_choice():
    R, idx_r, resp_r, next_r = _case()
    # the m-th oracle choice (index 1, r = 0.3) replaced by index 2 (oracle r = 0.2) while REPORTING 0.3: a checker that
    # trusts the reported value, or that never looks at a dropped m-th choice, lets this through
    assert _bad([[0, 2]], [[0.5, 0.3]], R, idx_r, resp_r, next_r) == 1
    assert _bad([[0, 2]], None, R, idx_r, resp_r, next_r, check_values=False) == 1
    # m = 1: wrong arg-max reported with the arg-max's value
    assert _bad([[1]], [[0.5]], R, idx_r[:, :1], resp_r[:, :1], np.array([0.3])) == 1


def test_ties_within_1e_6_may_resolve_either_way():
    R = np.array([[0.5, 0.25 + 4e-7, 0.25, 0.25 - 4e-7 - 0.0]])
    R = R / 1.0
    idx_r = np.array([[0, 1]], np.int32)
    resp_r = np.array([[0.5, R[0, 1]]])
    next_r = np.array([0.25])
    assert _bad([[0, 2]], [[0.5, 0.25]], R, idx_r, resp_r, next_r) == 0          # tie with the m-th: accepted
    assert _bad([[0, 3]], [[0.5, R[0, 3]]], R, idx_r, resp_r, next_r) == 0       # still within 1e-6 of the m-th
    R2 = R.copy()
    R2[0, 3] = 0.25 - 2e-6
    assert _bad([[0, 3]], [[0.5, R2[0, 3]]], R2, idx_r, resp_r, next_r) == 1     # beyond the tie width


def test_repeated_indices_fail():
    R, idx_r, resp_r, next_r = _case()
    assert _bad([[0, 0]], [[0.5, 0.5]], R, idx_r, resp_r, next_r) >= 1


def test_oracle_resp_at_picks_the_oracles_own_rows():
    rng = np.random.default_rng(3)
    N, D, K = 50, 3, 7
    X = rng.normal(size=(N, D)).astype(np.float32)
    mu = rng.normal(size=(K, D)).astype(np.float32)
    var = rng.uniform(0.5, 2.0, size=(K, D)).astype(np.float32)
    pi = rng.dirichlet(np.ones(K)).astype(np.float32)
    idx = rng.integers(0, K, size=(N, 3))
    R = orc.responsibilities(X, pi, mu, var)[0]
    got = oracle_resp_at(orc, X, pi, mu, var, idx, chunk=16)
    assert np.array_equal(got, np.take_along_axis(R, idx, axis=1))
