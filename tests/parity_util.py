"""Tolerances and comparison helpers shared by the GPU parity tests.

Tolerances (from the target statement of this build; "data scale" s = sqrt(mean over d of the global per-dimension
variance of X), float64):
  * mu:   |d mu_kd|  <= 1e-4 * s        for components with N_k >= 1
  * var:  |d var_kd| <= 1e-4 * s^2      for components with N_k >= 1
  * pi:   |d pi_k|   <= 1e-5            for every component
  * log-likelihood: relative 1e-5 after one step, 1e-4 along a free-running 30-iteration trace
  * top-m: identical index sets except where the responsibilities involved tie within 1e-6
Two modes: teacher-forced (every GPU step starts from the oracle's parameters of that iteration) and free-running
(both sides iterate from the same initial parameters).
"""
import numpy as np


def data_scale(X: np.ndarray) -> float:
    return float(np.sqrt(X.astype(np.float64).var(axis=0).mean()))


def assert_params_close(N, s, got, ref, Nk_ref, what=""):
    pi_g, mu_g, var_g = (np.asarray(a, np.float64) for a in got)
    pi_r, mu_r, var_r = (np.asarray(a, np.float64) for a in ref)
    dpi = np.abs(pi_g - pi_r).max()
    assert dpi <= 1e-5, f"{what}: max |d pi| = {dpi:.3e} > 1e-5"
    live = Nk_ref >= 1.0
    if live.any():
        dmu = np.abs(mu_g[live] - mu_r[live]).max()
        dvar = np.abs(var_g[live] - var_r[live]).max()
        assert dmu <= 1e-4 * s, f"{what}: max |d mu| = {dmu:.3e} > {1e-4 * s:.3e}"
        assert dvar <= 1e-4 * s * s, f"{what}: max |d var| = {dvar:.3e} > {1e-4 * s * s:.3e}"


def assert_stats_close(N, s, got, ref, what=""):
    """Statistics compared on the scale the parameter tolerances imply: N_k to 1e-5 N; S1 to 1e-4 s max(N_k, 1);
    S2 to 1e-4 s^2 max(N_k, 1) plus the matching share of the mean term."""
    Nk_g, S1_g, S2_g = (np.asarray(a, np.float64) for a in got)
    Nk_r, S1_r, S2_r = ref
    assert np.abs(Nk_g - Nk_r).max() <= 1e-5 * N, f"{what}: N_k off by {np.abs(Nk_g - Nk_r).max():.3e}"
    w = np.maximum(Nk_r, 1.0)[:, None]
    mean_abs = np.abs(S1_r) / w
    e1 = (np.abs(S1_g - S1_r) / w - 1e-5 * mean_abs).max()
    assert e1 <= 1e-4 * s, f"{what}: S1/N_k off by {e1:.3e} > {1e-4 * s:.3e}"
    e2 = (np.abs(S2_g - S2_r) / w - 3e-5 * (S2_r / w)).max()
    assert e2 <= 1e-4 * s * s, f"{what}: S2/N_k off by {e2:.3e} > {1e-4 * s * s:.3e}"


def assert_topm_matches(idx_g, resp_g, idx_r, resp_r, next_r, tie=1e-6, what=""):
    """Index sets equal except for ties within `tie` in responsibility; values within 1e-5 absolute + 1e-4 relative."""
    idx_g = np.asarray(idx_g)
    resp_g = np.asarray(resp_g, np.float64)
    N, m = idx_r.shape
    bad = 0
    for i in range(N):
        sg, sr = set(idx_g[i].tolist()), set(idx_r[i].tolist())
        if len(sg) != m:
            raise AssertionError(f"{what}: point {i} has repeated indices {idx_g[i]}")
        if sg != sr:
            # every oracle choice that the GPU dropped must tie with the oracle's (m+1)-th value or the m-th value
            thresh = resp_r[i, m - 1]
            for k in sr - sg:
                j = int(np.where(idx_r[i] == k)[0][0])
                if resp_r[i, j] - next_r[i] > tie and resp_r[i, j] - thresh > tie:
                    bad += 1
            for k in sg - sr:
                j = int(np.where(idx_g[i] == k)[0][0])
                if abs(resp_g[i, j] - thresh) > tie + 1e-4 * thresh and thresh - resp_g[i, j] > tie:
                    bad += 1
        else:
            ref_map = dict(zip(idx_r[i].tolist(), resp_r[i].tolist()))
            for j in range(m):
                r = ref_map[int(idx_g[i, j])]
                if abs(resp_g[i, j] - r) > 1e-5 + 1e-4 * r:
                    bad += 1
        # descending order up to the tie width
        if (np.diff(resp_g[i]) > tie + 1e-4 * resp_g[i, :-1]).any():
            bad += 1
    assert bad == 0, f"{what}: {bad} top-m disagreements beyond the tie rule"
