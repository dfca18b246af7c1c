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
    """Statistics compared on the scale the parameter tolerances imply: N_k to 1e-5 N; S1 / N_k to 1e-4 s; S2 / N_k to
    1e-4 s^2, each plus a small share (1e-5 / 3e-5) of its own size.

    Both sides are first moved to the data's centre c_d = sum_k S1_kd / sum_k N_k (S1' = S1 - c N_k,
    S2' = S2 - 2 c S1 + c^2 N_k, in float64): the parameters that follow from the statistics do not depend on where the
    origin is, and neither may the comparison -- about a far-away origin a difference of 1e-7 in N_k (harmless: it
    cancels in S1 / N_k and S2 / N_k) would show up multiplied by c^2, and the relative allowances would widen with c."""
    Nk_g, S1_g, S2_g = (np.asarray(a, np.float64) for a in got)
    Nk_r, S1_r, S2_r = (np.asarray(a, np.float64) for a in ref)
    assert np.abs(Nk_g - Nk_r).max() <= 1e-5 * N, f"{what}: N_k off by {np.abs(Nk_g - Nk_r).max():.3e}"
    c = S1_r.sum(0) / max(Nk_r.sum(), 1e-300)

    def centred(Nk, S1, S2):
        return S1 - c * Nk[:, None], S2 - 2.0 * c * S1 + c * c * Nk[:, None]

    S1_g, S2_g = centred(Nk_g, S1_g, S2_g)
    S1_r, S2_r = centred(Nk_r, S1_r, S2_r)
    # Each side's sums are divided by its OWN N_k (at least 1): what is compared is the weighted mean and the weighted
    # second moment a component implies.  A difference of 1e-6 in a component's total weight N_k scales all three of
    # its statistics alike, moves pi_k by 1e-6 pi_k and mu_k, var_k not at all; divided by the other side's N_k it would
    # show up multiplied by the component's distance from the centre squared.  (N_k itself is compared above.)
    wg, wr = np.maximum(Nk_g, 1.0)[:, None], np.maximum(Nk_r, 1.0)[:, None]
    e1 = (np.abs(S1_g / wg - S1_r / wr) - 1e-5 * np.abs(S1_r) / wr).max()
    assert e1 <= 1e-4 * s, f"{what}: S1/N_k off by {e1:.3e} > {1e-4 * s:.3e}"
    e2 = (np.abs(S2_g / wg - S2_r / wr) - 3e-5 * (S2_r / wr)).max()
    assert e2 <= 1e-4 * s * s, f"{what}: S2/N_k off by {e2:.3e} > {1e-4 * s * s:.3e}"


def oracle_resp_at(orc, X, pi, mu, var, idx, chunk=2048):
    """The oracle's responsibilities r_ik at the given indices idx [N, m] (float64 [N, m]), evaluated row block by
    row block so that the full N x K matrix of a large case is never held."""
    idx = np.asarray(idx).astype(np.int64)
    out = np.empty(idx.shape, np.float64)
    for lo in range(0, len(X), chunk):
        R = orc.responsibilities(X[lo:lo + chunk], pi, mu, var)[0]
        out[lo:lo + chunk] = np.take_along_axis(R, idx[lo:lo + chunk], axis=1)
    return out


def topm_disagreements(idx_g, resp_g, idx_r, resp_r, next_r, r_at_g, tie=1e-6, check_values=True):
    """Number of points whose top-m result breaks the rule below (a list of the reasons comes with it).

    The rule (ties within `tie` = 1e-6 in responsibility may resolve either way; everything is judged by the ORACLE's
    responsibilities, never by the values the GPU reports):
      * a GPU index outside the oracle's set is accepted iff the oracle's r at that index is within `tie` of the
        oracle's m-th largest r;
      * an oracle choice the GPU dropped (the m-th included) is accepted iff it is within `tie` of the oracle's
        (m+1)-th largest r;
      * every reported value agrees with the oracle's r at the same index to 1e-5 absolute + 1e-4 relative;
      * the reported values descend up to the tie width.
    r_at_g [N, m]: the oracle's r at the GPU's indices (oracle_resp_at)."""
    idx_g = np.asarray(idx_g)
    r_at_g = np.asarray(r_at_g, np.float64)
    N, m = idx_r.shape
    bad, why = 0, []
    for i in range(N):
        reasons = []
        sg, sr = set(idx_g[i].tolist()), set(idx_r[i].tolist())
        if len(sg) != m:
            reasons.append(f"repeated indices {idx_g[i].tolist()}")
        mth = resp_r[i, m - 1]
        for k in sr - sg:
            j = int(np.where(idx_r[i] == k)[0][0])
            if resp_r[i, j] - next_r[i] > tie:
                reasons.append(f"dropped oracle choice {k} (r={resp_r[i, j]:.3e}, (m+1)-th={next_r[i]:.3e})")
        for j in range(m):
            k = int(idx_g[i, j])
            if k not in sr and mth - r_at_g[i, j] > tie:
                reasons.append(f"extra index {k} (oracle r={r_at_g[i, j]:.3e}, m-th={mth:.3e})")
        if check_values:
            rg = np.asarray(resp_g[i], np.float64)
            if (np.abs(rg - r_at_g[i]) > 1e-5 + 1e-4 * r_at_g[i]).any():
                reasons.append(f"values {rg.tolist()} vs oracle {r_at_g[i].tolist()}")
            if (np.diff(rg) > tie + 1e-4 * rg[:-1]).any():
                reasons.append(f"values not descending {rg.tolist()}")
        else:           # indices only: the oracle's values at the GPU's indices must descend
            if (np.diff(r_at_g[i]) > tie).any():
                reasons.append(f"indices not in descending order of the oracle's r {r_at_g[i].tolist()}")
        if reasons:
            bad += 1
            if len(why) < 5:
                why.append(f"point {i}: " + "; ".join(reasons))
    return bad, why


def assert_topm_matches(idx_g, resp_g, idx_r, resp_r, next_r, r_at_g, tie=1e-6, what="", check_values=True):
    """See topm_disagreements."""
    bad, why = topm_disagreements(idx_g, resp_g, idx_r, resp_r, next_r, r_at_g, tie, check_values)
    assert bad == 0, f"{what}: {bad} top-m disagreements beyond the tie rule: " + " | ".join(why)
