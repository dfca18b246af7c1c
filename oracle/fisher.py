"""CPU oracle of Fisher-vector encoding under a diagonal Gaussian mixture: the use of the fused pattern (per-point
responsibilities combined into weighted statistics, one set per group of points instead of one global set) that the
paper's Discussion (Section 6) names.  The paper gives no formula; the definition taken is the standard one (the gradient
of a group's mean log-likelihood with respect to the means and the standard deviations, each coordinate scaled by the
inverse square root of its diagonal Fisher information, which is pi_k / sigma_kd^2 for a mean and 2 pi_k / sigma_kd^2
for a standard deviation).

TEST INFRASTRUCTURE ONLY: the tests call this; the product package never imports it.  Plain numpy in float64, the
definition written out point by point over the materialised responsibilities (Section 2's posterior), with no use of
the sufficient statistics the GPU path goes through:

    G_mu[k, d]    = 1 / (T sqrt(pi_k))   * sum_t r_tk (x_td - mu_kd) / sigma_kd
    G_sigma[k, d] = 1 / (T sqrt(2 pi_k)) * sum_t r_tk ((x_td - mu_kd)^2 / sigma_kd^2 - 1)

for a group of T points.  A component with pi_k = 0 has r = 0 for every point and gets zeros; an empty group gets
zeros.  No power or L2 normalisation is applied (that is the caller's).
"""
from __future__ import annotations

import numpy as np

from . import gmm_oracle


def fisher_vector(X, pi, mu, var):
    """Fisher vector of ONE group: float64 [2, K, D] (means part, then standard-deviation part)."""
    X = np.asarray(X, dtype=np.float32)
    pi64 = np.asarray(pi, dtype=np.float64)
    mu64 = np.asarray(mu, dtype=np.float64)
    sd = np.sqrt(np.asarray(var, dtype=np.float64))
    K, D = mu64.shape
    T = X.shape[0]
    out = np.zeros((2, K, D), np.float64)
    if T == 0:
        return out
    R, _ = gmm_oracle.responsibilities(X, pi, mu, var)                   # [T, K], the posterior of Section 2
    x = X.astype(np.float64)
    for k in range(K):
        if not pi64[k] > 0.0:
            continue
        z = (x - mu64[k][None, :]) / sd[k][None, :]                      # [T, D] standardised differences
        r = R[:, k][:, None]
        out[0, k] = (r * z).sum(0) / (T * np.sqrt(pi64[k]))
        out[1, k] = (r * (z * z - 1.0)).sum(0) / (T * np.sqrt(2.0 * pi64[k]))
    return out


def fisher_vectors(X, offsets, pi, mu, var):
    """Fisher vectors of G groups of consecutive rows: group g = rows offsets[g] .. offsets[g + 1] - 1; [G, 2, K, D]."""
    offsets = np.asarray(offsets, dtype=np.int64)
    X = np.asarray(X)
    return np.stack([fisher_vector(X[offsets[g]:offsets[g + 1]], pi, mu, var) for g in range(len(offsets) - 1)])


def mean_log_likelihood(X, pi, mu, var):
    """(1 / T) sum_t log p(x_t): what the Fisher vector differentiates."""
    _, lz = gmm_oracle.responsibilities(np.asarray(X, dtype=np.float32), pi, mu, var)
    return float(lz.mean())
