"""CPU oracle of one Lloyd (k-means) iteration, the warm start the paper uses before its EM iterations (Section 4.4,
experimental setup: 10 iterations of k-means, then Flash-GMM).

TEST INFRASTRUCTURE ONLY: the tests call this; the product package never imports it.  Plain numpy in float64, written
from the textbook definition with no blocking or reordering beyond a loop over chunks of points to bound memory:

* assignment: a point goes to the centroid at the smallest squared Euclidean distance (direct differences), ties to the
  smaller centroid index;
* update: a centroid becomes the mean of its points; a centroid without points keeps its position (the paper is silent;
  same reading as the frozen empty component of the mixture);
* inertia: the sum of the squared distances to the assigned (old) centroids.
"""
from __future__ import annotations

import numpy as np


def kmeans_step(X, centroids, chunk: int = 4096):
    """Returns (assign int64 [N], new_centroids float64 [K, D], counts int64 [K], inertia, gap float64 [N]).

    ``gap`` is the difference between a point's second smallest and smallest squared distance: where it is tiny, another
    precision may legitimately pick the other centroid."""
    X = np.asarray(X, dtype=np.float64)
    C = np.asarray(centroids, dtype=np.float64)
    N, D = X.shape
    K = C.shape[0]
    assign = np.empty(N, np.int64)
    best = np.empty(N, np.float64)
    gap = np.full(N, np.inf)
    for s in range(0, N, chunk):
        x = X[s:s + chunk]
        d2 = ((x[:, None, :] - C[None, :, :]) ** 2).sum(-1)          # [n, K], direct differences
        a = d2.argmin(1)                                             # first minimum = smaller index on ties
        assign[s:s + chunk] = a
        rows = np.arange(len(x))
        best[s:s + chunk] = d2[rows, a]
        if K > 1:
            d2[rows, a] = np.inf
            gap[s:s + chunk] = d2.min(1) - best[s:s + chunk]
    counts = np.bincount(assign, minlength=K).astype(np.int64)
    new = C.copy()
    for k in range(K):
        if counts[k] > 0:
            new[k] = X[assign == k].mean(0)
    return assign, new, counts, float(best.sum()), gap
