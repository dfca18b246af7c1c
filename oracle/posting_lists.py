"""CPU oracle of the IVF posting-list builder (paper Sections 4.2 and 4.3).

TEST INFRASTRUCTURE ONLY: the tests call this; the product package never imports it.  Plain Python / numpy, written
from the rule as the paper states it, with no blocking or reordering:

* Section 4.2 (drop-in hard assignment): a vector goes to the list of the cluster with the highest responsibility.
* Section 4.3 (multi-assignment): a vector goes to AT MOST ``max_lists`` clusters (the paper uses two): the top clusters
  whose responsibility exceeds tau, tau = 1 / K by default.

Reading adopted where the paper is silent: the best cluster always receives the vector (every vector has to be stored
somewhere; with tau = 1 / K its responsibility is at least 1 / K anyway, and an exact tie at 1 / K must not drop the
vector); further clusters are taken in the order of the top-m list while their responsibility is STRICTLY greater than
tau.  Lists hold point indices in ascending order; ``offsets`` is the exclusive prefix sum of the list lengths.
"""
from __future__ import annotations

import numpy as np


def posting_lists(idx, resp, K: int, tau: float | None = None, max_lists: int = 2):
    """idx [N, m] component indices (descending responsibility), resp [N, m] their responsibilities.

    Returns (offsets int64 [K + 1], items int64 [offsets[K]], mean_lists_per_vector)."""
    idx = np.asarray(idx)
    resp = np.asarray(resp, dtype=np.float32)          # the threshold test is taken in the precision of the input
    if idx.ndim != 2 or idx.shape != resp.shape:
        raise ValueError("idx and resp must both be [N, m]")
    N, m = idx.shape
    if not (1 <= max_lists <= m):
        raise ValueError("max_lists must be in [1, m]")
    thr = np.float32(1.0 / K if tau is None or tau <= 0 else tau)
    lists = [[] for _ in range(K)]
    for i in range(N):                                  # ascending i, so every list comes out ascending
        for j in range(max_lists):
            k = int(idx[i, j])
            if k < 0:
                break                                   # fewer than m components exist (m > K)
            if j == 0 or resp[i, j] > thr:
                lists[k].append(i)
            else:
                break                                   # responsibilities are descending: nothing further can pass
    offsets = np.zeros(K + 1, np.int64)
    for k in range(K):
        offsets[k + 1] = offsets[k] + len(lists[k])
    items = np.array([i for lst in lists for i in lst], dtype=np.int64)
    return offsets, items, (float(offsets[K]) / N if N else 0.0)
