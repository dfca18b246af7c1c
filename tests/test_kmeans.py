"""One Lloyd (k-means) iteration, the paper's warm start (Section 4.4 and the warm-start appendix: 10 iterations of k-means before the EM iterations):
pins of the CPU oracle, and parity of the CUDA step.

The oracle (oracle/kmeans.py) is pinned by closed forms, by separated clusters whose answer is known by construction,
and by scikit-learn's own single Lloyd iteration (an independent implementation).  The GPU step must give the same
assignment wherever the oracle's two smallest distances are not a near-tie, the same counts and centroids up to those
near-ties, and bit-identical results when repeated.
"""
import numpy as np
import pytest

from oracle.kmeans import kmeans_step


def _blobs(seed, N, D, K, spread=6.0, noise=1.0):
    rng = np.random.Generator(np.random.PCG64(seed))
    centers = rng.normal(0, spread, (K, D))
    lab = rng.integers(0, K, N)
    X = (centers[lab] + noise * rng.standard_normal((N, D))).astype(np.float32)
    return X, centers, lab


def test_single_centroid_is_the_mean_and_inertia_the_total_scatter():
    X, _, _ = _blobs(1, 500, 3, 1)
    c0 = np.array([[0.5, -1.0, 2.0]])
    a, new, counts, inertia, _ = kmeans_step(X, c0)
    X64 = X.astype(np.float64)
    assert np.all(a == 0) and counts.tolist() == [500]
    np.testing.assert_allclose(new[0], X64.mean(0), rtol=1e-13)
    assert inertia == pytest.approx(((X64 - c0) ** 2).sum(), rel=1e-13)


def test_separated_clusters_recover_their_own_means():
    # clusters 100 noise-widths apart, started at the true centres: every point keeps its cluster
    X, centers, lab = _blobs(2, 900, 4, 6, spread=100.0, noise=0.5)
    a, new, counts, inertia, gap = kmeans_step(X, centers)
    assert np.array_equal(a, lab)
    for k in range(6):
        np.testing.assert_allclose(new[k], X[lab == k].astype(np.float64).mean(0), rtol=1e-12)
    assert counts.tolist() == np.bincount(lab, minlength=6).tolist()
    assert inertia == pytest.approx(sum(((X[lab == k].astype(np.float64) - centers[k]) ** 2).sum() for k in range(6)))
    assert gap.min() > 1.0


def test_ties_go_to_the_smaller_index_and_an_empty_centroid_stays():
    X = np.array([[0.0, 0.0], [2.0, 0.0], [1.0, 0.0]], dtype=np.float32)          # the third point is equidistant
    C = np.array([[0.0, 0.0], [2.0, 0.0], [50.0, 50.0]])
    a, new, counts, inertia, gap = kmeans_step(X, C)
    assert a.tolist() == [0, 1, 0] and counts.tolist() == [2, 1, 0]
    np.testing.assert_allclose(new, [[0.5, 0.0], [2.0, 0.0], [50.0, 50.0]])
    assert inertia == pytest.approx(1.0) and gap[2] == 0.0


def test_lloyd_iteration_never_increases_inertia():
    X, _, _ = _blobs(3, 2000, 8, 12)
    C = X[:12].astype(np.float64)
    last = np.inf
    for _ in range(6):
        _, C, _, inertia, _ = kmeans_step(X, C)
        assert inertia <= last * (1 + 1e-12)
        last = inertia


def test_against_scikit_learn_single_lloyd_iteration():
    sk = pytest.importorskip("sklearn.cluster")
    X, _, _ = _blobs(4, 1500, 5, 9, spread=4.0)
    C = X[:9].astype(np.float64)
    km = sk.KMeans(n_clusters=9, init=C, n_init=1, max_iter=1, algorithm="lloyd", tol=0.0).fit(X.astype(np.float64))
    a, new, counts, inertia, gap = kmeans_step(X, C)
    # after one iteration scikit-learn holds the updated centres; its labels_ are those of a final extra assignment
    np.testing.assert_allclose(km.cluster_centers_, new, rtol=1e-6, atol=1e-6)
    a2, _, _, _, _ = kmeans_step(X, new)
    assert np.mean(km.labels_ == a2) == 1.0


# ------------------------------------------------------------------------------------------------------------------
# GPU parity
# ------------------------------------------------------------------------------------------------------------------

@pytest.mark.gpu
@pytest.mark.parametrize("N,D,K", [(1, 3, 1), (700, 5, 3), (5000, 16, 64), (40000, 128, 1024), (30011, 96, 300), (20000, 130, 70),
                                   (9000, 768, 300), (12000, 200, 1500)])
def test_gpu_kmeans_step_matches_oracle(N, D, K):
    import torch
    from paper_2606_10896_b200 import flashgmm as fg

    X, _, _ = _blobs(N + K, N, D, K, spread=3.0)
    rng = np.random.Generator(np.random.PCG64(5))
    C = X[rng.choice(N, K, replace=N < K)].astype(np.float32) if N >= K else X[[0] * K].astype(np.float32)
    a_r, new_r, counts_r, inertia_r, gap = kmeans_step(X, C.astype(np.float64))
    dev = "cuda:0"
    t = lambda v: torch.as_tensor(np.ascontiguousarray(v), device=dev)
    with fg.Context(0) as ctx:
        a_d, new_d, counts_d, inertia = ctx.gmm_kmeans_step(t(X), t(C))
        a_2, new_2, counts_2, inertia_2 = ctx.gmm_kmeans_step(t(X), t(C))
    assert torch.equal(a_d, a_2) and torch.equal(new_d, new_2) and torch.equal(counts_d, counts_2) and inertia == inertia_2
    a = a_d.cpu().numpy().astype(np.int64)
    scale = float(np.sqrt((X.astype(np.float64).var(0)).mean())) or 1.0
    # assignments agree wherever the two nearest centroids are not a near-tie in float32 distances
    near_tie = gap <= 1e-4 * (scale * scale * D)
    assert np.all((a == a_r) | near_tie), "assignment differs away from a tie"
    moved = int((a != a_r).sum())
    counts = counts_d.cpu().numpy()
    assert counts.sum() == N and np.abs(counts - counts_r).sum() <= 2 * moved
    if moved == 0:
        np.testing.assert_allclose(new_d.cpu().numpy(), new_r, rtol=0, atol=1e-4 * scale)
    assert abs(inertia - inertia_r) <= 1e-5 * abs(inertia_r) + 1e-6
