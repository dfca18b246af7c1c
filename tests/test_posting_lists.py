"""Posting-list builder (paper Sections 4.2-4.3): pins of the CPU oracle, and bit-exact parity of the CUDA builder.

The oracle (oracle/posting_lists.py) is pinned by a hand-worked example, by the definition applied directly to brute-force
responsibilities, and by structural invariants; the GPU builder must then reproduce the oracle's offsets and items
exactly (integers) on the same top-m input, at sizes that span many blocks and a ragged tail.
"""
from pathlib import Path

import numpy as np
import pytest

from oracle import gmm_oracle as orc
from oracle.posting_lists import posting_lists
from paper_2606_10896_b200 import synth

GOLDEN = Path(__file__).parent / "golden" / "posting_lists_small.txt"


def _golden():
    d = {}
    for line in GOLDEN.read_text().splitlines():
        if not line or line.startswith("#"):
            continue
        key, *vals = line.split()
        d[key] = vals
    return d


def test_hand_worked_example_multi_and_hard_assignment():
    g = _golden()
    K = int(g["K"][0])
    idx = np.array(g["idx"], dtype=np.int32).reshape(-1, 2)
    resp = np.array(g["resp"], dtype=np.float32).reshape(-1, 2)
    off, items, mean = posting_lists(idx, resp, K, None, 2)
    assert off.tolist() == [int(v) for v in g["offsets"]]
    assert items.tolist() == [int(v) for v in g["items"]]
    assert mean == pytest.approx(float(g["mean"][0]))
    off, items, mean = posting_lists(idx, resp, K, None, 1)
    assert off.tolist() == [int(v) for v in g["hard_offsets"]]
    assert items.tolist() == [int(v) for v in g["hard_items"]]
    assert mean == 1.0


def _tiny_mixture(seed, N=40, D=2, K=5):
    rng = np.random.Generator(np.random.PCG64(seed))
    mu = rng.normal(0, 1.5, (K, D))
    var = rng.uniform(0.5, 1.5, (K, D))
    pi = rng.dirichlet(np.ones(K) * 3)
    X = (mu[rng.integers(0, K, N)] + rng.standard_normal((N, D))).astype(np.float32)
    return X, pi.astype(np.float32), mu.astype(np.float32), var.astype(np.float32)


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_rule_applied_to_brute_force_responsibilities(seed):
    # The definition, written out on the full responsibility matrix from linear-space densities (no top-m, no log-sum-exp):
    # a vector is stored with its best cluster, and with its second best if that one's responsibility exceeds 1/K.
    X, pi, mu, var = _tiny_mixture(seed)
    K = len(pi)
    R, _ = orc.brute_force(X, pi, mu, var)
    expect = [[] for _ in range(K)]
    for i in range(len(X)):
        order = sorted(range(K), key=lambda k: (-R[i, k], k))
        expect[order[0]].append(i)
        if np.float32(R[i, order[1]]) > np.float32(1.0 / K):
            expect[order[1]].append(i)
    idx, resp, _ = orc.topm(X, pi, mu, var, 2)
    off, items, mean = posting_lists(idx, resp, K, None, 2)
    for k in range(K):
        assert items[off[k]:off[k + 1]].tolist() == sorted(expect[k])
    assert mean == pytest.approx(sum(len(e) for e in expect) / len(X))


def test_invariants():
    X, pi, mu, var = _tiny_mixture(9, N=200, D=3, K=7)
    K = len(pi)
    idx, resp, _ = orc.topm(X, pi, mu, var, 3)
    # hard assignment is a partition by argmax
    off, items, mean = posting_lists(idx, resp, K, None, 1)
    assert off[K] == len(X) and mean == 1.0
    assert sorted(items.tolist()) == list(range(len(X)))
    for k in range(K):
        assert np.all(idx[items[off[k]:off[k + 1]], 0] == k)
    # a threshold nothing exceeds gives the same partition; one everything exceeds gives max_lists entries per vector
    off1, items1, _ = posting_lists(idx, resp, K, 1.0, 3)
    assert off1.tolist() == off.tolist() and items1.tolist() == items.tolist()
    off3, items3, mean3 = posting_lists(idx, resp, K, 1e-30, 3)
    assert off3[K] == 3 * len(X) and mean3 == 3.0
    # lists are ascending without repeats, and the mean lies between 1 and max_lists
    off2, items2, mean2 = posting_lists(idx, resp, K, None, 2)
    assert 1.0 <= mean2 <= 2.0
    for k in range(K):
        lst = items2[off2[k]:off2[k + 1]]
        assert np.all(np.diff(lst) > 0)
    # raising tau can only remove entries
    assert posting_lists(idx, resp, K, 2.0 / K, 2)[0][K] <= off2[K] <= posting_lists(idx, resp, K, 0.5 / K, 2)[0][K]


# ------------------------------------------------------------------------------------------------------------------
# GPU parity: bit-exact against the oracle on the same top-m arrays
# ------------------------------------------------------------------------------------------------------------------

@pytest.mark.gpu
@pytest.mark.parametrize("N,D,K,m,max_lists,tau", [(1, 4, 3, 1, 1, None), (700, 8, 5, 2, 2, None), (20000, 16, 64, 2, 2, None),
                                                    (50000, 32, 1000, 4, 2, None), (30011, 16, 300, 4, 4, 0.5 / 300),
                                                    (30011, 16, 300, 3, 1, None), (9000, 8, 4096, 2, 2, None)])
def test_gpu_builder_matches_oracle_exactly(N, D, K, m, max_lists, tau):
    import torch
    from paper_2606_10896_b200 import flashgmm as fg

    rng = np.random.Generator(np.random.PCG64(N + K))
    mu = rng.normal(0, 2, (K, D)).astype(np.float32)
    var = rng.uniform(0.5, 2.0, (K, D)).astype(np.float32)
    pi = rng.dirichlet(np.ones(K)).astype(np.float32)
    X = (mu[rng.integers(0, K, N)] + 1.5 * rng.standard_normal((N, D))).astype(np.float32)
    dev = "cuda:0"
    t = lambda a: torch.as_tensor(np.ascontiguousarray(a), device=dev)
    with fg.Context(0) as ctx:
        idx_d, resp_d = ctx.gmm_assign_topm(t(X), t(pi), t(mu), t(var), m)
        off_d, items_d, total, mean = ctx.gmm_build_posting_lists(idx_d, resp_d, K, tau, max_lists)
        # a second build gives the same bytes (the placement is deterministic)
        off_2, items_2, total_2, _ = ctx.gmm_build_posting_lists(idx_d, resp_d, K, tau, max_lists)
    idx, resp = idx_d.cpu().numpy(), resp_d.cpu().numpy()
    off_r, items_r, mean_r = posting_lists(idx, resp, K, tau, max_lists)
    assert total == off_r[K] == total_2
    assert off_d.cpu().numpy().tolist() == off_r.tolist()
    assert items_d.cpu().numpy()[:total].tolist() == items_r.tolist()
    assert torch.equal(off_d, off_2) and torch.equal(items_d[:total], items_2[:total])
    assert mean == pytest.approx(mean_r)


@pytest.mark.gpu
def test_gpu_builder_rejects_bad_arguments():
    import torch
    from paper_2606_10896_b200 import flashgmm as fg

    idx = torch.zeros((10, 2), dtype=torch.int32, device="cuda:0")
    resp = torch.zeros((10, 2), dtype=torch.float32, device="cuda:0")
    with fg.Context(0) as ctx:
        for K, max_lists in [(0, 1), (4, 0), (4, 3), (1 << 20, 1)]:
            with pytest.raises(fg.GmmError) as err:
                ctx.gmm_build_posting_lists(idx, resp, K, None, max_lists)
            assert err.value.code in (fg.GMM_EINVAL, fg.GMM_EUNSUPPORTED)
