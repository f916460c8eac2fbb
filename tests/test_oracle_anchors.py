"""Pins of the anchor-construction oracle (Sec. 4.1, Eq. (2)) to things other than itself: library K-means from the
same start, brute force over subsets, the fixed-point and descent properties of Lloyd's iteration, closed forms."""
import itertools

import numpy as np
import pytest

from oracle import anchors as oa


def _blobs(seed, n_clusters, per, d, spread=0.3):
    rng = np.random.default_rng(seed)
    centres = rng.standard_normal((n_clusters, d)) * 2.0
    X = np.concatenate([centres[c] + spread * rng.standard_normal((per, d)) for c in range(n_clusters)])
    perm = rng.permutation(X.shape[0])
    return X[perm].astype(np.float32), centres


def _inertia(X, labels, mu):
    X = X.astype(np.float64)
    return float(((X - mu[labels]) ** 2).sum())


@pytest.mark.parametrize("seed,n,per,d", [(0, 3, 40, 8), (1, 5, 60, 32), (2, 4, 25, 3)])
def test_kmeans_matches_scikit_learn_from_the_same_start(seed, n, per, d):
    from sklearn.cluster import KMeans
    X, _ = _blobs(seed, n, per, d, spread=0.8)
    rng = np.random.default_rng(seed + 100)
    init = X[rng.choice(X.shape[0], n, replace=False)].astype(np.float64)       # a poor start: several rounds
    labels, mu, rounds = oa.kmeans(X, init, 100)
    km = KMeans(n_clusters=n, init=init, n_init=1, algorithm="lloyd", tol=0.0, max_iter=100).fit(X.astype(np.float64))
    assert rounds > 2
    assert np.array_equal(labels, km.labels_)
    assert np.abs(mu - km.cluster_centers_).max() < 1e-9


def test_kmeans_matches_scipy_from_the_same_start():
    from scipy.cluster.vq import kmeans2
    X, _ = _blobs(3, 4, 50, 6, spread=0.7)
    init = X[:4].astype(np.float64)
    labels, mu, _ = oa.kmeans(X, init, 200)
    c2, l2 = kmeans2(X.astype(np.float64), init, iter=200, minit="matrix")
    assert np.array_equal(labels, l2)
    assert np.abs(mu - c2).max() < 1e-9


def test_lloyd_fixed_point_and_descent():
    X, _ = _blobs(4, 5, 80, 16, spread=1.0)
    init = X[:5].astype(np.float64)
    prev = None
    for it in range(1, 12):                                   # inertia never rises from one round budget to the next
        labels, mu, rounds = oa.kmeans(X, init, it)
        cur = _inertia(X, labels, mu)
        assert prev is None or cur <= prev + 1e-9
        prev = cur
    labels, mu, rounds = oa.kmeans(X, init, 500)
    assert rounds < 500
    for c in range(5):                                        # every centroid is the mean of its members
        assert np.abs(mu[c] - X[labels == c].astype(np.float64).mean(axis=0)).max() < 1e-12
    d2 = ((X.astype(np.float64)[:, None, :] - mu[None]) ** 2).sum(-1)
    assert np.array_equal(labels, d2.argmin(axis=1))          # and every point sits with its nearest centroid


def test_one_cluster_is_the_global_mean():
    X, _ = _blobs(5, 1, 30, 4)
    labels, mu, rounds = oa.kmeans(X, np.zeros((1, 4)), 10)
    assert rounds == 2 and not labels.any()
    assert np.abs(mu[0] - X.astype(np.float64).mean(axis=0)).max() < 1e-13


def test_ties_go_to_the_lowest_index_and_empty_clusters_stay():
    X = np.array([[0.0, 0.0], [2.0, 0.0], [1.0, 0.0]], dtype=np.float32)       # the last point is midway
    init = np.array([[0.0, 0.0], [2.0, 0.0], [50.0, 50.0]])
    labels, _ = oa.assign(X, init)
    assert labels.tolist() == [0, 1, 0]
    labels, mu, _ = oa.kmeans(X, init, 10)
    assert np.array_equal(mu[2], [50.0, 50.0])                # no members: not moved
    assert np.allclose(mu[0], [0.5, 0.0]) and np.allclose(mu[1], [2.0, 0.0])


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_anchor_selection_is_the_brute_force_minimum_of_eq_2(seed):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((14, 3)).astype(np.float32)
    labels = np.array([0, 1] * 7, dtype=np.int32)
    mu = rng.standard_normal((2, 3))
    k = 3
    got = oa.select_anchors(X, labels, mu, k)
    for c in range(2):
        members = np.nonzero(labels == c)[0]
        dist = {i: float(np.linalg.norm(X[i].astype(np.float64) - mu[c])) for i in members}
        best = min(itertools.combinations(members, k), key=lambda S: sum(dist[i] for i in S))
        assert set(got[c].tolist()) == set(best)
        assert [dist[i] for i in got[c]] == sorted(dist[i] for i in got[c])     # nearest first


def test_anchor_selection_pads_small_clusters_and_orders_equal_distances_by_index():
    X = np.array([[1.0, 0.0], [0.0, 1.0], [-1.0, 0.0], [5.0, 5.0]], dtype=np.float32)
    labels = np.array([0, 0, 0, 1], dtype=np.int32)
    mu = np.array([[0.0, 0.0], [5.0, 5.0]])
    got = oa.select_anchors(X, labels, mu, 2)
    assert got.tolist() == [[0, 1], [3, -1]]


def test_build_anchors_recovers_planted_domains():
    """The workload's shape in small: n domains as Gaussian clusters; started from one sample of each domain, K-means
    returns the domains and the anchors are members of their own cluster, nearest first."""
    n, per, d, k = 5, 100, 64, 10
    X, centres = _blobs(7, n, per, d, spread=0.5)
    init = np.stack([X[np.argmin(((X - centres[c]) ** 2).sum(-1))] for c in range(n)]).astype(np.float64)
    r = oa.build_anchors(X, init, 50, k)
    assert sorted(np.bincount(r["labels"]).tolist()) == [per] * n
    for c in range(n):
        assert (r["labels"][r["anchors"][c]] == c).all()
        dist = np.linalg.norm(X[r["anchors"][c]].astype(np.float64) - r["centroids"][c], axis=1)
        assert (np.diff(dist) >= 0).all()
        others = np.setdiff1d(np.nonzero(r["labels"] == c)[0], r["anchors"][c])
        assert np.linalg.norm(X[others].astype(np.float64) - r["centroids"][c], axis=1).min() >= dist.max()
