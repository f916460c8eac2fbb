"""Anchor construction of the pre-inference stage - CPU oracle (test infrastructure only).

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import this module; it imports nothing from
the CUDA package.  Plain numpy in fp64, written from Sec. 4.1 ("Pre Inference"):

* the sampled last hidden vectors of all domains are clustered into n groups with the K-means algorithm, n = the
  number of domains (``kmeans``: Lloyd's iteration, the algorithm the name denotes; the paper does not say how it is
  started or stopped, so the starting centroids are an input and it stops when no assignment changes);
* for each cluster the k members nearest to the cluster centroid are its anchors, Eq. (2): the size-k subset S that
  minimises the sum of ||v - mu_i|| over S (``select_anchors``: that minimum is reached by the k smallest distances).

Pinned in ``tests/test_oracle_anchors.py`` against scikit-learn's and SciPy's K-means from the same start, brute force
over all subsets for Eq. (2), the fixed-point property of Lloyd's iteration and hand-made cases.
"""
from __future__ import annotations

from typing import List, Tuple

import numpy as np


def assign(X: np.ndarray, mu: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Nearest centroid of every point by squared Euclidean distance (lowest index on ties) and that distance."""
    X = np.asarray(X, dtype=np.float64)
    mu = np.asarray(mu, dtype=np.float64)
    d2 = np.empty((X.shape[0], mu.shape[0]), dtype=np.float64)
    for c in range(mu.shape[0]):
        diff = X - mu[c]
        d2[:, c] = np.einsum("ij,ij->i", diff, diff)
    labels = np.argmin(d2, axis=1).astype(np.int32)          # argmin returns the first of equal minima
    return labels, d2[np.arange(X.shape[0]), labels]


def kmeans(X: np.ndarray, init: np.ndarray, max_iter: int) -> Tuple[np.ndarray, np.ndarray, int]:
    """Lloyd's iteration from the centroids ``init`` [n][d].

    Each round assigns every point to its nearest centroid, stops if no assignment changed, else moves every centroid
    to the mean of its members (a centroid without members stays where it is).  Returns (labels int32 [N], centroids
    fp64 [n][d], number of assignment rounds)."""
    X = np.asarray(X, dtype=np.float64)
    mu = np.array(init, dtype=np.float64, copy=True)
    labels = None
    rounds = 0
    for _ in range(max_iter):
        new, _ = assign(X, mu)
        rounds += 1
        if labels is not None and np.array_equal(new, labels):
            break
        labels = new
        for c in range(mu.shape[0]):
            members = X[labels == c]
            if members.shape[0]:
                mu[c] = members.sum(axis=0) / members.shape[0]
    return labels, mu, rounds


def select_anchors(X: np.ndarray, labels: np.ndarray, mu: np.ndarray, k: int) -> np.ndarray:
    """Eq. (2): for each cluster the indices of its k members with the smallest ||v - mu_i|| (nearest first, lowest
    index first among equal distances); int32 [n][k], -1 where a cluster has fewer than k members."""
    X = np.asarray(X, dtype=np.float64)
    out = np.full((mu.shape[0], k), -1, dtype=np.int32)
    for c in range(mu.shape[0]):
        idx = np.nonzero(labels == c)[0]
        diff = X[idx] - mu[c]
        dist = np.sqrt(np.einsum("ij,ij->i", diff, diff))
        order = np.lexsort((idx, dist))                      # by distance, then by index
        take = idx[order[:k]]
        out[c, :take.shape[0]] = take
    return out


def build_anchors(X: np.ndarray, init: np.ndarray, max_iter: int, k: int):
    """The whole step: K-means, then Eq. (2) on its clusters.  Returns dict(labels, centroids, rounds, anchors)."""
    labels, mu, rounds = kmeans(X, init, max_iter)
    return {"labels": labels, "centroids": mu, "rounds": rounds, "anchors": select_anchors(X, labels, mu, k)}
