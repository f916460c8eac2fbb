"""Anchor construction (Sec. 4.1: K-means + Eq. (2)) on the GPU against the CPU oracle: cluster of every point,
round count and anchor indices exact, centroids to fp64 rounding."""
import numpy as np
import pytest
import torch

import synthetic_inputs as si
from oracle import anchors as oa

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kb():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2505_16162_b200 import build
    build.build()
    from paper_2505_16162_b200 import binding
    return binding


def _blobs(seed, n, per, d, spread):
    rng = np.random.default_rng(seed)
    centres = rng.standard_normal((n, d)) * 2.0
    X = np.concatenate([centres[c] + spread * rng.standard_normal((per, d)) for c in range(n)])
    return X[rng.permutation(X.shape[0])].astype(np.float32)


def _check(kb, X, init, max_rounds, k):
    want = oa.build_anchors(X, init.astype(np.float64), max_rounds, k)
    got = kb.knnssd_build_anchors(torch.tensor(X).cuda(), torch.tensor(init).cuda(), max_rounds, k)
    assert got["rounds"] == want["rounds"]
    assert np.array_equal(got["labels"], want["labels"])
    assert np.abs(got["centroids"].cpu().numpy() - want["centroids"]).max() < 1e-10
    assert np.array_equal(got["anchors"], want["anchors"])
    return want, got


# ragged sizes (points per block, columns per chunk, slices of the centroid sums), several rounds from a poor start
@pytest.mark.parametrize("seed,n,per,d,k", [(0, 3, 67, 70, 5), (1, 5, 131, 300, 10), (2, 16, 40, 33, 3), (3, 1, 50, 257, 4),
                                             (4, 4, 1100, 64, 10)])
def test_build_anchors_matches_oracle(kb, seed, n, per, d, k):
    X = _blobs(seed, n, per, d, spread=1.2)
    rng = np.random.default_rng(seed + 50)
    init = X[rng.choice(X.shape[0], n, replace=False)]
    want, _ = _check(kb, X, init, 100, k)
    assert want["rounds"] >= 2


@pytest.mark.parametrize("start", ["one per domain", "all from one domain"])
def test_paper_sized_problem(kb, start):
    """5 domains x 1000 sampled vectors of the 13B width, 10 anchors each."""
    n, per, d, k = 5, 1000, 5120, 10
    X = si.anchors(3, n, per, d, 0.5, normalise=False).numpy()
    init = X[::per].copy() if start == "one per domain" else X[:n].copy()
    want, got = _check(kb, X, init, 50, k)
    if start == "one per domain":
        assert np.bincount(want["labels"]).tolist() == [per] * n       # the planted domains come back
    assert got["ms_rounds"] > 0


def test_round_limit_small_and_empty_clusters(kb):
    X = _blobs(5, 3, 30, 20, spread=1.5)
    init = X[:3].copy()
    _check(kb, X, init, 1, 4)                                          # stopped by the limit: anchors against moved centroids
    _check(kb, X, init, 2, 4)
    far = np.concatenate([X[:2], np.full((1, 20), 1e3, dtype=np.float32)])
    want, got = _check(kb, X, far, 20, 4)                              # the third centroid never gets a member
    assert (want["anchors"][2] == -1).all()
    assert np.array_equal(got["centroids"][2].cpu().numpy(), far[2].astype(np.float64))
    tiny = np.concatenate([X[:5], X[:5]])                              # duplicates: equal distances, lowest index first
    _check(kb, tiny, tiny[:2].copy(), 20, 6)


def test_build_anchors_rejects_bad_arguments(kb):
    X = torch.zeros((40, 8), device="cuda")
    with pytest.raises(kb.KnnssdError) as e:
        kb.knnssd_build_anchors(X, torch.zeros((17, 8), device="cuda"), 5, 2)      # more clusters than supported
    assert e.value.status == 3
    with pytest.raises(kb.KnnssdError) as e:
        kb.knnssd_build_anchors(X[:3].contiguous(), torch.zeros((4, 8), device="cuda"), 5, 2)   # fewer points than clusters
    assert e.value.status == 1
    with pytest.raises(kb.KnnssdError) as e:
        kb.knnssd_build_anchors(X, torch.zeros((2, 8), device="cuda"), 0, 2)       # no rounds
    assert e.value.status == 1
