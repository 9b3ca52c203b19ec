"""Pins for the grouping oracle (Lloyd's K-means, Section 3.2): hand examples, the tie and empty-cluster
rules, two independent library implementations of the same iteration, and the descent property."""
import numpy as np
import pytest

from oracle import grouping as G
from paper_2408_05676_b200 import synth


def test_hand_example_on_a_line():
    X = np.asarray([[0.0], [1.0], [2.0], [10.0], [11.0], [12.0]])
    a, d2 = G.assign(X, np.asarray([[0.0], [10.0]]))
    assert a.tolist() == [0, 0, 0, 1, 1, 1] and d2[2].tolist() == [4.0, 64.0]
    C, a = G.lloyd(X, np.asarray([[0.0], [10.0]]), 3)
    assert C.ravel().tolist() == [1.0, 11.0] and a.tolist() == [0, 0, 0, 1, 1, 1]
    # a bad start is repaired: both centroids left of the data
    C, a = G.lloyd(X, np.asarray([[-1.0], [0.5]]), 5)
    assert C.ravel().tolist() == [1.0, 11.0]


def test_ties_go_to_the_smaller_index_and_empty_clusters_keep_their_centroid():
    a, _ = G.assign(np.asarray([[5.0, 0.0]]), np.asarray([[0.0, 0.0], [10.0, 0.0], [5.0, 5.0]]))
    assert a.tolist() == [0]
    X = np.asarray([[0.0], [1.0]])
    C = G.update(X, np.asarray([0, 0], np.int32), np.asarray([[0.0], [100.0]]))
    assert C.ravel().tolist() == [0.5, 100.0]


@pytest.mark.parametrize("n,dim,k,seed", [(3000, 8, 5, 1), (2000, 33, 12, 2)])
def test_matches_library_lloyd_iterations(n, dim, k, seed):
    from scipy.cluster.vq import kmeans2
    from sklearn.cluster import KMeans
    X, _ = synth.make_embeddings(n, dim, k, seed=seed)
    X = X.astype(np.float64)
    C0 = X[:k].copy()
    iters = 6
    C, a = G.lloyd(X, C0, iters)
    Cs, ls = kmeans2(X, C0.copy(), iter=iters, minit="matrix")
    assert np.abs(Cs - C).max() < 1e-9 and (ls == a).all()     # centroids and the last iteration's labels
    km = KMeans(n_clusters=k, init=C0.copy(), n_init=1, max_iter=iters, tol=0.0, algorithm="lloyd").fit(X)
    if km.n_iter_ == iters:                           # (it stops early once the assignment is stable)
        assert np.abs(km.cluster_centers_ - C).max() < 1e-6
    else:
        Cc, _ = G.lloyd(X, C0, km.n_iter_)
        assert np.abs(km.cluster_centers_ - Cc).max() < 1e-6


def test_objective_never_increases():
    X, _ = synth.make_embeddings(4000, 16, 9, seed=3)
    C = X[:9].astype(np.float64)
    last = np.inf
    for _ in range(8):
        a, d2 = G.assign(X, C)
        obj = d2[np.arange(len(a)), a].sum()
        assert obj <= last * (1 + 1e-12)
        last = obj
        C = G.update(X, a, C)
