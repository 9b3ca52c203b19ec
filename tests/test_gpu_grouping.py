"""laser_group_kmeans against the grouping oracle (Section 3.2, Collaborative-based Grouping): assignments
for given centroids must equal the oracle's except where a point's two nearest centroids are within fp32
rounding of each other (counted; none on this data), centroids within fp32 summation accuracy, and the
clusters found on synthetic mixture embeddings must be the generating components."""
import numpy as np
import pytest
import torch

from helpers import ensure_built
from oracle import grouping as G
from paper_2408_05676_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    ensure_built()
    from paper_2408_05676_b200 import binding
    return binding


def _near_ties(d2, a_gpu, a_ref, rel=1e-5):
    bad = np.nonzero(a_gpu != a_ref)[0]
    for i in bad:
        assert abs(d2[i, a_gpu[i]] - d2[i, a_ref[i]]) <= rel * d2[i, a_ref[i]], (i, d2[i, a_gpu[i]], d2[i, a_ref[i]])
    return len(bad)


@pytest.mark.parametrize("n,dim,k", [(20003, 64, 16), (5001, 40, 7), (333, 256, 3), (1, 5, 1)])
def test_one_iteration_and_ten(L, n, dim, k):
    X, comp = synth.make_embeddings(n, dim, k, seed=50 + dim)
    C0 = X[:k].copy()
    x = torch.as_tensor(X, device="cuda")
    # one iteration: assignment for the given centroids, new centroids, counts
    c = torch.as_tensor(C0, device="cuda").clone()
    a, cnt = L.group_kmeans(x, c, 1)
    a_ref, d2 = G.assign(X, C0)
    assert _near_ties(d2, a.cpu().numpy(), a_ref) == 0
    assert (cnt.cpu().numpy() == np.bincount(a_ref, minlength=k)).all()
    C1 = G.update(X, a_ref, C0)
    assert np.abs(c.cpu().numpy() - C1).max() <= 2e-5 * max(1.0, np.abs(C1).max())
    # ten iterations from the same start
    c = torch.as_tensor(C0, device="cuda").clone()
    a, cnt = L.group_kmeans(x, c, 10)
    C10, _ = G.lloyd(X, C0, 10)
    a10, d2 = G.assign(X, G.lloyd(X, C0, 9)[0])       # the last iteration assigns with the centroids before it
    flips = _near_ties(d2, a.cpu().numpy(), a10, rel=1e-3)
    assert flips <= max(1, n // 2000)
    assert np.abs(c.cpu().numpy() - C10).max() <= 1e-3 * max(1.0, np.abs(C10).max())
    assert int(cnt.sum()) == n


def test_groups_are_the_generating_components(L):
    n, dim, k = 50000, 64, 32
    X, comp = synth.make_embeddings(n, dim, k, seed=7)
    # start: one point of every component, so that no two starts share a component
    first = np.asarray([int(np.nonzero(comp == j)[0][0]) for j in range(k)])
    c = torch.as_tensor(X[first], device="cuda").clone()
    a, cnt = L.group_kmeans(torch.as_tensor(X, device="cuda"), c, 8)
    a = a.cpu().numpy()
    assert (a == comp).mean() > 0.99
    assert (cnt.cpu().numpy() == np.bincount(a, minlength=k)).all()
    with pytest.raises(L.LaserError):
        L.group_kmeans(torch.zeros(4, 300, device="cuda"), torch.zeros(2, 300, device="cuda"), 1)   # dim > 256
