"""Grouping oracle: Lloyd's iteration of K-means, the clustering the paper names for its
Collaborative-based Grouping (Section 3.2: users / items are embedded, the embeddings are clustered with
K-means, every cluster gets a retrieval pool of its own).

Test infrastructure only (see the package docstring).  Plain numpy in fp64.

One iteration: every point goes to its nearest centroid (squared Euclidean distance, ties to the
smaller cluster index), then every centroid becomes the mean of its points; a cluster that lost all of
its points keeps its centroid.
"""
from __future__ import annotations

from typing import Tuple

import numpy as np


def assign(X: np.ndarray, C: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """X [n, dim], C [k, dim] -> (cluster index int32[n], squared distances fp64 [n, k])."""
    X = np.asarray(X, dtype=np.float64)
    C = np.asarray(C, dtype=np.float64)
    d2 = np.zeros((X.shape[0], C.shape[0]))
    for j in range(C.shape[0]):
        diff = X - C[j]
        d2[:, j] = (diff * diff).sum(axis=1)
    return d2.argmin(axis=1).astype(np.int32), d2      # argmin returns the first (smallest) index of a tie


def update(X: np.ndarray, a: np.ndarray, C: np.ndarray) -> np.ndarray:
    """New centroids: the mean of each cluster's points; empty clusters keep theirs."""
    X = np.asarray(X, dtype=np.float64)
    new = np.asarray(C, dtype=np.float64).copy()
    for j in range(C.shape[0]):
        m = a == j
        if m.any():
            new[j] = X[m].mean(axis=0)
    return new


def lloyd(X: np.ndarray, C0: np.ndarray, iters: int) -> Tuple[np.ndarray, np.ndarray]:
    """`iters` iterations from centroids C0; returns (final centroids, assignment of the last iteration)."""
    C = np.asarray(C0, dtype=np.float64).copy()
    a = np.zeros(X.shape[0], np.int32)
    for _ in range(iters):
        a, _ = assign(X, C)
        C = update(X, a, C)
    return C, a
