"""CPU oracle of the offline task-partitioning step (test infrastructure only): K-means over sentence vectors.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module; it shares nothing with
the CUDA library.  Section 3.2 ("dynamic task partitioning") encodes every prompt as a 384-dimensional vector and
partitions the vectors with the K-means algorithm; the paper names the algorithm and gives no formula, so this is
Lloyd's iteration from its textbook definition, in float64, one plain loop per step:

    assign:  label_i = argmin_k  sum_d (x_id - c_kd)^2          (lowest k on ties)
    update:  c_k     = mean of the points with label k          (a centroid without points keeps its place)
    inertia = sum_i  min_k sum_d (x_id - c_kd)^2

The encoder, the dimensionality reduction and the datasets are outside the scope; inputs are synthetic.
"""
from __future__ import annotations

import numpy as np


def kmeans_assign(points, centroids):
    """(labels int32 [n], squared distance to the chosen centroid float64 [n])."""
    x = np.asarray(points, dtype=np.float64)
    c = np.asarray(centroids, dtype=np.float64)
    n, k = x.shape[0], c.shape[0]
    best = np.full(n, np.inf)
    labels = np.zeros(n, dtype=np.int32)
    for j in range(k):                                   # in index order: a later centroid must be strictly closer to win
        diff = x - c[j]
        dist = np.sum(diff * diff, axis=1)
        closer = dist < best
        labels[closer] = j
        best[closer] = dist[closer]
    return labels, best


def kmeans_update(points, labels, centroids):
    """(new centroids float64 [k][dim], counts int64 [k])."""
    x = np.asarray(points, dtype=np.float64)
    c = np.array(centroids, dtype=np.float64, copy=True)
    counts = np.zeros(c.shape[0], dtype=np.int64)
    for j in range(c.shape[0]):
        members = x[np.asarray(labels) == j]
        counts[j] = members.shape[0]
        if members.shape[0] > 0:
            c[j] = members.sum(axis=0) / members.shape[0]
    return c, counts


def kmeans_step(points, centroids):
    """One Lloyd iteration: (labels, new centroids, counts, inertia under the OLD centroids)."""
    labels, best = kmeans_assign(points, centroids)
    new_c, counts = kmeans_update(points, labels, centroids)
    return labels, new_c, counts, float(best.sum())


def kmeans(points, centroids, iters):
    """`iters` Lloyd iterations from the given centroids: (labels of the last assignment, centroids, inertia history)."""
    c = np.asarray(centroids, dtype=np.float64)
    hist = []
    labels = None
    for _ in range(iters):
        labels, c, _, inertia = kmeans_step(points, c)
        hist.append(inertia)
    return labels, c, hist
