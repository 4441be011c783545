"""Pins of the K-means oracle (offline task partitioning, Section 3.2) against things other than itself."""
import numpy as np
import pytest

from oracle import partition
from paper_2505_08600_b200 import synth


def test_assignment_against_scipy_vq():
    # scipy's vector-quantisation routine computes the same nearest-code assignment (Euclidean distance)
    from scipy.cluster.vq import vq
    x, _ = synth.make_sentence_vectors(3000, 384, 4, seed=11)
    c = x[[5, 77, 901, 2500]].astype(np.float64)
    labels, best = partition.kmeans_assign(x, c)
    code, dist = vq(x.astype(np.float64), c)
    assert (labels == code).all()
    np.testing.assert_allclose(np.sqrt(best), dist, rtol=1e-12, atol=1e-12)


def test_assignment_brute_force_on_tiny_inputs_and_ties_go_to_the_lowest_index():
    rng = np.random.default_rng(0)
    x = rng.integers(-3, 4, size=(40, 5)).astype(np.float64)          # small integers: exact arithmetic, real ties
    c = rng.integers(-3, 4, size=(6, 5)).astype(np.float64)
    c[4] = c[1]                                                       # a duplicate centroid never wins over the earlier copy
    labels, best = partition.kmeans_assign(x, c)
    for i in range(40):
        d = [sum((x[i][t] - c[j][t]) ** 2 for t in range(5)) for j in range(6)]
        assert best[i] == min(d)
        assert labels[i] == d.index(min(d))
    assert 4 not in labels.tolist() or (labels == 4).sum() == 0


def test_update_is_the_mean_and_an_empty_cluster_keeps_its_centroid():
    x = np.array([[0.0, 0.0], [2.0, 0.0], [10.0, 10.0]])
    c = np.array([[1.0, 1.0], [9.0, 9.0], [100.0, 100.0]])
    labels, new_c, counts, inertia = partition.kmeans_step(x, c)
    assert labels.tolist() == [0, 0, 1] and counts.tolist() == [2, 1, 0]
    np.testing.assert_array_equal(new_c, [[1.0, 0.0], [10.0, 10.0], [100.0, 100.0]])
    assert inertia == 2.0 + 2.0 + 2.0


def test_one_cluster_gives_the_mean_and_the_total_variance():
    x, _ = synth.make_sentence_vectors(500, 128, 3, seed=2)
    labels, new_c, counts, inertia = partition.kmeans_step(x, x[:1])
    assert (labels == 0).all() and counts.tolist() == [500]
    np.testing.assert_allclose(new_c[0], x.astype(np.float64).mean(axis=0), rtol=1e-12)
    _, _, _, inertia2 = partition.kmeans_step(x, new_c)
    np.testing.assert_allclose(inertia2, ((x.astype(np.float64) - new_c[0]) ** 2).sum(), rtol=1e-12)


def test_lloyd_iterations_never_increase_the_inertia_and_recover_separated_groups():
    x, task = synth.make_sentence_vectors(4000, 384, 4, seed=6, spread=0.5)
    first = [int(np.flatnonzero(task == t)[0]) for t in range(4)]     # one seed point from every group
    labels, c, hist = partition.kmeans(x, x[first], 8)
    assert all(b <= a + 1e-9 for a, b in zip(hist, hist[1:]))
    assert (labels == task).mean() > 0.98                             # the synthetic groups are as separable as the paper's tasks


def test_assignment_is_invariant_under_a_common_shift():
    x, _ = synth.make_sentence_vectors(800, 128, 4, seed=9)
    c = x[[1, 2, 3, 4]].astype(np.float64)
    shift = np.linspace(-1, 1, 128)
    l0, b0 = partition.kmeans_assign(x, c)
    l1, b1 = partition.kmeans_assign(x.astype(np.float64) + shift, c + shift)
    assert (l0 == l1).all()
    np.testing.assert_allclose(b0, b1, rtol=1e-9, atol=1e-12)
