"""K-means step of the CUDA library against the CPU oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

from oracle import partition
from paper_2505_08600_b200 import synth
from gpu_util import DEV

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sd():
    from paper_2505_08600_b200 import binding
    binding.lib()
    return binding


def _run(sd, x, c):
    n, dim = x.shape
    k = c.shape[0]
    labels = torch.full((max(n, 1),), -1, dtype=torch.int32, device=DEV)
    c_out = torch.zeros((k, dim), dtype=torch.float32, device=DEV)
    counts = torch.zeros((k,), dtype=torch.int64, device=DEV)
    inertia = torch.zeros((1,), dtype=torch.float64, device=DEV)
    xd = torch.from_numpy(x).to(DEV) if n else torch.zeros((0, dim), dtype=torch.float32, device=DEV)
    sd.sd_kmeans_step(xd, torch.from_numpy(c).to(DEV), labels, c_out, counts, inertia)
    torch.cuda.synchronize()
    return labels.cpu().numpy()[:n], c_out.cpu().numpy(), counts.cpu().numpy(), float(inertia.item())


CASES = [  # n, dim, k   (several blocks and a ragged tail; one warp's worth; fewer points than warps)
    (10007, 384, 4), (5000, 384, 2), (3001, 384, 3), (777, 128, 8), (2049, 256, 5), (33, 512, 1), (3, 384, 4),
]


@pytest.mark.parametrize("n,dim,k", CASES)
def test_kmeans_step_matches_the_oracle(sd, n, dim, k):
    x, task = synth.make_sentence_vectors(n, dim, max(k, 2), seed=n)
    c = np.ascontiguousarray(x[np.linspace(0, n - 1, k).astype(int)] + np.float32(0.01))
    labels, c_out, counts, inertia = _run(sd, x, c)
    l_ref, best = partition.kmeans_assign(x, c)
    # the decision is an argmin of fp32 sums on the device and of fp64 sums in the oracle: equal wherever the two
    # smallest distances differ by more than fp32 summation noise, and a valid nearest centroid everywhere
    xd, cd = x.astype(np.float64), c.astype(np.float64)
    dist = ((xd[:, None, :] - cd[None, :, :]) ** 2).sum(axis=2)
    two = np.sort(dist, axis=1)[:, :2] if k > 1 else np.stack([dist[:, 0], np.full(n, np.inf)], axis=1)
    clear = two[:, 1] - two[:, 0] > 1e-5 * (1.0 + two[:, 0])
    assert n < 1000 or clear.mean() > 0.99
    assert (labels[clear] == l_ref[clear]).all()
    assert (dist[np.arange(n), labels] <= two[:, 0] + 1e-5 * (1.0 + two[:, 0])).all()
    # update, counts and inertia for the labels the device chose (identical to the oracle's where clear)
    new_c, cnt_ref = partition.kmeans_update(x, labels, c)
    assert counts.tolist() == cnt_ref.tolist()
    np.testing.assert_allclose(c_out, new_c, rtol=0, atol=2e-6)
    np.testing.assert_allclose(inertia, dist[np.arange(n), labels].sum(), rtol=2e-6)


def test_kmeans_empty_input_duplicate_centroid_and_reproducibility(sd):
    x, _ = synth.make_sentence_vectors(4096, 384, 4, seed=1)
    c = np.ascontiguousarray(x[[0, 1, 0, 3]])                          # centroid 2 duplicates centroid 0: it never wins
    labels, c_out, counts, inertia = _run(sd, x, c)
    assert counts[2] == 0 and (labels != 2).all()
    np.testing.assert_array_equal(c_out[2], c[2])                      # an empty cluster keeps its centroid
    again = _run(sd, x, c)
    assert (again[0] == labels).all() and (again[1] == c_out).all() and again[3] == inertia      # bit-identical from run to run
    l0, c0, n0, i0 = _run(sd, x[:0], c)
    assert n0.tolist() == [0, 0, 0, 0] and i0 == 0.0
    np.testing.assert_array_equal(c0, c)


def test_kmeans_iterations_follow_the_oracle_and_rejects_unsupported_shapes(sd):
    x, task = synth.make_sentence_vectors(20000, 384, 4, seed=6, spread=0.5)
    first = [int(np.flatnonzero(task == t)[0]) for t in range(4)]
    c = np.ascontiguousarray(x[first])
    _, c_ref, hist = partition.kmeans(x, c, 5)
    cur, hist_gpu = c, []
    for _ in range(5):
        labels, cur, counts, inertia = _run(sd, x, cur)
        hist_gpu.append(inertia)
    np.testing.assert_allclose(hist_gpu, hist, rtol=1e-5)
    np.testing.assert_allclose(cur, c_ref, rtol=0, atol=1e-5)
    assert (labels == task).mean() > 0.98
    with pytest.raises(RuntimeError):
        _run(sd, np.zeros((8, 100), dtype=np.float32), np.zeros((2, 100), dtype=np.float32))      # dim not a multiple of 128
    with pytest.raises(RuntimeError):
        _run(sd, x[:64], np.ascontiguousarray(x[:9]))                                             # more than 8 clusters
