"""sd_accept against the oracle on shared p, q, x and Philox counters: decisions and emitted
tokens must be identical, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_08600_b200 import synth
from gpu_util import DEV, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sd():
    from paper_2505_08600_b200 import binding
    binding.lib()
    return binding


def _run_gpu(sd, target, q, x, T, seed, it, sid, is_logits):
    B, g1, V = target.shape
    n_acc = torch.full((B,), -9, dtype=torch.int32, device=DEV)
    out = torch.full((B, g1), -9, dtype=torch.int32, device=DEV)
    sd.sd_accept(to_dev(target), to_dev(q) if g1 > 1 else None, to_dev(x) if g1 > 1 else None, T, seed,
                 to_dev(it), to_dev(sid), n_acc, out, is_logits)
    torch.cuda.synchronize()
    return n_acc.cpu().numpy(), out.cpu().numpy()


def _make_case(B, gamma, V, sigma, seed):
    """target logits ~ N(0, 1.43^2); draft = softmax(target + N(0, sigma^2)) (the accept microbenchmark recipe)."""
    tl = synth.make_logits((B, gamma + 1, V), seed=seed, stream=1, std=1.43).astype(np.float64)
    noise = synth.make_logits((B, gamma, V), seed=seed, stream=2, std=sigma).astype(np.float64)
    p = oracle.softmax_T(tl, 1.0)
    q = oracle.softmax_T(tl[:, :gamma] + noise, 1.0)
    x = np.zeros((B, gamma), dtype=np.int32)
    for b in range(B):
        for s in range(gamma):
            x[b, s] = oracle.sample_icdf(q[b, s], oracle.uniform24(seed, b, s, 99, 0))
    return p, q, x


@pytest.mark.parametrize("B,gamma,V,sigma", [
    (4, 4, 1024, 0.5), (3, 5, 32000, 1.0), (8, 8, 32000, 0.5), (16, 5, 32000, 2.0), (5, 1, 8, 1.0),
    (2, 15, 1000, 0.25), (64, 3, 999, 0.5),
])
def test_accept_bit_exact_on_probabilities(sd, B, gamma, V, sigma):
    seed = 1000 + B * 31 + gamma
    p, q, x = _make_case(B, gamma, V, sigma, seed)
    it = (np.arange(B, dtype=np.uint32) * 7 + 3).astype(np.uint32)
    sid = (np.arange(B, dtype=np.uint32)[::-1] + 11).astype(np.uint32)
    n_gpu, out_gpu = _run_gpu(sd, p, q, x, 1.0, seed, it, sid, is_logits=0)
    for b in range(B):
        n_ref, out_ref = oracle.accept(p[b], q[b], x[b], seed, int(it[b]), int(sid[b]))
        assert n_gpu[b] == n_ref
        assert out_gpu[b].tolist() == out_ref.tolist()
    assert len(set(n_gpu.tolist())) > 1 or B < 4        # the cases exercise both accepts and rejects


def test_accept_edge_cases_bit_exact(sd):
    V, gamma, seed = 64, 3, 5
    p, q, x = _make_case(6, gamma, V, 1.0, seed)
    q[0] = p[0, :gamma]                                   # q == p: everything accepted, bonus token from p_gamma
    q[1] = 0; q[1, :, 5] = 1.0; x[1] = 5                  # one-hot draft
    p[2] = 0; p[2, :, 0:2] = 0.5; q[2] = 0; q[2, :, 2:6] = 0.25; x[2] = [2, 3, 4]     # disjoint supports
    p[3, 0] = q[3, 0]; x[3, 0] = int(np.argmax(q[3, 0]))  # first slot surely accepted
    q[4, :, :] = 0; q[4, :, 7] = 1.0; x[4] = 9            # drafts with q(x) = 0 are accepted (0 <= p)
    p[5, 1] = q[5, 1]                                      # residual of slot 1 vanishes if it is rejected (cannot be)
    it = np.arange(6, dtype=np.uint32); sid = np.zeros(6, dtype=np.uint32)
    n_gpu, out_gpu = _run_gpu(sd, p, q, x, 1.0, seed, it, sid, is_logits=0)
    for b in range(6):
        n_ref, out_ref = oracle.accept(p[b], q[b], x[b], seed, int(it[b]), 0)
        assert (n_gpu[b], out_gpu[b].tolist()) == (n_ref, out_ref.tolist()), b
    assert n_gpu[0] == gamma and n_gpu[2] == 0 and out_gpu[2, 0] in (0, 1) and n_gpu[4] == gamma


def test_accept_gamma_zero_is_plain_sampling(sd):
    V, seed = 500, 8
    p = oracle.softmax_T(synth.make_logits((4, 1, V), seed=1).astype(np.float64), 1.0)
    it = np.arange(4, dtype=np.uint32); sid = np.full(4, 2, dtype=np.uint32)
    n_gpu, out_gpu = _run_gpu(sd, p, None, None, 1.0, seed, it, sid, is_logits=0)
    for b in range(4):
        assert n_gpu[b] == 0
        assert out_gpu[b, 0] == oracle.sample_icdf(p[b, 0], oracle.uniform24(seed, b, 0, 2, 2))


def test_accept_residual_vanishes_falls_back_to_target(sd):
    # p and q differ by less than 2^-32 everywhere after a rejection: the integer residual is empty
    V, seed = 8, 3
    p = np.full((1, 2, V), 0.125, dtype=np.float32)
    q = np.full((1, 1, V), 0.125, dtype=np.float32)
    q[0, 0, 0] = np.float32(0.125) + np.float32(2.0**-26)     # q(x) slightly above p(x): rejected when u is ~1
    x = np.zeros((1, 1), dtype=np.int32)
    hits = 0
    for it in range(3000):
        n_ref, out_ref = oracle.accept(p[0], q[0], x[0], seed, it, 0)
        if n_ref == 0:
            hits += 1
            n_gpu, out_gpu = _run_gpu(sd, p, q, x, 1.0, seed, np.array([it], dtype=np.uint32), np.zeros(1, dtype=np.uint32), 0)
            assert n_gpu[0] == 0 and out_gpu[0].tolist() == out_ref.tolist()
            if hits >= 3:
                break


@pytest.mark.parametrize("T", [1.0, 0.7, 0.0])
def test_accept_from_logits_fused_softmax(sd, T):
    """With logits the kernel builds p itself in fp32; decisions agree with the oracle wherever the
    comparison is not within rounding distance, and emitted tokens are valid draws."""
    B, gamma, V, seed = 12, 5, 32000, 77
    tl = synth.make_logits((B, gamma + 1, V), seed=seed, stream=1, std=1.43)
    noise = synth.make_logits((B, gamma, V), seed=seed, stream=2, std=0.5)
    p = oracle.softmax_T(tl.astype(np.float64), T)
    q = oracle.softmax_T((tl[:, :gamma] + noise).astype(np.float64), T)
    x = np.zeros((B, gamma), dtype=np.int32)
    for b in range(B):
        for s in range(gamma):
            k = oracle.sample_icdf(q[b, s], oracle.uniform24(seed, b, s, b, 0))
            x[b, s] = k
    it = np.arange(B, dtype=np.uint32); sid = np.arange(B, dtype=np.uint32)
    n_gpu, out_gpu = _run_gpu(sd, tl, q, x, T, seed, it, sid, is_logits=1)
    agree = 0
    for b in range(B):
        n_ref, out_ref = oracle.accept(p[b], q[b], x[b], seed, b, b)
        # margin of every decision up to the oracle's stopping slot
        safe = True
        for s in range(min(n_ref + 1, gamma)):
            u = oracle.uniform24(seed, b, s, b, 1) / 2**24
            lhs, rhs = u * float(q[b, s, x[b, s]]), float(p[b, s, x[b, s]])
            if abs(lhs - rhs) <= 1e-5 * max(rhs, 1e-30):
                safe = False
        if safe:
            assert n_gpu[b] == n_ref
            assert out_gpu[b, :n_ref].tolist() == out_ref[:n_ref].tolist()
        y = int(out_gpu[b, n_gpu[b]])
        assert 0 <= y < V and (out_gpu[b, n_gpu[b] + 1:] == -1).all()
        if T == 0.0:
            assert out_gpu[b].tolist() == out_ref.tolist()
        agree += int(out_gpu[b].tolist() == out_ref.tolist())
    assert agree >= B - 2
