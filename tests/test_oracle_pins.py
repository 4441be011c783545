"""Pins of the CPU oracle against what the paper and the mathematics fix (CPU only)."""
import math
from fractions import Fraction

import numpy as np
import pytest
import scipy.special
import scipy.stats

import oracle
from paper_2505_08600_b200 import synth


# ----------------------------------------------------------------------------
# Philox4x32-10: published known-answer vectors
# ----------------------------------------------------------------------------
def test_philox_known_answers(golden_dir):
    rows = [l.split() for l in open(f"{golden_dir}/philox4x32_10_kat.txt") if not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(t, 16) for t in r]
        out = oracle.philox4x32_10(v[:4], v[4:6])
        assert [int(o) for o in out] == v[6:]


def test_uniform24_range_and_layout():
    # u_int = (word0 >> 8) + 1 of Philox(counter=(iter, slot, seq, purpose), key=seed)
    seed = 0x0123456789ABCDEF
    for it, slot, seq, purpose in [(0, 0, 0, 0), (7, 3, 2, 1), (2**32 - 1, 5, 9, 2)]:
        w = oracle.philox4x32_10([it, slot, seq, purpose], [seed & 0xFFFFFFFF, seed >> 32])
        assert oracle.uniform24(seed, it, slot, seq, purpose) == (int(w[0]) >> 8) + 1
    us = np.array([oracle.uniform24(5, i, 0, 0, 1) for i in range(20000)])
    assert us.min() >= 1 and us.max() <= 2**24
    assert abs(us.mean() / 2**24 - 0.5) < 0.01


# ----------------------------------------------------------------------------
# Sampler: exact inverse CDF (brute force with rationals on tiny vocabularies)
# ----------------------------------------------------------------------------
def _exact_token(w, u_int):
    wi = [int(Fraction(float(x)) * 2**32) for x in w]     # floor of the exact product
    tot = sum(wi)
    if tot == 0:
        return -1
    u = Fraction(u_int, 2**24)
    run = 0
    for k, x in enumerate(wi):
        run += x
        if Fraction(run, tot) >= u:
            return k
    raise AssertionError


def test_sampler_matches_exact_inverse_cdf():
    rng = np.random.default_rng(0)
    for trial in range(40):
        V = int(rng.integers(1, 9))
        w = rng.random(V).astype(np.float32)
        w[rng.random(V) < 0.3] = 0.0
        if trial % 5 == 0:
            w = (w / max(w.sum(), 1e-9)).astype(np.float32)
        for u_int in [1, 2, 2**24, 2**24 - 1, 2**23] + [int(x) for x in rng.integers(1, 2**24 + 1, 30)]:
            assert oracle.sample_icdf(w, u_int) == _exact_token(w, u_int)


def test_sampler_strata_sizes_exact():
    # token k owns exactly floor(C_k 2^24 / tot) - floor(C_{k-1} 2^24 / tot) of the 2^24 values of u_int
    w = np.array([0.5, 0.0, 0.25, 0.125, 0.0625, 0.0625], dtype=np.float32)
    wi = [int(Fraction(float(x)) * 2**32) for x in w]
    tot, run, lo = sum(wi), 0, 0
    for k, x in enumerate(wi):
        run += x
        hi = (run * 2**24) // tot          # last u_int that maps to a token <= k
        if x == 0:
            assert hi == lo                 # zero-weight tokens own nothing
            continue
        assert oracle.sample_icdf(w, lo + 1) == k
        assert oracle.sample_icdf(w, hi) == k
        if hi < 2**24:
            assert oracle.sample_icdf(w, hi + 1) > k
        lo = hi
    assert lo == 2**24
    assert oracle.sample_icdf(np.zeros(4, dtype=np.float32), 17) == -1


# ----------------------------------------------------------------------------
# Softmax with temperature
# ----------------------------------------------------------------------------
def test_softmax_properties():
    rng = np.random.default_rng(1)
    l = rng.standard_normal(50) * 3
    for T in (0.7, 1.0, 2.0):
        p = oracle.softmax_T(l, T).astype(np.float64)
        assert abs(p.sum() - 1) < 1e-6
        np.testing.assert_allclose(p, oracle.softmax_T(l + 123.0, T), rtol=1e-6)     # shift invariance
        np.testing.assert_allclose(p, scipy.special.softmax(l / T), rtol=1e-6, atol=1e-9)
        # ratio law: p_i / p_j = exp((l_i - l_j) / T)
        assert abs(p[3] / p[7] - math.exp((l[3] - l[7]) / T)) < 1e-5 * p[3] / p[7]
    two = oracle.softmax_T(np.array([0.3, -1.1]), 0.5)
    assert abs(two[0] - 1 / (1 + math.exp(-(0.3 + 1.1) / 0.5))) < 1e-7      # logistic closed form
    g = oracle.softmax_T(np.array([1.0, 5.0, 5.0, 2.0]), 0.0)
    assert g.tolist() == [0, 1, 0, 0]                                           # greedy, lowest index on ties


# ----------------------------------------------------------------------------
# Accept rule
# ----------------------------------------------------------------------------
P06 = np.array([0.525, 0.125, 0.1, 0.1, 0.05, 0.05, 0.025, 0.025], dtype=np.float32)
P08 = np.array([0.325, 0.125, 0.125, 0.125, 0.1, 0.1, 0.05, 0.05], dtype=np.float32)
QU = np.full(8, 0.125, dtype=np.float32)


def test_alpha_of_fixtures():
    assert abs(float(np.minimum(P06, QU).sum()) - 0.6) < 1e-6
    assert abs(float(np.minimum(P08, QU).sum()) - 0.8) < 1e-6


def test_alpha_terms_closed_forms():
    """Eq. 1's alpha for one slot, sum_k min(p(k), q(k)): exact values on the fixtures, 1 for q == p, 0 for disjoint supports,
    symmetric in its arguments, one value per slot."""
    p = np.stack([P06, P08, QU, P06])
    q = np.stack([QU, QU, QU])
    np.testing.assert_allclose(oracle.alpha_terms(p, q), [0.6, 0.8, 1.0], atol=1e-7)
    a = np.array([[0.5, 0.5, 0, 0, 0, 0, 0, 0]], dtype=np.float32)
    b = np.array([[0, 0, 0.25, 0.75, 0, 0, 0, 0]], dtype=np.float32)
    assert oracle.alpha_terms(a, b).tolist() == [0.0]
    np.testing.assert_allclose(oracle.alpha_terms(P06[None], P08[None]), oracle.alpha_terms(P08[None], P06[None]), atol=0)
    # 1 - total variation distance
    np.testing.assert_allclose(oracle.alpha_terms(P06[None], P08[None]), [1.0 - 0.5 * np.abs(P06.astype(np.float64) - P08).sum()], atol=1e-7)


@pytest.mark.parametrize("alpha,p", [(0.6, P06), (0.8, P08)])
def test_alpha_is_the_acceptance_frequency_of_judged_slots(alpha, p):
    """What the sum of minima estimates is the frequency with which a judged slot is accepted: slot s is judged iff all
    slots before it were accepted, so an iteration with n accepts judges min(n + 1, gamma) slots."""
    gamma, iters = 4, 400_000
    emitted, accepted, _ = oracle.mc_fixed(p, QU, gamma, iters, seed=99)
    # judged = sum over iterations of min(n + 1, gamma) = emitted - (iterations that accepted everything)
    # P(n = gamma) = alpha^gamma, so E[judged] = E[n + 1] - alpha^gamma
    judged_expect = iters * ((1 - alpha ** (gamma + 1)) / (1 - alpha) - alpha ** gamma)
    freq = accepted / judged_expect
    se = math.sqrt(alpha * (1 - alpha) / judged_expect) * 2     # judged is itself random: generous
    assert abs(freq - alpha) < 4 * se + 2e-3, (freq, alpha)
    assert abs(float(oracle.alpha_terms(p[None], QU[None])[0]) - alpha) < 1e-6


@pytest.mark.parametrize("alpha,p", [(0.6, P06), (0.8, P08)])
@pytest.mark.parametrize("gamma", [1, 2, 3, 4, 5, 6, 7, 8])
def test_eq1_expected_tokens_monte_carlo(alpha, p, gamma):
    """Eq. 1: expected tokens per iteration (1 - a^(g+1)) / (1 - a); speedup divides by (g c + 1)."""
    iters = 1_000_000 if gamma == 5 else 250_000
    emitted, accepted, _ = oracle.mc_fixed(p, QU, gamma, iters, seed=1234 + gamma)
    mean = emitted / iters
    expect = (1 - alpha ** (gamma + 1)) / (1 - alpha)
    # variance of the truncated geometric count, bounded by that of the untruncated one
    se = math.sqrt(alpha / (1 - alpha) ** 2 / iters)
    assert abs(mean - expect) < 4 * se, (mean, expect, se)
    for c in (0.02, 0.11):
        modelled = mean / (gamma * c + 1)            # walltime model: one target pass = 1, one draft pass = c
        eq1 = (1 - alpha ** (gamma + 1)) / ((1 - alpha) * (gamma * c + 1))
        assert abs(modelled - eq1) < 4 * se
    assert emitted == iters + accepted              # tokens = accepted drafts + one corrected/bonus token


def test_q_equal_p_accepts_everything():
    rng = np.random.default_rng(2)
    V, gamma = 64, 6
    for trial in range(200):
        p = oracle.softmax_T(rng.standard_normal((gamma + 1, V)) * 2, 1.0)
        q = p[:gamma].copy()
        x = rng.integers(0, V, gamma).astype(np.int32)
        n, out = oracle.accept(p, q, x, seed=trial, it=trial * 7, seq=3)
        assert n == gamma
        assert out[:gamma].tolist() == x.tolist()
        assert 0 <= out[gamma] < V


def test_zero_target_probability_never_accepted_and_zero_draft_probability_always():
    V, gamma = 8, 1
    p = np.zeros((2, V), dtype=np.float32); p[:, 0] = 1.0
    q = np.zeros((1, V), dtype=np.float32); q[0, 1] = 1.0
    for it in range(100):
        n, out = oracle.accept(p, q, np.array([1], dtype=np.int32), seed=9, it=it, seq=0)
        assert n == 0 and out[0] == 0            # p(x) = 0 < u q(x): reject, residual is one-hot at 0
        n, out = oracle.accept(p, q, np.array([0], dtype=np.int32), seed=9, it=it, seq=0)
        assert n == 1                             # q(x) = 0: 0 <= p(x) holds


CHI2_CASES = [
    (P06, QU),
    (P08, QU),
    (np.array([0.5, 0.5, 0, 0, 0, 0, 0, 0], dtype=np.float32), np.array([0, 0, 0.25, 0.25, 0.25, 0.25, 0, 0], dtype=np.float32)),
    (P06, np.array([0, 0, 0, 1, 0, 0, 0, 0], dtype=np.float32)),
    (QU, P06),
]


@pytest.mark.parametrize("case", range(len(CHI2_CASES)))
def test_first_emitted_token_follows_target_distribution(case):
    """Defining property of the cited verification rule: the output law equals p."""
    p, q = CHI2_CASES[case]
    iters = 1_000_000
    _, _, hist = oracle.mc_fixed(p, q, gamma=3, iters=iters, seed=77 + case)
    assert hist.sum() == iters
    support = p > 0
    assert hist[~support].sum() == 0
    expected = p[support].astype(np.float64) / p[support].sum() * iters
    chi2 = float(((hist[support] - expected) ** 2 / expected).sum())
    dof = int(support.sum()) - 1
    assert chi2 < scipy.stats.chi2.ppf(0.999, dof), (chi2, hist)


def test_chi_square_test_has_power():
    # a planted mistake (resampling from p instead of the residual) must fail the same test
    p, q = P06, QU
    rng = np.random.default_rng(5)
    iters = 200_000
    x = rng.choice(8, size=iters, p=q.astype(np.float64) / q.astype(np.float64).sum())
    acc = rng.random(iters) * q[x] <= p[x]
    y = np.where(acc, x, rng.choice(8, size=iters, p=p.astype(np.float64) / p.astype(np.float64).sum()))
    hist = np.bincount(y, minlength=8)
    expected = p.astype(np.float64) * iters
    assert float(((hist - expected) ** 2 / expected).sum()) > scipy.stats.chi2.ppf(0.999, 7)


# ----------------------------------------------------------------------------
# Metric definitions: Eq. 2 and tau, pinned by Table 1
# ----------------------------------------------------------------------------
def test_table1_fixes_tau_includes_bonus_token(golden_dir):
    rows = [l.split() for l in open(f"{golden_dir}/table1_acceptance.txt") if not l.startswith("#")]
    assert len(rows) == 16
    for g, _, _, ar, tau in rows:
        g, ar, tau = int(g), float(ar), float(tau)
        assert abs(tau - (1 + g * ar)) <= g * 0.005 + 0.005 + 1e-9      # printed to two decimals
        assert abs(tau - g * ar) > 0.5                                   # the other reading fails


# ----------------------------------------------------------------------------
# Primitives: closed forms and invariants
# ----------------------------------------------------------------------------
def test_rmsnorm_rope_silu_closed_forms():
    L = oracle.lib()
    rng = np.random.default_rng(3)
    x = rng.standard_normal(96)
    g = (rng.random(96) + 0.5).astype(np.float32)
    y = np.empty(96)
    L.orc_rmsnorm(x.ctypes.data, g.ctypes.data, 96, 0.0, y.ctypes.data)
    assert abs(np.mean((y / g) ** 2) - 1) < 1e-12                       # unit mean square before the gain
    y2 = np.empty(96)
    L.orc_rmsnorm((5 * x).ctypes.data, g.ctypes.data, 96, 0.0, y2.ctypes.data)
    np.testing.assert_allclose(y, y2, rtol=1e-12)                         # scale invariance
    L.orc_rmsnorm(x.ctypes.data, g.ctypes.data, 96, 1e-5, y2.ctypes.data)
    np.testing.assert_allclose(y2, x * g / math.sqrt(np.mean(x * x) + 1e-5), rtol=1e-12)

    v = np.array([1.0, 0.0]); L.orc_rope(v.ctypes.data, 1, 2, 1, 10000.0)
    np.testing.assert_allclose(v, [math.cos(1), math.sin(1)], atol=1e-15)  # head_dim 2: angle = pos
    v = np.array([1.0, 2.0, 0.0, 0.0]); L.orc_rope(v.ctypes.data, 1, 4, 3, 10000.0)
    th1 = 3 * 10000.0 ** (-2 / 4)                                          # pair (1, 3) turns by pos * base^(-2/4)
    np.testing.assert_allclose(v, [math.cos(3), 2 * math.cos(th1), math.sin(3), 2 * math.sin(th1)], atol=1e-14)
    a = rng.standard_normal(2 * 64); b = rng.standard_normal(2 * 64)
    def rot(z, pos):
        z = z.copy(); L.orc_rope(z.ctypes.data, 2, 64, pos, 10000.0); return z
    np.testing.assert_allclose(rot(a, 0), a, atol=0)                       # position 0 is the identity
    assert abs(np.linalg.norm(rot(a, 17)) - np.linalg.norm(a)) < 1e-12     # rotation keeps norms
    d1 = float(rot(a, 9) @ rot(b, 4)); d2 = float(rot(a, 105) @ rot(b, 100))
    assert abs(d1 - d2) < 1e-10                                            # only the offset matters

    assert L.orc_silu(0.0) == 0.0
    for z in (0.3, 2.0, 11.0):
        assert abs(L.orc_silu(z) - L.orc_silu(-z) - z) < 1e-12
        assert abs(L.orc_silu(z) - z / (1 + math.exp(-z))) < 1e-15
    assert abs(L.orc_silu(40.0) - 40.0) < 1e-12


def test_linear_against_library_matmul_both_dtypes():
    rng = np.random.default_rng(4)
    W = (rng.standard_normal((37, 53)) * 0.1).astype(np.float32)
    X = rng.standard_normal((5, 53))
    Y = np.empty((5, 37))
    oracle.lib().orc_linear(W.ctypes.data, 0, 37, 53, X.ctypes.data, 5, Y.ctypes.data)
    np.testing.assert_allclose(Y, X @ W.astype(np.float64).T, rtol=1e-12, atol=1e-13)
    Wb = synth.f32_to_bf16_bits(W)
    oracle.lib().orc_linear(Wb.ctypes.data, 1, 37, 53, X.ctypes.data, 5, Y.ctypes.data)
    np.testing.assert_allclose(Y, X @ synth.bf16_bits_to_f32(Wb).astype(np.float64).T, rtol=1e-12, atol=1e-13)
    # bf16 bit patterns widen exactly: 0x3F80 is 1.0, 0xC000 is -2.0
    one = np.array([[0x3F80, 0xC000]], dtype=np.uint16); x = np.array([[3.0, 0.5]]); y = np.empty((1, 1))
    oracle.lib().orc_linear(one.ctypes.data, 1, 1, 2, x.ctypes.data, 1, y.ctypes.data)
    assert y[0, 0] == 2.0


def test_attention_head_against_library_softmax():
    rng = np.random.default_rng(6)
    q = rng.standard_normal(32); K = rng.standard_normal((19, 32)); V = rng.standard_normal((19, 32))
    ref = scipy.special.softmax(K @ q / math.sqrt(32)) @ V
    np.testing.assert_allclose(oracle.attention_head(q, K, V), ref, rtol=1e-12, atol=1e-14)
    # one position: the value itself; identical keys: the mean of the values
    np.testing.assert_allclose(oracle.attention_head(q, K[:1], V[:1]), V[0], atol=1e-15)
    np.testing.assert_allclose(oracle.attention_head(q, np.tile(K[:1], (5, 1)), V[:5]), V[:5].mean(axis=0), atol=1e-14)
