"""Pins of the Mamba classifier oracle against closed forms, brute force and library routines."""
import numpy as np
import pytest

from oracle import classifier_mamba as om
from paper_2505_08600_b200 import synth


def test_scan_with_constant_inputs_is_a_geometric_series():
    # dt, A, B, C, v constant: h_t = b (1 - a^(t+1)) / (1 - a) with a = exp(dt A), b = dt v B
    P, Di, N = 40, 3, 2
    dt = np.full((P, Di), 0.3); v = np.tile([1.0, -2.0, 0.5], (P, 1))
    A = -np.array([[1.0, 2.0], [0.5, 3.0], [1.5, 0.1]])
    B = np.tile([0.7, -0.2], (P, 1)); C = np.tile([1.1, 0.4], (P, 1)); D = np.array([0.0, 1.0, -1.0])
    y = om.selective_scan(v, dt, A, B, C, D)
    a = np.exp(0.3 * A)
    for t in range(P):
        h = (0.3 * v[0])[:, None] * B[0][None, :] * (1 - a ** (t + 1)) / (1 - a)
        np.testing.assert_allclose(y[t], h @ C[0] + D * v[0], rtol=1e-12)


def test_scan_against_the_unrolled_sum_on_tiny_inputs():
    # y_t = sum_{s<=t} C_t . (prod_{r=s+1..t} exp(dt_r A)) (dt_s v_s B_s)  +  D v_t, written out with plain loops
    rng = np.random.default_rng(3)
    P, Di, N = 7, 2, 3
    v, dt = rng.standard_normal((P, Di)), rng.random((P, Di)) * 0.5 + 0.01
    A, B, C, D = -rng.random((Di, N)) * 2, rng.standard_normal((P, N)), rng.standard_normal((P, N)), rng.standard_normal(Di)
    y = om.selective_scan(v, dt, A, B, C, D)
    for t in range(P):
        for c in range(Di):
            tot = D[c] * v[t, c]
            for n in range(N):
                for s in range(t + 1):
                    decay = 1.0
                    for r in range(s + 1, t + 1):
                        decay *= np.exp(dt[r, c] * A[c, n])
                    tot += C[t, n] * decay * dt[s, c] * v[s, c] * B[s, n]
            assert abs(y[t, c] - tot) < 1e-12


def test_causal_convolution_against_numpy_convolve():
    rng = np.random.default_rng(1)
    u, w, b = rng.standard_normal((30, 4)), rng.standard_normal((4, 4)), rng.standard_normal(4)
    out = om.causal_depthwise_conv(u, w, b)
    for c in range(4):      # correlation with the taps = convolution with the reversed taps, first P outputs
        ref = np.convolve(u[:, c], w[c][::-1])[:30] + b[c]
        np.testing.assert_allclose(out[:, c], ref, rtol=1e-12, atol=1e-12)


def test_activations_against_library_routines():
    from scipy.special import expit, log1p
    x = np.linspace(-40, 40, 401)
    np.testing.assert_allclose(om.silu(x), x * expit(x), rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(om.softplus(x), np.logaddexp(0.0, x), rtol=1e-12)


def _weights(**kw):
    return synth.make_mamba_classifier(vocab=200, d_model=32, d_state=4, d_conv=4, expand=2, n_classes=3, seed=5, **kw)


def test_layer_is_causal_and_the_pool_is_the_mean_of_the_per_token_outputs():
    w = _weights()
    toks = synth.make_prompt(200, 24, seed=2)
    scores, pooled, o = om.forward(w, toks)
    np.testing.assert_allclose(pooled, o.mean(axis=0), rtol=1e-13)
    np.testing.assert_allclose(scores, w["w_fc"].astype(np.float64) @ pooled + w["b_fc"], rtol=1e-13)
    t2 = toks.copy(); t2[17] = (t2[17] + 1) % 200
    _, _, o2 = om.forward(w, t2)
    np.testing.assert_array_equal(o[:17], o2[:17])                    # nothing before the changed token moves
    assert np.abs(o[17:] - o2[17:]).max() > 0
    _, _, o3 = om.forward(w, toks[:10])                               # a prefix of the prompt gives the prefix of the outputs
    np.testing.assert_allclose(o3, o[:10], rtol=1e-12, atol=1e-15)


def test_without_state_input_the_layer_is_the_gated_skip_path():
    # B = 0 (zero rows of W_x for B): h stays 0, so y_t = D v_t and o_t = W_out (D v_t silu(z_t))
    w = _weights()
    R, N = w["w_dt"].shape[1], w["a_log"].shape[1]
    w["w_x"] = w["w_x"].copy(); w["w_x"][R:R + N] = 0.0
    toks = synth.make_prompt(200, 12, seed=4)
    _, _, o = om.forward(w, toks)
    f = {k: np.asarray(a, dtype=np.float64) for k, a in w.items()}
    Di = f["w_dt"].shape[0]
    uz = f["embed"][toks] @ f["w_in"].T
    v = om.silu(om.causal_depthwise_conv(uz[:, :Di], f["w_conv"], f["b_conv"]))
    ref = (f["d_skip"] * v * om.silu(uz[:, Di:])) @ f["w_out"].T
    np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-15)


def test_single_token_prompt_written_out():
    w = _weights()
    f = {k: np.asarray(a, dtype=np.float64) for k, a in w.items()}
    Di, R = f["w_dt"].shape; N = f["a_log"].shape[1]
    tok = 7
    uz = f["w_in"] @ f["embed"][tok]
    v = om.silu(f["b_conv"] + f["w_conv"][:, -1] * uz[:Di])            # only the last tap sees the token
    xd = f["w_x"] @ v
    dt = np.log1p(np.exp(f["w_dt"] @ xd[:R] + f["b_dt"]))
    h = (dt * v)[:, None] * xd[R:R + N][None, :]                       # h_{-1} = 0: the decay term vanishes
    y = h @ xd[R + N:] + f["d_skip"] * v
    o = f["w_out"] @ (y * om.silu(uz[Di:]))
    scores, pooled, _ = om.forward(w, [tok])
    np.testing.assert_allclose(pooled, o, rtol=1e-12)
    assert om.classify(w, [tok])[0] == int(np.argmax(f["w_fc"] @ o + f["b_fc"]))
