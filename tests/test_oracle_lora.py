"""Pins of the low-rank adapter oracle: the merged matrix against the factored product through a library matmul."""
import numpy as np

import oracle
from oracle import lora
from paper_2505_08600_b200 import synth

DIMS = dict(n_layers=2, d_model=64, n_heads=2, n_kv_heads=1, head_dim=32, d_ffn=96, vocab=50)


def test_merged_matrix_equals_base_plus_factored_update_applied_to_vectors():
    rng = np.random.default_rng(0)
    w, a, b = rng.standard_normal((24, 40)), rng.standard_normal((4, 40)), rng.standard_normal((24, 4))
    x = rng.standard_normal((5, 40))
    merged = lora.adapted_matrix(w, a, b, 0.5)
    np.testing.assert_allclose(x @ merged.T, x @ w.T + 0.5 * (x @ a.T) @ b.T, rtol=1e-12, atol=1e-12)
    np.testing.assert_array_equal(lora.adapted_matrix(w, a, np.zeros_like(b), 3.0), w)       # B = 0: the base matrix
    assert np.linalg.matrix_rank(merged - w) == 4                                              # the update has rank r


def test_bf16_factors_enter_with_their_exact_values_and_zero_adapter_is_the_base_model():
    base = synth.make_weights(DIMS, seed=0, model_index=1, dtype="bf16")
    ad = synth.make_lora(DIMS, 8, task=0, seed=0)
    a, b = ad["wo"][1]
    m = lora.merged_weights(DIMS, base, ad, 2.0)
    ref = synth.bf16_bits_to_f32(base["wo"][1]).astype(np.float64) + 2.0 * synth.bf16_bits_to_f32(b).astype(np.float64) @ synth.bf16_bits_to_f32(a).astype(np.float64)
    np.testing.assert_allclose(m["wo"][1], ref, rtol=1e-7)
    # the stacked matrices share one A: the key rows of the update are B's key rows times A
    a, b = ad["qkv"][0]
    dq, dkv = 64, 32
    ref_k = synth.bf16_bits_to_f32(base["wk"][0]).astype(np.float64) + 2.0 * synth.bf16_bits_to_f32(b[dq:dq + dkv]).astype(np.float64) @ synth.bf16_bits_to_f32(a).astype(np.float64)
    np.testing.assert_allclose(m["wk"][0], ref_k, rtol=1e-7)
    zero = {k: None for k in ("qkv", "wo", "gu", "wd")}
    m0 = lora.merged_weights(DIMS, base, zero, 2.0)
    toks = synth.make_prompt(50, 9, seed=1)
    l_base = oracle.OracleModel(DIMS, base).forward_full(toks)
    l_zero = oracle.OracleModel(DIMS, m0).forward_full(toks)
    np.testing.assert_allclose(l_zero, l_base, rtol=0, atol=1e-12)
    l_ad = oracle.OracleModel(DIMS, m).forward_full(toks)
    assert np.abs(l_ad - l_base).max() > 1e-3                                                  # an adapter changes the model


def test_scale_is_linear_in_the_update():
    base = synth.make_weights(DIMS, seed=0, model_index=1, dtype="f32")
    ad = synth.make_lora(DIMS, 8, task=1, seed=0, dtype="f32")
    m1, m2 = lora.merged_weights(DIMS, base, ad, 1.0), lora.merged_weights(DIMS, base, ad, 2.0)
    np.testing.assert_allclose(m2["wg"][0].astype(np.float64) - base["wg"][0], 2.0 * (m1["wg"][0].astype(np.float64) - base["wg"][0]), atol=1e-6)
