"""Pins of the oracle's transformer, classifier and decoding loop (CPU only)."""
import numpy as np
import pytest
import scipy.special

import oracle
from paper_2505_08600_b200 import synth

MICRO = dict(n_layers=2, d_model=64, n_heads=4, n_kv_heads=2, head_dim=16, d_ffn=96, vocab=50)
MICRO_DRAFT = dict(n_layers=1, d_model=32, n_heads=2, n_kv_heads=2, head_dim=16, d_ffn=48, vocab=50)


def _model(dims, seed=0, idx=0, dtype="f32", std=0.3):
    # a larger std than 0.02 makes attention and the FFN matter at these tiny widths
    return oracle.OracleModel(dims, synth.make_weights(dims, seed=seed, model_index=idx, dtype=dtype, std=std))


def test_cached_forward_equals_full_recompute_with_rollback():
    m = _model(MICRO)
    toks = synth.make_prompt(50, 24, seed=3)
    full = m.forward_full(toks)
    c = m.new_cache(40)
    a = c.forward(toks[:10], 0)                       # prefill chunk
    b = c.forward(toks[10:11], 10)                    # one decode step
    # speculate 5 wrong tokens, then roll back by overwriting the same positions
    c.forward(np.array([1, 2, 3, 4, 5], dtype=np.int32), 11)
    d = c.forward(toks[11:24], 11)
    got = np.concatenate([a, b, d])
    np.testing.assert_allclose(got, full, rtol=1e-9, atol=1e-10)


def test_causality_and_single_token_closed_form():
    m = _model(MICRO)
    toks = synth.make_prompt(50, 12, seed=4)
    full = m.forward_full(toks)
    toks2 = toks.copy(); toks2[8:] = (toks2[8:] + 7) % 50
    full2 = m.forward_full(toks2)
    np.testing.assert_allclose(full[:8], full2[:8], rtol=1e-12, atol=0)     # the future is invisible
    assert np.abs(full[8:] - full2[8:]).max() > 1e-3

    # one token: softmax over a single score is 1, so attention returns v whatever q and k are
    w = m.w
    f64 = lambda a: a.astype(np.float64)
    rms = lambda x: x / np.sqrt(np.mean(x * x) + 1e-5)
    h = f64(w["embed"][toks[0]])
    for l in range(MICRO["n_layers"]):
        v = f64(w["wv"][l]) @ rms(h)                                        # [n_kv*hd]
        o = np.concatenate([v[(hh // 2) * 16:(hh // 2 + 1) * 16] for hh in range(4)])   # GQA: 2 query heads per kv head
        h = h + f64(w["wo"][l]) @ o
        b = rms(h)
        g = f64(w["wg"][l]) @ b
        h = h + f64(w["wd"][l]) @ (g / (1 + np.exp(-g)) * (f64(w["wu"][l]) @ b))
    logits = f64(w["lm_head"]) @ rms(h)
    np.testing.assert_allclose(m.forward_full(toks[:1])[0], logits, rtol=1e-10, atol=1e-12)


def test_uniform_attention_special_case():
    # with Wq = 0 every score is 0, attention is the running mean of the values
    wts = synth.make_weights(MICRO, seed=1, std=0.3)
    for l in range(2):
        wts["wq"][l][:] = 0
    m = oracle.OracleModel(MICRO, wts)
    toks = synth.make_prompt(50, 7, seed=5)
    f64 = lambda a: a.astype(np.float64)
    rms = lambda x: x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + 1e-5)
    h = f64(wts["embed"][toks])                                             # [n, d]
    for l in range(2):
        v = rms(h) @ f64(wts["wv"][l]).T                                    # [n, 32]
        vm = np.cumsum(v, axis=0) / np.arange(1, 8)[:, None]
        o = np.concatenate([vm[:, (hh // 2) * 16:(hh // 2 + 1) * 16] for hh in range(4)], axis=1)
        h = h + o @ f64(wts["wo"][l]).T
        b = rms(h)
        g = b @ f64(wts["wg"][l]).T
        h = h + (scipy.special.expit(g) * g * (b @ f64(wts["wu"][l]).T)) @ f64(wts["wd"][l]).T
    np.testing.assert_allclose(m.forward_full(toks), rms(h) @ f64(wts["lm_head"]).T, rtol=1e-9, atol=1e-11)


def test_matrix_form_restatement_with_library_routines():
    # whole network through numpy matmul / scipy softmax, rotary as complex multiplication
    m = _model(MICRO, seed=2)
    w, n = m.w, 9
    toks = synth.make_prompt(50, n, seed=6)
    f64 = lambda a: a.astype(np.float64)
    rms = lambda x: x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + 1e-5)

    def rot(x, heads):                                                      # [n, heads*16]
        x = x.reshape(n, heads, 2, 8)
        z = (x[:, :, 0] + 1j * x[:, :, 1]) * np.exp(1j * np.arange(n)[:, None, None] * 10000.0 ** (-np.arange(8) / 8.0))
        return np.stack([z.real, z.imag], axis=2).reshape(n, heads * 16)

    h = f64(w["embed"][toks])
    mask = np.triu(np.full((n, n), -np.inf), 1)
    for l in range(2):
        a = rms(h)
        q, k, v = rot(a @ f64(w["wq"][l]).T, 4), rot(a @ f64(w["wk"][l]).T, 2), a @ f64(w["wv"][l]).T
        o = np.empty((n, 64))
        for hh in range(4):
            kv = hh // 2
            s = q[:, hh * 16:(hh + 1) * 16] @ k[:, kv * 16:(kv + 1) * 16].T / 4.0 + mask
            o[:, hh * 16:(hh + 1) * 16] = scipy.special.softmax(s, axis=1) @ v[:, kv * 16:(kv + 1) * 16]
        h = h + o @ f64(w["wo"][l]).T
        b = rms(h)
        g = b @ f64(w["wg"][l]).T
        h = h + (scipy.special.expit(g) * g * (b @ f64(w["wu"][l]).T)) @ f64(w["wd"][l]).T
    np.testing.assert_allclose(m.forward_full(toks), rms(h) @ f64(w["lm_head"]).T, rtol=1e-9, atol=1e-11)


def test_bf16_weights_are_the_same_values_as_their_fp32_expansion():
    wb = synth.make_weights(MICRO, seed=3, dtype="bf16", std=0.3)
    wf = {k: ([synth.bf16_bits_to_f32(a) if a.dtype == np.uint16 else a for a in v] if isinstance(v, list)
              else (synth.bf16_bits_to_f32(v) if v.dtype == np.uint16 else v)) for k, v in wb.items()}
    toks = synth.make_prompt(50, 6, seed=7)
    a = oracle.OracleModel(MICRO, wb).forward_full(toks)
    b = oracle.OracleModel(MICRO, wf).forward_full(toks)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("gamma", [1, 3, 5])
def test_greedy_speculative_equals_greedy_autoregressive(gamma):
    """T = 0: whatever the draft proposes, the output is the target's own greedy continuation."""
    t = _model(MICRO, seed=0)
    d = _model(MICRO_DRAFT, seed=0, idx=1)
    prompt = synth.make_prompt(50, 9, seed=8)
    toks, cnt, _ = oracle.spec_decode(t, d, prompt, max_new=20, gamma=gamma, T=0.0, seed=1)
    seq = list(prompt)
    for _ in range(20):                                   # independent route: full recompute + argmax
        seq.append(int(np.argmax(t.forward_full(np.array(seq, dtype=np.int32))[-1])))
    assert toks.tolist() == seq
    assert cnt["emitted"] == cnt["accepted"] + cnt["iterations"]


def test_self_draft_accepts_everything():
    # draft == target: q == p bit for bit, so every draft is accepted and tau = gamma + 1
    t = _model(MICRO, seed=0)
    d = _model(MICRO, seed=0)
    prompt = synth.make_prompt(50, 5, seed=9)
    _, cnt, tr = oracle.spec_decode(t, d, prompt, max_new=24, gamma=3, T=1.0, seed=4, trace_iters=10)
    assert cnt["accepted"] == cnt["drafted"]
    assert (tr["n_acc"] == 3).all()
    assert cnt["emitted"] / cnt["iterations"] == 4.0


def test_counters_identity_and_trace_consistency():
    t = _model(MICRO, seed=0)
    d = _model(MICRO_DRAFT, seed=0, idx=1)
    prompt = synth.make_prompt(50, 7, seed=10)
    gamma = 4
    toks, cnt, tr = oracle.spec_decode(t, d, prompt, max_new=40, gamma=gamma, T=1.0, seed=11,
                                       trace_iters=64, trace_probs=True, trace_logits=True)
    ar = cnt["accepted"] / cnt["drafted"]                 # Eq. 2
    tau = cnt["emitted"] / cnt["iterations"]
    assert abs(tau - (1 + gamma * ar)) < 1e-12
    assert len(toks) == 7 + 40
    # replay: the trace's tokens rebuild the sequence, and each iteration's accept is reproducible
    seq = list(prompt)
    for it in range(len(tr["n_acc"])):
        assert tr["len_before"][it] == len(seq)
        n, out = oracle.accept(tr["p"][it], tr["q"][it], tr["x"][it], seed=11, it=it, seq=0)
        assert n == tr["n_acc"][it]
        assert out[: n + 1].tolist() == tr["out_tok"][it][: n + 1].tolist()
        # the verify rows are the target's logits for [last token, drafts] given the history
        rows = np.array(seq + list(tr["x"][it]), dtype=np.int32)
        full = t.forward_full(rows)[len(seq) - 1:]
        np.testing.assert_allclose(tr["logits"][it], full, rtol=1e-8, atol=1e-9)
        seq += out[: n + 1].tolist()
    assert seq[: len(toks)] == toks.tolist()
    # the run's estimate of Eq. 1's alpha: sum over judged slots (s <= min(n, gamma - 1)) of sum_k min(p_s, q_s)
    a_sum, judged = 0.0, 0
    for it in range(len(tr["n_acc"])):
        n = int(tr["n_acc"][it])
        terms = np.minimum(tr["p"][it][:gamma].astype(np.float64), tr["q"][it].astype(np.float64)).sum(axis=1)
        a_sum += float(terms[: min(n + 1, gamma)].sum())
        judged += min(n + 1, gamma)
    assert tr["judged"] == judged
    assert abs(tr["alpha_sum"] - a_sum) < 1e-9


def test_route_prompt_mlp_and_forced_task():
    wts = synth.make_weights(MICRO, seed=0, std=0.3)
    clf = synth.make_classifier(64, 16, 3, seed=0)
    toks = synth.make_prompt(50, 11, seed=12)
    k, probs = oracle.route_prompt(wts["embed"], toks, clf["w1"], clf["b1"], clf["w2"], clf["b2"])
    e = wts["embed"][toks].astype(np.float64).mean(axis=0)
    z = np.maximum(clf["w1"].astype(np.float64) @ e + clf["b1"], 0)
    o = clf["w2"].astype(np.float64) @ z + clf["b2"]
    assert k == int(np.argmax(o))
    np.testing.assert_allclose(probs, scipy.special.softmax(o), rtol=1e-10)
    # Sec. 2.1: an explicit task type goes straight to that draft
    k2, _ = oracle.route_prompt(wts["embed"], toks, clf["w1"], clf["b1"], clf["w2"], clf["b2"], forced_task=2)
    assert k2 == 2
