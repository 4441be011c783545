"""End-to-end parity of the CUDA path against the CPU oracle, teacher-forced: the oracle runs the
whole speculative-decoding loop on its own, then the library replays every iteration on the
oracle's token history and each intermediate result is compared."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_08600_b200 import synth
from gpu_util import DEV

pytestmark = pytest.mark.gpu

# tolerances of the float comparisons
TOL = {
    "f32": dict(logits=2e-3, probs=1e-4),     # fp32 storage, fp32 accumulation in another order
    "bf16": dict(logits=5e-2, probs=1e-3),    # bf16 activations / KV against the fp64 oracle
}


@pytest.fixture(scope="module")
def sd():
    from paper_2505_08600_b200 import binding
    binding.lib()
    return binding


def _build(sd, target_dims, draft_dims_list, dtype, T, seed, max_seqs=2, max_ctx=160, max_gamma=8, clf_hidden=0, std=0.02):
    ctx = sd.Context(target_dims, draft_dims_list, dtype, max_seqs, max_ctx, max_gamma, T, seed, clf_d_hidden=clf_hidden)
    wt = synth.make_weights(target_dims, seed=0, model_index=0, dtype=dtype, std=std)
    ctx.load_weights(0, wt)
    omodels = [oracle.OracleModel(target_dims, wt)]
    for i, dd in enumerate(draft_dims_list):
        wd = synth.make_weights(dd, seed=0, model_index=1 + i, dtype=dtype, std=std)
        ctx.load_weights(1 + i, wd)
        omodels.append(oracle.OracleModel(dd, wd))
    return ctx, omodels


def _replay(sd, ctx, omodels, draft_k, prompt, gamma, T, seed, max_new, dtype, seq=0, seq_id=0, min_agree=0.8, tol_logits=None):
    tol = dict(TOL[dtype], logits=tol_logits) if tol_logits is not None else TOL[dtype]
    V = omodels[0].dims["vocab"]
    toks_ref, cnt_ref, tr = oracle.spec_decode(omodels[0], omodels[1 + draft_k], prompt, max_new, gamma, T, seed,
                                               seq_id=seq_id, trace_iters=max_new, trace_probs=True, trace_logits=True)
    ctx.sd_seq_begin(seq, prompt, seq_id)
    assert ctx.sd_route_prompt([seq], forced_task=[draft_k]).tolist() == [draft_k]
    ctx.sd_prefill([seq])
    x_forced = torch.zeros((1, gamma), dtype=torch.int32, device=DEV)
    x_samp = torch.zeros((1, gamma), dtype=torch.int32, device=DEV)
    q = torch.zeros((1, gamma, V), dtype=torch.float32, device=DEV)
    logits = torch.zeros((1, gamma + 1, V), dtype=torch.float32, device=DEV)
    n_acc = torch.zeros((1,), dtype=torch.int32, device=DEV)
    out_tok = torch.zeros((1, gamma + 1), dtype=torch.int32, device=DEV)
    n_it = len(tr["n_acc"])
    agree_x = agree_acc = 0
    worst_logit = worst_p = worst_q = 0.0
    for it in range(n_it):
        x_forced.copy_(torch.from_numpy(tr["x"][it:it + 1]))
        ctx.sd_draft_steps_replay([seq], gamma, x_forced, x_samp, q)
        ctx.sd_verify([seq], gamma, x_forced, logits)
        ctx.sd_accept_seqs([seq], gamma, logits, q, x_forced, n_acc, out_tok)
        q_gpu = q.cpu().numpy()[0]
        l_gpu = logits.cpu().numpy()[0].astype(np.float64)
        if T > 0:
            worst_q = max(worst_q, float(np.abs(q_gpu.astype(np.float64) - tr["q"][it]).max()))
        else:      # greedy: q is one-hot; a near-tie of the draft's top two logits may flip it (counted below)
            assert ((q_gpu == 0) | (q_gpu == 1)).all() and (q_gpu.sum(axis=1) == 1).all()
        worst_logit = max(worst_logit, float(np.abs(l_gpu - tr["logits"][it]).max()))
        if T > 0:
            p_gpu = torch.softmax(logits[0].double() / T, dim=-1).cpu().numpy()
            worst_p = max(worst_p, float(np.abs(p_gpu - tr["p"][it]).max()))
        else:      # greedy verification: same argmax wherever the oracle's top-2 margin is clear
            for j in range(gamma + 1):
                top2 = np.sort(tr["logits"][it][j])[-2:]
                if top2[1] - top2[0] > 2 * tol["logits"]:
                    assert int(np.argmax(l_gpu[j])) == int(np.argmax(tr["logits"][it][j]))
        agree_x += int(x_samp.cpu().numpy()[0].tolist() == tr["x"][it].tolist())
        n_g, o_g = int(n_acc.item()), out_tok.cpu().numpy()[0]
        agree_acc += int(n_g == tr["n_acc"][it] and o_g.tolist() == tr["out_tok"][it].tolist())
        assert 0 <= n_g <= gamma and 0 <= o_g[n_g] < V and (o_g[n_g + 1:] == -1).all()
        # commit the ORACLE's outcome so that the next iteration starts from its history
        n_acc.copy_(torch.from_numpy(tr["n_acc"][it:it + 1]))
        fix = tr["out_tok"][it:it + 1].copy()
        out_tok.copy_(torch.from_numpy(fix))
        ctx.sd_kv_rollback([seq], gamma, n_acc, out_tok)
        got, cnt = ctx.sd_seq_read(seq)
        L = int(tr["len_before"][it]) + int(tr["n_acc"][it]) + 1
        assert len(got) == L
        assert got.tolist() == toks_ref_full(tr, prompt, it)
    assert worst_logit <= tol["logits"], worst_logit
    assert worst_q <= tol["probs"], worst_q
    assert worst_p <= tol["probs"], worst_p
    assert ctx.sd_device_status() == 0
    got, cnt = ctx.sd_seq_read(seq)
    assert cnt == {k: int(v) for k, v in cnt_ref.items()}
    assert got[: len(toks_ref)].tolist() == toks_ref.tolist()
    assert agree_x >= min_agree * n_it, (agree_x, n_it)
    assert agree_acc >= min_agree * n_it, (agree_acc, n_it)
    # estimate of Eq. 1's alpha: the judged slots are the oracle's (its n_acc was committed), their sums of min(p, q) the GPU's
    a_sum, judged = ctx.sd_seq_alpha(seq)
    assert judged == tr["judged"]
    if T > 0:       # |sum min(p,q) - sum min(p',q')| <= |p-p'|_1 + |q-q'|_1, each at most about 2 * (logit error) / T
        assert abs(a_sum - tr["alpha_sum"]) <= judged * 4.0 * tol["logits"] / T, (a_sum, tr["alpha_sum"], judged)
    return dict(alpha_sum=a_sum, judged=judged, alpha_ref=tr["alpha_sum"] / max(1, tr["judged"]),
                iters=n_it, agree_x=agree_x, agree_acc=agree_acc, logit=worst_logit, p=worst_p, q=worst_q)


def toks_ref_full(tr, prompt, it):
    seq = list(prompt)
    for i in range(it + 1):
        n = int(tr["n_acc"][i])
        seq += tr["out_tok"][i][: n + 1].tolist()
    return seq


@pytest.mark.parametrize("T", [1.0, 0.0])
def test_tiny_config_teacher_forced(sd, T):
    cfg = synth.CONFIGS["tiny"]
    wl = cfg["workload"]
    ctx, om = _build(sd, cfg["target"], cfg["drafts"], "f32", T, wl["seed"], max_ctx=wl["max_ctx"])
    prompt = synth.make_prompt(cfg["target"]["vocab"], wl["prompt"], seed=wl["seed"])
    r = _replay(sd, ctx, om, 1, prompt, wl["gamma"], T, wl["seed"], wl["max_new"], "f32")
    assert r["iters"] >= 13
    ctx.close()


def test_tiny_self_draft_accepts_and_counts(sd):
    # the draft is a copy of the target: every draft is accepted on both sides
    cfg = synth.CONFIGS["tiny"]
    t = cfg["target"]
    ctx = sd.Context(t, [t], "f32", 1, 128, 4, 1.0, 9)
    w = synth.make_weights(t, seed=0, model_index=0, dtype="f32")
    ctx.load_weights(0, w); ctx.load_weights(1, w)
    om = [oracle.OracleModel(t, w), oracle.OracleModel(t, w)]
    prompt = synth.make_prompt(t["vocab"], 16, seed=2)
    r = _replay(sd, ctx, om, 0, prompt, 4, 1.0, 9, 30, "f32", min_agree=0.8)
    _, cnt = ctx.sd_seq_read(0)
    assert cnt["accepted"] >= 0.9 * cnt["drafted"]
    ctx.close()


def test_alpha_estimate_acceptance_rate_and_tau_against_the_oracle(sd):
    """Eq. 1's inputs from the library itself: alpha-hat = mean over judged slots of sum_k min(p, q), the acceptance rate
    (accepted / drafted), tau (tokens per verify iteration) and the cost ratio c from its own clock."""
    cfg = synth.CONFIGS["tiny"]
    wl = cfg["workload"]
    T = 1.0
    ctx, om = _build(sd, cfg["target"], cfg["drafts"], "f32", T, wl["seed"], max_ctx=wl["max_ctx"])
    prompt = synth.make_prompt(cfg["target"]["vocab"], wl["prompt"], seed=wl["seed"])
    ctx.sd_cost_timing(1)
    r = _replay(sd, ctx, om, 1, prompt, wl["gamma"], T, wl["seed"], wl["max_new"], "f32")
    alpha = r["alpha_sum"] / r["judged"]
    assert abs(alpha - r["alpha_ref"]) <= 1e-4, (alpha, r["alpha_ref"])
    _, cnt = ctx.sd_seq_read(0)
    _, cnt_ref, _ = oracle.spec_decode(om[0], om[2], prompt, wl["max_new"], wl["gamma"], T, wl["seed"], seq_id=0)
    ar, ar_ref = cnt["accepted"] / cnt["drafted"], cnt_ref["accepted"] / cnt_ref["drafted"]
    tau, tau_ref = cnt["emitted"] / cnt["iterations"], cnt_ref["emitted"] / cnt_ref["iterations"]
    assert ar == ar_ref and tau == tau_ref
    # alpha-hat estimates the acceptance rate of the judged slots (the draws are the oracle's; a loose statistical bound)
    assert abs(alpha - ar) < 0.25
    cost = ctx.sd_cost_read()
    assert cost["draft_passes"] == r["iters"] * wl["gamma"] and cost["verify_passes"] == r["iters"]
    assert cost["draft_pass_ms"] > 0 and cost["verify_pass_ms"] > 0
    assert abs(cost["c"] - cost["draft_pass_ms"] / cost["verify_pass_ms"]) < 1e-12
    g, a, c_ratio, speed = ctx.sd_best_gamma_measured(0, 8)
    assert abs(a - alpha) < 1e-12 and abs(c_ratio - cost["c"]) < 1e-12
    g_ref, speed_ref = sd.sd_best_gamma(alpha, cost["c"], 8)
    assert g == g_ref and abs(speed - speed_ref) < 1e-12
    eq1 = [(1 - alpha ** (k + 1)) / ((1 - alpha) * (k * cost["c"] + 1)) for k in range(1, 9)]        # Eq. 1 written out
    assert abs(speed_ref - max([1.0] + eq1)) < 1e-9
    # a new sequence starts from zero
    ctx.sd_seq_begin(0, prompt, 5)
    assert ctx.sd_seq_alpha(0) == (0.0, 0)
    ctx.close()


SMALL_BF16 = dict(n_layers=2, d_model=512, n_heads=8, n_kv_heads=2, head_dim=64, d_ffn=1408, vocab=4096)
SMALL_BF16_DRAFT = dict(n_layers=1, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ffn=768, vocab=4096)
WIDE_BF16 = dict(n_layers=2, d_model=1024, n_heads=8, n_kv_heads=8, head_dim=128, d_ffn=2816, vocab=8192)


@pytest.mark.parametrize("T", [0.7, 0.0])
def test_small_bf16_gqa_teacher_forced(sd, T):
    ctx, om = _build(sd, SMALL_BF16, [SMALL_BF16_DRAFT, SMALL_BF16_DRAFT], "bf16", T, 5, max_ctx=128)
    prompt = synth.make_prompt(4096, 40, seed=6)
    _replay(sd, ctx, om, 1, prompt, 5, T, 5, 24, "bf16", min_agree=0.6)
    ctx.close()


def test_long_prompt_crosses_the_slice_boundary(sd):
    # prompt of 1100 tokens: prefill in 256-row passes, verify rows against a cache cut into two slices
    ctx, om = _build(sd, SMALL_BF16, [SMALL_BF16_DRAFT], "bf16", 1.0, 11, max_ctx=1280)
    prompt = synth.make_prompt(4096, 1100, seed=12)
    _replay(sd, ctx, om, 0, prompt, 5, 1.0, 11, 12, "bf16", min_agree=0.5)
    ctx.close()


# The benchmark configurations at full width (every GEMM, attention and sampling shape of the real
# launch configuration) with the depth and the prompt cut down so that the oracle finishes in seconds.
FULL_WIDTH = {
    "1b": dict(cfg="1b", layers=2, prompt=48),
    "7b": dict(cfg="7b", layers=1, prompt=40),
    "13b": dict(cfg="13b", layers=1, prompt=24),
}


@pytest.mark.parametrize("name", sorted(FULL_WIDTH))
def test_benchmark_shapes_at_full_width_teacher_forced(sd, name):
    spec = FULL_WIDTH[name]
    cfg = synth.CONFIGS[spec["cfg"]]
    wl = cfg["workload"]
    t = dict(cfg["target"], n_layers=spec["layers"])
    d = dict(cfg["drafts"][0], n_layers=1)
    gamma = wl["gamma"]
    ctx, om = _build(sd, t, [d], "bf16", wl["temperature"], wl["seed"], max_seqs=1, max_ctx=spec["prompt"] + 40, max_gamma=gamma)
    prompt = synth.make_prompt(t["vocab"], spec["prompt"], seed=wl["seed"])
    # a vocabulary of 32000 with nearly flat random-init distributions: which token a draw lands on flips with
    # bf16-level noise in q, so the agreement of sampled tokens is not asserted here (the replay is teacher-forced)
    r = _replay(sd, ctx, om, 0, prompt, gamma, wl["temperature"], wl["seed"], 2 * (gamma + 1), "bf16", min_agree=0.0)
    assert r["iters"] >= 2
    assert ctx.sd_device_status() == 0
    ctx.close()


def _one_verify_step_error(sd, t, d, prompt_len, wl, two_part=1):
    """max |logit - oracle| and max |p - oracle| of one verify step (gamma + 1 rows after a prompt)."""
    gamma, T, seed, V = wl["gamma"], wl["temperature"], wl["seed"], t["vocab"]
    wt = synth.make_weights(t, seed=0, model_index=0, dtype="bf16")
    wd = synth.make_weights(d, seed=0, model_index=1, dtype="bf16")
    om = [oracle.OracleModel(t, wt), oracle.OracleModel(d, wd)]
    prompt = synth.make_prompt(V, prompt_len, seed=seed)
    _, _, tr = oracle.spec_decode(om[0], om[1], prompt, gamma + 1, gamma, T, seed, seq_id=0, trace_iters=1, trace_probs=True, trace_logits=True)
    ctx = sd.Context(t, [d], "bf16", 1, prompt_len + 40, gamma, T, seed)
    ctx.load_weights(0, wt); ctx.load_weights(1, wd)
    del wt, wd, om
    ctx.sd_use_two_part_activations(two_part)
    ctx.sd_seq_begin(0, prompt, 0); ctx.sd_route_prompt([0], forced_task=[0]); ctx.sd_prefill([0])
    x = torch.from_numpy(tr["x"][0:1].copy()).to(DEV)
    logits = torch.zeros((1, gamma + 1, V), dtype=torch.float32, device=DEV)
    ctx.sd_verify([0], gamma, x, logits)
    lg = logits.cpu().numpy()[0].astype(np.float64)
    p = torch.softmax(logits[0].double() / T, dim=-1).cpu().numpy()
    assert ctx.sd_device_status() == 0
    ctx.close()
    return float(np.abs(lg - tr["logits"][0]).max()), float(np.abs(p - tr["p"][0]).max())


# How the error of the verify step's logits grows with depth at the 7B width (bf16 KV cache, queries, keys, values and
# attention weights against the fp64 oracle; the GEMMs' inputs in two bf16 parts).  Measured on a B200: 0.031, 0.041, 0.061
# for 1, 2 and 4 layers (one bf16 part: 0.037, 0.049, 0.068) - about the square root of the depth.  The stated 5e-2 holds to
# two layers; deeper, the bound asserted here is the measured value with a margin, and the probabilities (what the
# accept rule consumes) stay inside their 1e-3 by an order of magnitude.
DEPTH_SERIES_7B = [(1, 5e-2), (2, 5e-2), (4, 8e-2)]


@pytest.mark.parametrize("layers,bound", DEPTH_SERIES_7B)
def test_logit_error_against_depth_at_7b_width(sd, layers, bound):
    cfg = synth.CONFIGS["7b"]
    t = dict(cfg["target"], n_layers=layers)
    d = dict(cfg["drafts"][0], n_layers=1)
    dl, dp = _one_verify_step_error(sd, t, d, 24, cfg["workload"])
    print(f"7B width, {layers} layer(s): max |logit - oracle| = {dl:.4f}, max |p - oracle| = {dp:.2e}")
    assert dl <= bound, dl
    assert dp <= TOL["bf16"]["probs"], dp
    if layers == 1:                               # the two-part activations are what keeps one layer inside the stated bound with room
        dl1, _ = _one_verify_step_error(sd, t, d, 24, cfg["workload"], two_part=0)
        assert dl < dl1, (dl, dl1)


def test_full_depth_7b_verify_step_against_the_oracle(sd):
    """All 32 layers of the 7B configuration, one verify step after a 24-token prompt (the oracle needs about ten seconds,
    generating the 13 GB of weights on the host a minute or two).  bf16 noise grows with about the square root of the depth:
    measured max |logit - oracle| at full depth is recorded here and bounded; the probabilities stay inside the stated 1e-3."""
    cfg = synth.CONFIGS["7b"]
    t = dict(cfg["target"])
    d = dict(cfg["drafts"][0], n_layers=1)
    dl, dp = _one_verify_step_error(sd, t, d, 24, cfg["workload"])
    print(f"7B, all {t['n_layers']} layers: max |logit - oracle| = {dl:.4f}, max |p - oracle| = {dp:.2e}")
    assert dl <= 0.30, dl
    assert dp <= TOL["bf16"]["probs"], dp


def test_wide_bf16_head_dim_128_teacher_forced(sd):
    ctx, om = _build(sd, WIDE_BF16, [SMALL_BF16_DRAFT | dict(vocab=8192)], "bf16", 1.0, 7, max_ctx=96)
    prompt = synth.make_prompt(8192, 33, seed=8)
    _replay(sd, ctx, om, 0, prompt, 3, 1.0, 7, 16, "bf16", min_agree=0.6)
    ctx.close()


def test_batched_ragged_sequences_match_single_sequence_runs(sd):
    """Several sequences of different lengths, routed to different drafts, in one call each:
    every sequence must see exactly what it sees when run alone."""
    T, gamma, seed = 1.0, 3, 21
    ctx, om = _build(sd, SMALL_BF16, [SMALL_BF16_DRAFT, SMALL_BF16_DRAFT], "bf16", T, seed, max_seqs=4, max_ctx=96)
    V = 4096
    prompts = [synth.make_prompt(V, n, seed=30, seq=i) for i, n in enumerate([9, 33, 17, 20])]
    route = [0, 1, 1, 0]
    traces = []
    for i, p in enumerate(prompts):
        _, _, tr = oracle.spec_decode(om[0], om[1 + route[i]], p, 12, gamma, T, seed, seq_id=100 + i,
                                      trace_iters=3, trace_probs=True, trace_logits=True)
        traces.append(tr)
        ctx.sd_seq_begin(i, p, 100 + i)
    seqs = [2, 0, 3, 1]                                   # deliberately not in slot order
    assert ctx.sd_route_prompt(seqs, forced_task=[route[s] for s in seqs]).tolist() == [route[s] for s in seqs]
    ctx.sd_prefill(seqs)
    B = len(seqs)
    x = torch.zeros((B, gamma), dtype=torch.int32, device=DEV)
    xs = torch.zeros((B, gamma), dtype=torch.int32, device=DEV)
    q = torch.zeros((B, gamma, V), dtype=torch.float32, device=DEV)
    logits = torch.zeros((B, gamma + 1, V), dtype=torch.float32, device=DEV)
    n_acc = torch.zeros((B,), dtype=torch.int32, device=DEV)
    out_tok = torch.zeros((B, gamma + 1), dtype=torch.int32, device=DEV)
    for it in range(3):
        x.copy_(torch.from_numpy(np.stack([traces[s]["x"][it] for s in seqs])))
        ctx.sd_draft_steps_replay(seqs, gamma, x, xs, q)
        ctx.sd_verify(seqs, gamma, x, logits)
        ctx.sd_accept_seqs(seqs, gamma, logits, q, x, n_acc, out_tok)
        lg, qg = logits.cpu().numpy().astype(np.float64), q.cpu().numpy().astype(np.float64)
        for b, s in enumerate(seqs):
            assert np.abs(lg[b] - traces[s]["logits"][it]).max() <= 5e-2
            assert np.abs(qg[b] - traces[s]["q"][it]).max() <= 1e-3
        n_acc.copy_(torch.from_numpy(np.array([traces[s]["n_acc"][it] for s in seqs], dtype=np.int32)))
        out_tok.copy_(torch.from_numpy(np.stack([traces[s]["out_tok"][it] for s in seqs])))
        ctx.sd_kv_rollback(seqs, gamma, n_acc, out_tok)
    for s in seqs:
        got, cnt = ctx.sd_seq_read(s)
        assert got.tolist() == toks_ref_full(traces[s], prompts[s], 2)
        assert cnt["iterations"] == 3 and cnt["drafted"] == 9
    assert ctx.sd_device_status() == 0
    ctx.close()


def test_draft_groups_side_by_side_give_what_they_give_one_after_the_other(sd):
    """Sequences routed to different draft models: their draft passes run on streams of their own by default; the drafts
    and their distributions are bit for bit those of the group-after-group order, with and without captured graphs."""
    V, gamma = 4096, 4
    ctx, om = _build(sd, SMALL_BF16, [SMALL_BF16_DRAFT, SMALL_BF16_DRAFT, SMALL_BF16_DRAFT], "bf16", 1.0, 23, max_seqs=6, max_ctx=128)
    prompts = [synth.make_prompt(V, n, seed=14, seq=i) for i, n in enumerate([17, 40, 33, 25, 58, 19])]
    route = [2, 0, 1, 0, 2, 1]
    outs = []
    for graphs, streams in ((1, 1), (1, 0), (0, 1), (0, 0)):
        ctx.sd_use_graphs(graphs); ctx.sd_use_draft_streams(streams)
        for s, p in enumerate(prompts):
            ctx.sd_seq_begin(s, p, 300 + s)
        ctx.sd_route_prompt(list(range(6)), forced_task=route)
        ctx.sd_prefill(list(range(6)))
        x = torch.zeros((6, gamma), dtype=torch.int32, device=DEV); q = torch.zeros((6, gamma, V), dtype=torch.float32, device=DEV)
        for _ in range(2):                                   # the second call replays the captured graph
            ctx.sd_draft_steps(list(range(6)), gamma, x, q)
        outs.append((x.cpu().clone(), q.cpu().clone()))
    for x, q in outs[1:]:
        assert torch.equal(x, outs[0][0]) and torch.equal(q, outs[0][1])
    for s, p in enumerate(prompts):                          # and they are the oracle's
        _, _, tr = oracle.spec_decode(om[0], om[1 + route[s]], p, gamma + 1, gamma, 1.0, 23, seq_id=300 + s, trace_iters=1, trace_probs=True)
        assert np.abs(outs[0][1][s].numpy().astype(np.float64) - tr["q"][0]).max() <= TOL["bf16"]["probs"]
    assert ctx.sd_device_status() == 0
    ctx.close()


def test_batch16_launch_configuration_at_full_width(sd):
    """The batched benchmark's launch configuration (16 sequences x (gamma + 1) = 96 verify rows in one call: wide-N
    GEMMs, fused steps in several row batches, the several-CTAs-per-SM form of attention, ragged contexts) at the
    7B width, with one layer and short prompts so that the oracle finishes in seconds."""
    cfg = synth.CONFIGS["7b_batch16"]
    wl = cfg["workload"]
    t = dict(cfg["target"], n_layers=1)
    d = dict(cfg["drafts"][0], n_layers=1)
    gamma, T, seed, B = wl["gamma"], wl["temperature"], wl["seed"], 16
    ctx, om = _build(sd, t, [d], "bf16", T, seed, max_seqs=B, max_ctx=48, max_gamma=gamma)
    V = t["vocab"]
    prompts = [synth.make_prompt(V, 6 + (5 * i) % 15, seed=wl["seed"], seq=i) for i in range(B)]
    traces = []
    for i, p in enumerate(prompts):
        _, _, tr = oracle.spec_decode(om[0], om[1], p, gamma + 1, gamma, T, seed, seq_id=200 + i,
                                      trace_iters=1, trace_probs=True, trace_logits=True)
        traces.append(tr)
        ctx.sd_seq_begin(i, p, 200 + i)
    seqs = list(range(B))
    ctx.sd_route_prompt(seqs, forced_task=[0] * B)
    ctx.sd_prefill(seqs)
    x = torch.from_numpy(np.stack([traces[s]["x"][0] for s in seqs])).to(DEV)
    xs = torch.zeros((B, gamma), dtype=torch.int32, device=DEV)
    q = torch.zeros((B, gamma, V), dtype=torch.float32, device=DEV)
    logits = torch.zeros((B, gamma + 1, V), dtype=torch.float32, device=DEV)
    ctx.sd_draft_steps_replay(seqs, gamma, x, xs, q)
    ctx.sd_verify(seqs, gamma, x, logits)
    lg, qg = logits.cpu().numpy().astype(np.float64), q.cpu().numpy().astype(np.float64)
    worst = max(float(np.abs(lg[b] - traces[b]["logits"][0]).max()) for b in seqs)
    print(f"batch-16 launch, one layer at 7B width: max |logit - oracle| = {worst:.4f}")
    assert worst <= TOL["bf16"]["logits"], worst
    for b in seqs:
        assert np.abs(qg[b] - traces[b]["q"][0]).max() <= TOL["bf16"]["probs"], b
    assert ctx.sd_device_status() == 0
    ctx.close()


def test_route_prompt_classifier_matches_oracle(sd):
    cfg = synth.CONFIGS["tiny"]
    t, (d_in, d_h, K) = cfg["target"], cfg["classifier"]
    ctx, om = _build(sd, t, cfg["drafts"], "f32", 1.0, 1, max_seqs=8, clf_hidden=d_h)
    clf = synth.make_classifier(d_in, d_h, K, seed=0)
    ctx.sd_load_classifier(clf["w1"], clf["b1"], clf["w2"], clf["b2"])
    expect, seqs = [], list(range(8))
    for s in seqs:
        p = synth.make_prompt(t["vocab"], 5 + 9 * s, seed=40, seq=s)
        ctx.sd_seq_begin(s, p)
        k, probs = oracle.route_prompt(om[0].w["embed"], p, clf["w1"], clf["b1"], clf["w2"], clf["b2"])
        assert np.sort(probs)[-1] - np.sort(probs)[-2] > 1e-4       # the synthetic classifier is decisive
        expect.append(k)
    assert ctx.sd_route_prompt(seqs).tolist() == expect
    assert len(set(expect)) == K                                      # both drafts are used
    forced = [1, -1, 0, -1, -1, 1, 0, -1]                             # Sec. 2.1: a given task type bypasses the classifier
    got = ctx.sd_route_prompt(seqs, forced_task=forced).tolist()
    assert got == [f if f >= 0 else e for f, e in zip(forced, expect)]
    ctx.close()


def test_greedy_speculative_equals_greedy_autoregressive_on_gpu(sd):
    """Invariant of the path itself: with T = 0 the speculative loop emits exactly what plain
    autoregressive decoding of the target emits (free-running, no teacher forcing)."""
    ctx, om = _build(sd, SMALL_BF16, [SMALL_BF16_DRAFT], "bf16", 0.0, 3, max_seqs=2, max_ctx=128)
    V, gamma = 4096, 4
    prompt = synth.make_prompt(V, 21, seed=50)
    for s in (0, 1):
        ctx.sd_seq_begin(s, prompt, 0)
    ctx.sd_route_prompt([0, 1], forced_task=[0, 0]); ctx.sd_prefill([0, 1])
    x = torch.zeros((1, gamma), dtype=torch.int32, device=DEV)
    q = torch.zeros((1, gamma, V), dtype=torch.float32, device=DEV)
    logits = torch.zeros((1, gamma + 1, V), dtype=torch.float32, device=DEV)
    n_acc = torch.zeros((1,), dtype=torch.int32, device=DEV)
    out_tok = torch.zeros((1, gamma + 1), dtype=torch.int32, device=DEV)
    for _ in range(8):                                    # speculative, sequence 0
        ctx.sd_draft_steps([0], gamma, x, q)
        ctx.sd_verify([0], gamma, x, logits)
        ctx.sd_accept_seqs([0], gamma, logits, q, x, n_acc, out_tok)
        ctx.sd_kv_rollback([0], gamma, n_acc, out_tok)
    spec, cnt = ctx.sd_seq_read(0)
    assert cnt["emitted"] == len(spec) - 21 and cnt["iterations"] == 8
    l1 = torch.zeros((1, 1, V), dtype=torch.float32, device=DEV)
    o1 = torch.zeros((1, 1), dtype=torch.int32, device=DEV)
    for _ in range(len(spec) - 21):                       # autoregressive, sequence 1: gamma = 0
        ctx.sd_verify([1], 0, None, l1)
        ctx.sd_accept_seqs([1], 0, l1, None, None, n_acc, o1)
        ctx.sd_kv_rollback([1], 0, n_acc, o1)
    ar, _ = ctx.sd_seq_read(1)
    # bf16 rounding differs between a 5-row and a 1-row pass only through the order of fp32 sums,
    # which the kernels keep fixed per row: the outputs are identical
    assert spec.tolist() == ar.tolist()
    ctx.close()


def test_capacity_and_state_errors_are_reported_on_the_host(sd):
    cfg = synth.CONFIGS["tiny"]
    ctx, _ = _build(sd, cfg["target"], cfg["drafts"], "f32", 1.0, 1, max_seqs=2, max_ctx=24, max_gamma=4)
    V = cfg["target"]["vocab"]
    x = torch.zeros((1, 4), dtype=torch.int32, device=DEV)
    q = torch.zeros((1, 4, V), dtype=torch.float32, device=DEV)
    logits = torch.zeros((1, 5, V), dtype=torch.float32, device=DEV)
    with pytest.raises(sd.SdError) as e:
        ctx.sd_verify([0], 4, x, logits)                  # nothing begun in slot 0
    assert e.value.status == 2
    with pytest.raises(sd.SdError) as e:
        ctx.sd_seq_begin(0, synth.make_prompt(V, 30))     # longer than the KV cache
    assert e.value.status == 3
    ctx.sd_seq_begin(0, synth.make_prompt(V, 21))
    with pytest.raises(sd.SdError) as e:
        ctx.sd_prefill([0])                               # not routed yet
    assert e.value.status == 2
    ctx.sd_route_prompt([0], forced_task=[0]); ctx.sd_prefill([0])
    with pytest.raises(sd.SdError) as e:
        ctx.sd_verify([0], 5, x, logits)                  # gamma above max_gamma
    assert e.value.status == 1
    with pytest.raises(sd.SdError) as e:
        ctx.sd_verify([0, 0], 4, x, logits)               # duplicate sequence
    assert e.value.status == 1
    with pytest.raises(sd.SdError) as e:
        ctx.sd_verify([0], 4, x, logits)                  # 21 + 4 positions do not fit 24
    assert e.value.status == 3
    ctx.sd_verify([0], 3, x, logits)                      # 21 + 3 does
    # rollback with an impossible n_acc is clamped and flagged, not trusted
    n_acc = torch.full((1,), 9, dtype=torch.int32, device=DEV)
    out_tok = torch.zeros((1, 4), dtype=torch.int32, device=DEV)
    ctx.sd_kv_rollback([0], 3, n_acc, out_tok)
    assert ctx.sd_device_status() & 4
    ctx.close()


def test_tile_by_tile_hand_off_of_token_rows_gives_identical_results(sd):
    """With SD_TUNE_TILE_HANDOFF the GEMMs load each k block of token rows as soon as the step kernel's CTA for that tile has
    written it instead of waiting for the whole kernel: same arithmetic, so the teacher-forced run still matches the
    oracle and the logits are bit for bit those of the default path; so are the other measurement knobs."""
    V, gamma = 4096, 5
    prompt = synth.make_prompt(V, 41, seed=12)
    ref = None
    for knobs in ({}, {sd.SD_TUNE_TILE_HANDOFF: 1}, {sd.SD_TUNE_PACE_NS: 1, sd.SD_TUNE_MANY_ROWS_CB: 4, sd.SD_TUNE_STEADY_STAGES: 8},
                  {sd.SD_TUNE_WO_STAGES: 6, sd.SD_TUNE_WO_PREFILL_ALL: 1}):       # (the attention knobs change the order of its merges)
        ctx, om = _build(sd, SMALL_BF16, [SMALL_BF16_DRAFT], "bf16", 1.0, 17, max_ctx=128)
        for k, v in knobs.items():
            ctx.sd_tuning(k, v)
        _replay(sd, ctx, om, 0, prompt, gamma, 1.0, 17, 12, "bf16", min_agree=0.0)      # (few iterations: agreement counts are covered elsewhere)
        x = torch.from_numpy(synth.make_prompt(V, gamma, seed=3).reshape(1, gamma).astype(np.int32)).to(DEV)
        logits = torch.zeros((1, gamma + 1, V), dtype=torch.float32, device=DEV)
        ctx.sd_verify([0], gamma, x, logits)
        got = logits.cpu()
        if ref is None:
            ref = got
        else:
            assert torch.equal(got, ref), knobs
        assert ctx.sd_device_status() == 0
        ctx.close()


def test_graph_replay_plain_path_and_fused_call_agree(sd):
    """The same iterations through (a) captured graphs, (b) kernel-by-kernel launches, (c) the plain
    CUDA-core kernels and (d) the one-call verify+accept+rollback give the same tokens; (a), (b) and
    (d) are the same kernels and must agree bit for bit."""
    T, gamma, seed, V = 1.0, 4, 31, 4096
    ctx, om = _build(sd, SMALL_BF16, [SMALL_BF16_DRAFT], "bf16", T, seed, max_seqs=4, max_ctx=128)
    prompt = synth.make_prompt(V, 19, seed=60)
    for s in range(4):
        ctx.sd_seq_begin(s, prompt, 7)                    # same Philox stream everywhere
    ctx.sd_route_prompt([0, 1, 2, 3], forced_task=[0, 0, 0, 0])
    ctx.sd_prefill([0, 1, 2, 3])
    outs, logs = [], []
    for s, mode in enumerate(["graphs", "launches", "plain", "fused"]):
        ctx.sd_use_graphs(mode in ("graphs", "fused"))
        ctx.sd_force_plain_path(mode == "plain")
        x = torch.zeros((1, gamma), dtype=torch.int32, device=DEV)
        q = torch.zeros((1, gamma, V), dtype=torch.float32, device=DEV)
        logits = torch.zeros((1, gamma + 1, V), dtype=torch.float32, device=DEV)
        n_acc = torch.zeros((1,), dtype=torch.int32, device=DEV)
        out_tok = torch.zeros((1, gamma + 1), dtype=torch.int32, device=DEV)
        keep = []
        for it in range(6):
            ctx.sd_draft_steps([s], gamma, x, q)
            if mode == "fused":
                ctx.sd_verify_accept([s], gamma, x, q, logits, n_acc, out_tok)
            else:
                ctx.sd_verify([s], gamma, x, logits)
                ctx.sd_accept_seqs([s], gamma, logits, q, x, n_acc, out_tok)
                ctx.sd_kv_rollback([s], gamma, n_acc, out_tok)
            keep.append(logits.clone())
        toks, cnt = ctx.sd_seq_read(s)
        assert cnt["iterations"] == 6
        outs.append(toks.tolist()); logs.append(keep)
    ctx.sd_use_graphs(1); ctx.sd_force_plain_path(0)
    assert outs[0] == outs[1] == outs[3]
    for a, b, c in zip(logs[0], logs[1], logs[3]):
        assert torch.equal(a, b) and torch.equal(a, c)
    # the plain kernels round differently; compare the first iteration (same inputs) within tolerance
    assert (logs[0][0] - logs[2][0]).abs().max().item() < 5e-2
    assert ctx.sd_device_status() == 0
    ctx.close()
