"""Drafts as one base model plus a low-rank adapter per task, against the oracle's merged-weight models (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import lora
from paper_2505_08600_b200 import synth
from gpu_util import DEV
from test_gpu_model import SMALL_BF16, TOL, _replay

pytestmark = pytest.mark.gpu

BASE_DRAFT = dict(n_layers=2, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ffn=768, vocab=4096)
N_TASKS, RANK, SCALE = 3, 16, 2.0
MATS = {"qkv": 0, "wo": 1, "gu": 2, "wd": 3}


@pytest.fixture(scope="module")
def sd():
    from paper_2505_08600_b200 import binding
    binding.lib()
    return binding


def _build(sd, T, seed, max_seqs=3, load_adapters=True):
    ctx = sd.Context(SMALL_BF16, [BASE_DRAFT], "bf16", max_seqs, 160, 5, T, seed, lora_adapters=N_TASKS, lora_rank=RANK, lora_scale=SCALE)
    wt = synth.make_weights(SMALL_BF16, seed=0, model_index=0, dtype="bf16")
    wb = synth.make_weights(BASE_DRAFT, seed=0, model_index=1, dtype="bf16")
    ctx.load_weights(0, wt)
    ctx.load_weights(1, wb)
    om = [oracle.OracleModel(SMALL_BF16, wt)]
    for task in range(N_TASKS):
        ad = synth.make_lora(BASE_DRAFT, RANK, task, seed=0)
        if load_adapters:
            for name, mat in MATS.items():
                for l, (a, b) in enumerate(ad[name]):
                    ctx.sd_load_lora(task, l, mat, a, b)
        else:
            ad = {k: None for k in MATS}
        om.append(oracle.OracleModel(BASE_DRAFT, lora.merged_weights(BASE_DRAFT, wb, ad, SCALE)))
    return ctx, om, wt, wb


@pytest.mark.parametrize("task", [0, 1, 2])
def test_each_task_teacher_forced_against_its_merged_model(sd, task):
    ctx, om, _, _ = _build(sd, 1.0, 11)
    prompt = synth.make_prompt(4096, 37, seed=3 + task)
    r = _replay(sd, ctx, om, task, prompt, 4, 1.0, 11, 20, "bf16", min_agree=0.6)
    assert r["iters"] >= 4
    ctx.close()


def test_adapters_differ_and_unloaded_adapters_are_the_base_draft(sd):
    # draft distributions of the three tasks for the same prompt differ by far more than the tolerance; with no
    # adapter loaded every task gives the base draft's distribution, bit for bit the one of a context without adapters
    prompt = synth.make_prompt(4096, 30, seed=2)
    V, gamma = 4096, 3
    qs = []
    for loaded in (True, False):
        ctx, om, wt, wb = _build(sd, 1.0, 5, load_adapters=loaded)
        for task in range(N_TASKS):
            ctx.sd_seq_begin(0, prompt, 7)
            ctx.sd_route_prompt([0], forced_task=[task])
            ctx.sd_prefill([0])
            x = torch.zeros((1, gamma), dtype=torch.int32, device=DEV); q = torch.zeros((1, gamma, V), dtype=torch.float32, device=DEV)
            ctx.sd_draft_steps([0], gamma, x, q)
            qs.append(q.cpu().numpy()[0, 0])
        ctx.close()
    assert np.abs(qs[0] - qs[1]).max() > 0.01 * qs[0].max() and np.abs(qs[1] - qs[2]).max() > 0.01 * qs[1].max()
    assert (qs[3] == qs[4]).all() and (qs[4] == qs[5]).all()
    plain = sd.Context(SMALL_BF16, [BASE_DRAFT], "bf16", 1, 160, 5, 1.0, 5)
    plain.load_weights(0, wt); plain.load_weights(1, wb)
    plain.sd_seq_begin(0, prompt, 7); plain.sd_route_prompt([0], forced_task=[0]); plain.sd_prefill([0])
    x = torch.zeros((1, gamma), dtype=torch.int32, device=DEV); q = torch.zeros((1, gamma, V), dtype=torch.float32, device=DEV)
    plain.sd_draft_steps([0], gamma, x, q)
    np.testing.assert_allclose(q.cpu().numpy()[0, 0], qs[3], rtol=0, atol=1e-7)
    plain.close()


def test_sequences_of_different_tasks_share_one_draft_pass(sd):
    # three sequences, three tasks, one sd_draft_steps call: every sequence gets what it gets when it runs alone
    gamma, V = 4, 4096
    prompts = [synth.make_prompt(V, n, seed=9, seq=i) for i, n in enumerate([21, 40, 33])]
    tasks = [2, 0, 1]
    ctx, om, _, _ = _build(sd, 1.0, 13)
    for s, p in enumerate(prompts):
        ctx.sd_seq_begin(s, p, 100 + s)
    assert ctx.sd_route_prompt([0, 1, 2], forced_task=tasks).tolist() == tasks
    ctx.sd_prefill([0, 1, 2])
    x = torch.zeros((3, gamma), dtype=torch.int32, device=DEV); q = torch.zeros((3, gamma, V), dtype=torch.float32, device=DEV)
    n0 = ctx.sd_launch_count()
    ctx.sd_use_graphs(0)
    ctx.sd_draft_steps([0, 1, 2], gamma, x, q)
    launches_together = ctx.sd_launch_count() - n0
    q_all, x_all = q.cpu().numpy(), x.cpu().numpy()
    ctx.close()
    for s, p in enumerate(prompts):
        _, _, tr = oracle.spec_decode(om[0], om[1 + tasks[s]], p, gamma + 1, gamma, 1.0, 13, seq_id=100 + s, trace_iters=1, trace_probs=True)
        assert np.abs(q_all[s].astype(np.float64) - tr["q"][0]).max() <= TOL["bf16"]["probs"]
    # alone
    ctx, _, _, _ = _build(sd, 1.0, 13)
    ctx.sd_use_graphs(0)
    for s, p in enumerate(prompts):
        ctx.sd_seq_begin(s, p, 100 + s)
        ctx.sd_route_prompt([s], forced_task=[tasks[s]])
        ctx.sd_prefill([s])
        x1 = torch.zeros((1, gamma), dtype=torch.int32, device=DEV); q1 = torch.zeros((1, gamma, V), dtype=torch.float32, device=DEV)
        n0 = ctx.sd_launch_count()
        ctx.sd_draft_steps([s], gamma, x1, q1)
        launches_alone = ctx.sd_launch_count() - n0
        # (six rows together feed the GEMMs in two bf16 parts, two rows alone in one: equal up to bf16 rounding of the activations)
        np.testing.assert_allclose(q1.cpu().numpy()[0], q_all[s], rtol=0, atol=2e-5)
    assert launches_together == launches_alone                     # three tasks cost the launches of one
    assert ctx.sd_device_status() == 0
    ctx.close()


def test_configuration_errors_are_reported(sd):
    with pytest.raises(RuntimeError):                              # adapters and tasks must agree; rank a multiple of 8
        sd.Context(SMALL_BF16, [BASE_DRAFT], "bf16", 1, 64, 4, 1.0, 1, lora_adapters=3, lora_rank=12, lora_scale=1.0)
    with pytest.raises(RuntimeError):                              # 9 adapters of rank 16 do not fit one tile
        sd.Context(SMALL_BF16, [BASE_DRAFT], "bf16", 1, 64, 4, 1.0, 1, lora_adapters=9, lora_rank=16, lora_scale=1.0)
    ctx = sd.Context(SMALL_BF16, [BASE_DRAFT], "bf16", 1, 64, 4, 1.0, 1)
    with pytest.raises(RuntimeError):                              # no adapters in this context
        ctx.sd_load_lora(0, 0, 0, np.zeros((16, 256), dtype=np.uint16), np.zeros((768, 16), dtype=np.uint16))
    ctx.close()
