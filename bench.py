#!/usr/bin/env python
"""Benchmark of the verify step (target pass over gamma+1 rows + accept/reject + KV rollback).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 7b|all] [--impl reference] [--gamma-sweep 1..10]

One JSON line on stdout.  `value` is verify-step tokens/s: B * (gamma + 1) query positions per
sd_verify + sd_accept_seqs + sd_kv_rollback, timed with CUDA events on the library's stream with
inputs resident in HBM.  The path does not shard: with N > 1 every rank runs an independent replica.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2505_08600_b200 import replicas, synth  # noqa: E402

GEMM_TRAFFIC_PER_WEIGHT_BYTE = 1.0073      # measured: (dram read + write) / weight bytes of k_gemm_streamk
METRIC = "verify_step_tokens_per_s"
UNIT = "tokens/s"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def eq1_speedup(alpha, gamma, c):
    return (1 - alpha ** (gamma + 1)) / ((1 - alpha) * (gamma * c + 1))


# ------------------------------------------------------------------------------------------
# CPU baseline: the oracle as it stands, on a bounded sample of the same verify step
# ------------------------------------------------------------------------------------------
def oracle_sample(cfg_name, sample_layers=2, min_seconds=10.0, max_reps=64):
    """Times the oracle's cached forward over gamma+1 rows at the config's shapes with only
    `sample_layers` of the layers, and the lm_head alone, then scales to the full depth.
    Repeats until about `min_seconds` of CPU work have been timed."""
    import oracle
    cfg = synth.CONFIGS[cfg_name]
    wl, t = cfg["workload"], dict(cfg["target"])
    gamma = wl["gamma"]
    n_prompt = wl["prompt"] if isinstance(wl["prompt"], int) else (wl["prompt"][0] + wl["prompt"][1]) // 2
    B = wl["batch"]
    full_layers = t["n_layers"]
    t["n_layers"] = sample_layers
    w = synth.make_weights(t, seed=0, model_index=0, dtype=cfg["dtype"])
    m = oracle.OracleModel(t, w)
    cache = m.new_cache(n_prompt + gamma + 1)
    rng = np.random.default_rng(0)
    cache.k[:] = rng.standard_normal(cache.k.shape[0])          # attention cost does not depend on the values
    cache.v[:] = rng.standard_normal(cache.v.shape[0])
    toks = synth.make_prompt(t["vocab"], gamma + 1, seed=1)
    cores = len(os.sched_getaffinity(0))
    t_with, t_layers = [], []
    while len(t_with) < max_reps and sum(t_with) + sum(t_layers) < min_seconds:
        t0 = time.perf_counter(); cache.forward(toks, n_prompt - 1, want_logits=True); t_with.append(time.perf_counter() - t0)
        t0 = time.perf_counter(); cache.forward(toks, n_prompt - 1, want_logits=False); t_layers.append(time.perf_counter() - t0)
    tl, tw = min(t_layers), min(t_with)
    step_s = B * (tl / sample_layers * full_layers + (tw - tl))  # sequences are independent: B of them cost B times one
    return dict(value=B * (gamma + 1) / step_s, unit=UNIT, cores=cores, kind="oracle",
                sample=f"{sample_layers} of {full_layers} layers + lm_head at full width, {gamma + 1} rows, context {n_prompt}, "
                       f"one sequence, best of {len(t_with)} repeats; scaled by layers and batch {B}",
                seconds_measured=round(sum(t_with) + sum(t_layers), 2), step_seconds_scaled=round(step_s, 2))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    for _ in range(args.warmup if args.warmup < 2 else 1):
        oracle_sample(args.config, min_seconds=1.0)
    for _ in range(max(1, min(args.steps, 5))):
        vals.append(oracle_sample(args.config, min_seconds=5.0))
    v = statistics.median(x["value"] for x in vals)
    cb = dict(vals[0]); cb["value"] = v
    wl = synth.CONFIGS[args.config]["workload"]
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": len(vals),
        "warmup": args.warmup, "ms_per_step": 1000.0 * wl["batch"] * (wl["gamma"] + 1) / v, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.config}: verify step, oracle on host cores, bounded sample"},
        "cpu_baseline": cb, "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------
def device_weights(torch, dims, dtype, seed, model_index, dev):
    """Random-init weights generated on the device, tensor by tensor (N(0, 0.02), gains 1)."""
    g = torch.Generator(device=dev)
    g.manual_seed(seed * 1000003 + model_index)
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    shapes = synth.mat_shapes(dims)

    def normal(shape):
        return (torch.randn(shape, generator=g, device=dev, dtype=torch.float32) * 0.02).to(td).contiguous()

    yield "embed", 0, normal((dims["vocab"], dims["d_model"]))
    yield "lm_head", 0, normal((dims["vocab"], dims["d_model"]))
    ones = torch.ones(dims["d_model"], device=dev, dtype=torch.float32)
    yield "final_norm", 0, ones
    for l in range(dims["n_layers"]):
        for name in synth.LAYER_MATS:
            yield name, l, normal(shapes[name])
        yield "norm1", l, ones
        yield "norm2", l, ones


class ClockSampler:
    Q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
        "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, gpu_id):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_id), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "20"], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
        os.unlink(self.f.name)
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.strip().lower() == "active":
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def setup(args, gamma_max, steps_per_phase):
    """Context with the config's models (random-init, generated on the device), its sequences begun, routed and prefilled.
    Prompts are shortened where the config's cache could not hold `steps_per_phase` verify steps after them."""
    import torch
    import torch.distributed as dist
    from paper_2505_08600_b200 import binding as sd

    rank, world, local = replicas.rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    if local >= torch.cuda.device_count():
        raise SystemExit(f"bench.py: rank {rank} wants cuda:{local}, the node has {torch.cuda.device_count()} GPU(s)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    torch.cuda.set_stream(torch.cuda.Stream(dev))           # a capturable (non-default) stream for everything below
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)      # only for the barrier and the max over ranks
    cfg = synth.CONFIGS[args.config]
    wl, tdims = cfg["workload"], cfg["target"]
    B, V, T, seed = wl["batch"], tdims["vocab"], wl["temperature"], wl["seed"]
    need = (gamma_max + 1) * steps_per_phase + gamma_max + 8
    if isinstance(wl["prompt"], int):
        lens = [wl["prompt"]] * B
    else:
        lens = synth.make_prompt_lengths(B, wl["prompt"][0], wl["prompt"][1], seed=seed).tolist()
    if max(lens) + need > wl["max_ctx"] and wl["max_ctx"] - need >= max(lens) // 2:
        lens = [min(n, wl["max_ctx"] - need) for n in lens]          # the timed steps end at the config's cache size
    max_ctx = max(wl["max_ctx"], max(lens) + need)

    lora = getattr(args, "lora", False)
    drafts = [cfg["drafts"][0]] if lora else list(cfg["drafts"])       # --lora: one base draft + one rank-16 adapter per task
    ctx = sd.Context(tdims, drafts, cfg["dtype"], B, max_ctx, max(gamma_max, 1), T, seed, clf_d_hidden=cfg["classifier"][1], device=dev,
                     lora_adapters=len(cfg["drafts"]) if lora else 0, lora_rank=16 if lora else 0, lora_scale=2.0 if lora else 0.0)
    for mid, dims in enumerate([tdims] + drafts):
        for name, l, tensor in device_weights(torch, dims, cfg["dtype"], 0, mid, dev):
            ctx.sd_load_tensor(mid, sd.TENSOR_KIND[name], l, tensor)
    if lora:
        dd = drafts[0]
        dq, dkv = dd["n_heads"] * dd["head_dim"], dd["n_kv_heads"] * dd["head_dim"]
        shapes = [(dq + 2 * dkv, dd["d_model"]), (dd["d_model"], dq), (2 * dd["d_ffn"], dd["d_model"]), (dd["d_model"], dd["d_ffn"])]
        g = torch.Generator(device=dev); g.manual_seed(77)
        for task in range(len(cfg["drafts"])):
            for l in range(dd["n_layers"]):
                for mat, (n_out, n_in) in enumerate(shapes):
                    a = (torch.randn((16, n_in), generator=g, device=dev) * 0.05).to(torch.bfloat16).contiguous()
                    b = (torch.randn((n_out, 16), generator=g, device=dev) * 0.05).to(torch.bfloat16).contiguous()
                    ctx.sd_load_lora(task, l, mat, a, b)
    clf = synth.make_classifier(*cfg["classifier"], seed=0)
    ctx.sd_load_classifier(clf["w1"], clf["b1"], clf["w2"], clf["b2"])
    torch.cuda.synchronize()

    seqs = list(range(B))
    prompts = [synth.make_prompt(V, lens[s], seed=seed, seq=s) for s in seqs]
    for s in seqs:
        ctx.sd_seq_begin(s, prompts[s], s)
    n_drafts = len(cfg["drafts"])
    routed = ctx.sd_route_prompt(seqs) if B == 1 else ctx.sd_route_prompt(seqs, forced_task=[s % n_drafts for s in seqs])
    ctx.sd_prefill(seqs)

    def rewind():        # back to the prompts (the caches keep their prefix), so that every phase sees the same contexts
        for s in seqs:
            ctx.sd_seq_force(s, prompts[s], lens[s] - 1, 0)

    return dict(torch=torch, dist=dist, sd=sd, rank=rank, world=world, local=local, dev=dev, cfg=cfg, ctx=ctx, seqs=seqs, lens=lens,
                routed=routed, rewind=rewind, max_ctx=max_ctx)


STEP_AFTER = {0: "lm_head", 1: "qkv", 2: "residual", 3: "swiglu"}
LAYER_LAUNCHES = ["gemm qkv", "step qkv", "attention", "gemm wo", "step wo", "gemm gate_up", "step gate_up", "gemm down", "step down"]


def in_graph_timeline(ctx, cfg, step_fn, esz):
    """Time stamps taken inside the kernels while the step runs as it always runs (captured graph, overlapping
    dependent launches): per launch of a layer, averaged over the inner layers, in microseconds after the layer's QKV
    GEMM issued its first MMA.  A GEMM's in-graph duration is counted from the moment its token rows exist (the kernel
    before it has finished) to its last CTA finishing; weights requested before that moment are part of the overlap."""
    t = cfg["target"]
    nl, per = t["n_layers"], len(LAYER_LAUNCHES)
    ctx.sd_launch_stamps(1)
    for _ in range(3):
        step_fn()
    st, kinds = ctx.sd_launch_stamps_read()
    ctx.sd_launch_stamps(0)
    if len(kinds) < nl * per + 2 or nl < 4:
        return None
    st = st.astype(np.int64)
    cols = ["start", "dep_first", "dep_last", "data_first", "data_last", "done_first", "done_last"]
    inner = range(1, nl - 1)
    rows = np.array([[[(st[l * per + j][k] - st[l * per][3]) / 1e3 if st[l * per + j][k] else np.nan for k in range(7)]
                      for j in range(per)] for l in inner])
    with np.errstate(all="ignore"):
        import warnings
        with warnings.catch_warnings():
            warnings.simplefilter("ignore", RuntimeWarning)
            avg = np.nanmean(rows, axis=0)           # (columns a kind of launch never reports stay NaN)
    period = float(np.mean([(st[(l + 1) * per][3] - st[l * per][3]) / 1e3 for l in inner]))
    table = {name: {c: (None if np.isnan(avg[j][k]) else round(float(avg[j][k]), 2)) for k, c in enumerate(cols)} for j, name in enumerate(LAYER_LAUNCHES)}
    gemm_us = 0.0
    for j, name in enumerate(LAYER_LAUNCHES):
        if name.startswith("gemm"):
            gemm_us += float(avg[j][6] - avg[j][1])
    # the lm_head GEMM: the last GEMM record of the pass
    lm = st[nl * per]
    lm_us = (lm[6] - lm[1]) / 1e3
    return {"layer_period_us": round(period, 2), "gemm_us_per_layer": round(gemm_us, 2), "lm_head_gemm_us": round(float(lm_us), 2),
            "columns": "us after the layer's QKV GEMM had its first stage: first CTA start; first/last CTA saw its dependency; "
                       "first/last CTA had its first stage (GEMM); first/last CTA done",
            "launches": table}


def run_gpu(args):
    K, W = args.steps, args.warmup
    n_iter_phase = min(10, K)
    cfg0 = synth.CONFIGS[args.config]
    gamma = args.gamma if args.gamma is not None else cfg0["workload"]["gamma"]
    env = setup(args, gamma, K + W + args.profile_steps + 4)
    torch, dist, sd, ctx = env["torch"], env["dist"], env["sd"], env["ctx"]
    rank, world, local, dev, cfg, seqs, lens, routed, rewind = (env[k] for k in ("rank", "world", "local", "dev", "cfg", "seqs", "lens", "routed", "rewind"))
    wl, tdims = cfg["workload"], cfg["target"]
    B, V, T, seed = wl["batch"], tdims["vocab"], wl["temperature"], wl["seed"]

    x = torch.zeros((B, gamma), dtype=torch.int32, device=dev)
    q = torch.zeros((B, gamma, V), dtype=torch.float32, device=dev)
    logits = torch.zeros((B, gamma + 1, V), dtype=torch.float32, device=dev)
    n_acc = torch.zeros((B,), dtype=torch.int32, device=dev)
    out_tok = torch.zeros((B, gamma + 1), dtype=torch.int32, device=dev)
    ctx.sd_draft_steps(seqs, gamma, x, q)          # the drafts every timed verify step scores (values do not change its cost)
    torch.cuda.synchronize()
    rewind()

    def verify_step():          # sd_verify + sd_accept_seqs + sd_kv_rollback as one captured launch sequence
        ctx.sd_verify_accept(seqs, gamma, x, q, logits, n_acc, out_tok)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(v):
        return replicas.max_over_ranks(v, world, dev)

    stream = torch.cuda.current_stream(dev)
    # ---- phase A: the headline, device-resident inputs
    try:
        gpu_id = str(torch.cuda.get_device_properties(dev).uuid)
        gpu_id = gpu_id if gpu_id.startswith("GPU-") else "GPU-" + gpu_id
    except Exception:
        gpu_id = str(local)
    sampler = ClockSampler(gpu_id)                 # samples cover the warm-up steps (the same launches) and the timed steps
    for _ in range(W):
        verify_step()
    l0 = ctx.sd_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.profiler.start()                 # a profiler told to wait for this range sees the timed steps only
    ev0.record(stream)
    for _ in range(K):
        verify_step()
    ev1.record(stream)
    barrier()
    torch.cuda.profiler.stop()
    ms_total = max_over_ranks(ev0.elapsed_time(ev1))
    clocks = sampler.stop()
    launches = ctx.sd_launch_count() - l0
    ms_step = ms_total / K
    value = replicas.whole_job_tokens_per_s(world, B, gamma, ms_step)
    ctx.sd_seq_read(0)
    n_ctx = [int(ctx.sd_seq_read(s)[0].shape[0]) for s in seqs]          # context lengths at the end of the timed steps

    # ---- per-kernel split of the same step (events between launches; separate from the timed run)
    ctx.sd_profile(1)
    for _ in range(args.profile_steps):
        verify_step()
    prof = ctx.sd_profile_read()
    ctx.sd_profile(0)
    rewind()
    esz0 = 2 if cfg["dtype"] == "bf16" else 4
    tl = in_graph_timeline(ctx, cfg, verify_step, esz0) if cfg["dtype"] == "bf16" else None
    rewind()
    esz = 2 if cfg["dtype"] == "bf16" else 4
    weight_bytes = synth.param_count(tdims, streamed_only=True) * esz
    kv_bytes = sum(n_ctx) * 2 * tdims["n_layers"] * tdims["n_kv_heads"] * tdims["head_dim"] * esz
    peak, peak_kind = _peaks()
    # Per-launch durations come from CUDA events recorded between the launches of the profiling pass just above.  An
    # event between two kernels keeps the second from starting early, so these are durations of launches run one after
    # the other: `achieved` is the conservative figure.  In the timed step consecutive launches overlap (programmatic
    # dependent launch); `overlapped` apportions the timed step by the shares of the split.
    split = {k: v["ms"] / args.profile_steps for k, v in prof.items()}
    n_gemm = 4 * tdims["n_layers"] + 1
    gemm_ms = split["linear"]
    achieved = weight_bytes / (gemm_ms * 1e-3) / 1e9
    total_split = max(sum(split.values()), 1e-9)
    gemm_share = split["linear"] / total_split
    in_step_ms = ms_step * gemm_share
    pair_ms = ms_step * (split["linear"] + split["fused_step"]) / total_split
    roofline = {"bound": "hbm", "kernel": f"k_gemm_streamk ({n_gemm} launches per verify step, all weight matrices once)",
                "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                "avg_launch_us": gemm_ms * 1e3 / n_gemm, "timing": "CUDA events around each launch (launches serialised)",
                # dram read+write per weight byte from the ncu capture summarised in profiles/gemm_streamk_1b_ncu_full.md
                "traffic": weight_bytes * GEMM_TRAFFIC_PER_WEIGHT_BYTE / n_gemm, "traffic_unit": "bytes per launch (average)",
                "algorithmic_bytes_per_launch": weight_bytes / n_gemm, "launches_per_step": n_gemm,
                "algorithmic_bytes_per_step": weight_bytes,
                "overlapped": {"kernel_share_of_split": gemm_share, "kernel_ms_in_step": in_step_ms,
                               # the same bytes over the GEMMs plus the small kernels that sum their pieces and apply the step after them
                               "with_fused_steps": {"ms_in_step": pair_ms, "gbs": weight_bytes / (pair_ms * 1e-3) / 1e9,
                                                    "frac": weight_bytes / (pair_ms * 1e-3) / 1e9 / peak}},
                "whole_step": {"bytes": weight_bytes + kv_bytes, "gbs": (weight_bytes + kv_bytes) / (ms_step * 1e-3) / 1e9,
                               "frac_of_peak": (weight_bytes + kv_bytes) / (ms_step * 1e-3) / 1e9 / peak,
                               "frac_of_nominal_8tbs": (weight_bytes + kv_bytes) / (ms_step * 1e-3) / 1e9 / 8000.0},
                "split_ms_per_step_serialised": split}
    if tl:
        # in-graph: the GEMM launches' own time from "token rows exist" to "last CTA done", summed over the step
        lm_bytes = tdims["vocab"] * tdims["d_model"] * esz
        layer_bytes = (weight_bytes - lm_bytes) / tdims["n_layers"]
        g_ms = (tl["gemm_us_per_layer"] * tdims["n_layers"] + tl["lm_head_gemm_us"]) * 1e-3
        roofline["in_graph"] = {"gemm_ms_in_step": g_ms, "gbs": weight_bytes / (g_ms * 1e-3) / 1e9, "frac": weight_bytes / (g_ms * 1e-3) / 1e9 / peak,
                                "layer_period_us": tl["layer_period_us"], "layer_bytes": layer_bytes,
                                "layer_us_at_peak": layer_bytes / (peak * 1e9) * 1e6,
                                "timing": "time stamps inside the kernels of the captured step (sd_launch_stamps), inner layers averaged",
                                "timeline": tl["launches"], "columns": tl["columns"]}

    # ---- e2e: drafts and results in pinned host memory, copies inside the timed region
    xh = x.cpu().pin_memory(); qh = q.cpu().pin_memory()
    nh = torch.zeros((B,), dtype=torch.int32).pin_memory(); oh = torch.zeros((B, gamma + 1), dtype=torch.int32).pin_memory()
    for _ in range(W):
        ctx.sd_verify_accept_host(seqs, gamma, xh, qh, nh, oh)
    barrier()
    t0 = time.perf_counter()
    ev0.record(stream)
    for _ in range(K):
        ctx.sd_verify_accept_host(seqs, gamma, xh, qh, nh, oh)
    ev1.record(stream)
    barrier()
    e2e_ms = max_over_ranks(max(ev0.elapsed_time(ev1), (time.perf_counter() - t0) * 1e3)) / K
    e2e = {"value": replicas.whole_job_tokens_per_s(world, B, gamma, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
           "h2d_bytes_per_step": int(xh.numel() * 4 + qh.numel() * 4), "d2h_bytes_per_step": int(nh.numel() * 4 + oh.numel() * 4)}
    ctx.sd_seq_read(0)
    rewind()

    # ---- sustained: the same step for about two seconds (blocks of K steps from the same contexts), clocks sampled throughout
    sustained = None
    if world == 1 and args.sustained_s > 0:
        sampler2 = ClockSampler(gpu_id)
        blocks, tot_ms, t_end = 0, 0.0, time.perf_counter() + args.sustained_s
        while time.perf_counter() < t_end:
            rewind()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(K):
                verify_step()
            b.record(stream)
            torch.cuda.synchronize()
            tot_ms += a.elapsed_time(b); blocks += 1
        sustained = {"ms_per_step": tot_ms / (blocks * K), "steps": blocks * K, "seconds": round(args.sustained_s, 1), "clocks": sampler2.stop()}
        rewind()

    # ---- whole iterations and the cost ratio c of Eq. 1
    def timed(fn, n):
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    def iteration():
        ctx.sd_draft_steps(seqs, gamma, x, q)
        verify_step()

    ctx.sd_draft_steps(seqs, gamma, x, q)
    draft_ms = timed(lambda: ctx.sd_draft_steps(seqs, gamma, x, q), 3) / gamma
    l1 = torch.zeros((B, 1, V), dtype=torch.float32, device=dev)
    ctx.sd_target_step(seqs, l1)
    decode_ms = timed(lambda: ctx.sd_target_step(seqs, l1), 3)
    iter_ms = timed(iteration, n_iter_phase)
    c = draft_ms / decode_ms
    extras = {"draft_step_ms": draft_ms, "target_decode_step_ms": decode_ms, "iteration_ms": iter_ms, "c": c,
              "verify_over_decode": ms_step / decode_ms,
              "eq1_speedup": {f"alpha={a}": eq1_speedup(a, gamma, c) for a in (0.6, 0.8)},
              "best_gamma": {f"alpha={a}": dict(zip(("gamma", "speedup"), sd.sd_best_gamma(a, c, 15))) for a in (0.6, 0.8)},
              "routed_drafts": [int(r) for r in routed], "drafts": "one base draft + low-rank adapters (rank 16)" if getattr(args, "lora", False) else "separate models"}
    status = ctx.sd_device_status()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = oracle_sample(args.config)

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": cfg["dtype"], "data": "synthetic",
            "config": {"workload": f"{args.config}: batch {B}, gamma {gamma}, prompt {lens if B > 1 else lens[0]}, "
                                   f"target {tdims['n_layers']}x{tdims['d_model']}, verify step = sd_verify + sd_accept_seqs + sd_kv_rollback",
                       "context_at_end_of_timed_steps": n_ctx if B > 1 else n_ctx[0],
                       "l2": "weights (>= 2 GB per step) far exceed the 126 MB L2; no flush", "replicas": world,
                       "device_status": status},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu, "sustained": sustained, **extras,
        }))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def run_gamma_sweep(args):
    """Verify step, draft step and Eq. 1 against gamma at one configuration (one GPU): for every gamma of the range the
    verify step is timed like the headline (device-resident inputs, CUDA events), the cost ratio c comes from the
    library's own clock (sd_cost_read) and alpha-hat from its accumulator (sd_seq_alpha)."""
    lo, hi = (int(v) for v in args.gamma_sweep.split(".."))
    K, W = args.steps, args.warmup
    env = setup(args, hi, K + W + 8)
    torch, sd, ctx, dev, cfg, seqs, rewind = (env[k] for k in ("torch", "sd", "ctx", "dev", "cfg", "seqs", "rewind"))
    wl, tdims = cfg["workload"], cfg["target"]
    B, V = wl["batch"], tdims["vocab"]
    stream = torch.cuda.current_stream(dev)
    l1 = torch.zeros((B, 1, V), dtype=torch.float32, device=dev)
    rows = []
    for gamma in range(lo, hi + 1):
        x = torch.zeros((B, gamma), dtype=torch.int32, device=dev)
        q = torch.zeros((B, gamma, V), dtype=torch.float32, device=dev)
        logits = torch.zeros((B, gamma + 1, V), dtype=torch.float32, device=dev)
        n_acc = torch.zeros((B,), dtype=torch.int32, device=dev)
        out_tok = torch.zeros((B, gamma + 1), dtype=torch.int32, device=dev)
        rewind()
        for _ in range(3):                          # graphs captured, caches warm
            ctx.sd_draft_steps(seqs, gamma, x, q)
            ctx.sd_verify_accept(seqs, gamma, x, q, logits, n_acc, out_tok)
            ctx.sd_target_step(seqs, l1)
        rewind()
        ctx.sd_cost_timing(1)
        ctx.sd_cost_read(reset=1)
        for _ in range(5):                          # whole iterations on the library's clock: c, and alpha-hat of these drafts
            ctx.sd_draft_steps(seqs, gamma, x, q)
            ctx.sd_verify_accept(seqs, gamma, x, q, logits, n_acc, out_tok)
        for _ in range(5):
            ctx.sd_target_step(seqs, l1)
        cost = ctx.sd_cost_read(reset=1)
        ctx.sd_cost_timing(0)
        a_sum, judged = ctx.sd_seq_alpha(0)
        rewind()
        ctx.sd_draft_steps(seqs, gamma, x, q)
        rewind()
        for _ in range(W):
            ctx.sd_verify_accept(seqs, gamma, x, q, logits, n_acc, out_tok)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(K):
            ctx.sd_verify_accept(seqs, gamma, x, q, logits, n_acc, out_tok)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / K
        c = cost["c"]
        rows.append({"gamma": gamma, "verify_step_ms": ms, "verify_step_tokens_per_s": B * (gamma + 1) / (ms * 1e-3),
                     "draft_pass_ms": cost["draft_pass_ms"], "target_pass_ms": cost["target_pass_ms"], "verify_pass_ms_library_clock": cost["verify_pass_ms"],
                     "c": c, "verify_over_decode": ms / cost["target_pass_ms"] if cost["target_pass_ms"] else None,
                     "alpha_hat_random_init": a_sum / judged if judged else None,
                     "eq1_speedup": {f"alpha={a}": eq1_speedup(a, gamma, c) for a in (0.6, 0.8)},
                     # Eq. 1 takes the verify pass to cost one decode pass; with the measured verify pass instead:
                     "speedup_with_measured_verify": {f"alpha={a}": (1 - a ** (gamma + 1)) / (1 - a) * cost["target_pass_ms"] /
                                                      (gamma * cost["draft_pass_ms"] + ms) for a in (0.6, 0.8)} if cost["target_pass_ms"] else None})
    c_mean = sum(r["c"] for r in rows) / len(rows)
    status = ctx.sd_device_status()
    print(json.dumps({"metric": "gamma_sweep", "unit": "per gamma", "n_gpus": 1, "steps": K, "warmup": W, "dtype": cfg["dtype"], "data": "synthetic",
                      "config": {"workload": f"{args.config}: batch {B}, gamma {lo}..{hi}, prompt {env['lens'] if B > 1 else env['lens'][0]}", "device_status": status},
                      "best_gamma": {f"alpha={a}": dict(zip(("gamma", "speedup"), sd.sd_best_gamma(a, c_mean, hi))) for a in (0.6, 0.8)},
                      "c_mean": c_mean, "sweep": rows}))
    ctx.close()


def run_kmeans_bench(args):
    """One Lloyd iteration over synthetic sentence vectors (offline task partitioning): 2,097,152 x 384 fp32 points
    (3.2 GB, far beyond L2), 4 clusters; bound by the one pass over the points."""
    import torch
    from paper_2505_08600_b200 import binding as sd
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    n, dim, k = 2 * 1024 * 1024, 384, 4
    g = torch.Generator(device=dev); g.manual_seed(6)
    centers = torch.nn.functional.normalize(torch.randn((k, dim), generator=g, device=dev), dim=1)
    task = torch.randint(0, k, (n,), generator=g, device=dev)
    x = torch.nn.functional.normalize(centers[task] + torch.randn((n, dim), generator=g, device=dev) * (0.6 / dim ** 0.5), dim=1).contiguous()
    c = x[:k].clone()
    labels = torch.zeros((n,), dtype=torch.int32, device=dev)
    c_out = torch.zeros_like(c); counts = torch.zeros((k,), dtype=torch.int64, device=dev); inertia = torch.zeros((1,), dtype=torch.float64, device=dev)
    for _ in range(max(3, args.warmup)):
        sd.sd_kmeans_step(x, c, labels, c_out, counts, inertia)
    torch.cuda.synchronize()
    K = max(5, min(args.steps, 50))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(torch.cuda.current_stream())
    for _ in range(K):
        sd.sd_kmeans_step(x, c, labels, c_out, counts, inertia)
    e1.record(torch.cuda.current_stream()); torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / K
    peak, kind = _peaks()
    bytes_ = n * dim * 4 + n * 4
    # the oracle on a bounded sample of the same points
    from oracle import partition
    xs = x[: 200000].cpu().numpy(); cs = c.cpu().numpy()
    t0 = time.perf_counter(); reps = 0
    while time.perf_counter() - t0 < 10.0:
        partition.kmeans_step(xs, cs); reps += 1
    cpu_pts = reps * xs.shape[0] / (time.perf_counter() - t0)
    print(json.dumps({"metric": "kmeans_points_per_s", "unit": "points/s", "value": n / (ms * 1e-3), "ms_per_step": ms, "n_gpus": 1, "steps": K,
                      "dtype": "f32", "data": "synthetic", "config": {"workload": f"K-means step: {n} x {dim} fp32 points, {k} clusters (labels + new centroids + inertia)"},
                      "roofline": {"bound": "hbm", "achieved": bytes_ / (ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s", "frac": bytes_ / (ms * 1e-3) / 1e9 / peak,
                                   "peak_kind": f"of {kind}", "algorithmic_bytes_per_launch": bytes_, "traffic": None},
                      "counts": counts.cpu().tolist(), "inertia": float(inertia.item()),
                      "cpu_baseline": {"value": cpu_pts, "unit": "points/s", "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                                       "sample": f"{xs.shape[0]} of the points, {reps} repeats"}}))


def run_mamba_bench(args):
    """The Mamba-based prompt classifier on a batch the size of the paper's test set: 400 prompts of 32..512 tokens
    (uniform), vocabulary 21128, d_model 128, 16 states, 4 classes; all 400 scored by one call."""
    import torch
    from paper_2505_08600_b200 import binding as sd
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    vocab, n_prompts = 21128, 400
    w = synth.make_mamba_classifier(vocab, d_model=128, d_state=16, d_conv=4, expand=2, n_classes=4, seed=0)
    clf = sd.MambaClassifier(w)
    lens = synth.make_prompt_lengths(n_prompts, 32, 512, seed=8)
    starts = np.concatenate([[0], np.cumsum(lens)[:-1]]).astype(np.int64)
    tokens_h = np.concatenate([synth.make_prompt(vocab, int(n), seed=8, seq=i) for i, n in enumerate(lens)])
    tokens = torch.from_numpy(tokens_h).to(dev)
    for _ in range(max(3, args.warmup)):
        scores, labels = clf.classify(tokens, starts, lens)
    torch.cuda.synchronize()
    K = max(5, min(args.steps, 50))
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(torch.cuda.current_stream())
    for _ in range(K):
        scores, labels = clf.classify(tokens, starts, lens)
    e1.record(torch.cuda.current_stream()); torch.cuda.synchronize()
    ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3) / K          # the call uploads small host tables: wall time counts
    T = int(lens.sum())
    D, Di, N, R, Kc = 128, 256, 16, 8, 4
    flop = T * 2.0 * (2 * Di * D + Kc * Di + (R + 2 * N) * Di + R * Di + 2 * 3 * Di * N) + n_prompts * 2.0 * (D * Di + 4 * D)
    alu_peak = 148 * 128 * 2 * 1.965e9                                           # fp32 lanes x 2 flop x clock
    from oracle import classifier_mamba as om
    t0 = time.perf_counter(); done = 0
    while time.perf_counter() - t0 < 10.0 and done < n_prompts:
        om.classify(w, tokens_h[starts[done]: starts[done] + lens[done]]); done += 1
    cpu_s = (time.perf_counter() - t0) / done
    agree = sum(int(om.classify(w, tokens_h[starts[i]: starts[i] + lens[i]])[0] == int(labels[i])) for i in range(min(done, 25)))
    print(json.dumps({"metric": "mamba_classifier_prompts_per_s", "unit": "prompts/s", "value": n_prompts / (ms * 1e-3), "ms_per_step": ms,
                      "ms_per_prompt": ms / n_prompts, "n_gpus": 1, "steps": K, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": f"{n_prompts} prompts, {T} tokens (32..512 each), vocab {vocab}, d_model 128, 16 states, 4 classes, one call"},
                      "roofline": {"bound": "alu", "achieved": flop / (ms * 1e-3) / 1e12, "peak": alu_peak / 1e12, "unit": "TFLOP/s",
                                   "frac": flop / (ms * 1e-3) / alu_peak, "peak_kind": "148 SMs x 128 fp32 lanes x 2 x 1.965 GHz", "traffic": None},
                      "labels_agree_with_oracle": f"{agree} of {min(done, 25)}",
                      "cpu_baseline": {"value": 1.0 / cpu_s, "unit": "prompts/s", "cores": len(os.sched_getaffinity(0)), "kind": "oracle", "sample": f"the first {done} prompts"}}))


def run_prefill_bench(args):
    """Prefill of one 512-token prompt of the configuration's target model (the contraction-bound regime): forward over the
    prompt in batches of at most 256 rows through the same weight GEMM as the verify step, no logits.  The draft's prefill
    runs in the same call and is timed with it; flops counted are the target's weight GEMMs only."""
    env = setup(args, 1, 8)
    torch, ctx, dev, cfg, seqs = (env[k] for k in ("torch", "ctx", "dev", "cfg", "seqs"))
    t = cfg["target"]
    n = env["lens"][0]
    prompt = synth.make_prompt(t["vocab"], n, seed=3)
    stream = torch.cuda.current_stream(dev)

    def once():
        ctx.sd_seq_begin(0, prompt, 0)
        ctx.sd_route_prompt([0], forced_task=[0])
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        ctx.sd_prefill([0])
        e1.record(stream); torch.cuda.synchronize()
        return e0.elapsed_time(e1)
    for _ in range(3):
        once()
    K = max(3, min(args.steps, 10))
    ms = sorted(once() for _ in range(K))[K // 2]
    layer_params = synth.param_count(t, streamed_only=True) - t["vocab"] * t["d_model"]
    flop = 2.0 * layer_params * (n - 1)
    peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
    peak = float(peaks.get("bf16_tflops", 1590.0))
    print(json.dumps({"metric": "prefill_tokens_per_s", "unit": "tokens/s", "value": (n - 1) / (ms * 1e-3), "ms_per_step": ms, "n_gpus": 1, "steps": K,
                      "dtype": cfg["dtype"], "data": "synthetic",
                      "config": {"workload": f"{args.config}: prefill of one {n}-token prompt (target {t['n_layers']}x{t['d_model']} and its routed draft), rows in batches of <= 256"},
                      "roofline": {"bound": "tensor", "achieved": flop / (ms * 1e-3) / 1e12, "peak": peak, "unit": "TFLOP/s", "frac": flop / (ms * 1e-3) / 1e12 / peak,
                                   "peak_kind": "of measured" if peaks else "of fallback", "traffic": None,
                                   "note": "the draft's prefill and the attention over the prompt are inside the timed call; flops are the target's layer GEMMs"},
                      "device_status": ctx.sd_device_status()}))
    ctx.close()


def run_accept_microbench(args):
    """Accept / reject / resample kernel alone at the 13B configuration's shape (8 sequences, gamma 8, vocab 32000):
    draft distributions are softmax(target_logits + N(0, sigma^2)) so that sigma sets the acceptance rate."""
    import torch
    from paper_2505_08600_b200 import binding as sd
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    wl, t = synth.CONFIGS["13b"]["workload"], synth.CONFIGS["13b"]["target"]
    B, gamma, V, T = wl["batch"], wl["gamma"], t["vocab"], wl["temperature"]
    g = torch.Generator(device=dev); g.manual_seed(5)
    logits = torch.randn((B, gamma + 1, V), generator=g, device=dev) * (0.02 * t["d_model"] ** 0.5)   # spread of random-init logits
    p = torch.softmax(logits.double() / T, dim=-1)
    n_acc = torch.zeros((B,), dtype=torch.int32, device=dev); out_tok = torch.zeros((B, gamma + 1), dtype=torch.int32, device=dev)
    seq_id = torch.arange(B, dtype=torch.int32, device=dev)
    out = []
    for sigma in (0.5, 1.0, 2.0):
        q = torch.softmax((logits[:, :gamma] + sigma * torch.randn((B, gamma, V), generator=g, device=dev)).double() / T, dim=-1).float().contiguous()
        alpha_hat = float(torch.minimum(p[:, :gamma].float(), q).sum(-1).mean())
        x = torch.multinomial(q.reshape(-1, V), 1, generator=g).reshape(B, gamma).to(torch.int32)
        hist = [0] * (gamma + 1)
        its = 200
        it = torch.zeros((B,), dtype=torch.int32, device=dev)
        for i in range(3):
            sd.sd_accept(logits, q, x, T, 5, it, seq_id, n_acc, out_tok, target_is_logits=1)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(torch.cuda.current_stream())
        for i in range(its):
            sd.sd_accept(logits, q, x, T, 5, it, seq_id, n_acc, out_tok, target_is_logits=1)
        e1.record(torch.cuda.current_stream()); torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / its * 1e3
        for i in range(64):                                   # acceptance statistics over fresh uniforms (the iteration is a Philox counter word)
            it.fill_(i)
            sd.sd_accept(logits, q, x, T, 5, it, seq_id, n_acc, out_tok, target_is_logits=1)
            for n in n_acc.cpu().tolist():
                hist[n] += 1
        tot = sum(hist)
        out.append({"sigma": sigma, "alpha_hat": alpha_hat, "kernel_us": us, "mean_accepted": sum(i * h for i, h in enumerate(hist)) / tot,
                    "n_acc_hist": [h / tot for h in hist]})
    print(json.dumps({"metric": "accept_kernel_us", "unit": "us per call", "config": {"workload": f"accept microbench: {B} sequences, gamma {gamma}, vocab {V}, T {T}"},
                      "bytes_touched_upper": B * (2 * gamma + 1) * V * 4, "results": out}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="7b", choices=sorted(synth.CONFIGS) + ["all"], help="'all': one JSON line per configuration, each in its own process")
    ap.add_argument("--gamma-sweep", default=None, metavar="LO..HI", help="time the verify and draft steps for every gamma of the range and exit")
    ap.add_argument("--gamma", type=int, default=None)
    ap.add_argument("--profile-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sustained-s", type=float, default=2.0, help="seconds of back-to-back verify steps for the sustained figure (0: skip)")
    ap.add_argument("--accept-microbench", action="store_true", help="time the accept kernel alone (sigma sweep) and exit")
    ap.add_argument("--lora", action="store_true", help="drafts = one base draft + one low-rank adapter per task (sequences of all tasks share each draft pass)")
    ap.add_argument("--prefill", action="store_true", help="time the prefill of one prompt of the configuration and exit")
    ap.add_argument("--mamba", action="store_true", help="time the Mamba-based prompt classifier on 400 synthetic prompts and exit")
    ap.add_argument("--kmeans", action="store_true", help="time one K-means step over synthetic sentence vectors and exit")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    launched = "WORLD_SIZE" in os.environ
    if args.config == "all":
        if launched and int(os.environ["WORLD_SIZE"]) > 1:
            raise SystemExit("--config all runs one process per configuration; start it without a launcher")
        rc = 0
        for name in synth.CONFIGS:
            argv = [sys.executable, os.path.abspath(__file__)] + [a for a in sys.argv[1:]]
            i = argv.index("--config")
            argv[i + 1] = name
            rc = rc or subprocess.run(argv).returncode
        sys.exit(rc)
    if args.impl == "ours" and args.gpus > 1 and not launched and not args.accept_microbench and not args.gamma_sweep and not args.kmeans and not args.mamba and not args.prefill:
        # no launcher: this process starts the N replicas itself (one per GPU) and passes rank 0's line through
        rc, out = replicas.spawn_local(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:])
        sys.stdout.write(out)
        sys.exit(rc)
    if args.accept_microbench:
        run_accept_microbench(args)
    elif args.kmeans:
        run_kmeans_bench(args)
    elif args.mamba:
        run_mamba_bench(args)
    elif args.prefill:
        run_prefill_bench(args)
    elif args.gamma_sweep:
        run_gamma_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
