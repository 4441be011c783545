"""Seeded synthetic inputs: model shapes, random-init weights, prompts, classifier weights.

This module only produces DATA.  It holds none of the method's arithmetic (no
softmax, no sampling rule, no transformer math) and is the one place that both
the CPU checker and the CUDA library are fed from.  Shapes follow the five
benchmark configurations; values stand in for the trained LLaMA weights and the
Wanjuan / ChemData prompts of the paper's Sec. 3.1, which are not available
offline: all matrices and embeddings are N(0, 0.02), norm gains are 1, prompts
are uniform-random token ids.
"""
from __future__ import annotations

import numpy as np


def _m(L, d, H, Hkv, hd, F, V):
    return dict(n_layers=L, d_model=d, n_heads=H, n_kv_heads=Hkv, head_dim=hd, d_ffn=F, vocab=V)


# name -> dict(dtype, target, drafts[list], classifier(d_in, d_hidden, n_classes), workload)
CONFIGS = {
    "tiny": dict(
        dtype="f32",
        target=_m(2, 256, 4, 4, 64, 688, 1024),
        drafts=[_m(1, 128, 2, 2, 64, 344, 1024)] * 2,
        classifier=(256, 64, 2),
        workload=dict(batch=1, prompt=32, gamma=4, max_new=64, temperature=1.0, seed=1, max_ctx=128),
    ),
    "1b": dict(
        dtype="bf16",
        target=_m(16, 2048, 32, 8, 64, 8192, 32000),
        drafts=[_m(2, 768, 12, 12, 64, 3072, 32000), _m(4, 768, 12, 12, 64, 3072, 32000),
                _m(6, 768, 12, 12, 64, 3072, 32000)],
        classifier=(2048, 256, 3),
        workload=dict(batch=1, prompt=128, gamma=5, max_new=128, temperature=0.7, seed=2, max_ctx=512),
    ),
    "7b": dict(
        dtype="bf16",
        target=_m(32, 4096, 32, 32, 128, 11008, 32000),
        drafts=[_m(12, 768, 12, 12, 64, 3072, 32000)] * 4,
        classifier=(4096, 512, 4),
        workload=dict(batch=1, prompt=512, gamma=5, max_new=128, temperature=1.0, seed=3, max_ctx=2048),
    ),
    "7b_batch16": dict(
        dtype="bf16",
        target=_m(32, 4096, 32, 32, 128, 11008, 32000),
        drafts=[_m(12, 768, 12, 12, 64, 3072, 32000)] * 4,
        classifier=(4096, 512, 4),
        workload=dict(batch=16, prompt=(256, 1024), gamma=5, max_new=128, temperature=1.0, seed=4, max_ctx=4096),
    ),
    "13b": dict(
        dtype="bf16",
        target=_m(40, 5120, 40, 40, 128, 13824, 32000),
        drafts=[_m(16, 1024, 16, 16, 64, 4096, 32000)] * 4,
        classifier=(5120, 512, 4),
        workload=dict(batch=8, prompt=8192 - 9, gamma=8, max_new=128, temperature=1.0, seed=5, max_ctx=8192),
    ),
}

LAYER_MATS = ("wq", "wk", "wv", "wo", "wg", "wu", "wd")


def mat_shapes(dims):
    d, dq, dkv, F = dims["d_model"], dims["n_heads"] * dims["head_dim"], dims["n_kv_heads"] * dims["head_dim"], dims["d_ffn"]
    return dict(wq=(dq, d), wk=(dkv, d), wv=(dkv, d), wo=(d, dq), wg=(F, d), wu=(F, d), wd=(d, F))


def param_count(dims, streamed_only=False):
    s = mat_shapes(dims)
    per_layer = sum(a * b for a, b in s.values())
    n = dims["n_layers"] * per_layer + dims["vocab"] * dims["d_model"]      # layers + lm_head
    if not streamed_only:
        n += dims["vocab"] * dims["d_model"] + (2 * dims["n_layers"] + 1) * dims["d_model"]
    return n


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even conversion of fp32 values to bf16 bit patterns (uint16)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + r) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def _rng(seed, stream):
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def _normal(shape, seed, stream, std, dtype):
    a = _rng(seed, stream).standard_normal(shape, dtype=np.float32) * np.float32(std)
    return f32_to_bf16_bits(a) if dtype == "bf16" else a


def make_weights(dims, seed=0, model_index=0, dtype="f32", std=0.02):
    """dict of numpy arrays: fp32, or uint16 bf16 bit patterns when dtype == 'bf16'.
    Norm gains are always fp32 ones.  model_index separates the random streams of
    target (0) and drafts (1..K)."""
    L, d, V = dims["n_layers"], dims["d_model"], dims["vocab"]
    shapes = mat_shapes(dims)
    base = model_index * 100000
    w = dict(
        embed=_normal((V, d), seed, base + 1, std, dtype),
        lm_head=_normal((V, d), seed, base + 2, std, dtype),
        final_norm=np.ones(d, dtype=np.float32),
        norm1=[np.ones(d, dtype=np.float32) for _ in range(L)],
        norm2=[np.ones(d, dtype=np.float32) for _ in range(L)],
    )
    for i, name in enumerate(LAYER_MATS):
        w[name] = [_normal(shapes[name], seed, base + 1000 + l * 16 + i, std, dtype) for l in range(L)]
    return w


def make_classifier(d_in, d_hidden, n_classes, seed=0):
    """fp32 MLP weights; N(0,1) matrices and N(0,0.01) biases so that class scores of
    different random prompts differ by far more than rounding noise."""
    g = _rng(seed, 777)
    return dict(
        w1=g.standard_normal((d_hidden, d_in), dtype=np.float32),
        b1=(g.standard_normal(d_hidden, dtype=np.float32) * np.float32(0.01)),
        w2=g.standard_normal((n_classes, d_hidden), dtype=np.float32),
        b2=(g.standard_normal(n_classes, dtype=np.float32) * np.float32(0.01)),
    )


def make_prompt(vocab, n_tokens, seed=1, seq=0):
    return _rng(seed, 5000 + seq).integers(0, vocab, size=n_tokens, dtype=np.int64).astype(np.int32)


def make_prompt_lengths(batch, lo, hi, seed=4):
    return _rng(seed, 4999).integers(lo, hi + 1, size=batch, dtype=np.int64).astype(np.int32)


def make_logits(shape, seed, stream=0, std=1.0):
    return _rng(seed, 9000 + stream).standard_normal(shape, dtype=np.float32) * np.float32(std)


def make_sentence_vectors(n, dim=384, n_tasks=4, seed=6, spread=0.6):
    """Stand-in for the sentence vectors of the offline partitioning step: n unit-length fp32 vectors of `dim`
    components in n_tasks groups (a random unit direction per task plus isotropic noise of relative size `spread`,
    renormalised), and the group of every vector.  Groups overlap a little, like the paper's 90-99 % clusterable tasks."""
    g = _rng(seed, 8800)
    centers = g.standard_normal((n_tasks, dim), dtype=np.float32)
    centers /= np.linalg.norm(centers, axis=1, keepdims=True)
    task = g.integers(0, n_tasks, size=n, dtype=np.int64).astype(np.int32)
    x = centers[task] + g.standard_normal((n, dim), dtype=np.float32) * np.float32(spread / np.sqrt(dim))
    x /= np.linalg.norm(x, axis=1, keepdims=True)
    return np.ascontiguousarray(x, dtype=np.float32), task


def make_mamba_classifier(vocab, d_model=128, d_state=16, d_conv=4, expand=2, n_classes=4, seed=0):
    """fp32 weights of the Mamba-based prompt classifier (embedding, one selective state-space layer, pooled output,
    fully connected layer), initialised the way the Mamba paper initialises its layer: A = -(1..N) per channel, step
    sizes softplus(b_dt) log-uniform in [1e-3, 1e-1], D = 1, projections N(0, 1/fan_in); embedding N(0, 1)."""
    g = _rng(seed, 7100)
    Di, R = expand * d_model, (d_model + 15) // 16

    def n(shape, std):
        return (g.standard_normal(shape, dtype=np.float32) * np.float32(std)).astype(np.float32)

    dt = np.exp(g.random(Di) * (np.log(0.1) - np.log(1e-3)) + np.log(1e-3))
    return dict(
        embed=n((vocab, d_model), 1.0),
        w_in=n((2 * Di, d_model), d_model ** -0.5),
        w_conv=n((Di, d_conv), d_conv ** -0.5), b_conv=n((Di,), 0.02),
        w_x=n((R + 2 * d_state, Di), Di ** -0.5),
        w_dt=n((Di, R), R ** -0.5), b_dt=(dt + np.log(-np.expm1(-dt))).astype(np.float32),      # inverse softplus
        a_log=np.log(np.tile(np.arange(1, d_state + 1, dtype=np.float32), (Di, 1))).astype(np.float32),
        d_skip=np.ones(Di, dtype=np.float32),
        w_out=n((d_model, Di), Di ** -0.5),
        w_fc=n((n_classes, d_model), 1.0), b_fc=n((n_classes,), 0.01),
    )


def make_lora(dims, rank, task, seed=0, std=0.05, dtype="bf16"):
    """One task's low-rank adapter for every layer of a draft: dict "qkv" / "wo" / "gu" / "wd" -> list over layers of
    (A [rank][in], B [out][rank]), N(0, std) entries (with alpha / r = 2 and rank 16 the update B A has about the spread
    of the N(0, 0.02) base weights, so tasks differ visibly), bf16 bit patterns unless dtype == 'f32'."""
    d, F = dims["d_model"], dims["d_ffn"]
    dq, dkv = dims["n_heads"] * dims["head_dim"], dims["n_kv_heads"] * dims["head_dim"]
    shapes = {"qkv": (dq + 2 * dkv, d), "wo": (d, dq), "gu": (2 * F, d), "wd": (d, F)}
    out = {}
    for i, (name, (n_out, n_in)) in enumerate(shapes.items()):
        out[name] = [(_normal((rank, n_in), seed, 600000 + task * 10000 + l * 16 + 2 * i, std, dtype),
                      _normal((n_out, rank), seed, 600000 + task * 10000 + l * 16 + 2 * i + 1, std, dtype)) for l in range(dims["n_layers"])]
    return out
