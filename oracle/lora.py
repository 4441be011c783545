"""CPU oracle of low-rank adapted drafts (test infrastructure only).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module; it shares nothing with
the CUDA library.  Section 2.3 builds every task's draft from one base draft by LoRA fine-tuning; the LoRA paper
defines the adapted matrix as

    W' = W + (alpha / r) * B A,        A [r][in],  B [out][r].

The oracle is that definition written out: the adapted matrices are formed in float64 and handed, as fp32 arrays, to
the ordinary oracle model (storing W' in fp32 rounds it by 6e-8 relative, three orders below the bf16 noise of the
path it is compared with; bf16 base weights and factors enter with their exact values).  An adapter is given per fused
matrix of a layer: "qkv" (one A for the stacked query, key and value rows), "wo", "gu" (one A for the stacked gate and
up rows), "wd".
"""
from __future__ import annotations

import numpy as np


def _f64(a):
    a = np.asarray(a)
    if a.dtype == np.uint16:                                  # bf16 bit patterns
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def adapted_matrix(w, a, b, scale):
    return _f64(w) + float(scale) * (_f64(b) @ _f64(a))


def merged_weights(dims, base, adapter, scale):
    """fp32 weight dict of the base model with one task's adapter folded in.  adapter: dict name -> list over layers of
    (A, B) or None, names "qkv", "wo", "gu", "wd"."""
    L = dims["n_layers"]
    dq = dims["n_heads"] * dims["head_dim"]
    dkv = dims["n_kv_heads"] * dims["head_dim"]
    F = dims["d_ffn"]
    out = dict(embed=_f64(base["embed"]).astype(np.float32), lm_head=_f64(base["lm_head"]).astype(np.float32),
               final_norm=np.asarray(base["final_norm"], dtype=np.float32),
               norm1=[np.asarray(g, dtype=np.float32) for g in base["norm1"]], norm2=[np.asarray(g, dtype=np.float32) for g in base["norm2"]])
    for name in ("wq", "wk", "wv", "wo", "wg", "wu", "wd"):
        out[name] = [None] * L

    def get(kind, l):
        lst = adapter.get(kind)
        return lst[l] if lst is not None and lst[l] is not None else None

    for l in range(L):
        ab = get("qkv", l)
        for name, lo, hi in (("wq", 0, dq), ("wk", dq, dq + dkv), ("wv", dq + dkv, dq + 2 * dkv)):
            w = _f64(base[name][l])
            if ab is not None:
                w = w + float(scale) * (_f64(ab[1])[lo:hi] @ _f64(ab[0]))
            out[name][l] = np.ascontiguousarray(w, dtype=np.float32)
        ab = get("gu", l)
        for name, lo, hi in (("wg", 0, F), ("wu", F, 2 * F)):
            w = _f64(base[name][l])
            if ab is not None:
                w = w + float(scale) * (_f64(ab[1])[lo:hi] @ _f64(ab[0]))
            out[name][l] = np.ascontiguousarray(w, dtype=np.float32)
        for kind, name in (("wo", "wo"), ("wd", "wd")):
            ab = get(kind, l)
            w = _f64(base[name][l]) if ab is None else adapted_matrix(base[name][l], ab[0], ab[1], scale)
            out[name][l] = np.ascontiguousarray(w, dtype=np.float32)
    return out
