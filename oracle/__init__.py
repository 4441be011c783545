"""ctypes front end of the CPU oracle (test infrastructure only).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares nothing with the CUDA library: the C file is compiled
with gcc on first use (``-O2 -ffp-contract=off``, never fast-math) and loaded
here.  Argument conventions follow the C file; arrays are numpy, C-contiguous.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sd_oracle.c")
_LIB = os.path.join(_HERE, "liborc.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + f".{os.getpid()}.tmp"
            subprocess.check_call(
                ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
                 "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


class Model(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
        ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ffn", C.c_int32),
        ("vocab", C.c_int32), ("wdtype", C.c_int32),
        ("rms_eps", C.c_double), ("rope_base", C.c_double),
        ("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
        ("wq", C.POINTER(C.c_void_p)), ("wk", C.POINTER(C.c_void_p)), ("wv", C.POINTER(C.c_void_p)),
        ("wo", C.POINTER(C.c_void_p)), ("wg", C.POINTER(C.c_void_p)), ("wu", C.POINTER(C.c_void_p)),
        ("wd", C.POINTER(C.c_void_p)),
        ("norm1", C.POINTER(C.c_void_p)), ("norm2", C.POINTER(C.c_void_p)),
    ]


class Cache(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("max_ctx", C.c_int32)]


class Counters(C.Structure):
    _fields_ = [("iterations", C.c_int64), ("drafted", C.c_int64),
                ("accepted", C.c_int64), ("emitted", C.c_int64)]


class Trace(C.Structure):
    _fields_ = [("cap_iters", C.c_int32), ("n_iters", C.c_int32),
                ("len_before", C.c_void_p), ("n_acc", C.c_void_p), ("x", C.c_void_p),
                ("out_tok", C.c_void_p), ("q", C.c_void_p), ("p", C.c_void_p),
                ("logits", C.c_void_p)]


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_philox4x32_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_philox4x32_10.restype = None
        L.orc_uniform24.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32]
        L.orc_uniform24.restype = C.c_uint32
        L.orc_argmax.argtypes = [C.c_void_p, C.c_int]
        L.orc_argmax.restype = C.c_int
        L.orc_softmax_T.argtypes = [C.c_void_p, C.c_int, C.c_double, C.c_void_p]
        L.orc_softmax_T.restype = None
        L.orc_sample_icdf.argtypes = [C.c_void_p, C.c_int, C.c_uint32]
        L.orc_sample_icdf.restype = C.c_int
        L.orc_accept.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_uint64,
                                 C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p]
        L.orc_accept.restype = None
        L.orc_forward_cached.argtypes = [C.POINTER(Model), C.POINTER(Cache), C.c_void_p, C.c_int,
                                         C.c_int, C.c_void_p]
        L.orc_forward_cached.restype = C.c_int
        L.orc_forward_full.argtypes = [C.POINTER(Model), C.c_void_p, C.c_int, C.c_void_p]
        L.orc_forward_full.restype = C.c_int
        L.orc_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_double, C.c_void_p]
        L.orc_rmsnorm.restype = None
        L.orc_rope.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_double]
        L.orc_rope.restype = None
        L.orc_silu.argtypes = [C.c_double]
        L.orc_silu.restype = C.c_double
        L.orc_linear.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p]
        L.orc_linear.restype = None
        L.orc_attention_head.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p]
        L.orc_attention_head.restype = None
        L.orc_route_prompt.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int,
                                       C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p,
                                       C.c_int, C.c_int, C.c_void_p]
        L.orc_route_prompt.restype = C.c_int
        L.orc_spec_decode.argtypes = [C.POINTER(Model), C.POINTER(Model), C.POINTER(Cache),
                                      C.POINTER(Cache), C.c_void_p, C.c_int, C.c_int, C.c_int,
                                      C.c_double, C.c_uint64, C.c_uint32, C.c_void_p,
                                      C.POINTER(Counters), C.POINTER(Trace), C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        L.orc_spec_decode.restype = C.c_int
        L.orc_alpha_terms.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        L.orc_alpha_terms.restype = None
        L.orc_mc_fixed.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int64, C.c_uint64,
                                   C.c_void_p, C.c_void_p]
        L.orc_mc_fixed.restype = C.c_int64
        _lib = L
    return _lib


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


# ----------------------------------------------------------------------------
# thin numpy wrappers
# ----------------------------------------------------------------------------

def philox4x32_10(ctr, key):
    ctr = np.ascontiguousarray(ctr, dtype=np.uint32)
    key = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_ptr(ctr), _ptr(key), _ptr(out))
    return out


def uniform24(seed, it, slot, seq, purpose):
    return int(lib().orc_uniform24(seed, it, slot, seq, purpose))


def softmax_T(logits, T):
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    flat = logits.reshape(-1, logits.shape[-1])
    out = np.empty(flat.shape, dtype=np.float32)
    for i in range(flat.shape[0]):
        lib().orc_softmax_T(_ptr(flat[i]), flat.shape[1], float(T), _ptr(out[i]))
    return out.reshape(logits.shape)


def sample_icdf(w, u_int):
    w = np.ascontiguousarray(w, dtype=np.float32)
    return int(lib().orc_sample_icdf(_ptr(w), w.shape[0], int(u_int)))


def accept(p, q, x, seed, it, seq):
    """p [gamma+1, V], q [gamma, V] fp32, x [gamma] -> (n, out_tok[gamma+1] with -1 padding)."""
    p = np.ascontiguousarray(p, dtype=np.float32)
    q = np.ascontiguousarray(q, dtype=np.float32)
    x = np.ascontiguousarray(x, dtype=np.int32)
    gamma, V = q.shape[0], p.shape[1]
    assert p.shape[0] == gamma + 1
    n = np.zeros(1, dtype=np.int32)
    out = np.full(gamma + 1, -1, dtype=np.int32)
    if gamma == 0:
        q = np.zeros((1, V), dtype=np.float32)
    lib().orc_accept(_ptr(p), _ptr(q), _ptr(x), gamma, V, int(seed), int(it), int(seq), _ptr(n), _ptr(out))
    out[int(n[0]) + 1:] = -1
    return int(n[0]), out


def alpha_terms(p, q):
    """p [gamma+1, V] (or [gamma, V]), q [gamma, V] fp32 -> sum_k min(p_s(k), q_s(k)) for every slot s (float64 [gamma])."""
    p = np.ascontiguousarray(p, dtype=np.float32)
    q = np.ascontiguousarray(q, dtype=np.float32)
    gamma, V = q.shape
    out = np.zeros(gamma, dtype=np.float64)
    lib().orc_alpha_terms(_ptr(p), _ptr(q), gamma, V, _ptr(out))
    return out


class OracleModel:
    """Holds numpy weights (fp32 arrays, or uint16 arrays of bf16 bit patterns) alive and
    exposes the C struct.  ``weights`` is the dict produced by the synthetic generator:
    embed, lm_head, final_norm, and per-layer lists wq wk wv wo wg wu wd norm1 norm2."""

    def __init__(self, dims: dict, weights: dict, rms_eps: float = 1e-5, rope_base: float = 10000.0):
        self.dims = dict(dims)
        self.w = weights
        emb = weights["embed"]
        wdtype = 1 if emb.dtype == np.uint16 else 0
        L = dims["n_layers"]
        self._arrs = {}
        m = Model()
        m.n_layers, m.d_model, m.n_heads = L, dims["d_model"], dims["n_heads"]
        m.n_kv_heads, m.head_dim, m.d_ffn = dims["n_kv_heads"], dims["head_dim"], dims["d_ffn"]
        m.vocab, m.wdtype = dims["vocab"], wdtype
        m.rms_eps, m.rope_base = rms_eps, rope_base
        m.embed = emb.ctypes.data
        m.lm_head = weights["lm_head"].ctypes.data
        assert weights["final_norm"].dtype == np.float32
        m.final_norm = weights["final_norm"].ctypes.data
        for name in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2"):
            arr = (C.c_void_p * L)(*[w.ctypes.data for w in weights[name]])
            self._arrs[name] = arr
            setattr(m, name, C.cast(arr, C.POINTER(C.c_void_p)))
        self.c = m

    def new_cache(self, max_ctx: int) -> "OracleCache":
        return OracleCache(self, max_ctx)

    def forward_full(self, tokens):
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        out = np.empty((tokens.shape[0], self.dims["vocab"]), dtype=np.float64)
        rc = lib().orc_forward_full(C.byref(self.c), _ptr(tokens), tokens.shape[0], _ptr(out))
        assert rc == 0
        return out


class OracleCache:
    def __init__(self, model: OracleModel, max_ctx: int):
        d = model.dims
        n = d["n_layers"] * max_ctx * d["n_kv_heads"] * d["head_dim"]
        self.k = np.zeros(n, dtype=np.float64)
        self.v = np.zeros(n, dtype=np.float64)
        self.model = model
        self.max_ctx = max_ctx
        self.c = Cache(self.k.ctypes.data, self.v.ctypes.data, max_ctx)

    def forward(self, tokens, pos0, want_logits=True):
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        out = np.empty((tokens.shape[0], self.model.dims["vocab"]), dtype=np.float64) if want_logits else None
        rc = lib().orc_forward_cached(C.byref(self.model.c), C.byref(self.c), _ptr(tokens),
                                      tokens.shape[0], int(pos0), _ptr(out))
        if rc != 0:
            raise ValueError("oracle cache capacity exceeded")
        return out


def attention_head(q, K, V):
    """q [hd], K, V [n_ctx, hd] (float64) -> softmax(q K^T / sqrt(hd)) V."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    K = np.ascontiguousarray(K, dtype=np.float64)
    V = np.ascontiguousarray(V, dtype=np.float64)
    out = np.empty(q.shape[0], dtype=np.float64)
    lib().orc_attention_head(_ptr(q), _ptr(K), _ptr(V), K.shape[0], q.shape[0], K.shape[1], _ptr(out))
    return out


def linear(W, X):
    """X [rows, n_in] float64, W [n_out, n_in] fp32 or uint16 bf16 bits -> X W^T (float64)."""
    X = np.ascontiguousarray(X, dtype=np.float64)
    W = np.ascontiguousarray(W)
    Y = np.empty((X.shape[0], W.shape[0]), dtype=np.float64)
    lib().orc_linear(_ptr(W), 1 if W.dtype == np.uint16 else 0, W.shape[0], W.shape[1], _ptr(X), X.shape[0], _ptr(Y))
    return Y


def route_prompt(embed, tokens, w1, b1, w2, b2, forced_task=-1):
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    wdtype = 1 if embed.dtype == np.uint16 else 0
    d_in = embed.shape[1]
    d_hidden, n_classes = w1.shape[0], w2.shape[0]
    for a in (w1, b1, w2, b2):
        assert a.dtype == np.float32 and a.flags.c_contiguous
    probs = np.zeros(n_classes, dtype=np.float64)
    k = lib().orc_route_prompt(_ptr(embed), wdtype, d_in, _ptr(tokens), tokens.shape[0],
                               _ptr(w1), _ptr(b1), d_hidden, _ptr(w2), _ptr(b2), n_classes,
                               int(forced_task), _ptr(probs))
    return int(k), probs


def spec_decode(target: OracleModel, draft: OracleModel | None, prompt, max_new, gamma, T, seed,
                seq_id=0, max_ctx=None, trace_iters=0, trace_probs=False, trace_logits=False):
    """Runs the whole loop for one sequence.  Returns (tokens, counters dict, trace dict|None)."""
    prompt = np.ascontiguousarray(prompt, dtype=np.int32)
    n_prompt = prompt.shape[0]
    cap = n_prompt + max_new + gamma + 2
    if max_ctx is None:
        max_ctx = cap
    toks = np.zeros(cap, dtype=np.int32)
    toks[:n_prompt] = prompt
    tc = target.new_cache(max_ctx)
    dc = draft.new_cache(max_ctx) if draft is not None else None
    V = target.dims["vocab"]
    cnt = Counters()
    alpha_sum, judged = C.c_double(0.0), C.c_int64(0)
    ln = np.zeros(1, dtype=np.int32)
    tr = None
    keep = {}
    if trace_iters > 0:
        tr = Trace()
        tr.cap_iters = trace_iters
        keep["len_before"] = np.zeros(trace_iters, dtype=np.int32)
        keep["n_acc"] = np.zeros(trace_iters, dtype=np.int32)
        keep["x"] = np.zeros((trace_iters, max(gamma, 1)), dtype=np.int32)[:, :gamma].copy()
        keep["out_tok"] = np.zeros((trace_iters, gamma + 1), dtype=np.int32)
        tr.len_before, tr.n_acc = keep["len_before"].ctypes.data, keep["n_acc"].ctypes.data
        tr.x, tr.out_tok = keep["x"].ctypes.data, keep["out_tok"].ctypes.data
        if trace_probs:
            keep["q"] = np.zeros((trace_iters, gamma, V), dtype=np.float32)
            keep["p"] = np.zeros((trace_iters, gamma + 1, V), dtype=np.float32)
            tr.q, tr.p = keep["q"].ctypes.data, keep["p"].ctypes.data
        if trace_logits:
            keep["logits"] = np.zeros((trace_iters, gamma + 1, V), dtype=np.float64)
            tr.logits = keep["logits"].ctypes.data
    rc = lib().orc_spec_decode(C.byref(target.c), C.byref(draft.c) if draft is not None else None,
                               C.byref(tc.c), C.byref(dc.c) if dc is not None else None,
                               _ptr(toks), n_prompt, int(max_new), int(gamma), float(T), int(seed),
                               int(seq_id), _ptr(ln), C.byref(cnt), C.byref(tr) if tr is not None else None,
                               C.byref(alpha_sum), C.byref(judged))
    if rc != 0:
        raise RuntimeError("oracle spec_decode failed (cache capacity?)")
    counters = dict(iterations=cnt.iterations, drafted=cnt.drafted, accepted=cnt.accepted, emitted=cnt.emitted)
    trace = None
    if tr is not None:
        n = tr.n_iters
        trace = {k: v[:n] for k, v in keep.items()}
        trace["alpha_sum"], trace["judged"] = float(alpha_sum.value), int(judged.value)      # estimate of Eq. 1's alpha: their ratio
    return toks[: int(ln[0])].copy(), counters, trace


def mc_fixed(p, q, gamma, iters, seed):
    """Monte Carlo with the same p, q in every slot.  Returns (emitted, accepted, hist of first token)."""
    p = np.ascontiguousarray(p, dtype=np.float32)
    q = np.ascontiguousarray(q, dtype=np.float32)
    V = p.shape[0]
    hist = np.zeros(V, dtype=np.int64)
    acc = np.zeros(1, dtype=np.int64)
    em = lib().orc_mc_fixed(_ptr(p), _ptr(q), V, int(gamma), int(iters), int(seed), _ptr(hist), _ptr(acc))
    return int(em), int(acc[0]), hist
