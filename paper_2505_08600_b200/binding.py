"""Thin ctypes binding of libsd.so: same names as include/sd.h, argument marshalling only.

PyTorch appears here for device memory and streams alone; every step of the path runs in
the library's kernels.  Importing this module without the built library raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsd.so")

SD_F32, SD_BF16 = 0, 1
SD_MAX_BATCH, SD_MAX_ROWS, SD_MAX_GAMMA = 64, 256, 15
T_EMBED, T_LM_HEAD, T_FINAL_NORM, T_WQ, T_WK, T_WV, T_WO, T_WG, T_WU, T_WD, T_NORM1, T_NORM2 = range(12)
TENSOR_KIND = dict(embed=T_EMBED, lm_head=T_LM_HEAD, final_norm=T_FINAL_NORM, wq=T_WQ, wk=T_WK, wv=T_WV,
                   wo=T_WO, wg=T_WG, wu=T_WU, wd=T_WD, norm1=T_NORM1, norm2=T_NORM2)


class ModelDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab", "dtype")] + \
               [("rms_eps", C.c_float), ("rope_base", C.c_float)]


class Config(C.Structure):
    _fields_ = [("max_seqs", C.c_int32), ("max_ctx", C.c_int32), ("max_gamma", C.c_int32), ("n_drafts", C.c_int32),
                ("temperature", C.c_float), ("seed", C.c_uint64), ("clf_d_hidden", C.c_int32), ("lora_adapters", C.c_int32),
                ("lora_rank", C.c_int32), ("lora_scale", C.c_float)]


class Counters(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("iterations", "drafted", "accepted", "emitted")]


class Cost(C.Structure):
    _fields_ = [("draft_pass_ms", C.c_double), ("verify_pass_ms", C.c_double), ("target_pass_ms", C.c_double), ("c", C.c_double),
                ("draft_passes", C.c_int64), ("verify_passes", C.c_int64), ("target_passes", C.c_int64)]


class MambaDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("vocab", "d_model", "d_state", "d_conv", "expand", "n_classes", "dt_rank")]


MAMBA_WEIGHT_NAMES = ("embed", "w_in", "w_conv", "b_conv", "w_x", "w_dt", "b_dt", "a_log", "d_skip", "w_out", "w_fc", "b_fc")


class MambaWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in MAMBA_WEIGHT_NAMES]


class MambaClassifier:
    """Device copy of the classifier's weights (fp32 numpy arrays in, CUDA tensors kept here) and its descriptor."""

    def __init__(self, weights, device="cuda:0"):
        self.t = {n: torch.from_numpy(np.ascontiguousarray(weights[n], dtype=np.float32)).to(device) for n in MAMBA_WEIGHT_NAMES}
        Di, R = weights["w_dt"].shape
        V, D = weights["embed"].shape
        self.desc = MambaDesc(V, D, weights["a_log"].shape[1], weights["w_conv"].shape[1], Di // D, weights["w_fc"].shape[0], R)
        self.w = MambaWeights(*[self.t[n].data_ptr() for n in MAMBA_WEIGHT_NAMES])
        self.device = self.t["embed"].device

    def workspace(self, total_tokens, n_prompts):
        need = lib().sd_mamba_workspace(C.byref(self.desc), int(total_tokens), int(n_prompts))
        return torch.empty(max(need, 1), dtype=torch.uint8, device=self.device), need

    def classify(self, tokens_dev, starts, lens, stream=None):
        """(scores [n][K] fp32 tensor, labels [n] int32 tensor) for prompts tokens_dev[starts[i] : starts[i] + lens[i]]."""
        n = len(lens)
        starts = np.ascontiguousarray(starts, dtype=np.int64); lens = np.ascontiguousarray(lens, dtype=np.int32)
        scores = torch.zeros((n, self.desc.n_classes), dtype=torch.float32, device=self.device)
        labels = torch.full((n,), -1, dtype=torch.int32, device=self.device)
        ws, need = self.workspace(int(lens.sum()), n)
        _check(lib().sd_mamba_classify(C.byref(self.desc), C.byref(self.w), _dp(tokens_dev), starts.ctypes.data_as(C.c_void_p),
                                       lens.ctypes.data_as(C.c_void_p), n, _dp(scores), _dp(labels), _dp(ws), need, _stream_ptr(stream)), "sd_mamba_classify")
        return scores, labels


class AcceptArgs(C.Structure):
    _fields_ = [("target", C.c_void_p), ("target_is_logits", C.c_int32), ("q", C.c_void_p), ("x", C.c_void_p),
                ("B", C.c_int32), ("gamma", C.c_int32), ("V", C.c_int32), ("temperature", C.c_float),
                ("seed", C.c_uint64), ("iter", C.c_void_p), ("seq_id", C.c_void_p), ("n_acc", C.c_void_p),
                ("out_tok", C.c_void_p), ("cuda_stream", C.c_void_p)]


# knobs of sd_tuning (see include/sd.h)
(SD_TUNE_WO_STAGES, SD_TUNE_WO_PREFILL_ALL, SD_TUNE_ATTN_WARPS, SD_TUNE_ATTN_CLUSTER, SD_TUNE_PACE_NS, SD_TUNE_PREFILL_STAGES,
 SD_TUNE_MANY_ROWS_CB, SD_TUNE_STEADY_STAGES, SD_TUNE_TILE_HANDOFF) = range(9)


class SdError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {lib().sd_status_str(status).decode()} ({status})")


_lib = None
_vp, _i, _sz = C.c_void_p, C.c_int, C.c_size_t

_PROTOS = {
    "sd_arena_bytes": (_sz, [C.POINTER(Config), C.POINTER(ModelDesc)]),
    "sd_create": (_i, [C.POINTER(Config), C.POINTER(ModelDesc), _vp, _vp, _sz, C.POINTER(_vp)]),
    "sd_destroy": (_i, [_vp]),
    "sd_load_tensor": (_i, [_vp, _i, _i, _i, _vp, _i]),
    "sd_load_lora": (_i, [_vp, _i, _i, _i, _vp, _vp, _i]),
    "sd_load_classifier": (_i, [_vp, _vp, _vp, _vp, _vp, _i]),
    "sd_seq_begin": (_i, [_vp, _i, _vp, _i, C.c_uint32]),
    "sd_prefill": (_i, [_vp, _vp, _i]),
    "sd_route_prompt": (_i, [_vp, _vp, _i, _vp, _vp]),
    "sd_draft_steps": (_i, [_vp, _vp, _i, _i, _vp, _vp]),
    "sd_draft_steps_replay": (_i, [_vp, _vp, _i, _i, _vp, _vp, _vp]),
    "sd_verify": (_i, [_vp, _vp, _i, _i, _vp, _vp]),
    "sd_accept": (_i, [C.POINTER(AcceptArgs)]),
    "sd_accept_seqs": (_i, [_vp, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp]),
    "sd_kv_rollback": (_i, [_vp, _vp, _i, _i, _vp, _vp]),
    "sd_verify_accept_host": (_i, [_vp, _vp, _i, _i, _vp, _vp, _vp, _vp]),
    "sd_verify_accept": (_i, [_vp, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp]),
    "sd_use_graphs": (_i, [_vp, _i]),
    "sd_tuning": (_i, [_vp, _i, _i]),
    "sd_use_draft_streams": (_i, [_vp, _i]),
    "sd_launch_stamps": (_i, [_vp, _i]),
    "sd_launch_stamps_read": (_i, [_vp, _vp, _vp, _i, C.POINTER(C.c_int32)]),
    "sd_seq_alpha": (_i, [_vp, _i, C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
    "sd_cost_timing": (_i, [_vp, _i]),
    "sd_cost_read": (_i, [_vp, C.POINTER(Cost), _i]),
    "sd_best_gamma_measured": (_i, [_vp, _i, _i, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_double)]),
    "sd_use_pass_kernel": (_i, [_vp, _i, _i, _i]),
    "sd_pass_tuning": (_i, [_vp, _vp, _vp, _i]),
    "sd_pass_stamps": (_i, [_vp, _vp, _sz]),
    "sd_pass_schedule_check": (_i, [_vp, _vp, _vp, _vp, C.c_char_p, _sz]),
    "sd_pass_schedule_blob": (_sz, [_vp, _vp, _vp, _vp, _sz]),
    "sd_force_plain_path": (_i, [_vp, _i]),
    "sd_use_two_part_activations": (_i, [_vp, _i]),
    "sd_launch_count": (_i, [_vp, C.POINTER(C.c_uint64)]),
    "sd_profile": (_i, [_vp, _i]),
    "sd_profile_read": (_i, [_vp, _vp, _vp]),
    "sd_seq_read": (_i, [_vp, _i, _vp, _i, C.POINTER(C.c_int32), C.POINTER(Counters)]),
    "sd_seq_force": (_i, [_vp, _i, _vp, _i, _i, C.c_uint32]),
    "sd_device_status": (_i, [_vp, C.POINTER(C.c_uint32)]),
    "sd_target_step": (_i, [_vp, _vp, _i, _vp]),
    "sd_op_linear": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _sz, _vp]),
    "sd_op_linear_workspace": (_sz, [_i, _i, _i, _i, _i]),
    "sd_op_linear_static": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp]),
    "sd_op_linear_wait_expiry": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _sz, _vp, _sz, C.c_uint64, _vp, _vp]),
    "sd_mamba_workspace": (_sz, [_vp, C.c_int64, _i]),
    "sd_mamba_classify": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _vp, _vp, _vp, _sz, _vp]),
    "sd_route_prompt_mamba": (_i, [_vp, _vp, _vp, _vp, _i, _vp, _sz, _vp]),
    "sd_kmeans_step": (_i, [_vp, C.c_int64, _i, _vp, _i, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "sd_kmeans_workspace": (_sz, [_i, _i]),
    "sd_op_attention": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _sz, _vp]),
    "sd_op_attention_runs": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _i, _vp, _sz, _vp]),
    "sd_op_attention_workspace": (_sz, [_i, _i, _i, _i]),
    "sd_op_philox": (_i, [_vp, _i, C.c_uint32, C.c_uint32, _vp, _vp]),
    "sd_op_softmax_sample": (_i, [_vp, _i, _i, C.c_float, _vp, _vp, _vp, _vp]),
    "sd_status_str": (C.c_char_p, [_i]),
    "sd_eq1_speedup": (C.c_double, [C.c_double, _i, C.c_double]),
    "sd_best_gamma": (_i, [C.c_double, C.c_double, _i, C.POINTER(C.c_double)]),
}


def lib():
    """Loads libsd.so; there is no fallback of any kind when it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is not built: run `python -m paper_2505_08600_b200.build`")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in _PROTOS.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def sd_pass_schedule_check(dims, rows, rows_per_seq, n_splits, want_logits=1, grid=148, waves=None, chunk_major=None):
    """Builds and replays the persistent kernel's schedule on the host; returns (status, info dict, message)."""
    shape = np.array([dims["n_layers"], dims["d_model"], dims["n_heads"], dims["n_kv_heads"], dims["head_dim"], dims["d_ffn"],
                      dims["vocab"], rows, rows_per_seq, n_splits, want_logits, grid], dtype=np.int32)
    info = np.zeros(8, dtype=np.int32)
    err = C.create_string_buffer(256)
    w = np.ascontiguousarray(waves, dtype=np.int32) if waves is not None else None
    cm = np.ascontiguousarray(chunk_major, dtype=np.int32) if chunk_major is not None else None
    st = lib().sd_pass_schedule_check(shape.ctypes.data_as(C.c_void_p), w.ctypes.data_as(C.c_void_p) if w is not None else None,
                                      cm.ctypes.data_as(C.c_void_p) if cm is not None else None, info.ctypes.data_as(C.c_void_p), err, 256)
    names = ("words_per_layer", "total_words", "slots0", "slots1", "max_seg", "max_section", "program_bytes", "units_per_layer")
    return st, dict(zip(names, info.tolist())), err.value.decode()


def sd_pass_schedule(dims, rows, rows_per_seq, n_splits, want_logits=1, grid=148, waves=None, chunk_major=None):
    """The persistent kernel's schedule as per-CTA lists: [{'segs': [body, tail], 'tasks': [body, tail]}], records as numpy structured arrays."""
    shape = np.array([dims["n_layers"], dims["d_model"], dims["n_heads"], dims["n_kv_heads"], dims["head_dim"], dims["d_ffn"],
                      dims["vocab"], rows, rows_per_seq, n_splits, want_logits, grid], dtype=np.int32)
    w = np.ascontiguousarray(waves, dtype=np.int32) if waves is not None else None
    cm = np.ascontiguousarray(chunk_major, dtype=np.int32) if chunk_major is not None else None
    wp = w.ctypes.data_as(C.c_void_p) if w is not None else None
    cp = cm.ctypes.data_as(C.c_void_p) if cm is not None else None
    n = lib().sd_pass_schedule_blob(shape.ctypes.data_as(C.c_void_p), wp, cp, None, 0)
    if n == 0:
        raise ValueError("no schedule for this shape")
    blob = np.zeros(n, dtype=np.uint8)
    lib().sd_pass_schedule_blob(shape.ctypes.data_as(C.c_void_p), wp, cp, blob.ctypes.data_as(C.c_void_p), n)
    seg_t = np.dtype([("tile", "<u2"), ("kb0", "<u2"), ("n_kb", "<u2"), ("mat", "u1"), ("flags", "u1"), ("dep", "<u2"),
                      ("dep_need", "<u2"), ("arrive", "<u2"), ("slot", "<u2")])
    task_t = np.dtype([("item", "<u4"), ("piece0", "<u4"), ("kind", "<u2"), ("mat", "<u2"), ("wait_word", "<u2"),
                       ("wait_need", "<u2"), ("done_word", "<u2"), ("n_pieces", "<u2")])
    offs = blob[: 4 * (grid + 1)].view("<u4")
    out = []
    for c in range(grid):
        sec = blob[offs[c]: offs[c + 1]]
        h = sec[:40].view("<u4")          # n_seg[2], n_task[2], seg_off[2], task_off[2], piece_off, bytes
        out.append(dict(segs=[sec[h[4 + k]: h[4 + k] + 16 * h[k]].view(seg_t) for k in range(2)],
                        tasks=[sec[h[6 + k]: h[6 + k] + 20 * h[2 + k]].view(task_t) for k in range(2)]))
    return out


def exported_symbols():
    return sorted(_PROTOS)


def _check(status, where):
    if status != 0:
        raise SdError(status, where)


def _stream_ptr(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _dp(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def _seqs(seqs):
    a = np.ascontiguousarray(seqs, dtype=np.int32)
    return a, a.ctypes.data_as(C.c_void_p), int(a.shape[0])


def _desc(dims, dtype, rms_eps=1e-5, rope_base=10000.0):
    return ModelDesc(dims["n_layers"], dims["d_model"], dims["n_heads"], dims["n_kv_heads"], dims["head_dim"],
                     dims["d_ffn"], dims["vocab"], SD_BF16 if dtype == "bf16" else SD_F32, rms_eps, rope_base)


class Context:
    """Owns one sd_ctx and the torch-allocated arena behind it.  Methods carry the names of
    the C calls and do nothing but marshal their arguments."""

    def __init__(self, target_dims, draft_dims, dtype, max_seqs, max_ctx, max_gamma, temperature, seed,
                 clf_d_hidden=0, device="cuda:0", stream=None, lora_adapters=0, lora_rank=0, lora_scale=0.0):
        """lora_adapters > 0: draft_dims holds ONE base draft shared by lora_adapters tasks (one low-rank adapter each)."""
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: this library has no CPU path")
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.L = lib()
        self.dtype = dtype
        self.dims = [target_dims] + list(draft_dims)
        self.vocab = target_dims["vocab"]
        n = len(self.dims)
        self._descs = (ModelDesc * n)(*[_desc(d, dtype) for d in self.dims])
        n_tasks = int(lora_adapters) if lora_adapters else n - 1
        self.cfg = Config(max_seqs, max_ctx, max_gamma, n_tasks, float(temperature), int(seed), int(clf_d_hidden),
                          int(lora_adapters), int(lora_rank), float(lora_scale))
        need = self.L.sd_arena_bytes(C.byref(self.cfg), self._descs)
        if need == 0:
            raise SdError(1, "sd_arena_bytes")
        self.arena = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
        base = (self.arena.data_ptr() + 255) & ~255
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        h = C.c_void_p()
        _check(self.L.sd_create(C.byref(self.cfg), self._descs, _stream_ptr(self.stream), C.c_void_p(base), need, C.byref(h)), "sd_create")
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            self.L.sd_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- loading
    def sd_load_lora(self, adapter, layer, mat, a, b):
        """a [r][in], b [out][r]: numpy uint16 arrays of bf16 bit patterns, or contiguous torch.bfloat16 CUDA tensors."""
        if isinstance(a, np.ndarray):
            a = np.ascontiguousarray(a, dtype=np.uint16); b = np.ascontiguousarray(b, dtype=np.uint16)
            pa, pb, dev = a.ctypes.data_as(C.c_void_p), b.ctypes.data_as(C.c_void_p), 0
        else:
            pa, pb, dev = _dp(a), _dp(b), 1
        _check(self.L.sd_load_lora(self.h, int(adapter), int(layer), int(mat), pa, pb, dev), "sd_load_lora")

    def sd_load_tensor(self, model_id, kind, layer, src):
        """src: numpy array (host) or torch CUDA tensor, already in the model's dtype
        (bf16 as uint16 bit patterns or torch.bfloat16)."""
        if isinstance(src, np.ndarray):
            src = np.ascontiguousarray(src)
            _check(self.L.sd_load_tensor(self.h, model_id, kind, layer, src.ctypes.data_as(C.c_void_p), 0), "sd_load_tensor")
        else:
            assert src.is_cuda and src.is_contiguous()
            _check(self.L.sd_load_tensor(self.h, model_id, kind, layer, _dp(src), 1), "sd_load_tensor")

    def load_weights(self, model_id, weights):
        for name, val in weights.items():
            kind = TENSOR_KIND[name]
            if isinstance(val, (list, tuple)):
                for l, a in enumerate(val):
                    self.sd_load_tensor(model_id, kind, l, a)
            else:
                self.sd_load_tensor(model_id, kind, 0, val)

    def sd_load_classifier(self, w1, b1, w2, b2):
        arrs = [np.ascontiguousarray(a, dtype=np.float32) for a in (w1, b1, w2, b2)]
        _check(self.L.sd_load_classifier(self.h, *[a.ctypes.data_as(C.c_void_p) for a in arrs], 0), "sd_load_classifier")

    # ---- sequences
    def sd_seq_begin(self, seq, prompt, seq_id=None):
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        _check(self.L.sd_seq_begin(self.h, seq, p.ctypes.data_as(C.c_void_p), p.shape[0], seq if seq_id is None else seq_id), "sd_seq_begin")

    def sd_route_prompt(self, seqs, forced_task=None):
        a, p, n = _seqs(seqs)
        out = np.zeros(n, dtype=np.int32)
        f = np.ascontiguousarray(forced_task, dtype=np.int32) if forced_task is not None else None
        _check(self.L.sd_route_prompt(self.h, p, n, f.ctypes.data_as(C.c_void_p) if f is not None else None,
                                      out.ctypes.data_as(C.c_void_p)), "sd_route_prompt")
        return out

    def sd_prefill(self, seqs):
        a, p, n = _seqs(seqs)
        _check(self.L.sd_prefill(self.h, p, n), "sd_prefill")

    # ---- the hot calls; tensors are preallocated CUDA tensors owned by the caller
    def sd_draft_steps(self, seqs, gamma, x, q):
        a, p, n = _seqs(seqs)
        _check(self.L.sd_draft_steps(self.h, p, n, gamma, _dp(x), _dp(q)), "sd_draft_steps")

    def sd_draft_steps_replay(self, seqs, gamma, x_forced, x_sampled, q):
        a, p, n = _seqs(seqs)
        _check(self.L.sd_draft_steps_replay(self.h, p, n, gamma, _dp(x_forced), _dp(x_sampled), _dp(q)), "sd_draft_steps_replay")

    def sd_verify(self, seqs, gamma, x, logits):
        a, p, n = _seqs(seqs)
        _check(self.L.sd_verify(self.h, p, n, gamma, _dp(x), _dp(logits)), "sd_verify")

    def sd_accept_seqs(self, seqs, gamma, logits, q, x, n_acc, out_tok):
        a, p, n = _seqs(seqs)
        _check(self.L.sd_accept_seqs(self.h, p, n, gamma, _dp(logits), _dp(q), _dp(x), _dp(n_acc), _dp(out_tok)), "sd_accept_seqs")

    def sd_kv_rollback(self, seqs, gamma, n_acc, out_tok):
        a, p, n = _seqs(seqs)
        _check(self.L.sd_kv_rollback(self.h, p, n, gamma, _dp(n_acc), _dp(out_tok)), "sd_kv_rollback")

    def sd_target_step(self, seqs, logits):
        a, p, n = _seqs(seqs)
        _check(self.L.sd_target_step(self.h, p, n, _dp(logits)), "sd_target_step")

    def sd_verify_accept_host(self, seqs, gamma, x_host, q_host, n_acc_host, out_tok_host):
        """x_host, q_host, n_acc_host, out_tok_host: CPU tensors (pinned for asynchronous copies)."""
        a, p, n = _seqs(seqs)
        _check(self.L.sd_verify_accept_host(self.h, p, n, gamma, _dp(x_host), _dp(q_host), _dp(n_acc_host), _dp(out_tok_host)),
               "sd_verify_accept_host")

    def sd_verify_accept(self, seqs, gamma, x, q, logits, n_acc, out_tok):
        a, p, n = _seqs(seqs)
        _check(self.L.sd_verify_accept(self.h, p, n, gamma, _dp(x), _dp(q), _dp(logits), _dp(n_acc), _dp(out_tok)), "sd_verify_accept")

    def sd_route_prompt_mamba(self, clf, seqs):
        seqs_a = np.ascontiguousarray(seqs, dtype=np.int32)
        lens_total = int(self.cfg.max_ctx) * len(seqs)
        ws, need = clf.workspace(lens_total, len(seqs))
        out = np.zeros(len(seqs), dtype=np.int32)
        _check(self.L.sd_route_prompt_mamba(self.h, C.byref(clf.desc), C.byref(clf.w), seqs_a.ctypes.data_as(C.c_void_p), len(seqs),
                                            _dp(ws), need, out.ctypes.data_as(C.c_void_p)), "sd_route_prompt_mamba")
        return out

    def sd_use_draft_streams(self, on):
        _check(self.L.sd_use_draft_streams(self.h, int(on)), "sd_use_draft_streams")

    def sd_tuning(self, knob, value):
        _check(self.L.sd_tuning(self.h, int(knob), int(value)), "sd_tuning")

    def sd_launch_stamps(self, enable):
        _check(self.L.sd_launch_stamps(self.h, int(enable)), "sd_launch_stamps")

    def sd_launch_stamps_read(self, cap=1024):
        """(stamps [n][8] uint64 nanoseconds, kinds [n] int32) of the most recent forward pass."""
        st = np.zeros((cap, 8), dtype=np.uint64)
        kinds = np.zeros(cap, dtype=np.int32)
        n = C.c_int32()
        _check(self.L.sd_launch_stamps_read(self.h, st.ctypes.data_as(C.c_void_p), kinds.ctypes.data_as(C.c_void_p), cap, C.byref(n)), "sd_launch_stamps_read")
        k = min(cap, n.value)
        return st[:k], kinds[:k]

    def sd_seq_alpha(self, seq):
        a, j = C.c_double(), C.c_int64()
        _check(self.L.sd_seq_alpha(self.h, int(seq), C.byref(a), C.byref(j)), "sd_seq_alpha")
        return a.value, j.value

    def sd_cost_timing(self, enable):
        _check(self.L.sd_cost_timing(self.h, int(enable)), "sd_cost_timing")

    def sd_cost_read(self, reset=0):
        c = Cost()
        _check(self.L.sd_cost_read(self.h, C.byref(c), int(reset)), "sd_cost_read")
        return {n: getattr(c, n) for n, _ in Cost._fields_}

    def sd_best_gamma_measured(self, seq, gamma_max):
        a, c, s = C.c_double(), C.c_double(), C.c_double()
        g = self.L.sd_best_gamma_measured(self.h, int(seq), int(gamma_max), C.byref(a), C.byref(c), C.byref(s))
        return g, a.value, c.value, s.value

    def sd_use_graphs(self, on):
        _check(self.L.sd_use_graphs(self.h, int(on)), "sd_use_graphs")

    def sd_use_pass_kernel(self, target_on, drafts_on=0, max_rows=0):
        _check(self.L.sd_use_pass_kernel(self.h, int(target_on), int(drafts_on), int(max_rows)), "sd_use_pass_kernel")

    def sd_pass_tuning(self, waves=None, chunk_major=None, stages=0):
        w = np.ascontiguousarray(waves, dtype=np.int32) if waves is not None else None
        cm = np.ascontiguousarray(chunk_major, dtype=np.int32) if chunk_major is not None else None
        _check(self.L.sd_pass_tuning(self.h, w.ctypes.data_as(C.c_void_p) if w is not None else None,
                                     cm.ctypes.data_as(C.c_void_p) if cm is not None else None, int(stages)), "sd_pass_tuning")

    def sd_pass_stamps(self, stamps):
        """stamps: int64 device tensor or None."""
        self._stamps = stamps
        _check(self.L.sd_pass_stamps(self.h, _dp(stamps), 0 if stamps is None else stamps.numel()), "sd_pass_stamps")

    def sd_use_two_part_activations(self, on):
        _check(self.L.sd_use_two_part_activations(self.h, int(on)), "sd_use_two_part_activations")

    def sd_force_plain_path(self, on):
        _check(self.L.sd_force_plain_path(self.h, int(on)), "sd_force_plain_path")

    def sd_launch_count(self):
        v = C.c_uint64()
        _check(self.L.sd_launch_count(self.h, C.byref(v)), "sd_launch_count")
        return v.value

    def sd_profile(self, enable):
        _check(self.L.sd_profile(self.h, int(enable)), "sd_profile")

    def sd_profile_read(self):
        ms = (C.c_float * 6)()
        n = (C.c_uint32 * 6)()
        _check(self.L.sd_profile_read(self.h, ms, n), "sd_profile_read")
        names = ("linear", "attention", "elementwise", "sampling", "state", "fused_step")
        return {k: dict(ms=float(ms[i]), launches=int(n[i])) for i, k in enumerate(names)}

    # ---- observation
    def sd_seq_read(self, seq, cap=None):
        cap = self.cfg.max_ctx + 1 if cap is None else cap
        toks = np.zeros(cap, dtype=np.int32)
        ln = C.c_int32()
        cnt = Counters()
        _check(self.L.sd_seq_read(self.h, seq, toks.ctypes.data_as(C.c_void_p), cap, C.byref(ln), C.byref(cnt)), "sd_seq_read")
        return toks[: min(cap, ln.value)].copy(), {k: getattr(cnt, k) for k in ("iterations", "drafted", "accepted", "emitted")}

    def sd_seq_force(self, seq, tokens, draft_kv_len, it):
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        _check(self.L.sd_seq_force(self.h, seq, t.ctypes.data_as(C.c_void_p), t.shape[0], int(draft_kv_len), int(it)), "sd_seq_force")

    def sd_device_status(self):
        f = C.c_uint32()
        st = self.L.sd_device_status(self.h, C.byref(f))
        if st not in (0, 6):                  # SD_ERR_TIMEOUT comes with the flags: the caller looks at them
            _check(st, "sd_device_status")
        return f.value


def sd_accept(target, q, x, temperature, seed, it, seq_id, n_acc, out_tok, target_is_logits, stream=None):
    """Stateless accept/reject: all arguments are CUDA tensors except the scalars."""
    B, g1, V = target.shape
    a = AcceptArgs(target.data_ptr(), int(target_is_logits), q.data_ptr() if q is not None else None,
                   x.data_ptr() if x is not None else None, B, g1 - 1, V, float(temperature), int(seed),
                   it.data_ptr(), seq_id.data_ptr(), n_acc.data_ptr(), out_tok.data_ptr(), _stream_ptr(stream).value)
    _check(lib().sd_accept(C.byref(a)), "sd_accept")


def sd_eq1_speedup(alpha, gamma, c):
    return float(lib().sd_eq1_speedup(float(alpha), int(gamma), float(c)))


def sd_best_gamma(alpha, c, gamma_max):
    """(gamma, speedup) maximising Eq. 1; gamma 0 when speculative decoding does not pay."""
    s = C.c_double()
    g = lib().sd_best_gamma(float(alpha), float(c), int(gamma_max), C.byref(s))
    return int(g), float(s.value)


def sd_op_linear(x, w, y, dtype, impl=0, stream=None):
    rows, n_in = x.shape
    n_out = w.shape[0]
    need = lib().sd_op_linear_workspace(rows, n_out, n_in, dtype, impl)
    ws = torch.empty(max(need, 1), dtype=torch.uint8, device=x.device)
    _check(lib().sd_op_linear(_dp(x), _dp(w), _dp(y), rows, n_out, n_in, dtype, impl, _dp(ws), need, _stream_ptr(stream)), "sd_op_linear")


def sd_op_linear_wait_expiry(x, w, y, wait_ns, stream=None):
    """The tensor-core linear with the fused step's bounded wait made to run out; returns the device status word."""
    rows, n_in = x.shape
    n_out = w.shape[0]
    need = lib().sd_op_linear_workspace(rows, n_out, n_in, SD_BF16, 2)
    ws = torch.empty(max(need, 1), dtype=torch.uint8, device=x.device)
    words = torch.zeros(((n_out + 127) // 128,), dtype=torch.int32, device=x.device)
    status = torch.zeros((1,), dtype=torch.int32, device=x.device)
    _check(lib().sd_op_linear_wait_expiry(_dp(x), _dp(w), _dp(y), rows, n_out, n_in, _dp(ws), need, _dp(words), words.numel(),
                                          int(wait_ns), _dp(status), _stream_ptr(stream)), "sd_op_linear_wait_expiry")
    torch.cuda.synchronize()
    return int(status.item()), words


def sd_op_linear_static(x, w, y, stream=None):
    """bf16 x [rows][n_in], w [n_out][n_in] -> fp32 y [rows][n_out]; the library's built-in scratch, no allocation."""
    rows, n_in = x.shape
    _check(lib().sd_op_linear_static(_dp(x), _dp(w), _dp(y), rows, w.shape[0], n_in, _stream_ptr(stream)), "sd_op_linear_static")


def sd_op_attention(q, kc, vc, out, row_slot, row_pos, n_heads, n_kv_heads, head_dim, max_ctx, dtype, stream=None, rows_per_seq=1):
    rows = q.shape[0]
    need = lib().sd_op_attention_workspace(rows, n_heads, head_dim, max_ctx)
    ws = torch.empty(max(need, 1), dtype=torch.uint8, device=q.device)
    _check(lib().sd_op_attention_runs(_dp(q), _dp(kc), _dp(vc), _dp(out), _dp(row_slot), _dp(row_pos), rows, int(rows_per_seq), n_heads,
                                      n_kv_heads, head_dim, max_ctx, dtype, _dp(ws), need, _stream_ptr(stream)), "sd_op_attention_runs")


def sd_kmeans_step(points, centroids, labels, centroids_out=None, counts_out=None, inertia_out=None, stream=None):
    """One Lloyd iteration on the device (all arguments CUDA tensors: fp32 points [n][dim], centroids [k][dim], int32 labels [n],
    optional fp32 centroids_out [k][dim], int64 counts_out [k], float64 inertia_out [1])."""
    n, dim = points.shape
    k = centroids.shape[0]
    need = lib().sd_kmeans_workspace(dim, k)
    ws = torch.empty(max(need, 1), dtype=torch.uint8, device=points.device)
    opt = lambda t: _dp(t) if t is not None else None
    _check(lib().sd_kmeans_step(_dp(points), n, dim, _dp(centroids), k, _dp(labels), opt(centroids_out), opt(counts_out), opt(inertia_out),
                                _dp(ws), need, _stream_ptr(stream)), "sd_kmeans_step")


def sd_op_philox(ctr, key0, key1, out, stream=None):
    _check(lib().sd_op_philox(_dp(ctr), ctr.shape[0], key0, key1, _dp(out), _stream_ptr(stream)), "sd_op_philox")


def sd_op_softmax_sample(logits, temperature, u_int, probs, tok, stream=None):
    rows, V = logits.shape
    _check(lib().sd_op_softmax_sample(_dp(logits), rows, V, float(temperature), _dp(u_int), _dp(probs), _dp(tok),
                                      _stream_ptr(stream)), "sd_op_softmax_sample")
