"""The C-ABI library loads without a GPU and exports everything include/sd.h declares."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def sdlib():
    from paper_2505_08600_b200 import build
    build.build()
    from paper_2505_08600_b200 import binding
    return binding


def _declared():
    text = open(os.path.join(ROOT, "include", "sd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sd_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(sdlib):
    names = _declared()
    assert {"sd_route_prompt", "sd_draft_steps", "sd_verify", "sd_accept", "sd_kv_rollback"} <= set(names)
    raw = C.CDLL(sdlib.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), f"{n} declared in sd.h but not exported"
    assert set(sdlib.exported_symbols()) == set(names)


def test_host_side_validation_needs_no_gpu(sdlib):
    L = sdlib.lib()
    dims = dict(n_layers=2, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ffn=688, vocab=1024)
    descs = (sdlib.ModelDesc * 2)(sdlib._desc(dims, "f32"), sdlib._desc(dims, "f32"))
    cfg = sdlib.Config(4, 128, 4, 1, 1.0, 1, 0, 0)
    small = L.sd_arena_bytes(C.byref(cfg), descs)
    assert small > 2 * 4 * (2 * 1024 * 256)                 # at least the embeddings of both models
    cfg2 = sdlib.Config(4, 256, 4, 1, 1.0, 1, 0, 0)
    assert L.sd_arena_bytes(C.byref(cfg2), descs) > small    # a longer KV cache needs more
    bad = sdlib.Config(65, 128, 4, 1, 1.0, 1, 0, 0)          # more slots than SD_MAX_BATCH
    assert L.sd_arena_bytes(C.byref(bad), descs) == 0
    bad_heads = dict(dims, n_heads=3)
    descs_bad = (sdlib.ModelDesc * 2)(sdlib._desc(bad_heads, "f32"), sdlib._desc(dims, "f32"))
    assert L.sd_arena_bytes(C.byref(cfg), descs_bad) == 0
    assert L.sd_accept(None) == 1                             # SD_ERR_INVALID_ARG
    h = C.c_void_p()
    assert L.sd_create(C.byref(cfg), descs, None, None, 0, C.byref(h)) == 1
    assert L.sd_status_str(3) == b"capacity exceeded"


def test_eq1_and_gamma_choice_on_the_host(sdlib):
    # Eq. 1 against its definition as an expected-token count, and the argmax against brute force
    for alpha in (0.0, 0.3, 0.6, 0.8, 0.95, 1.0):
        for c in (0.0, 0.02, 0.138, 0.5):
            best, best_s = 0, 1.0
            for g in range(0, 16):
                tokens = sum(alpha ** i for i in range(g + 1))        # 1 + alpha + ... + alpha^gamma
                want = tokens / (g * c + 1)
                assert abs(sdlib.sd_eq1_speedup(alpha, g, c) - want) < 1e-12
                if g >= 1 and want > best_s + 1e-15:
                    best, best_s = g, want
            got_g, got_s = sdlib.sd_best_gamma(alpha, c, 15)
            assert got_g == best and abs(got_s - best_s) < 1e-12
    assert sdlib.sd_best_gamma(0.1, 0.5, 15) == (0, 1.0)                  # a poor, expensive draft never pays
    assert sdlib.sd_eq1_speedup(-0.1, 3, 0.1) == 0.0
    # the paper's Table 1 relation: speedup = tau / (gamma c + 1) with tau = expected tokens per iteration
    assert abs(sdlib.sd_eq1_speedup(0.8, 5, 0.0) - (1 - 0.8 ** 6) / 0.2) < 1e-12
