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
