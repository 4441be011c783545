"""Host logic of the persistent streaming kernel: its static schedule is built and replayed on the CPU (no GPU needed)."""
import numpy as np
import pytest

from paper_2505_08600_b200 import binding as sd
from paper_2505_08600_b200 import synth

SHAPES = [("1b", 6, 6, 4), ("1b", 1, 1, 4), ("7b", 6, 6, 4), ("7b", 16, 8, 2), ("7b", 9, 9, 1), ("13b", 9, 9, 4), ("13b", 32, 2, 1)]


@pytest.mark.parametrize("name,rows,rps,ns", SHAPES)
def test_schedule_builds_and_replays(name, rows, rps, ns):
    dims = synth.CONFIGS[name]["target"]
    st, info, msg = sd.sd_pass_schedule_check(dims, rows, rps, ns)
    assert st == 0, msg
    d, H, Hkv, hd, F = dims["d_model"], dims["n_heads"], dims["n_kv_heads"], dims["head_dim"], dims["d_ffn"]
    units = ((H + 2 * Hkv) * hd // 128) * (d // 64) + (d // 128) * (H * hd // 64) + (2 * F // 128) * (d // 64) + (d // 128) * (F // 64)
    assert info["units_per_layer"] == units                     # every 128 x 64 weight block of a layer, once
    assert info["max_section"] <= 8192 and info["total_words"] < 65536


@pytest.mark.parametrize("waves,cm", [([1, 1, 1, 1, 1], [0] * 5), ([2, 2, 4, 2, 2], [0] * 5), ([2, 2, 4, 2, 2], [1] * 5), ([4, 2, 8, 4, 2], [1, 0, 1, 0, 0])])
def test_schedule_covers_every_block_once_and_balances(waves, cm):
    dims = synth.CONFIGS["7b"]["target"]
    G = 148
    prog = sd.sd_pass_schedule(dims, 6, 6, 4, 1, G, waves, cm)
    d, H, Hkv, hd, F, V = dims["d_model"], dims["n_heads"], dims["n_kv_heads"], dims["head_dim"], dims["d_ffn"], dims["vocab"]
    nt = [(H + 2 * Hkv) * hd // 128, d // 128, 2 * F // 128, d // 128, V // 128]
    kb = [d // 64, H * hd // 64, d // 64, F // 64, d // 64]
    seen = [np.zeros((nt[m], kb[m]), dtype=np.int32) for m in range(5)]
    per_cta = np.zeros(G, dtype=np.int64)
    pieces = [np.zeros(nt[m], dtype=np.int32) for m in range(5)]
    for c in range(G):
        for k in range(2):
            for sg in prog[c]["segs"][k]:
                m = int(sg["mat"])
                seen[m][int(sg["tile"]), int(sg["kb0"]): int(sg["kb0"]) + int(sg["n_kb"])] += 1
                per_cta[c] += int(sg["n_kb"]) if k == 0 else 0
                pieces[m][int(sg["tile"])] += (int(sg["flags"]) >> 3) & 1            # the segment that leaves the CTA's piece
    for m in range(5):
        assert (seen[m] == 1).all(), m
        assert (pieces[m] >= 1).all()
    assert per_cta.max() - per_cta.min() <= 2 * len(waves) * 4          # the blocks of a layer are spread evenly over the CTAs
    # every tile is reduced by exactly one task, which expects as many pieces as there are segments that leave one
    for m in range(5):
        expect = np.zeros(nt[m], dtype=np.int32)
        for c in range(G):
            for k in range(2):
                for tk in prog[c]["tasks"][k]:
                    if int(tk["kind"]) == 0 and int(tk["mat"]) == m:
                        assert expect[int(tk["item"])] == 0
                        expect[int(tk["item"])] = int(tk["n_pieces"])
        assert (expect == pieces[m]).all(), m


def test_unsupported_shapes_are_refused():
    dims = dict(synth.CONFIGS["7b"]["target"])
    dims["head_dim"] = 96
    st, _, msg = sd.sd_pass_schedule_check(dims, 6, 6, 4)
    assert st != 0 and msg
