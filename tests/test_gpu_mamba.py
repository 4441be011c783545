"""Mamba-based prompt classifier of the CUDA library against the CPU oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

from oracle import classifier_mamba as om
from paper_2505_08600_b200 import synth
from gpu_util import DEV

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sd():
    from paper_2505_08600_b200 import binding
    binding.lib()
    return binding


def _compare(sd, w, lens, vocab, seed):
    clf = sd.MambaClassifier(w)
    prompts = [synth.make_prompt(vocab, n, seed=seed, seq=i) for i, n in enumerate(lens)]
    gap = 5                                                      # prompts sit apart in the token buffer, as sequences do in the library
    starts, flat, at = [], [], 0
    for p in prompts:
        starts.append(at); flat += p.tolist() + [vocab - 1] * gap; at += len(p) + gap
    tokens = torch.tensor(flat, dtype=torch.int32, device=DEV)
    scores, labels = clf.classify(tokens, starts, lens)
    torch.cuda.synchronize()
    scores, labels = scores.cpu().numpy().astype(np.float64), labels.cpu().numpy()
    for i, p in enumerate(prompts):
        ref, _, _ = om.forward(w, p)
        tol = 2e-4 * (1.0 + np.abs(ref).max())                   # fp32 sums over up to 1000 tokens against fp64
        np.testing.assert_allclose(scores[i], ref, rtol=0, atol=tol)
        top2 = np.sort(ref)[-2:]
        if top2[1] - top2[0] > 2 * tol:
            assert labels[i] == int(np.argmax(ref))
        assert labels[i] == int(np.argmax(scores[i].astype(np.float32)))
    return scores, labels


def test_classifier_at_the_default_sizes_ragged_prompts_across_chunk_boundaries(sd):
    vocab = 3000
    w = synth.make_mamba_classifier(vocab, d_model=128, d_state=16, d_conv=4, expand=2, n_classes=4, seed=1)
    _compare(sd, w, [1, 2, 3, 4, 5, 63, 64, 65, 128, 129, 200, 1000], vocab, seed=3)


def test_short_prompts_only_take_the_single_chunk_path(sd):
    vocab = 500
    w = synth.make_mamba_classifier(vocab, d_model=128, d_state=16, d_conv=4, expand=2, n_classes=3, seed=2)
    _compare(sd, w, [32, 17, 64, 1], vocab, seed=4)


def test_other_sizes(sd):
    vocab = 300
    w = synth.make_mamba_classifier(vocab, d_model=48, d_state=5, d_conv=3, expand=1, n_classes=2, seed=7)      # odd sizes: 48 channels, 5 states, 3 taps
    _compare(sd, w, [70, 9, 300], vocab, seed=5)
    w = synth.make_mamba_classifier(vocab, d_model=256, d_state=8, d_conv=4, expand=2, n_classes=5, seed=8)
    _compare(sd, w, [150, 40], vocab, seed=6)


def test_long_prompt_many_chunks_and_batch_independence(sd):
    vocab = 1000
    w = synth.make_mamba_classifier(vocab, d_model=128, d_state=16, d_conv=4, expand=2, n_classes=4, seed=3)
    s_all, _ = _compare(sd, w, [4100, 77], vocab, seed=9)
    clf = sd.MambaClassifier(w)
    p1 = synth.make_prompt(vocab, 77, seed=9, seq=1)
    s1, _ = clf.classify(torch.from_numpy(p1).to(DEV), [0], [77])
    assert (s1.cpu().numpy()[0] == s_all[1].astype(np.float32)).all()          # a prompt's scores do not depend on its neighbours


def test_routing_through_the_context_and_unsupported_sizes(sd):
    cfg = synth.CONFIGS["tiny"]
    t = cfg["target"]
    ctx = sd.Context(t, cfg["drafts"], "f32", 3, 128, 4, 1.0, 9)
    w = synth.make_mamba_classifier(t["vocab"], d_model=64, d_state=8, d_conv=4, expand=2, n_classes=len(cfg["drafts"]), seed=4)
    clf = sd.MambaClassifier(w)
    prompts = [synth.make_prompt(t["vocab"], n, seed=6, seq=i) for i, n in enumerate([20, 70, 33])]
    for s, p in enumerate(prompts):
        ctx.sd_seq_begin(s, p, s)
    got = ctx.sd_route_prompt_mamba(clf, [0, 1, 2])
    want = [om.classify(w, p)[0] for p in prompts]
    margins = [np.sort(om.classify(w, p)[1])[-1] - np.sort(om.classify(w, p)[1])[-2] for p in prompts]
    for g, r, mg in zip(got.tolist(), want, margins):
        assert mg < 1e-3 or g == r
    ctx.sd_prefill([0, 1, 2])                                              # routed sequences continue down the normal path
    ctx.close()
    big = synth.make_mamba_classifier(100, d_model=64, d_state=32, d_conv=4, expand=2, n_classes=2, seed=1)      # 32 states: not supported
    with pytest.raises(RuntimeError):
        sd.MambaClassifier(big).classify(torch.zeros(8, dtype=torch.int32, device=DEV), [0], [8])
