"""Single-operator parity of the CUDA library against the CPU oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_08600_b200 import synth
from gpu_util import DEV, quantize, to_dev, widen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sd():
    from paper_2505_08600_b200 import binding
    binding.lib()
    return binding


def test_philox_known_answers_on_device(sd, golden_dir):
    rows = [[int(t, 16) for t in l.split()] for l in open(f"{golden_dir}/philox4x32_10_kat.txt") if not l.startswith("#")]
    for r in rows:
        ctr = to_dev(np.array([r[:4]], dtype=np.uint32))
        out = torch.zeros((1, 4), dtype=torch.int32, device=DEV)
        sd.sd_op_philox(ctr, r[4], r[5], out)
        assert out.cpu().numpy().view(np.uint32)[0].tolist() == r[6:]
    # a batch of counters against the oracle's generator
    rng = np.random.default_rng(0)
    ctr = rng.integers(0, 2**32, size=(257, 4), dtype=np.uint64).astype(np.uint32)
    out = torch.zeros((257, 4), dtype=torch.int32, device=DEV)
    sd.sd_op_philox(to_dev(ctr), 0xDEADBEEF, 0x12345678, out)
    got = out.cpu().numpy().view(np.uint32)
    for i in range(257):
        assert got[i].tolist() == oracle.philox4x32_10(ctr[i], [0xDEADBEEF, 0x12345678]).tolist()


LINEAR_SHAPES = [  # rows, n_out, n_in
    (1, 8, 8), (5, 37, 64), (6, 1024, 256), (8, 688, 256), (9, 256, 688), (17, 130, 344), (6, 300, 1000),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("rows,n_out,n_in", LINEAR_SHAPES)
def test_linear_plain_kernel(sd, dtype, rows, n_out, n_in):
    x = quantize(synth.make_logits((rows, n_in), seed=11, stream=rows), dtype)
    w = quantize(synth.make_logits((n_out, n_in), seed=12, stream=n_out, std=0.05), dtype)
    ref = oracle.linear(w, widen(x))
    y = torch.full((rows, n_out), float("nan"), dtype=torch.float32, device=DEV)
    sd.sd_op_linear(to_dev(x), to_dev(w), y, sd.SD_BF16 if dtype == "bf16" else sd.SD_F32, impl=1)
    got = y.cpu().numpy().astype(np.float64)
    # fp32 accumulation of n_in products of magnitude ~0.05: a few 1e-6 at most
    np.testing.assert_allclose(got, ref, rtol=0, atol=2e-5 * np.sqrt(n_in / 64))


ATTN_CASES = [  # H, Hkv, hd, max_ctx, positions of the rows
    (4, 4, 64, 40, [0, 1, 7, 39]),
    (4, 2, 64, 300, [5, 128, 129, 255, 299]),
    (8, 2, 128, 700, [0, 63, 64, 65, 511, 699]),
    (2, 1, 16, 33, [32, 31, 0]),
    # long caches: several slices per head merged by the last CTA (odd and even slice counts), rows inside one slice
    (4, 2, 128, 2600, [0, 1023, 1024, 1025, 2047, 2599]),
    (4, 4, 64, 4100, [4099, 3000, 17, 1024]),
    (2, 2, 128, 8192, [8191, 4096, 100]),
    # many (head, row, slice) items: several CTAs per SM, the four-warp form of the kernel (single slice, and merged slices)
    (32, 32, 128, 700, [0, 63, 64, 127, 128, 300, 511, 640, 698, 699]),
    (16, 16, 64, 2100, [2099, 1024, 1023, 17, 2048, 700, 1500]),
    (32, 32, 64, 4200, [4199, 2048, 2047, 17, 4096, 700, 3000, 1]),      # four-warp form with three merged slices
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("H,Hkv,hd,max_ctx,positions", ATTN_CASES)
def test_attention_over_cache(sd, dtype, H, Hkv, hd, max_ctx, positions):
    n_slots, rows = 3, len(positions)
    q = quantize(synth.make_logits((rows, H, hd), seed=21, stream=hd), dtype)
    kc = quantize(synth.make_logits((n_slots, Hkv, max_ctx, hd), seed=22, stream=hd), dtype)
    vc = quantize(synth.make_logits((n_slots, Hkv, max_ctx, hd), seed=23, stream=hd), dtype)
    row_slot = np.array([(2 * r + 1) % n_slots for r in range(rows)], dtype=np.int32)
    row_pos = np.array(positions, dtype=np.int32)
    out = torch.zeros((rows, H, hd), dtype=torch.bfloat16 if dtype == "bf16" else torch.float32, device=DEV)
    sd.sd_op_attention(to_dev(q), to_dev(kc), to_dev(vc), out, to_dev(row_slot), to_dev(row_pos), H, Hkv, hd, max_ctx,
                       sd.SD_BF16 if dtype == "bf16" else sd.SD_F32)
    got = out.float().cpu().numpy().astype(np.float64)
    qf, kf, vf = widen(q), widen(kc), widen(vc)
    for r in range(rows):
        for h in range(H):
            kvh = h // (H // Hkv)
            n_ctx = positions[r] + 1
            ref = oracle.attention_head(qf[r, h], kf[row_slot[r], kvh, :n_ctx], vf[row_slot[r], kvh, :n_ctx])
            tol = 2e-2 if dtype == "bf16" else 2e-5          # bf16 output rounding: 2^-9 relative on values up to ~3
            np.testing.assert_allclose(got[r, h], ref, rtol=0, atol=tol)


def test_attention_launch_of_the_eight_sequence_long_cache_configuration(sd):
    """The attention launch of the 13B-class workload as the verify step issues it: 8 sequences x 9 rows, 40 heads of
    128, caches of 8192 positions, the rows at the last nine positions.  The oracle scores sampled (row, head) pairs."""
    B, g1, H, hd, max_ctx = 8, 9, 40, 128, 8192
    rows = B * g1
    q = quantize(synth.make_logits((rows, H, hd), seed=41, stream=hd), "bf16")
    base_k = quantize(synth.make_logits((H, max_ctx, hd), seed=42, stream=hd), "bf16")
    base_v = quantize(synth.make_logits((H, max_ctx, hd), seed=43, stream=hd), "bf16")
    # sequence b's cache is the base block rolled by 97 * b positions (eight distinct caches from one generated block)
    kc = torch.empty((B, H, max_ctx, hd), dtype=torch.bfloat16, device=DEV)
    vc = torch.empty((B, H, max_ctx, hd), dtype=torch.bfloat16, device=DEV)
    bk, bv = to_dev(base_k), to_dev(base_v)
    for b in range(B):
        kc[b] = torch.roll(bk, 97 * b, dims=1)
        vc[b] = torch.roll(bv, 97 * b, dims=1)
    row_slot = np.repeat(np.arange(B, dtype=np.int32), g1)
    row_pos = np.tile(np.arange(max_ctx - g1, max_ctx, dtype=np.int32), B)
    out = torch.zeros((rows, H, hd), dtype=torch.bfloat16, device=DEV)
    sd.sd_op_attention(to_dev(q), kc, vc, out, to_dev(row_slot), to_dev(row_pos), H, H, hd, max_ctx, sd.SD_BF16, rows_per_seq=g1)
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    # the same rows one by one (every row its own pass over the cache) give the same numbers up to the output's rounding
    out1 = torch.zeros_like(out)
    sd.sd_op_attention(to_dev(q), kc, vc, out1, to_dev(row_slot), to_dev(row_pos), H, H, hd, max_ctx, sd.SD_BF16)
    assert (out.float() - out1.float()).abs().max().item() <= 2e-2
    qf, kf, vf = widen(q), widen(base_k), widen(base_v)
    rng = np.random.default_rng(7)
    picks = {(0, 0), (rows - 1, H - 1), (g1 - 1, 17), (g1, 3)} | {(int(rng.integers(rows)), int(rng.integers(H))) for _ in range(28)}
    for r, h in sorted(picks):
        b, n_ctx = int(row_slot[r]), int(row_pos[r]) + 1
        ref = oracle.attention_head(qf[r, h], np.roll(kf[h], 97 * b, axis=0)[:n_ctx], np.roll(vf[h], 97 * b, axis=0)[:n_ctx])
        np.testing.assert_allclose(got[r, h], ref, rtol=0, atol=2e-2)
    # rows of one sequence differ only by the causal bound: the last row sees eight more keys than the first
    assert np.abs(got[0] - got[g1 - 1]).max() > 0


def test_attention_inactive_row_gives_zeros(sd):
    H, hd, max_ctx = 2, 64, 16
    q = synth.make_logits((2, H, hd), seed=1)
    kc = synth.make_logits((1, H, max_ctx, hd), seed=2)
    out = torch.ones((2, H, hd), dtype=torch.float32, device=DEV)
    sd.sd_op_attention(to_dev(q), to_dev(kc), to_dev(kc), out, to_dev(np.zeros(2, dtype=np.int32)),
                       to_dev(np.array([-1, 3], dtype=np.int32)), H, H, hd, max_ctx, sd.SD_F32)
    o = out.cpu().numpy()
    assert (o[0] == 0).all() and np.abs(o[1]).max() > 0


@pytest.mark.parametrize("V", [8, 1000, 1024, 32000])
@pytest.mark.parametrize("T", [1.0, 0.7, 0.0])
def test_softmax_and_draw(sd, V, T):
    rows = 7
    logits = synth.make_logits((rows, V), seed=31, stream=V, std=2.0)
    u = np.array([oracle.uniform24(3, r, 0, 0, 0) for r in range(rows)], dtype=np.uint32)
    u[0], u[1] = 1, 2**24
    probs = torch.zeros((rows, V), dtype=torch.float32, device=DEV)
    tok = torch.full((rows,), -7, dtype=torch.int32, device=DEV)
    sd.sd_op_softmax_sample(to_dev(logits), T, to_dev(u), probs, tok)
    p_ref = oracle.softmax_T(logits.astype(np.float64), T)
    p_gpu = probs.cpu().numpy()
    assert np.abs(p_gpu.astype(np.float64) - p_ref).max() <= 1e-3          # the stated probability tolerance
    assert np.abs(p_gpu.astype(np.float64) - p_ref).max() <= 2e-6          # what fp32 arithmetic actually gives
    t_gpu = tok.cpu().numpy()
    same = 0
    for r in range(rows):
        t_ref = oracle.sample_icdf(p_ref[r], int(u[r]))
        same += int(t_ref == t_gpu[r])
        # the draw must be right for the oracle's CDF up to the rounding of the probabilities
        cdf = np.cumsum(p_ref[r].astype(np.float64))
        uu = u[r] / 2**24
        k = int(t_gpu[r])
        assert 0 <= k < V and p_ref[r][k] > 0
        assert (cdf[k - 1] if k else 0.0) - 1e-4 < uu <= cdf[k] + 1e-4
    if T == 0.0:
        assert same == rows
        assert (t_gpu == np.argmax(logits, axis=1)).all()
    else:
        assert same >= rows - 1


TC_SHAPES = [  # rows, n_out, n_in: single tile, several tiles + ragged tail, split tiles, wide token counts
    (6, 128, 64), (6, 128, 4096), (1, 256, 512), (6, 1024, 256), (16, 300, 1000), (6, 4096, 4096),
    (5, 12288, 1024), (17, 640, 2304), (96, 1152, 768), (72, 4096, 1024), (200, 256, 512), (256, 384, 320),
    (6, 32000, 512), (2, 11008, 1024), (6, 1024, 11008),
]


@pytest.mark.parametrize("rows,n_out,n_in", TC_SHAPES)
def test_linear_tensor_core_kernel(sd, rows, n_out, n_in):
    x = quantize(synth.make_logits((rows, n_in), seed=13, stream=rows), "bf16")
    w = quantize(synth.make_logits((n_out, n_in), seed=14, stream=n_out % 1000, std=0.05), "bf16")
    y = torch.full((rows, n_out), float("nan"), dtype=torch.float32, device=DEV)
    sd.sd_op_linear(to_dev(x), to_dev(w), y, sd.SD_BF16, impl=2)
    torch.cuda.synchronize()
    got = y.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    # the oracle computes sampled rows and columns one by one at the larger sizes
    rng = np.random.default_rng(rows * 7 + n_out)
    cols = np.arange(n_out) if n_out * n_in <= 2**22 else np.unique(np.concatenate(
        [rng.integers(0, n_out, 192), [0, 127, 128, n_out - 1, n_out - 129 if n_out > 129 else 0]]))
    ref = oracle.linear(np.ascontiguousarray(w[cols]), widen(x))
    np.testing.assert_allclose(got[:, cols], ref, rtol=0, atol=2e-5 * np.sqrt(n_in / 64))
    # same answer on a second run: the reduction order is fixed
    y2 = torch.zeros_like(y)
    sd.sd_op_linear(to_dev(x), to_dev(w), y2, sd.SD_BF16, impl=2)
    assert torch.equal(y, y2)


def test_bounded_wait_runs_out_and_the_fallback_finishes_the_job(sd):
    """The step after the GEMM watches arrival words for a bounded time.  Here nobody counts into them (the GEMM is not told
    to), the limit is 1 ms: every tile's CTA must give up, wait for the GEMM's grid instead, still produce the right
    result, and report SD_DEV_WAIT_EXPIRED.  Nothing hangs, nothing faults."""
    rows, n_out, n_in = 6, 1024, 2048
    x = quantize(synth.make_logits((rows, n_in), seed=41, stream=1), "bf16")
    w = quantize(synth.make_logits((n_out, n_in), seed=42, stream=2, std=0.05), "bf16")
    ref = torch.full((rows, n_out), float("nan"), dtype=torch.float32, device=DEV)
    sd.sd_op_linear(to_dev(x), to_dev(w), ref, sd.SD_BF16, impl=2)
    got = torch.full((rows, n_out), float("nan"), dtype=torch.float32, device=DEV)
    status, words = sd.sd_op_linear_wait_expiry(to_dev(x), to_dev(w), got, wait_ns=1_000_000)
    assert status & 8                                      # SD_DEV_WAIT_EXPIRED
    assert torch.equal(got, ref)
    assert int(words.abs().sum()) == 0                     # the words are left at zero
    np.testing.assert_allclose(got.cpu().numpy().astype(np.float64), oracle.linear(w, widen(x)), rtol=0, atol=2e-5 * np.sqrt(n_in / 64))
