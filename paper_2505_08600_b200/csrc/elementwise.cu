// Small memory-bound kernels around the GEMMs: token embedding + row planning, RMSNorm,
// rotary embedding + KV append, residual add, SwiGLU, and the per-sequence state updates.
#include "kernels.h"
#include "pass_stream.h"

namespace sd {

// ------------------------------------------------------------------ embedding + row plan
// One block per query row.  Works out which sequence, position and token the row stands for
// (the state lives on the device, so the host never needs the current lengths), records
// them for the later kernels of the pass and loads the embedding row as fp32.
template <typename T>
__global__ void k_embed(SeqState S, SeqList list, RowPlan plan, const T* __restrict__ embed, int d, int vocab,
                        float* __restrict__ h, int32_t* __restrict__ row_slot, int32_t* __restrict__ row_pos,
                        const float* __restrict__ gain, bf16* __restrict__ xn, float* __restrict__ ssq,
                        const float* __restrict__ rcos, const float* __restrict__ rsin, int half,
                        float* __restrict__ row_cos, float* __restrict__ row_sin, int tagged_m_pad, const uint32_t* __restrict__ epoch, int lo_off) {
    __shared__ float red[32];
    const int r = blockIdx.x;
    const int i = r / plan.rows_per_seq, j = r % plan.rows_per_seq;
    const int slot = list.ids[i], b = list.out[i];
    const int len = S.len[slot];
    const int32_t* toks = S.tokens + (size_t)slot * S.tok_stride;
    int pos, tok;
    switch (plan.kind) {
        case PLAN_PREFILL: pos = plan.pos0 + j; tok = toks[pos]; break;
        case PLAN_VERIFY:                       // rows: last token, then the gamma drafts
            pos = len - 1 + j;
            tok = (j == 0) ? toks[len - 1] : plan.x[(size_t)b * plan.gamma + (j - 1)];
            break;
        case PLAN_DRAFT_FIRST:                  // two rows: the token missed after a full accept, the last token
            pos = len - 2 + j;
            if (pos < S.dkv[slot] || pos < 0) { pos = -1; tok = 0; } else tok = toks[pos];
            break;
        case PLAN_DRAFT_NEXT: pos = len - 1 + plan.step; tok = plan.x[(size_t)b * plan.gamma + (plan.step - 1)]; break;
        default: pos = len - 1; tok = toks[len - 1]; break;   // PLAN_TARGET_STEP
    }
    if (pos >= S.max_ctx) { if (threadIdx.x == 0) atomicOr(S.status, SD_DEV_BAD_POS); pos = -1; }
    if (tok < 0 || tok >= vocab) { if (threadIdx.x == 0) atomicOr(S.status, SD_DEV_BAD_TOKEN); tok = 0; }
    if (threadIdx.x == 0) { row_slot[r] = slot; row_pos[r] = pos; row_slot[SD_MAX_ROWS + r] = S.draft_id[slot]; }      // (the row's task follows the slots)
    if (row_cos)                         // the row's rotary factors, so that the step after the QKV GEMM needs no dependent lookup
        for (int k = threadIdx.x; k < half; k += blockDim.x) {
            row_cos[(size_t)r * half + k] = pos >= 0 ? rcos[(size_t)pos * half + k] : 1.f;
            row_sin[(size_t)r * half + k] = pos >= 0 ? rsin[(size_t)pos * half + k] : 0.f;
        }
    const T* e = embed + (size_t)tok * d;
    float ss = 0.f;
    if (tagged_m_pad) {
        // For the persistent streaming kernel: h, the first norm's operand and the row's sum of squares as tagged 64-bit
        // words (payload + the pass's tag), the operand as [k block][row][32 words of two bf16].
        const uint32_t tag = pass_tag(*epoch, 0, 1);
        tagged_t* th = reinterpret_cast<tagged_t*>(h);
        tagged_t* txn = reinterpret_cast<tagged_t*>(xn);
        for (int k = 2 * threadIdx.x; k < d; k += 2 * blockDim.x) {
            const float v0 = to_f32<T>(e[k]), v1 = to_f32<T>(e[k + 1]);
            th[(size_t)r * d + k] = ((tagged_t)tag << 32) | __float_as_uint(v0);
            th[(size_t)r * d + k + 1] = ((tagged_t)tag << 32) | __float_as_uint(v1);
            const uint32_t lo = __bfloat16_as_ushort(__float2bfloat16_rn(v0 * gain[k])), hi = __bfloat16_as_ushort(__float2bfloat16_rn(v1 * gain[k + 1]));
            txn[xtagged_index(r, k, tagged_m_pad)] = ((tagged_t)tag << 32) | lo | (hi << 16);
            ss += v0 * v0 + v1 * v1;
        }
        ss = block_sum(ss, red);
        if (threadIdx.x == 0) reinterpret_cast<tagged_t*>(ssq)[(size_t)r * 64] = ((tagged_t)tag << 32) | __float_as_uint(ss);
        return;
    }
    for (int k = threadIdx.x; k < d; k += blockDim.x) {
        const float v = to_f32<T>(e[k]);
        h[(size_t)r * d + k] = v;
        if (gain) {
            const float x = v * gain[k];
            const bf16 hi = __float2bfloat16_rn(x);
            xn[(size_t)r * d + k] = hi;
            if (lo_off) xn[(size_t)(r + lo_off) * d + k] = __float2bfloat16_rn(x - __bfloat162float(hi));
            ss += v * v;
        }
    }
    if (gain) {                          // first half of the first layer's RMSNorm: the 1/rms factor follows the GEMM
        ss = block_sum(ss, red);
        if (threadIdx.x == 0) ssq[(size_t)r * 64] = ss;
    }
}

cudaError_t launch_embed(const SeqState& S, const SeqList& list, const RowPlan& plan, int n_rows,
                         const void* embed, int dtype, int d, int vocab,
                         float* h, int32_t* row_slot, int32_t* row_pos, const float* gain, void* xn, float* ssq,
                         const float* rope_cos, const float* rope_sin, int half, float* row_cos, float* row_sin, int tagged_m_pad,
                         const uint32_t* epoch, cudaStream_t st, int lo_off) {
    if (dtype == SD_BF16)
        k_embed<bf16><<<n_rows, 256, 0, st>>>(S, list, plan, (const bf16*)embed, d, vocab, h, row_slot, row_pos, gain, (bf16*)xn, ssq,
                                              rope_cos, rope_sin, half, row_cos, row_sin, tagged_m_pad, epoch, lo_off);
    else
        k_embed<float><<<n_rows, 256, 0, st>>>(S, list, plan, (const float*)embed, d, vocab, h, row_slot, row_pos, nullptr, nullptr, nullptr,
                                               nullptr, nullptr, 0, nullptr, nullptr, 0, nullptr, 0);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ RMSNorm
template <typename T>
__global__ void k_rmsnorm(const float* __restrict__ h, const float* __restrict__ gain, T* __restrict__ xn, int d,
                          float eps, int row_stride, int row_offset) {
    __shared__ float red[32];
    const float* x = h + (size_t)(blockIdx.x * row_stride + row_offset) * d;
    float ss = 0.f;
    for (int k = threadIdx.x; k < d; k += blockDim.x) { float v = x[k]; ss += v * v; }
    ss = block_sum(ss, red);
    const float inv = rsqrtf(ss / (float)d + eps);
    for (int k = threadIdx.x; k < d; k += blockDim.x)
        xn[(size_t)blockIdx.x * d + k] = from_f32<T>(x[k] * inv * gain[k]);
}

cudaError_t launch_rmsnorm(const float* h, const float* gain, void* xn, int dtype, int n_rows, int d, float eps,
                           int row_stride, int row_offset, cudaStream_t st) {
    if (dtype == SD_BF16) k_rmsnorm<bf16><<<n_rows, 256, 0, st>>>(h, gain, (bf16*)xn, d, eps, row_stride, row_offset);
    else k_rmsnorm<float><<<n_rows, 256, 0, st>>>(h, gain, (float*)xn, d, eps, row_stride, row_offset);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ rotary embedding + KV append
// grid (rows, n_heads + 2 n_kv_heads), head_dim/2 threads.  Query heads are rotated and kept,
// key heads are rotated and appended to the cache, value heads are appended as they are.
// Cache layout of one layer: [slot][kv_head][position][head_dim].
template <typename T>
__global__ void k_rope_kv(const float* __restrict__ qkv, T* __restrict__ q_out, T* __restrict__ kc, T* __restrict__ vc,
                          const int32_t* __restrict__ row_slot, const int32_t* __restrict__ row_pos,
                          int H, int Hkv, int hd, int max_ctx, const float* __restrict__ rcos,
                          const float* __restrict__ rsin, uint32_t* status) {
    const int r = blockIdx.x, head = blockIdx.y, i = threadIdx.x, half = hd >> 1;
    const int pos = row_pos[r];
    if (pos < 0) return;
    const int n_all = (H + 2 * Hkv) * hd;
    const float* src = qkv + (size_t)r * n_all + (size_t)head * hd;
    float a = src[i], b = src[i + half];
    if (head < H + Hkv) {
        float c = rcos[(size_t)pos * half + i], s = rsin[(size_t)pos * half + i];
        float ra = a * c - b * s, rb = a * s + b * c;
        a = ra; b = rb;
    }
    T* dst;
    if (head < H) dst = q_out + ((size_t)r * H + head) * hd;
    else {
        const int kvh = (head - H) % Hkv;
        T* base = (head < H + Hkv) ? kc : vc;
        dst = base + (((size_t)row_slot[r] * Hkv + kvh) * max_ctx + pos) * hd;
    }
    dst[i] = from_f32<T>(a);
    dst[i + half] = from_f32<T>(b);
}

cudaError_t launch_rope_kv(const float* qkv, void* q_out, void* kc, void* vc, int dtype,
                           const int32_t* row_slot, const int32_t* row_pos, int n_rows,
                           int H, int Hkv, int hd, int max_ctx, const float* rcos, const float* rsin,
                           uint32_t* status, cudaStream_t st) {
    dim3 grid(n_rows, H + 2 * Hkv);
    if (dtype == SD_BF16) k_rope_kv<bf16><<<grid, hd / 2, 0, st>>>(qkv, (bf16*)q_out, (bf16*)kc, (bf16*)vc, row_slot, row_pos, H, Hkv, hd, max_ctx, rcos, rsin, status);
    else k_rope_kv<float><<<grid, hd / 2, 0, st>>>(qkv, (float*)q_out, (float*)kc, (float*)vc, row_slot, row_pos, H, Hkv, hd, max_ctx, rcos, rsin, status);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ residual add, SwiGLU
__global__ void k_residual_add(float* __restrict__ h, const float* __restrict__ y, size_t n) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) h[i] += y[i];
}
cudaError_t launch_residual_add(float* h, const float* y, size_t n, cudaStream_t st) {
    k_residual_add<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(h, y, n);
    return cudaGetLastError();
}

template <typename T>
__global__ void k_swiglu(const float* __restrict__ gu, T* __restrict__ act, int F, int interleaved) {
    const int r = blockIdx.y;
    const int f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= F) return;
    const int ig = interleaved ? (f / 64) * 128 + f % 64 : f, iu = interleaved ? ig + 64 : F + f;
    float g = gu[(size_t)r * 2 * F + ig], u = gu[(size_t)r * 2 * F + iu];
    act[(size_t)r * F + f] = from_f32<T>(g / (1.f + expf(-g)) * u);
}
cudaError_t launch_swiglu(const float* gu, void* act, int dtype, int n_rows, int F, int interleaved, cudaStream_t st) {
    dim3 grid((F + 255) / 256, n_rows);
    if (dtype == SD_BF16) k_swiglu<bf16><<<grid, 256, 0, st>>>(gu, (bf16*)act, F, interleaved);
    else k_swiglu<float><<<grid, 256, 0, st>>>(gu, (float*)act, F, interleaved);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ per-sequence state
__global__ void k_set_state(SeqState S, int slot, int len, int tkv, int dkv, uint32_t iter, uint32_t seq_id, int reset) {
    S.len[slot] = len; S.tkv[slot] = tkv; S.dkv[slot] = dkv; S.iter[slot] = iter;
    if (reset) {
        S.seq_id[slot] = seq_id; S.n_prompt[slot] = len;
        for (int i = 0; i < 4; ++i) S.counters[slot * 4 + i] = 0;
        S.alpha_sum[slot] = 0.0; S.judged[slot] = 0;
    }
}
cudaError_t launch_set_state(const SeqState& S, int slot, int len, int tkv, int dkv, uint32_t iter, uint32_t seq_id,
                             int reset_counters, cudaStream_t st) {
    k_set_state<<<1, 1, 0, st>>>(S, slot, len, tkv, dkv, iter, seq_id, reset_counters);
    return cudaGetLastError();
}

// Commit of one iteration.  Nothing in either KV cache moves: the lengths shrink and the
// next append lands on the rejected positions.
__global__ void k_rollback(SeqState S, SeqList list, int gamma, const int32_t* __restrict__ n_acc,
                           const int32_t* __restrict__ out_tok, const float* __restrict__ alpha_terms) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= list.n) return;
    const int slot = list.ids[i], b = list.out[i];
    int n = n_acc[b];
    if (n < 0 || n > gamma) { atomicOr(S.status, SD_DEV_BAD_NACC); n = n < 0 ? 0 : gamma; }
    const int L = S.len[slot];
    if (L + n + 1 > S.tok_stride) { atomicOr(S.status, SD_DEV_BAD_POS); return; }
    int32_t* toks = S.tokens + (size_t)slot * S.tok_stride;
    for (int s = 0; s <= n; ++s) toks[L + s] = out_tok[(size_t)b * (gamma + 1) + s];
    S.tkv[slot] = L + n;
    S.dkv[slot] = min(L + n, L + gamma - 1);
    S.len[slot] = L + n + 1;
    S.iter[slot] += 1;
    S.counters[slot * 4 + 0] += 1;
    S.counters[slot * 4 + 1] += gamma;
    S.counters[slot * 4 + 2] += n;
    S.counters[slot * 4 + 3] += n + 1;
    if (alpha_terms) {                          // the judged slots, in order: run-to-run identical sums
        double a = 0.0;
        const int nj = min(n + 1, gamma);
        for (int s = 0; s < nj; ++s) a += (double)alpha_terms[(size_t)b * gamma + s];
        S.alpha_sum[slot] += a;
        S.judged[slot] += nj;
    }
}
cudaError_t launch_rollback(const SeqState& S, const SeqList& list, int gamma, const int32_t* n_acc,
                            const int32_t* out_tok, const float* alpha_terms, cudaStream_t st) {
    k_rollback<<<1, 64, 0, st>>>(S, list, gamma, n_acc, out_tok, alpha_terms);
    return cudaGetLastError();
}

}  // namespace sd
