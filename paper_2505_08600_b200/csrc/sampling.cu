// Vocabulary-wide kernels: softmax with temperature, the exact integer inverse-CDF draw, the
// draft's per-step sampler and the fused accept / reject / resample kernel.
#include <cooperative_groups.h>

#include "gemm_tc.h"
#include "kernels.h"

namespace sd {

__global__ void k_philox(const uint32_t* __restrict__ ctr, int n, uint32_t k0, uint32_t k1, uint32_t* __restrict__ out) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    uint32_t o[4];
    philox4x32_10(ctr[4 * i], ctr[4 * i + 1], ctr[4 * i + 2], ctr[4 * i + 3], k0, k1, o);
    for (int j = 0; j < 4; ++j) out[4 * i + j] = o[j];
}
cudaError_t launch_philox(const uint32_t* ctr, int n, uint32_t k0, uint32_t k1, uint32_t* out, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    k_philox<<<(n + 127) / 128, 128, 0, st>>>(ctr, n, k0, k1, out);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- block-wide helpers
struct BlockScratch {
    float red[32];
    unsigned long long scan[32];
    unsigned long long total;
    int tok;
    int idx;
};

__device__ __forceinline__ int block_min_int(int v, BlockScratch& sh) {
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    int* r = reinterpret_cast<int*>(sh.red);
    if (lane == 0) r[w] = v;
    __syncthreads();
    int x = (threadIdx.x < nw) ? r[threadIdx.x] : 0x7fffffff;
    if (w == 0) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x = min(x, __shfl_xor_sync(0xffffffffu, x, o));
        if (lane == 0) sh.idx = x;
    }
    __syncthreads();
    return sh.idx;
}

// lowest index of the maximum of f(k), k in [0, V)
template <class F>
__device__ __forceinline__ int block_argmax(F f, int V, BlockScratch& sh, float* max_out) {
    float m = -INFINITY;
    for (int k = threadIdx.x; k < V; k += blockDim.x) m = fmaxf(m, f(k));
    m = block_max(m, sh.red);
    int best = 0x7fffffff;
    for (int k = threadIdx.x; k < V; k += blockDim.x) if (f(k) == m) { best = k; break; }
    if (max_out) *max_out = m;
    return block_min_int(best, sh);
}

// Exact inverse CDF over integer weights floor(w(k) * 2^32): returns the first k whose running
// sum reaches ceil(u_int * total / 2^24), or -1 when every weight is zero.  Each thread owns a
// contiguous chunk; integer addition is associative, so the split cannot change the answer.
template <class F>
__device__ __forceinline__ int block_icdf(F w, int V, uint32_t u_int, BlockScratch& sh) {
    const int t = threadIdx.x, lane = t & 31, wid = t >> 5, nw = (blockDim.x + 31) >> 5;
    const int chunk = (V + blockDim.x - 1) / blockDim.x;
    const int k0 = min(V, t * chunk), k1 = min(V, k0 + chunk);
    unsigned long long local = 0;
    {   // every thread starts its chunk at a different offset, so that a vocabulary row staged in shared
        // memory is read without bank conflicts (the order inside a sum of integers does not matter)
        const int n = k1 - k0;
        int i = n > 0 ? t % n : 0;
        for (int c = 0; c < n; ++c) { local += __float2ull_rz(w(k0 + i) * 4294967296.0f); i = (i + 1 == n) ? 0 : i + 1; }
    }
    unsigned long long incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    __syncthreads();
    if (lane == 31) sh.scan[wid] = incl;
    if (t == 0) sh.tok = -1;
    __syncthreads();
    if (wid == 0) {
        unsigned long long v = lane < nw ? sh.scan[lane] : 0ull, s = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            unsigned long long u = __shfl_up_sync(0xffffffffu, s, o);
            if (lane >= o) s += u;
        }
        sh.scan[lane] = s - v;                       // exclusive prefix of each warp
        if (lane == 31) sh.total = s;
    }
    __syncthreads();
    const unsigned long long tot = sh.total;
    if (tot == 0ull) return -1;
    incl += sh.scan[wid];
    const unsigned long long excl = incl - local;
    const unsigned long long thr = ((unsigned long long)u_int * tot + 16777215ull) >> 24;
    if (excl < thr && thr <= incl) {
        unsigned long long run = excl;
        for (int k = k0; k < k1; ++k) {
            run += __float2ull_rz(w(k) * 4294967296.0f);
            if (run >= thr) { sh.tok = k; break; }
        }
    }
    __syncthreads();
    return sh.tok;
}

// Copies one vocabulary row into shared memory with every load in flight at once (the later
// passes over the row - max, sum, probabilities, CDF - then cost no memory round trips).
__device__ __forceinline__ void stage_row(const float* __restrict__ src, float* __restrict__ dst, int V) {
    if ((V & 3) == 0 && (reinterpret_cast<uintptr_t>(src) & 15) == 0) {
        const float4* s4 = reinterpret_cast<const float4*>(src);
        float4* d4 = reinterpret_cast<float4*>(dst);
        const int n4 = V >> 2;
        for (int k0 = 0; k0 < n4; k0 += 8 * blockDim.x) {
            float4 v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) { const int k = k0 + i * blockDim.x + threadIdx.x; if (k < n4) v[i] = __ldcg(s4 + k); }
#pragma unroll
            for (int i = 0; i < 8; ++i) { const int k = k0 + i * blockDim.x + threadIdx.x; if (k < n4) d4[k] = v[i]; }
        }
    } else {
        for (int k = threadIdx.x; k < V; k += blockDim.x) dst[k] = __ldcg(src + k);
    }
    __syncthreads();
}
constexpr int STAGE_MAX_BYTES = 200 * 1024;      // a row of up to 51200 fp32 values fits beside the static shared memory

// Dynamic shared memory for one staged row, or 0 when the vocabulary is too large to stage.
static size_t row_stage_bytes(int V) { return (size_t)V * 4 <= (size_t)STAGE_MAX_BYTES ? (size_t)V * 4 : 0; }

// ---------------------------------------------------------------- softmax + draw (draft steps)
// One block per row.  probs = softmax(logits / T) (one-hot argmax when T == 0) is written out,
// then one token is drawn from the written fp32 values.
__device__ __forceinline__ int softmax_sample_row(const float* __restrict__ l_global, int V, float T, uint32_t u_int,
                                                  float* __restrict__ probs, BlockScratch& sh, float* rowbuf) {
    const float* l = l_global;
    if (rowbuf) { stage_row(l_global, rowbuf, V); l = rowbuf; }
    if (T == 0.f) {
        int a = block_argmax([&](int k) { return l[k]; }, V, sh, nullptr);
        for (int k = threadIdx.x; k < V; k += blockDim.x) probs[k] = (k == a) ? 1.f : 0.f;
        return a;
    }
    float m = -INFINITY;
    for (int k = threadIdx.x; k < V; k += blockDim.x) m = fmaxf(m, l[k]);
    m = block_max(m, sh.red);
    float s = 0.f;
    // one division each for 1/T and 1/sum, then multiplications: an IEEE division per element costs about as much as
    // the exponential itself, and the result differs from e / sum by an ulp (the probability tolerance is 1e-3)
    const float inv_T = 1.f / T;
    for (int k = threadIdx.x; k < V; k += blockDim.x) s += expf((l[k] - m) * inv_T);
    s = block_sum(s, sh.red);
    const float inv_s = 1.f / s;
    for (int k = threadIdx.x; k < V; k += blockDim.x) {
        const float pk = expf((l[k] - m) * inv_T) * inv_s;
        probs[k] = pk;
        if (rowbuf) rowbuf[k] = pk;                      // the draw below reads the same fp32 values
    }
    __syncthreads();
    const float* pr = rowbuf ? rowbuf : probs;
    int tok = block_icdf([&](int k) { return pr[k]; }, V, u_int, sh);
    if (tok < 0) tok = block_argmax([&](int k) { return pr[k]; }, V, sh, nullptr);
    return tok;
}

__global__ void __launch_bounds__(1024) k_softmax_sample_explicit(const float* __restrict__ logits, int V, float T,
                                                                  const uint32_t* __restrict__ u_int,
                                                                  float* __restrict__ probs, int32_t* __restrict__ tok, int staged) {
    extern __shared__ __align__(16) float rowbuf[];
    __shared__ BlockScratch sh;
    const int r = blockIdx.x;
    int k = softmax_sample_row(logits + (size_t)r * V, V, T, u_int[r], probs + (size_t)r * V, sh, staged ? rowbuf : nullptr);
    if (threadIdx.x == 0) tok[r] = k;
}
cudaError_t launch_softmax_sample_explicit(const float* logits, int rows, int V, float T, const uint32_t* u_int,
                                           float* probs, int32_t* tok, cudaStream_t st) {
    if (rows <= 0) return cudaSuccess;
    const size_t smem = row_stage_bytes(V);
    cudaError_t e = cudaFuncSetAttribute(k_softmax_sample_explicit, cudaFuncAttributeMaxDynamicSharedMemorySize, STAGE_MAX_BYTES);
    if (e != cudaSuccess) return e;
    k_softmax_sample_explicit<<<rows, 1024, smem, st>>>(logits, V, T, u_int, probs, tok, smem > 0);
    return cudaGetLastError();
}

__global__ void __launch_bounds__(1024) k_draft_sample(const float* __restrict__ logits, SeqState S, SeqList list, int V, float T,
                                                       uint64_t seed, int step, int gamma, float* __restrict__ q_out,
                                                       int32_t* __restrict__ x_out, int staged) {
    extern __shared__ __align__(16) float rowbuf[];
    __shared__ BlockScratch sh;
    const int i = blockIdx.x, slot = list.ids[i], b = list.out[i];
    const uint32_t u = uniform24(seed, S.iter[slot], (uint32_t)step, S.seq_id[slot], DRAW_DRAFT);
    int k = softmax_sample_row(logits + (size_t)i * V, V, T, u, q_out + ((size_t)b * gamma + step) * V, sh, staged ? rowbuf : nullptr);
    if (threadIdx.x == 0) x_out[(size_t)b * gamma + step] = k;
}
cudaError_t launch_draft_sample(const float* logits, const SeqState& S, const SeqList& list, int V, float T,
                                uint64_t seed, int step, int gamma, float* q_out, int32_t* x_out, cudaStream_t st) {
    if (list.n <= 0) return cudaSuccess;
    const size_t smem = row_stage_bytes(V);
    cudaError_t e = cudaFuncSetAttribute(k_draft_sample, cudaFuncAttributeMaxDynamicSharedMemorySize, STAGE_MAX_BYTES);
    if (e != cudaSuccess) return e;
    k_draft_sample<<<list.n, 1024, smem, st>>>(logits, S, list, V, T, seed, step, gamma, q_out, x_out, smem > 0);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- accept / reject / resample
// One thread-block cluster per sequence, one CTA per target row (two when gamma + 1 > 8).
// Every CTA works out the softmax statistics of its row(s) and, for a draft slot, the accept
// test u_s * q_s(x_s) <= p_s(x_s) with a single rounded fp32 multiply.  The flags are exchanged
// through distributed shared memory; the CTA that owns the first rejected row n (or row gamma
// after gamma accepts) draws the next token from the residual max(0, p_n - q_n), or from
// p_gamma itself, and writes the result.
constexpr int ACC_ROWS_PER_CTA = 2;

__global__ void __launch_bounds__(1024) k_accept(AcceptParams P, int csize, int staged) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ __align__(16) float rowbuf[];            // one target row (when it fits): every pass over it reads shared memory
    __shared__ BlockScratch sh;
    __shared__ float row_max[ACC_ROWS_PER_CTA], row_inv[ACC_ROWS_PER_CTA];      // max of the row's logits, 1 / sum of its exponentials
    __shared__ int row_arg[ACC_ROWS_PER_CTA];
    __shared__ int flag_sh[ACC_ROWS_PER_CTA];
    __shared__ int n_sh;
    pdl_launch_dependents();
    const int i = blockIdx.x / csize, rank = blockIdx.x % csize;
    const int idx = P.use_list ? P.list.ids[i] : i;
    const int b = P.use_list ? P.list.out[i] : i;
    const int V = P.V, gamma = P.gamma;
    const float T = P.T;
    const float inv_T = T > 0.f ? 1.f / T : 0.f;
    const float* tgt = P.target + (size_t)b * (gamma + 1) * V;
    const float* q = P.q + (size_t)b * gamma * V;
    const int32_t* x = P.x + (size_t)b * gamma;
    const bool logits = P.target_is_logits != 0;
    pdl_wait();                                   // target rows, drafts and per-sequence state come from earlier kernels

    int cur = -1;                                 // which of this CTA's rows the buffer holds
    auto ensure = [&](int j, int li) {
        if (staged && cur != li) { __syncthreads(); stage_row(tgt + (size_t)j * V, rowbuf, V); cur = li; }
    };
    auto val = [&](int j, int k) -> float { return staged ? rowbuf[k] : tgt[(size_t)j * V + k]; };
    auto prob = [&](int j, int li, int k) -> float {          // li: index of row j among this CTA's rows
        if (logits && T == 0.f) return k == row_arg[li] ? 1.f : 0.f;
        const float v = val(j, k);
        if (!logits) return v;
        return expf((v - row_max[li]) * inv_T) * row_inv[li];      // (multiplications by 1/T and 1/sum: see softmax_sample_row)
    };

    for (int li = 0; li < ACC_ROWS_PER_CTA; ++li) {
        const int j = rank + li * csize;
        if (j > gamma) break;                                   // uniform in the CTA
        ensure(j, li);
        if (logits) {
            if (T == 0.f) {
                int a = block_argmax([&](int k) { return val(j, k); }, V, sh, nullptr);
                if (threadIdx.x == 0) row_arg[li] = a;
            } else {
                float m = -INFINITY;
                for (int k = threadIdx.x; k < V; k += blockDim.x) m = fmaxf(m, val(j, k));
                m = block_max(m, sh.red);
                float sum = 0.f;
                for (int k = threadIdx.x; k < V; k += blockDim.x) sum += expf((val(j, k) - m) * inv_T);
                sum = block_sum(sum, sh.red);
                if (threadIdx.x == 0) { row_max[li] = m; row_inv[li] = 1.f / sum; }
            }
            __syncthreads();
        }
        if (P.alpha_terms && j < gamma) {                       // Eq. 1's alpha for this slot: the draft is kept with probability sum_k min(p, q)
            const float* __restrict__ qj = q + (size_t)j * V;
            float a = 0.f;
            const int stride = blockDim.x;
            int k = threadIdx.x;
            for (; k + 3 * stride < V; k += 4 * stride) {             // four independent loads of q in flight per thread
                const float q0 = __ldg(qj + k), q1 = __ldg(qj + k + stride), q2 = __ldg(qj + k + 2 * stride), q3 = __ldg(qj + k + 3 * stride);
                a += fminf(prob(j, li, k), q0);
                a += fminf(prob(j, li, k + stride), q1);
                a += fminf(prob(j, li, k + 2 * stride), q2);
                a += fminf(prob(j, li, k + 3 * stride), q3);
            }
            for (; k < V; k += stride) a += fminf(prob(j, li, k), __ldg(qj + k));
            a = block_sum(a, sh.red);
            if (threadIdx.x == 0) P.alpha_terms[(size_t)b * gamma + j] = a;
        }
        if (threadIdx.x == 0 && j < gamma) {
            int ok = 0;
            const int xs = x[j];
            if (xs >= 0 && xs < V) {                            // an impossible token counts as rejected
                const uint32_t ui = uniform24(P.seed, P.iter[idx], (uint32_t)j, P.seq_id[idx], DRAW_ACCEPT);
                const float u = (float)ui * (1.0f / 16777216.0f);
                const float lhs = __fmul_rn(u, q[(size_t)j * V + xs]);
                ok = lhs <= prob(j, li, xs);
            }
            flag_sh[li] = ok;
        }
    }
    cluster.sync();                                             // every CTA's flags are in place
    if (threadIdx.x == 0) {
        int n = 0;
        while (n < gamma) {
            const int* remote = cluster.map_shared_rank(flag_sh, n % csize);
            if (!remote[n / csize]) break;
            ++n;
        }
        n_sh = n;
    }
    __syncthreads();
    const int n = n_sh;
    if (n % csize == rank) {                                    // this CTA holds the statistics of row n
        const int li = n / csize;
        const uint32_t ui = uniform24(P.seed, P.iter[idx], (uint32_t)n, P.seq_id[idx], DRAW_RESAMPLE);
        const float* qn = q + (size_t)(n < gamma ? n : 0) * V;
        int y;
        if (staged) {
            // the weights of the draw replace the row in shared memory (one coalesced pass over q), then the
            // integer CDF runs on them; residual all zero -> the target distribution itself -> its argmax
            ensure(n, li);
            for (int k = threadIdx.x; k < V; k += blockDim.x) {
                const float pk = prob(n, li, k);
                rowbuf[k] = n < gamma ? fmaxf(__fsub_rn(pk, qn[k]), 0.f) : pk;
            }
            __syncthreads();
            y = block_icdf([&](int k) { return rowbuf[k]; }, V, ui, sh);
            if (y < 0 && n < gamma) {
                cur = -1;
                ensure(n, li);
                for (int k = threadIdx.x; k < V; k += blockDim.x) rowbuf[k] = prob(n, li, k);
                __syncthreads();
                y = block_icdf([&](int k) { return rowbuf[k]; }, V, ui, sh);
            }
            if (y < 0) y = block_argmax([&](int k) { return rowbuf[k]; }, V, sh, nullptr);
        } else {
            if (n < gamma) {
                y = block_icdf([&](int k) { return fmaxf(__fsub_rn(prob(n, li, k), qn[k]), 0.f); }, V, ui, sh);
                if (y < 0) y = block_icdf([&](int k) { return prob(n, li, k); }, V, ui, sh);
            } else {
                y = block_icdf([&](int k) { return prob(n, li, k); }, V, ui, sh);
            }
            if (y < 0) y = block_argmax([&](int k) { return prob(n, li, k); }, V, sh, nullptr);
        }
        if (threadIdx.x == 0) P.n_acc[b] = n;
        for (int s = threadIdx.x; s <= gamma; s += blockDim.x)
            P.out_tok[(size_t)b * (gamma + 1) + s] = s < n ? x[s] : (s == n ? y : -1);
    }
    cluster.sync();                                             // no CTA leaves while its flags may still be read
}

cudaError_t launch_accept(const AcceptParams& p, int dependent, cudaStream_t st) {
    if (p.B <= 0) return cudaSuccess;
    int csize = 1;
    while (csize < p.gamma + 1 && csize < 8) csize <<= 1;      // portable cluster sizes only
    if (csize * ACC_ROWS_PER_CTA < p.gamma + 1) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    const size_t smem = row_stage_bytes(p.V);
    cudaError_t e = cudaFuncSetAttribute(k_accept, cudaFuncAttributeMaxDynamicSharedMemorySize, STAGE_MAX_BYTES);
    if (e != cudaSuccess) return e;
    cfg.gridDim = dim3(p.B * csize); cfg.blockDim = dim3(1024); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = csize; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, k_accept, p, csize, (int)(smem > 0));
}

}  // namespace sd
