// The Mamba-based prompt classifier (Section 2.4, Section 3.3.3): embedding -> one selective state-space layer ->
// average pooling over the prompt -> fully connected layer -> argmax.  Everything is fp32.
//
// The layer's recurrence h_t = a_t * h_{t-1} + b_t is linear in h, so a prompt is cut into chunks of MB_CHUNK tokens
// that are scanned side by side: (A) every chunk is scanned from a zero state and leaves its end state and the product
// of its decays, (B) a short serial pass over a prompt's chunks turns those into the state each chunk starts from,
// (C) every chunk is scanned again from that state and emits the gated outputs.  Prompts of one chunk skip (A) and (B).
// The pooled vector is the mean over tokens of W_out g_t, which is W_out applied to the mean of g_t: the kernels sum
// g_t per channel (chunks in order) and apply W_out and the classification layer once per prompt.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <vector>

#include "../../include/sd.h"

namespace sd {
namespace {

constexpr int MB_CHUNK = 64;         // tokens per chunk of the scan
constexpr int MB_TOK_TILE = 16;      // tokens per CTA of the input projection
constexpr int MB_MAX_N = 16;         // state size kept in registers
constexpr int MB_MAX_CONV = 8;

struct MambaDims { int V, D, Di, N, R, Kc, K; };

struct ChunkRec { int32_t prompt, tok0, n_tok, pos0; };      // tok0: index into the flattened token list; pos0: position of the chunk's first token in its prompt

__device__ __forceinline__ float silu_f(float x) { return x / (1.f + expf(-x)); }
__device__ __forceinline__ float softplus_f(float x) { return x > 20.f ? x : log1pf(expf(x)); }

// Where every flattened token comes from and its position in its prompt, from the chunk records (one CTA per chunk).
__global__ void k_mamba_tables(const ChunkRec* __restrict__ chunks, const int64_t* __restrict__ starts, int64_t* __restrict__ tok_src,
                               int32_t* __restrict__ tok_pos) {
    const ChunkRec ch = chunks[blockIdx.x];
    for (int i = threadIdx.x; i < ch.n_tok; i += blockDim.x) {
        tok_src[ch.tok0 + i] = starts[ch.prompt] + ch.pos0 + i;
        tok_pos[ch.tok0 + i] = ch.pos0 + i;
    }
}

// u, z = split(W_in E[token]) for a tile of tokens.  One thread per output feature; the tile's embedding rows sit in
// shared memory, and W_in passes through shared memory in blocks of 256 rows x 32 columns so that global loads are
// coalesced (a warp reads 128 contiguous bytes of one row) and every thread then walks its own row without bank
// conflicts (rows padded to 33 words).
__global__ void __launch_bounds__(256)
k_mamba_in(MambaDims m, const int32_t* __restrict__ tokens, const int64_t* __restrict__ tok_src, int T, const float* __restrict__ embed,
           const float* __restrict__ w_in, float* __restrict__ u, float* __restrict__ z) {
    extern __shared__ __align__(16) float in_smem[];
    float* e_s = in_smem;                                // [MB_TOK_TILE][D]
    float* w_s = in_smem + MB_TOK_TILE * m.D;            // [256][36]: rows padded to 36 words (16-byte aligned, conflict-free float4 reads)
    const int t0 = blockIdx.x * MB_TOK_TILE, nt = min(MB_TOK_TILE, T - t0);
    for (int i = threadIdx.x; i < MB_TOK_TILE * m.D; i += blockDim.x) {
        const int tt = i / m.D, d = i % m.D;
        float e = 0.f;                                   // rows past the end of the token list are zero
        if (tt < nt) {
            int tok = tokens[tok_src[t0 + tt]];
            tok = min(max(tok, 0), m.V - 1);
            e = embed[(size_t)tok * m.D + d];
        }
        e_s[tt * m.D + d] = e;
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int j0 = 0; j0 < 2 * m.Di; j0 += 256) {
        const int j = j0 + threadIdx.x;
        float acc[MB_TOK_TILE];
#pragma unroll
        for (int tt = 0; tt < MB_TOK_TILE; ++tt) acc[tt] = 0.f;
        for (int d0 = 0; d0 < m.D; d0 += 32) {
            __syncthreads();                             // the previous block of W (and, the first time, e_s) is settled
            for (int rr = warp; rr < 256; rr += 8) {     // warp per row: lanes along the row
                const int row = j0 + rr;
                w_s[rr * 36 + lane] = (row < 2 * m.Di && d0 + lane < m.D) ? w_in[(size_t)row * m.D + d0 + lane] : 0.f;
            }
            __syncthreads();
            const int nd = min(32, m.D - d0);
            if ((m.D & 3) == 0) {                        // four columns at a time: one 16-byte read of W and of every token's embedding
                for (int dd = 0; dd < nd; dd += 4) {
                    const float4 w = *reinterpret_cast<const float4*>(w_s + threadIdx.x * 36 + dd);
#pragma unroll
                    for (int tt = 0; tt < MB_TOK_TILE; ++tt) {
                        const float4 e = *reinterpret_cast<const float4*>(e_s + tt * m.D + d0 + dd);
                        acc[tt] = fmaf(w.x, e.x, acc[tt]); acc[tt] = fmaf(w.y, e.y, acc[tt]);
                        acc[tt] = fmaf(w.z, e.z, acc[tt]); acc[tt] = fmaf(w.w, e.w, acc[tt]);
                    }
                }
            } else {
                for (int dd = 0; dd < nd; ++dd) {
                    const float w = w_s[threadIdx.x * 36 + dd];
#pragma unroll
                    for (int tt = 0; tt < MB_TOK_TILE; ++tt) acc[tt] = fmaf(w, e_s[tt * m.D + d0 + dd], acc[tt]);
                }
            }
        }
        if (j < 2 * m.Di) {
            float* dst = j < m.Di ? u : z;
            const int c = j < m.Di ? j : j - m.Di;
#pragma unroll
            for (int tt = 0; tt < MB_TOK_TILE; ++tt) if (tt < nt) dst[(size_t)(t0 + tt) * m.Di + c] = acc[tt];
        }
    }
}

// Per tile of MB_CP_TILE tokens: causal depthwise convolution + SiLU, the projections to (r, B, C), the step size.
// A tile shares every weight it reads (each row of W_x is read once per tile and used for all its tokens).
constexpr int MB_CP_TILE = 8;
__global__ void __launch_bounds__(256)
k_mamba_conv_proj(MambaDims m, int T, const int32_t* __restrict__ tok_pos /*position inside its prompt*/,
                  const float* __restrict__ u, const float* __restrict__ w_conv, const float* __restrict__ b_conv,
                  const float* __restrict__ w_x, const float* __restrict__ w_dt, const float* __restrict__ b_dt,
                  float* __restrict__ v, float* __restrict__ dt, float* __restrict__ bc) {
    extern __shared__ float sm[];                        // v [tile][Di], x_dbl [tile][R + 2N]
    const int n_x = m.R + 2 * m.N;
    float* v_s = sm;
    float* xd_s = sm + MB_CP_TILE * m.Di;
    const int t0 = blockIdx.x * MB_CP_TILE, nt = min(MB_CP_TILE, T - t0);
    for (int idx = threadIdx.x; idx < MB_CP_TILE * m.Di; idx += blockDim.x) {
        const int tt = idx / m.Di, c = idx % m.Di;
        float val = 0.f;
        if (tt < nt) {
            const int t = t0 + tt, pos = tok_pos[t];
            float acc = b_conv[c];
            for (int j = 0; j < m.Kc; ++j) {
                const int back = m.Kc - 1 - j;           // tap j looks `back` tokens back; nothing before the prompt's first token
                if (back <= pos) acc = fmaf(w_conv[(size_t)c * m.Kc + j], u[(size_t)(t - back) * m.Di + c], acc);
            }
            val = silu_f(acc);
            v[(size_t)t * m.Di + c] = val;
        }
        v_s[idx] = val;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    for (int o = warp; o < n_x; o += n_warps) {
        float acc[MB_CP_TILE];
#pragma unroll
        for (int tt = 0; tt < MB_CP_TILE; ++tt) acc[tt] = 0.f;
        for (int c = lane; c < m.Di; c += 32) {
            const float w = w_x[(size_t)o * m.Di + c];
#pragma unroll
            for (int tt = 0; tt < MB_CP_TILE; ++tt) acc[tt] = fmaf(w, v_s[tt * m.Di + c], acc[tt]);
        }
#pragma unroll
        for (int tt = 0; tt < MB_CP_TILE; ++tt) {
#pragma unroll
            for (int s = 16; s > 0; s >>= 1) acc[tt] += __shfl_xor_sync(0xffffffffu, acc[tt], s);
            if (lane == 0 && tt < nt) {
                xd_s[tt * n_x + o] = acc[tt];
                if (o >= m.R) bc[(size_t)(t0 + tt) * 2 * m.N + (o - m.R)] = acc[tt];
            }
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < nt * m.Di; idx += blockDim.x) {
        const int tt = idx / m.Di, c = idx % m.Di;
        float acc = b_dt[c];
        for (int r = 0; r < m.R; ++r) acc = fmaf(w_dt[(size_t)c * m.R + r], xd_s[tt * n_x + r], acc);
        dt[(size_t)(t0 + tt) * m.Di + c] = softplus_f(acc);
    }
}

// One chunk x 64 channels.  EMIT = false: scan from zero, leave the end state and the product of the decays.
// EMIT = true: scan from the chunk's starting state and leave the chunk's sum over tokens of y_t * silu(z_t).
template <bool EMIT>
__global__ void __launch_bounds__(64)
k_mamba_scan(MambaDims m, const ChunkRec* __restrict__ chunks, const float* __restrict__ v, const float* __restrict__ dt,
             const float* __restrict__ bc, const float* __restrict__ z, const float* __restrict__ a_log, const float* __restrict__ d_skip,
             float* __restrict__ end_state /*[chunk][Di][N]*/, float* __restrict__ decay /*[chunk][Di][N]*/,
             const float* __restrict__ start_state /*[chunk][Di][N] or nullptr = zero*/, float* __restrict__ chunk_sum /*[chunk][Di]*/) {
    __shared__ float bc_s[MB_CHUNK][2 * MB_MAX_N];
    const ChunkRec ch = chunks[blockIdx.x];
    const int c = blockIdx.y * 64 + threadIdx.x;
    for (int i = threadIdx.x; i < ch.n_tok * 2 * m.N; i += blockDim.x) bc_s[i / (2 * m.N)][i % (2 * m.N)] = bc[(size_t)ch.tok0 * 2 * m.N + i];
    __syncthreads();
    if (c >= m.Di) return;
    float A[MB_MAX_N], h[MB_MAX_N], p[MB_MAX_N];
#pragma unroll
    for (int n = 0; n < MB_MAX_N; ++n) {
        A[n] = n < m.N ? -expf(a_log[(size_t)c * m.N + n]) : 0.f;
        h[n] = (EMIT && start_state && n < m.N) ? start_state[((size_t)blockIdx.x * m.Di + c) * m.N + n] : 0.f;
        p[n] = 1.f;
    }
    const float dsk = d_skip[c];
    float sum = 0.f;
    for (int tt = 0; tt < ch.n_tok; ++tt) {
        const size_t ti = (size_t)(ch.tok0 + tt) * m.Di + c;
        const float d = dt[ti], x = v[ti], dx = d * x;
        float y = 0.f;
#pragma unroll
        for (int n = 0; n < MB_MAX_N; ++n) {
            if (n < m.N) {
                const float a = expf(d * A[n]);
                h[n] = fmaf(a, h[n], dx * bc_s[tt][n]);
                if (EMIT) y = fmaf(h[n], bc_s[tt][m.N + n], y); else p[n] *= a;
            }
        }
        if (EMIT) sum += (y + dsk * x) * silu_f(z[ti]);
    }
    if (EMIT) chunk_sum[(size_t)blockIdx.x * m.Di + c] = sum;
    else {
#pragma unroll
        for (int n = 0; n < MB_MAX_N; ++n) if (n < m.N) {
            end_state[((size_t)blockIdx.x * m.Di + c) * m.N + n] = h[n];
            decay[((size_t)blockIdx.x * m.Di + c) * m.N + n] = p[n];
        }
    }
}

// The state each chunk starts from: serial over the chunks of a prompt, one thread per (channel, state).
__global__ void k_mamba_carry(MambaDims m, const int32_t* __restrict__ prompt_chunk0 /*[n_prompts + 1]*/, const float* __restrict__ end_state,
                              const float* __restrict__ decay, float* __restrict__ start_state) {
    const int i = blockIdx.y * blockDim.x + threadIdx.x;
    if (i >= m.Di * m.N) return;
    float s = 0.f;
    for (int ch = prompt_chunk0[blockIdx.x]; ch < prompt_chunk0[blockIdx.x + 1]; ++ch) {
        const size_t at = (size_t)ch * m.Di * m.N + i;
        start_state[at] = s;
        s = fmaf(decay[at], s, end_state[at]);
    }
}

// Per prompt: mean over tokens of the gated outputs (chunks in order), W_out, the classification layer, argmax.
__global__ void k_mamba_head(MambaDims m, const int32_t* __restrict__ prompt_chunk0, const int32_t* __restrict__ lens,
                             const float* __restrict__ chunk_sum, const float* __restrict__ w_out, const float* __restrict__ w_fc,
                             const float* __restrict__ b_fc, float* __restrict__ scores, int32_t* __restrict__ labels) {
    extern __shared__ float hs[];                        // g mean [Di], pooled [D], scores [K]
    float* g_s = hs;
    float* o_s = hs + m.Di;
    float* sc_s = o_s + m.D;
    const int pr = blockIdx.x;
    const float inv = 1.f / (float)lens[pr];
    for (int c = threadIdx.x; c < m.Di; c += blockDim.x) {
        float s = 0.f;
        for (int ch = prompt_chunk0[pr]; ch < prompt_chunk0[pr + 1]; ++ch) s += chunk_sum[(size_t)ch * m.Di + c];
        g_s[c] = s * inv;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    for (int d = warp; d < m.D; d += n_warps) {
        float acc = 0.f;
        for (int c = lane; c < m.Di; c += 32) acc = fmaf(w_out[(size_t)d * m.Di + c], g_s[c], acc);
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
        if (lane == 0) o_s[d] = acc;
    }
    __syncthreads();
    for (int k = warp; k < m.K; k += n_warps) {
        float acc = 0.f;
        for (int d = lane; d < m.D; d += 32) acc = fmaf(w_fc[(size_t)k * m.D + d], o_s[d], acc);
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
        if (lane == 0) { acc += b_fc[k]; sc_s[k] = acc; if (scores) scores[(size_t)pr * m.K + k] = acc; }
    }
    __syncthreads();
    if (threadIdx.x == 0 && labels) {
        int best = 0;
        for (int k = 1; k < m.K; ++k) if (sc_s[k] > sc_s[best]) best = k;        // lowest index on ties
        labels[pr] = best;
    }
}

size_t al(size_t v) { return (v + 255) & ~(size_t)255; }

bool dims_ok(const sd_mamba_desc* d, MambaDims& m) {
    if (!d || d->vocab < 1 || d->d_model < 1 || d->d_state < 1 || d->d_conv < 1 || d->expand < 1 || d->n_classes < 1 || d->dt_rank < 1) return false;
    m = MambaDims{d->vocab, d->d_model, d->expand * d->d_model, d->d_state, d->dt_rank, d->d_conv, d->n_classes};
    return true;
}

struct Layout { size_t u, z, v, dt, bc, end_state, decay, start_state, chunk_sum, tok_src, tok_pos, chunks, prompt_chunk0, lens, starts, total; };

Layout layout(const MambaDims& m, int64_t T, int64_t n_chunks, int n_prompts) {
    Layout L;
    size_t o = 0;
    auto take = [&](size_t bytes) { const size_t at = o; o += al(bytes); return at; };
    L.u = take((size_t)T * m.Di * 4); L.z = take((size_t)T * m.Di * 4); L.v = take((size_t)T * m.Di * 4); L.dt = take((size_t)T * m.Di * 4);
    L.bc = take((size_t)T * 2 * m.N * 4);
    L.end_state = take((size_t)n_chunks * m.Di * m.N * 4); L.decay = take((size_t)n_chunks * m.Di * m.N * 4);
    L.start_state = take((size_t)n_chunks * m.Di * m.N * 4);
    L.chunk_sum = take((size_t)n_chunks * m.Di * 4);
    L.tok_src = take((size_t)T * 8); L.tok_pos = take((size_t)T * 4);
    L.chunks = take((size_t)n_chunks * sizeof(ChunkRec));
    L.prompt_chunk0 = take((size_t)(n_prompts + 1) * 4); L.lens = take((size_t)n_prompts * 4); L.starts = take((size_t)n_prompts * 8);
    L.total = o;
    return L;
}

}  // namespace
}  // namespace sd

extern "C" size_t sd_mamba_workspace(const sd_mamba_desc* desc, int64_t total_tokens, int n_prompts) {
    sd::MambaDims m;
    if (!sd::dims_ok(desc, m) || total_tokens < 0 || n_prompts < 0) return 0;
    // every prompt may end with a partly filled chunk
    const int64_t n_chunks = total_tokens / sd::MB_CHUNK + n_prompts;
    return sd::layout(m, total_tokens, n_chunks, n_prompts).total;
}

extern "C" sd_status sd_mamba_classify(const sd_mamba_desc* desc, const sd_mamba_weights* w, const int32_t* tokens_dev,
                                       const int64_t* starts_host, const int32_t* lens_host, int n_prompts, float* scores_dev,
                                       int32_t* labels_dev, void* workspace_dev, size_t workspace_bytes, void* cuda_stream) {
    using namespace sd;
    MambaDims m;
    if (!dims_ok(desc, m) || !w || !tokens_dev || !starts_host || !lens_host || n_prompts < 0 || (!scores_dev && !labels_dev)) return SD_ERR_INVALID_ARG;
    if (!w->embed || !w->w_in || !w->w_conv || !w->b_conv || !w->w_x || !w->w_dt || !w->b_dt || !w->a_log || !w->d_skip || !w->w_out || !w->w_fc || !w->b_fc)
        return SD_ERR_INVALID_ARG;
    if (m.N > MB_MAX_N || m.Kc > MB_MAX_CONV || m.Di > 1024 || m.D > 512 || m.R + 2 * m.N > 256 || m.K > 64) return SD_ERR_UNSUPPORTED;
    if (n_prompts == 0) return SD_OK;
    int64_t T = 0;
    for (int i = 0; i < n_prompts; ++i) {
        if (lens_host[i] < 1 || starts_host[i] < 0) return SD_ERR_INVALID_ARG;
        T += lens_host[i];
    }
    if (T > (int64_t)1 << 30) return SD_ERR_CAPACITY;
    if (!workspace_dev || workspace_bytes < sd_mamba_workspace(desc, T, n_prompts)) return SD_ERR_CAPACITY;
    // host tables: the chunks of every prompt (the per-token tables are filled on the device from them)
    std::vector<int32_t> prompt_chunk0((size_t)n_prompts + 1);
    std::vector<ChunkRec> chunks;
    int64_t t = 0;
    int max_len = 0;
    for (int i = 0; i < n_prompts; ++i) {
        prompt_chunk0[i] = (int32_t)chunks.size();
        max_len = lens_host[i] > max_len ? lens_host[i] : max_len;
        for (int p = 0; p < lens_host[i]; p += MB_CHUNK) {
            const int n = lens_host[i] - p < MB_CHUNK ? lens_host[i] - p : MB_CHUNK;
            chunks.push_back(ChunkRec{i, (int32_t)t, n, p});
            t += n;
        }
    }
    prompt_chunk0[n_prompts] = (int32_t)chunks.size();
    const int64_t n_chunks = (int64_t)chunks.size();
    const Layout L = layout(m, T, T / MB_CHUNK + n_prompts, n_prompts);
    char* base = (char*)workspace_dev;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    auto up = [&](size_t at, const void* src, size_t bytes) { return cudaMemcpyAsync(base + at, src, bytes, cudaMemcpyHostToDevice, st) == cudaSuccess; };
    if (!up(L.chunks, chunks.data(), (size_t)n_chunks * sizeof(ChunkRec)) || !up(L.prompt_chunk0, prompt_chunk0.data(), (size_t)(n_prompts + 1) * 4) ||
        !up(L.lens, lens_host, (size_t)n_prompts * 4) || !up(L.starts, starts_host, (size_t)n_prompts * 8))
        return SD_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SD_ERR_CUDA;      // the host tables above go out of scope
    float* u = (float*)(base + L.u); float* z = (float*)(base + L.z); float* v = (float*)(base + L.v); float* dt = (float*)(base + L.dt);
    float* bc = (float*)(base + L.bc);
    const ChunkRec* chunks_d = (const ChunkRec*)(base + L.chunks);
    const int32_t* pc0 = (const int32_t*)(base + L.prompt_chunk0);

    k_mamba_tables<<<(unsigned)n_chunks, 64, 0, st>>>(chunks_d, (const int64_t*)(base + L.starts), (int64_t*)(base + L.tok_src), (int32_t*)(base + L.tok_pos));
    const size_t in_smem_bytes = ((size_t)MB_TOK_TILE * m.D + 256 * 36) * 4;      // up to 66 KB at d_model 512: above the default limit
    if (cudaFuncSetAttribute(k_mamba_in, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)in_smem_bytes) != cudaSuccess) return SD_ERR_CUDA;
    k_mamba_in<<<(unsigned)((T + MB_TOK_TILE - 1) / MB_TOK_TILE), 256, in_smem_bytes, st>>>(
        m, tokens_dev, (const int64_t*)(base + L.tok_src), (int)T, w->embed, w->w_in, u, z);
    k_mamba_conv_proj<<<(unsigned)((T + MB_CP_TILE - 1) / MB_CP_TILE), 256, (size_t)MB_CP_TILE * (m.Di + m.R + 2 * m.N) * 4, st>>>(
        m, (int)T, (const int32_t*)(base + L.tok_pos), u, w->w_conv, w->b_conv, w->w_x, w->w_dt, w->b_dt, v, dt, bc);
    const dim3 sgrid((unsigned)n_chunks, (unsigned)((m.Di + 63) / 64));
    const float* start = nullptr;
    if (max_len > MB_CHUNK) {
        k_mamba_scan<false><<<sgrid, 64, 0, st>>>(m, chunks_d, v, dt, bc, z, w->a_log, w->d_skip, (float*)(base + L.end_state), (float*)(base + L.decay),
                                                  nullptr, nullptr);
        k_mamba_carry<<<dim3((unsigned)n_prompts, (unsigned)((m.Di * m.N + 255) / 256)), 256, 0, st>>>(
            m, pc0, (const float*)(base + L.end_state), (const float*)(base + L.decay), (float*)(base + L.start_state));
        start = (const float*)(base + L.start_state);
    }
    k_mamba_scan<true><<<sgrid, 64, 0, st>>>(m, chunks_d, v, dt, bc, z, w->a_log, w->d_skip, nullptr, nullptr, start, (float*)(base + L.chunk_sum));
    k_mamba_head<<<(unsigned)n_prompts, 256, (size_t)(m.Di + m.D + m.K) * 4, st>>>(
        m, pc0, (const int32_t*)(base + L.lens), (const float*)(base + L.chunk_sum), w->w_out, w->w_fc, w->b_fc, scores_dev, labels_dev);
    return cudaGetLastError() == cudaSuccess ? SD_OK : SD_ERR_CUDA;
}
