// Split-KV attention for the verify / draft rows (bf16 cache, head_dim 64 or 128).
//
// A block of consecutive query rows of one sequence (the gamma+1 verify rows) times the query
// heads that share one KV head is scored against one slice of that head's cache; every slice
// is streamed from HBM once, whatever the number of rows.  Slices leave unnormalised partial
// outputs with their running max and sum; a second small kernel merges them.
// Cache layout of one layer: [slot][kv_head][position][head_dim].
#include "kernels.h"

namespace sd {

namespace {

constexpr int ATT_THREADS = 128;
constexpr int NQ_MAX = 32;          // query vectors per CTA: rows in the block x heads per KV head
constexpr int QCHUNK = 8;           // query vectors accumulated at once in the value pass

__device__ __forceinline__ void unpack8(const uint4& u, float f[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w[i] << 16); f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
}

struct AttnParams {
    const bf16* q; const bf16* kc; const bf16* vc;
    const int32_t* row_slot; const int32_t* row_pos;
    float* part_o;      // [rows][H][n_splits][hd]
    float* part_ml;     // [rows][H][n_splits][2]
    int n_rows, rows_per_seq, rows_per_block, H, Hkv, max_ctx, split_len, n_splits;
};

template <int HD>
__global__ void __launch_bounds__(ATT_THREADS) k_attn_split(AttnParams P) {
    extern __shared__ float sm[];
    constexpr int LPP = 8;                       // lanes that share one key position
    constexpr int EPL = HD / LPP;                // elements of a key each of them holds (8 or 16)
    const int split = blockIdx.x, kvh = blockIdx.y;
    const int group = P.H / P.Hkv;
    const int bps = (P.rows_per_seq + P.rows_per_block - 1) / P.rows_per_block;     // query blocks per sequence
    const int r0 = (blockIdx.z / bps) * P.rows_per_seq + (blockIdx.z % bps) * P.rows_per_block;
    const int nr = min(P.rows_per_block, P.rows_per_seq - (int)(blockIdx.z % bps) * P.rows_per_block);
    const int nq = nr * group;
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    float* qs = sm;                              // [nq][HD] scaled queries
    float* sc = qs + NQ_MAX * HD;                // [nq][split_len] scores, then probabilities
    float* red = sc + NQ_MAX * P.split_len;      // [4][QCHUNK][HD] cross-warp reduction of the value pass
    __shared__ int pos_sm[NQ_MAX];
    __shared__ float m_sm[NQ_MAX], l_sm[NQ_MAX];

    int max_pos = -1;
    for (int j = 0; j < nr; ++j) max_pos = max(max_pos, P.row_pos[r0 + j]);
    const int p_begin = split * P.split_len;
    const int p_end = min(p_begin + P.split_len, max_pos + 1);
    const int np = p_end - p_begin;              // positions of this slice (<= 0: nothing to do)
    if (np <= 0) {
        for (int i = t; i < nq; i += ATT_THREADS) {
            const int r = r0 + i / group, h = kvh * group + i % group;
            float* ml = P.part_ml + (((size_t)r * P.H + h) * P.n_splits + split) * 2;
            ml[0] = -INFINITY; ml[1] = 0.f;
        }
        return;
    }
    const int slot = P.row_slot[r0];
    const bf16* K = P.kc + (((size_t)slot * P.Hkv + kvh) * P.max_ctx + p_begin) * HD;
    const bf16* V = P.vc + (((size_t)slot * P.Hkv + kvh) * P.max_ctx + p_begin) * HD;

    const float scale = rsqrtf((float)HD);
    for (int i = t; i < nq * HD; i += ATT_THREADS) {
        const int j = i / HD, e = i % HD;
        const int r = r0 + j / group, h = kvh * group + j % group;
        qs[j * HD + e] = __bfloat162float(P.q[((size_t)r * P.H + h) * HD + e]) * scale;
    }
    if (t < nq) pos_sm[t] = P.row_pos[r0 + t / group];
    __syncthreads();

    // ---- scores: eight lanes per key position, 16 positions per round
    const int grp = t / LPP, gl = t % LPP;
    for (int pb = 0; pb < np; pb += ATT_THREADS / LPP) {
        const int p = pb + grp;
        float kf[EPL];
        if (p < np) {
#pragma unroll
            for (int c = 0; c < EPL / 8; ++c) {
                const uint4 u = *reinterpret_cast<const uint4*>(K + (size_t)p * HD + c * 64 + gl * 8);
                unpack8(u, kf + 8 * c);
            }
        } else {
#pragma unroll
            for (int e = 0; e < EPL; ++e) kf[e] = 0.f;
        }
        for (int j = 0; j < nq; ++j) {
            float s = 0.f;
#pragma unroll
            for (int c = 0; c < EPL / 8; ++c) {
                const float4 qa = *reinterpret_cast<const float4*>(qs + j * HD + c * 64 + gl * 8);
                const float4 qb4 = *reinterpret_cast<const float4*>(qs + j * HD + c * 64 + gl * 8 + 4);
                s = fmaf(kf[8 * c + 0], qa.x, s); s = fmaf(kf[8 * c + 1], qa.y, s);
                s = fmaf(kf[8 * c + 2], qa.z, s); s = fmaf(kf[8 * c + 3], qa.w, s);
                s = fmaf(kf[8 * c + 4], qb4.x, s); s = fmaf(kf[8 * c + 5], qb4.y, s);
                s = fmaf(kf[8 * c + 6], qb4.z, s); s = fmaf(kf[8 * c + 7], qb4.w, s);
            }
            s += __shfl_xor_sync(0xffffffffu, s, 1);
            s += __shfl_xor_sync(0xffffffffu, s, 2);
            s += __shfl_xor_sync(0xffffffffu, s, 4);
            if (gl == 0 && p < np) sc[j * P.split_len + p] = (p_begin + p <= pos_sm[j]) ? s : -INFINITY;
        }
    }
    __syncthreads();

    // ---- per-query max and sum over the slice; scores become probabilities relative to the slice max
    for (int j = warp; j < nq; j += ATT_THREADS / 32) {
        float m = -INFINITY;
        for (int p = lane; p < np; p += 32) m = fmaxf(m, sc[j * P.split_len + p]);
        m = warp_max(m);
        float l = 0.f;
        for (int p = lane; p < np; p += 32) {
            const float e = (m == -INFINITY) ? 0.f : __expf(sc[j * P.split_len + p] - m);
            sc[j * P.split_len + p] = e;
            l += e;
        }
        l = warp_sum(l);
        if (lane == 0) { m_sm[j] = m; l_sm[j] = l; }
    }
    __syncthreads();

    // ---- values: 16 (HD 128) or 8 (HD 64) threads span a value row, eight elements each
    constexpr int TPR = HD / 8;                  // threads per value row
    constexpr int PGROUPS = ATT_THREADS / TPR;   // positions in flight per step
    const int vg = t / TPR, ve = (t % TPR) * 8;
    for (int j0 = 0; j0 < nq; j0 += QCHUNK) {
        const int nj = min(QCHUNK, nq - j0);
        float acc[QCHUNK][8];
#pragma unroll
        for (int j = 0; j < QCHUNK; ++j)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[j][e] = 0.f;
        for (int p = vg; p < np; p += PGROUPS) {
            float vf[8];
            unpack8(*reinterpret_cast<const uint4*>(V + (size_t)p * HD + ve), vf);
#pragma unroll
            for (int j = 0; j < QCHUNK; ++j) {
                if (j < nj) {
                    const float w = sc[(j0 + j) * P.split_len + p];
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[j][e] = fmaf(w, vf[e], acc[j][e]);
                }
            }
        }
        // position groups inside a warp first (TPR 16: two groups, TPR 8: four), then across warps
#pragma unroll
        for (int j = 0; j < QCHUNK; ++j)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                float v = acc[j][e];
                v += __shfl_xor_sync(0xffffffffu, v, 16);
                if (TPR == 8) v += __shfl_xor_sync(0xffffffffu, v, 8);
                acc[j][e] = v;
            }
        __syncthreads();
        if (lane < TPR) {
#pragma unroll
            for (int j = 0; j < QCHUNK; ++j)
#pragma unroll
                for (int e = 0; e < 8; ++e) red[(warp * QCHUNK + j) * HD + lane * 8 + e] = acc[j][e];
        }
        __syncthreads();
        for (int i = t; i < nj * HD; i += ATT_THREADS) {
            const int j = i / HD, e = i % HD;
            const float v = red[(0 * QCHUNK + j) * HD + e] + red[(1 * QCHUNK + j) * HD + e] +
                            red[(2 * QCHUNK + j) * HD + e] + red[(3 * QCHUNK + j) * HD + e];
            const int jq = j0 + j, r = r0 + jq / group, h = kvh * group + jq % group;
            P.part_o[(((size_t)r * P.H + h) * P.n_splits + split) * HD + e] = v;
        }
    }
    for (int i = t; i < nq; i += ATT_THREADS) {
        const int r = r0 + i / group, h = kvh * group + i % group;
        float* ml = P.part_ml + (((size_t)r * P.H + h) * P.n_splits + split) * 2;
        ml[0] = m_sm[i]; ml[1] = l_sm[i];
    }
}

// Merge of the slices of one (row, head): out = sum_s e^(m_s - M) O_s / sum_s e^(m_s - M) l_s.
template <int HD>
__global__ void k_attn_combine(const float* __restrict__ part_o, const float* __restrict__ part_ml, bf16* __restrict__ out,
                               int H, int n_splits) {
    const int r = blockIdx.x, h = blockIdx.y, e = threadIdx.x;
    const float* ml = part_ml + ((size_t)r * H + h) * n_splits * 2;
    const float* o = part_o + ((size_t)r * H + h) * n_splits * HD;
    float M = -INFINITY;
    for (int s = 0; s < n_splits; ++s) M = fmaxf(M, ml[2 * s]);
    float acc = 0.f, den = 0.f;
    if (M != -INFINITY) {
        for (int s = 0; s < n_splits; ++s) {
            const float m = ml[2 * s];
            if (m == -INFINITY) continue;
            const float w = __expf(m - M);
            den = fmaf(w, ml[2 * s + 1], den);
            acc = fmaf(w, o[(size_t)s * HD + e], acc);
        }
    }
    out[((size_t)r * H + h) * HD + e] = __float2bfloat16_rn(den > 0.f ? acc / den : 0.f);
}

int pick_split_len(int max_ctx) {
    int len = 64;
    while ((max_ctx + len - 1) / len > 32) len += 64;
    return len;
}

}  // namespace

bool attention_split_supported(int dtype, int H, int Hkv, int hd) {
    return dtype == SD_BF16 && (hd == 64 || hd == 128) && H / Hkv <= NQ_MAX;
}

size_t attention_split_workspace(int rows, int H, int hd, int max_ctx) {
    const int n_splits = (max_ctx + pick_split_len(max_ctx) - 1) / pick_split_len(max_ctx);
    return sizeof(float) * (size_t)rows * H * n_splits * (hd + 2);
}

// Rows come in runs of rows_per_seq consecutive rows of one sequence (n_rows is a multiple of it);
// ctx_bound: no row sees a position >= ctx_bound (bounds the number of slices launched).
cudaError_t launch_attention_split(const void* q, const void* kc, const void* vc, void* out, const int32_t* row_slot,
                                   const int32_t* row_pos, int n_rows, int rows_per_seq, int H, int Hkv, int hd,
                                   int max_ctx, int ctx_bound, void* workspace, size_t workspace_bytes, cudaStream_t st) {
    if (n_rows <= 0) return cudaSuccess;
    ctx_bound = std::max(1, std::min(ctx_bound, max_ctx));
    AttnParams P;
    P.q = (const bf16*)q; P.kc = (const bf16*)kc; P.vc = (const bf16*)vc;
    P.row_slot = row_slot; P.row_pos = row_pos;
    if (rows_per_seq < 1 || n_rows % rows_per_seq) return cudaErrorInvalidValue;
    P.n_rows = n_rows; P.rows_per_seq = rows_per_seq; P.H = H; P.Hkv = Hkv; P.max_ctx = max_ctx;
    P.rows_per_block = std::max(1, std::min(rows_per_seq, NQ_MAX / (H / Hkv)));
    const int bps = (rows_per_seq + P.rows_per_block - 1) / P.rows_per_block;
    P.split_len = pick_split_len(ctx_bound);
    P.n_splits = (ctx_bound + P.split_len - 1) / P.split_len;
    const size_t need = sizeof(float) * (size_t)n_rows * H * P.n_splits * (hd + 2);
    if (need > workspace_bytes) return cudaErrorInvalidValue;
    P.part_o = (float*)workspace;
    P.part_ml = P.part_o + (size_t)n_rows * H * P.n_splits * hd;
    const size_t smem = sizeof(float) * ((size_t)NQ_MAX * hd + (size_t)NQ_MAX * P.split_len + (size_t)4 * QCHUNK * hd);
    dim3 grid(P.n_splits, Hkv, (n_rows / rows_per_seq) * bps);
    cudaError_t e;
    if (hd == 128) {
        if ((e = cudaFuncSetAttribute(k_attn_split<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        k_attn_split<128><<<grid, ATT_THREADS, smem, st>>>(P);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        k_attn_combine<128><<<dim3(n_rows, H), 128, 0, st>>>(P.part_o, P.part_ml, (bf16*)out, H, P.n_splits);
    } else {
        if ((e = cudaFuncSetAttribute(k_attn_split<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        k_attn_split<64><<<grid, ATT_THREADS, smem, st>>>(P);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        k_attn_combine<64><<<dim3(n_rows, H), 64, 0, st>>>(P.part_o, P.part_ml, (bf16*)out, H, P.n_splits);
    }
    return cudaGetLastError();
}

}  // namespace sd
