// Interface of the tensor-core weight-streaming GEMM (gemm_tc.cu) and of the fixed-order
// reduction its consumers use.
#pragma once
#include <algorithm>

#include "common.cuh"

namespace sd {

struct alignas(64) TensorMap { uint8_t bytes[128]; };     // opaque TMA descriptor (CUtensorMap)

// Work split of one GEMM: (row tile, k block) pairs numbered tile-major are divided evenly
// over `grid` CTAs; CTA i owns pairs [i*T/grid, (i+1)*T/grid) and writes one partial
// accumulator per tile it touches into slot i*max_seg + j (j counts its tiles in order).
struct GemmGeom {
    int m_tok, m_pad, n_out, K;
    int n_tiles, kb_per_tile;
    int grid, max_seg, stages;
};

bool gemm_tc_supported(int m_tok, int n_out, int K);
GemmGeom gemm_geometry(int m_tok, int n_out, int K, int n_sm);
size_t gemm_partials_bytes(const GemmGeom& g);
bool make_tensor_map_bf16(TensorMap* out, const void* base, int rows, int K, int box_rows);
cudaError_t launch_gemm_streamk(const TensorMap& tm_w, const TensorMap& tm_x, const GemmGeom& g, float* partials,
                                uint32_t* status, cudaStream_t st);
struct RowScale;
// y[i][n] = scale(row) * sum of segments, row = i * row_stride + row_offset, i < n_out_rows
cudaError_t launch_reduce_plain(const float* partials, const GemmGeom& g, float* y, int n_out_rows, int row_stride,
                                int row_offset, const RowScale& rs, cudaStream_t st);

// fused.cu: consumers that fold the step after the GEMM into the reduction of its partials
cudaError_t launch_prep_norm(const float* h, const float* gain, void* xn, float* ssq, int n_rows, int d, cudaStream_t st);
cudaError_t launch_cons_qkv_rope(const float* partials, const GemmGeom& g, const RowScale& rs, void* q_out, void* kc, void* vc,
                                 const int32_t* row_slot, const int32_t* row_pos, int n_rows, int H, int Hkv, int hd,
                                 int max_ctx, const float* rcos, const float* rsin, cudaStream_t st);
cudaError_t launch_cons_residual(const float* partials, const GemmGeom& g, float* h, const float* gain_next, void* xn,
                                 float* ssq, int n_rows, cudaStream_t st);
cudaError_t launch_cons_swiglu(const float* partials, const GemmGeom& g, const RowScale& rs, void* act, int n_rows, int F,
                               cudaStream_t st);

// RMSNorm folded around a GEMM: the GEMM's input rows are h * gain (no 1/rms factor), the
// factor rsqrt(mean(h^2) + eps) of each row multiplies the GEMM's output instead.  The sum of
// squares of a row arrives in n_parts pieces (one per 128-wide tile of the kernel that wrote h).
struct RowScale {
    const float* ssq;       // [row][SSQ_STRIDE]; nullptr: no scaling
    int n_parts;
    float inv_d, eps;
};
constexpr int SSQ_STRIDE = 64;

__device__ __forceinline__ float row_scale(const RowScale& rs, int row) {
    if (!rs.ssq) return 1.f;
    float ss = 0.f;
    for (int i = 0; i < rs.n_parts; ++i) ss += rs.ssq[(size_t)row * SSQ_STRIDE + i];
    return rsqrtf(ss * rs.inv_d + rs.eps);
}

// Sum of the partial accumulators that cover output (token m, feature n), always in the
// order of the CTAs that produced them.  (T * grid < 2^32 is checked by gemm_geometry.)
__device__ __forceinline__ float gemm_reduce(const float* __restrict__ partials, const GemmGeom& g, int m, int n) {
    const uint32_t tile = (uint32_t)n >> 7, r = (uint32_t)n & 127u, KB = (uint32_t)g.kb_per_tile;
    const uint32_t T = (uint32_t)g.n_tiles * KB, G = (uint32_t)g.grid;
    const uint32_t ua = tile * KB, ub = ua + KB - 1;
    const uint32_t i_first = ((ua + 1) * G + T - 1) / T - 1;
    const uint32_t i_last = ((ub + 1) * G + T - 1) / T - 1;
    float acc = 0.f;
    for (uint32_t i = i_first; i <= i_last; ++i) {
        const uint32_t j = tile - (i * T / G) / KB;
        acc += partials[(((size_t)i * g.max_seg + j) * g.m_pad + m) * 128 + r];
    }
    return acc;
}

}  // namespace sd
