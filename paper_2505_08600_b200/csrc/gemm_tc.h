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
cudaError_t launch_reduce_plain(const float* partials, const GemmGeom& g, float* y, cudaStream_t st);

// Sum of the partial accumulators that cover output (token m, feature n), always in the
// order of the CTAs that produced them.
__device__ __forceinline__ float gemm_reduce(const float* __restrict__ partials, const GemmGeom& g, int m, int n) {
    const int tile = n >> 7, r = n & 127;
    const unsigned long long T = (unsigned long long)g.n_tiles * g.kb_per_tile, G = g.grid;
    const unsigned long long ua = (unsigned long long)tile * g.kb_per_tile, ub = ua + g.kb_per_tile - 1;
    const int i_first = (int)(((ua + 1) * G + T - 1) / T) - 1;
    const int i_last = (int)(((ub + 1) * G + T - 1) / T) - 1;
    float acc = 0.f;
    for (int i = i_first; i <= i_last; ++i) {
        const int j = tile - (int)((i * T / G) / g.kb_per_tile);
        acc += partials[(((size_t)i * g.max_seg + j) * g.m_pad + m) * 128 + r];
    }
    return acc;
}

}  // namespace sd
