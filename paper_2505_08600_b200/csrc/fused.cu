// Consumers of the tensor-core GEMM's partial accumulators.  Each one adds the segments of an
// output in their fixed order and applies, in the same pass, the elementwise step that follows
// the GEMM in the decoder layer, so that no intermediate fp32 matrix goes through memory.
// RMSNorm is split around the GEMMs: the kernel that updates the residual stream h writes
// h * gain as the next GEMM's bf16 input plus per-tile sums of squares, and the consumer of
// that GEMM multiplies by rsqrt(mean(h^2) + eps).
#include "gemm_tc.h"
#include "kernels.h"

namespace sd {

// First layer: xn = bf16(h * gain), ssq[row][0] = sum h^2.  One block per row.
__global__ void __launch_bounds__(512) k_prep_norm(const float* __restrict__ h, const float* __restrict__ gain,
                                                   bf16* __restrict__ xn, float* __restrict__ ssq, int d) {
    __shared__ float red[32];
    const int r = blockIdx.x;
    float ss = 0.f;
    for (int k = threadIdx.x; k < d; k += blockDim.x) {
        const float v = h[(size_t)r * d + k];
        xn[(size_t)r * d + k] = __float2bfloat16_rn(v * gain[k]);
        ss += v * v;
    }
    ss = block_sum(ss, red);
    if (threadIdx.x == 0) ssq[(size_t)r * SSQ_STRIDE] = ss;
}
cudaError_t launch_prep_norm(const float* h, const float* gain, void* xn, float* ssq, int n_rows, int d, cudaStream_t st) {
    k_prep_norm<<<n_rows, 512, 0, st>>>(h, gain, (bf16*)xn, ssq, d);
    return cudaGetLastError();
}

// QKV projection -> 1/rms factor -> rotary embedding -> query buffer / KV-cache append (bf16).
// grid (128-feature tiles, rows), 128 threads; a tile holds one head (head_dim 128) or two (64).
__global__ void __launch_bounds__(128) k_cons_qkv_rope(const float* __restrict__ partials, GemmGeom g, RowScale rs,
                                                       bf16* __restrict__ q_out, bf16* __restrict__ kc, bf16* __restrict__ vc,
                                                       const int32_t* __restrict__ row_slot, const int32_t* __restrict__ row_pos,
                                                       int H, int Hkv, int hd, int max_ctx,
                                                       const float* __restrict__ rcos, const float* __restrict__ rsin) {
    __shared__ float val[128];
    const int r = blockIdx.y, t = threadIdx.x, n = blockIdx.x * 128 + t;
    const int pos = row_pos[r];
    if (pos < 0) return;
    val[t] = n < g.n_out ? gemm_reduce(partials, g, r, n) * row_scale(rs, r) : 0.f;
    __syncthreads();
    if (n >= g.n_out) return;
    const int head = n / hd, i = n % hd, half = hd >> 1;
    if (i >= half) return;
    float a = val[t], b = val[t + half];
    if (head < H + Hkv) {
        const float c = rcos[(size_t)pos * half + i], s = rsin[(size_t)pos * half + i];
        const float ra = a * c - b * s, rb = a * s + b * c;
        a = ra; b = rb;
    }
    bf16* dst;
    if (head < H) dst = q_out + ((size_t)r * H + head) * hd;
    else {
        const int kvh = (head - H) % Hkv;
        bf16* base = (head < H + Hkv) ? kc : vc;
        dst = base + (((size_t)row_slot[r] * Hkv + kvh) * max_ctx + pos) * hd;
    }
    dst[i] = __float2bfloat16_rn(a);
    dst[i + half] = __float2bfloat16_rn(b);
}

cudaError_t launch_cons_qkv_rope(const float* partials, const GemmGeom& g, const RowScale& rs, void* q_out, void* kc, void* vc,
                                 const int32_t* row_slot, const int32_t* row_pos, int n_rows, int H, int Hkv, int hd,
                                 int max_ctx, const float* rcos, const float* rsin, cudaStream_t st) {
    if (128 % hd) return cudaErrorInvalidValue;            // a head must not straddle two tiles
    dim3 grid(g.n_tiles, n_rows);
    k_cons_qkv_rope<<<grid, 128, 0, st>>>(partials, g, rs, (bf16*)q_out, (bf16*)kc, (bf16*)vc, row_slot, row_pos, H, Hkv, hd, max_ctx, rcos, rsin);
    return cudaGetLastError();
}

// Output / down projection -> residual add; also prepares the next norm: xn = bf16(h * gain_next)
// and the tile's share of sum h^2.  grid (tiles, rows), 128 threads.  gain_next == nullptr: h only.
__global__ void __launch_bounds__(128) k_cons_residual(const float* __restrict__ partials, GemmGeom g, float* __restrict__ h,
                                                       const float* __restrict__ gain_next, bf16* __restrict__ xn,
                                                       float* __restrict__ ssq) {
    __shared__ float red[32];
    const int r = blockIdx.y, n = blockIdx.x * 128 + threadIdx.x, d = g.n_out;
    float v = 0.f;
    if (n < d) {
        v = h[(size_t)r * d + n] + gemm_reduce(partials, g, r, n);
        h[(size_t)r * d + n] = v;
        if (gain_next) xn[(size_t)r * d + n] = __float2bfloat16_rn(v * gain_next[n]);
    }
    if (!gain_next) return;
    const float ss = block_sum(v * v, red);
    if (threadIdx.x == 0) ssq[(size_t)r * SSQ_STRIDE + blockIdx.x] = ss;
}

cudaError_t launch_cons_residual(const float* partials, const GemmGeom& g, float* h, const float* gain_next, void* xn,
                                 float* ssq, int n_rows, cudaStream_t st) {
    if (g.n_tiles > SSQ_STRIDE) return cudaErrorInvalidValue;
    dim3 grid(g.n_tiles, n_rows);
    k_cons_residual<<<grid, 128, 0, st>>>(partials, g, h, gain_next, (bf16*)xn, ssq);
    return cudaGetLastError();
}

// Gate/up projection -> 1/rms factor -> SwiGLU: act[r][f] = silu(gate_f) * up_f, gate rows [0, F), up rows [F, 2F).
__global__ void k_cons_swiglu(const float* __restrict__ partials, GemmGeom g, RowScale rs, bf16* __restrict__ act, int F) {
    const int r = blockIdx.y, f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= F) return;
    const float sc = row_scale(rs, r);
    const float gt = gemm_reduce(partials, g, r, f) * sc, up = gemm_reduce(partials, g, r, F + f) * sc;
    act[(size_t)r * F + f] = __float2bfloat16_rn(gt / (1.f + expf(-gt)) * up);
}

cudaError_t launch_cons_swiglu(const float* partials, const GemmGeom& g, const RowScale& rs, void* act, int n_rows, int F,
                               cudaStream_t st) {
    dim3 grid((F + 127) / 128, n_rows);
    k_cons_swiglu<<<grid, 128, 0, st>>>(partials, g, rs, (bf16*)act, F);
    return cudaGetLastError();
}

}  // namespace sd
