// Attention of the new query rows over the KV cache (grouped-query heads).
// Cache layout of one layer: [slot][kv_head][position][head_dim]; row r sees positions
// 0..row_pos[r] of slot row_slot[r] (its own key/value was appended just before).
#include "kernels.h"

namespace sd {

template <typename T> __device__ __forceinline__ float dot_row(const T* __restrict__ k, const float* __restrict__ q, int hd);
template <> __device__ __forceinline__ float dot_row<bf16>(const bf16* __restrict__ k, const float* __restrict__ q, int hd) {
    float s = 0.f;
    for (int i = 0; i < hd; i += 8) {
        uint4 u = *reinterpret_cast<const uint4*>(k + i);
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            s = fmaf(__uint_as_float(w[j] << 16), q[i + 2 * j], s);
            s = fmaf(__uint_as_float(w[j] & 0xffff0000u), q[i + 2 * j + 1], s);
        }
    }
    return s;
}
template <> __device__ __forceinline__ float dot_row<float>(const float* __restrict__ k, const float* __restrict__ q, int hd) {
    float s = 0.f;
    for (int i = 0; i < hd; i += 4) {
        float4 u = *reinterpret_cast<const float4*>(k + i);
        s = fmaf(u.x, q[i], s); s = fmaf(u.y, q[i + 1], s); s = fmaf(u.z, q[i + 2], s); s = fmaf(u.w, q[i + 3], s);
    }
    return s;
}

// Plain two-pass kernel: one block per (row, query head); scores for the whole context sit in
// shared memory, softmax is exact (max, then sum), then the value rows are blended.
template <typename T>
__global__ void __launch_bounds__(128) k_attention_plain(const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc,
                                                         T* __restrict__ out, const int32_t* __restrict__ row_slot,
                                                         const int32_t* __restrict__ row_pos, int H, int Hkv, int hd, int max_ctx) {
    extern __shared__ float smem[];
    __shared__ float red[32];
    float* qs = smem;              // [hd]
    float* sc = smem + hd;         // [n_ctx]
    const int r = blockIdx.x, h = blockIdx.y, t = threadIdx.x;
    const int pos = row_pos[r];
    T* o = out + ((size_t)r * H + h) * hd;
    if (pos < 0) { for (int i = t; i < hd; i += blockDim.x) o[i] = from_f32<T>(0.f); return; }
    const int n_ctx = pos + 1, kvh = h / (H / Hkv);
    const size_t base = ((size_t)row_slot[r] * Hkv + kvh) * (size_t)max_ctx * hd;
    const T* K = kc + base;
    const T* V = vc + base;
    const float scale = rsqrtf((float)hd);
    for (int i = t; i < hd; i += blockDim.x) qs[i] = to_f32<T>(q[((size_t)r * H + h) * hd + i]) * scale;
    __syncthreads();
    float mx = -INFINITY;
    for (int p = t; p < n_ctx; p += blockDim.x) {
        float s = dot_row<T>(K + (size_t)p * hd, qs, hd);
        sc[p] = s;
        mx = fmaxf(mx, s);
    }
    mx = block_max(mx, red);
    float den = 0.f;
    for (int p = t; p < n_ctx; p += blockDim.x) { float e = expf(sc[p] - mx); sc[p] = e; den += e; }
    den = block_sum(den, red);
    const float inv = 1.f / den;
    for (int i = t; i < hd; i += blockDim.x) {
        float acc = 0.f;
        for (int p = 0; p < n_ctx; ++p) acc = fmaf(sc[p], to_f32<T>(V[(size_t)p * hd + i]), acc);
        o[i] = from_f32<T>(acc * inv);
    }
}

size_t attention_workspace_bytes(int rows, int n_heads, int head_dim, int max_ctx) {
    (void)rows; (void)n_heads; (void)head_dim; (void)max_ctx;
    return 0;
}

cudaError_t launch_attention(const void* q, const void* kc, const void* vc, void* out, int dtype,
                             const int32_t* row_slot, const int32_t* row_pos, int n_rows,
                             int H, int Hkv, int hd, int max_ctx, void* workspace, size_t workspace_bytes, cudaStream_t st) {
    (void)workspace; (void)workspace_bytes;
    if (n_rows <= 0) return cudaSuccess;
    const size_t smem = sizeof(float) * (size_t)(hd + max_ctx);
    if (smem > 200 * 1024) return cudaErrorInvalidValue;
    dim3 grid(n_rows, H);
    cudaError_t e;
    if (dtype == SD_BF16) {
        if (smem > 48 * 1024 && (e = cudaFuncSetAttribute(k_attention_plain<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        k_attention_plain<bf16><<<grid, 128, smem, st>>>((const bf16*)q, (const bf16*)kc, (const bf16*)vc, (bf16*)out, row_slot, row_pos, H, Hkv, hd, max_ctx);
    } else {
        if (smem > 48 * 1024 && (e = cudaFuncSetAttribute(k_attention_plain<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        k_attention_plain<float><<<grid, 128, smem, st>>>((const float*)q, (const float*)kc, (const float*)vc, (float*)out, row_slot, row_pos, H, Hkv, hd, max_ctx);
    }
    return cudaGetLastError();
}

}  // namespace sd
