// y[rows][n_out] (fp32) = x[rows][n_in] * W[n_out][n_in]^T on CUDA cores.
// The plain path: any shape, fp32 or bf16 storage, fp32 accumulation.  One warp owns one
// weight row and streams it once per tile of up to eight token rows.
#include "kernels.h"

namespace sd {

template <typename T> struct Vec8;
template <> struct Vec8<bf16> {
    static __device__ __forceinline__ void load(const bf16* p, float v[8]) {
        uint4 u = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) { v[2 * i] = __uint_as_float(w[i] << 16); v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
    }
};
template <> struct Vec8<float> {
    static __device__ __forceinline__ void load(const float* p, float v[8]) {
        float4 a = __ldg(reinterpret_cast<const float4*>(p)), b = __ldg(reinterpret_cast<const float4*>(p) + 1);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    }
};

template <typename T, int MT>
__global__ void __launch_bounds__(256) k_linear_simt(const T* __restrict__ x, const T* __restrict__ w, float* __restrict__ y,
                                                     int rows, int n_out, int n_in) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o = blockIdx.x * 8 + warp;
    if (o >= n_out) return;
    const T* wr = w + (size_t)o * n_in;
    const int k_vec = n_in & ~7;
    for (int r0 = 0; r0 < rows; r0 += MT) {
        float acc[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[m] = 0.f;
        for (int k = lane * 8; k < k_vec; k += 256) {
            float wv[8];
            Vec8<T>::load(wr + k, wv);
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                if (r0 + m < rows) {
                    float xv[8];
                    Vec8<T>::load(x + (size_t)(r0 + m) * n_in + k, xv);
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[m] = fmaf(wv[i], xv[i], acc[m]);
                }
            }
        }
        for (int k = k_vec + lane; k < n_in; k += 32) {            // ragged tail of the reduction
            float wv = to_f32<T>(wr[k]);
#pragma unroll
            for (int m = 0; m < MT; ++m)
                if (r0 + m < rows) acc[m] = fmaf(wv, to_f32<T>(x[(size_t)(r0 + m) * n_in + k]), acc[m]);
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            float s = warp_sum(acc[m]);
            if (lane == 0 && r0 + m < rows) y[(size_t)(r0 + m) * n_out + o] = s;
        }
    }
}

cudaError_t launch_linear_simt(const void* x, const void* w, float* y, int rows, int n_out, int n_in, int dtype,
                               cudaStream_t st) {
    if (rows <= 0 || n_out <= 0) return cudaSuccess;
    // 128-bit loads need rows of x and W to start on 16-byte (bf16) / 32-byte (fp32) boundaries
    const int align = dtype == SD_BF16 ? 8 : 4;
    if (n_in % align != 0) return cudaErrorInvalidValue;
    const int grid = (n_out + 7) / 8;
    if (dtype == SD_BF16) k_linear_simt<bf16, 8><<<grid, 256, 0, st>>>((const bf16*)x, (const bf16*)w, y, rows, n_out, n_in);
    else k_linear_simt<float, 8><<<grid, 256, 0, st>>>((const float*)x, (const float*)w, y, rows, n_out, n_in);
    return cudaGetLastError();
}

}  // namespace sd
