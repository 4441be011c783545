// One Lloyd iteration of K-means over dense fp32 vectors (the offline task-partitioning step, Section 3.2:
// 384-dimensional sentence vectors, a handful of clusters).
//
// With K <= 8 centroids the step is a single pass over the points and is bound by that pass (4 K flop per loaded
// byte-quad: far below the ALU ridge), so the kernel is a streaming one, not a tensor-core contraction: a warp takes
// whole points, every lane owns dim / 32 columns (float4 loads, one coalesced row per warp), the centroids sit in
// shared memory, squared distances are summed in fp32 and reduced with shuffles.  The same pass accumulates, per warp
// and in registers, the sum of the points of every cluster; warps of a block are added in warp order, blocks in block
// order by a second small kernel: the new centroids, the counts and the inertia are identical from run to run.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sd.h"

namespace sd {
namespace {

constexpr int KM_MAX_K = 8;
constexpr int KM_WARPS = 8;
constexpr int KM_DEPTH = 6;            // points of a warp in flight

// Two fp32 values in one 64-bit register and the packed arithmetic of sm_100 on them: each instruction is two
// independent IEEE operations (same results as the scalar forms), which halves the instructions per loaded byte.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 f2_sub(f32x2 a, f32x2 b) { f32x2 r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ f32x2 f2_add(f32x2 a, f32x2 b) { f32x2 r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ f32x2 f2_fma(f32x2 a, f32x2 b, f32x2 c) { f32x2 r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c)); return r; }
__device__ __forceinline__ float f2_hsum(f32x2 v) { float a, b; asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); return a + b; }

template <int NV, int KM>          // KM: compiled cluster bound (4 or 8); with 4 the centroids are kept in registers
__global__ void __launch_bounds__(32 * KM_WARPS, (KM == 4 && NV <= 3) ? 2 : 1)
k_kmeans_assign(const float* __restrict__ pts, long long n, int k, const float* __restrict__ cent, int32_t* __restrict__ labels,
                float* __restrict__ part_sums, long long* __restrict__ part_counts, double* __restrict__ part_inertia) {
    constexpr int DIM = 128 * NV;
    extern __shared__ __align__(16) float km_smem[];
    float* cs = km_smem;                       // [k][DIM] centroids
    float* acc_s = km_smem + KM * DIM;         // [k][DIM] the block's sums
    __shared__ long long cnt_s[KM];
    __shared__ double inertia_s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < k * DIM; i += blockDim.x) cs[i] = cent[i];
    __syncthreads();

    // Up to four centroids: every lane keeps its columns of them in registers (shared memory could not feed four
    // centroid reads per point at the rate the points arrive); more: read from shared memory.
    constexpr bool CREG = KM == 4;
    ulonglong2 creg[CREG ? KM : 1][CREG ? NV : 1];
    if (CREG) {
#pragma unroll
        for (int kk = 0; kk < KM; ++kk)
#pragma unroll
            for (int v = 0; v < NV; ++v)
                creg[CREG ? kk : 0][CREG ? v : 0] = kk < k ? *reinterpret_cast<const ulonglong2*>(cs + kk * DIM + (v * 32 + lane) * 4) : make_ulonglong2(0ull, 0ull);
    }
    ulonglong2 acc[KM][NV];                     // (the bit pattern 0 is +0.0f twice)
#pragma unroll
    for (int kk = 0; kk < KM; ++kk)
#pragma unroll
        for (int v = 0; v < NV; ++v) acc[kk][v] = make_ulonglong2(0ull, 0ull);
    int cnt[KM];                                // points of this warp per cluster (a warp sees n / (8 * blocks) points)
#pragma unroll
    for (int kk = 0; kk < KM; ++kk) cnt[kk] = 0;
    double inertia = 0.0;

    // Every lane copies its own columns of the next KM_DEPTH - 1 points of its warp into shared memory with
    // asynchronous 16-byte copies and reads back only what it copied itself: no barrier, and enough bytes in flight per SM
    // (warps x depth x row) to cover the memory latency at full bandwidth.
    const long long total_warps = (long long)gridDim.x * KM_WARPS;
    const long long i0 = (long long)blockIdx.x * KM_WARPS + warp;
    float* ring = acc_s + KM * DIM + (size_t)warp * KM_DEPTH * DIM + lane * 4;     // [KM_DEPTH][DIM] of this warp, this lane's first column
    const uint32_t ring_sa = (uint32_t)__cvta_generic_to_shared(ring);
    const float* src_next = pts + i0 * DIM + lane * 4;                            // the next point to request and its index
    long long idx_next = i0;
    const long long src_step = total_warps * DIM;
    int slot_next = 0;
    auto stage = [&]() {
        if (idx_next < n) {
#pragma unroll
            for (int v = 0; v < NV; ++v)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring_sa + (uint32_t)(slot_next * DIM + v * 128) * 4u), "l"(src_next + v * 128) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");                      // (an empty group past the end keeps the count uniform)
        idx_next += total_warps; src_next += src_step;
        slot_next = slot_next + 1 == KM_DEPTH ? 0 : slot_next + 1;
    };
    for (int t = 0; t < KM_DEPTH - 1; ++t) stage();
    int slot = 0;
    for (long long i = i0; i < n; i += total_warps) {
        stage();
        asm volatile("cp.async.wait_group %0;" ::"n"(KM_DEPTH - 1) : "memory");    // this point has landed
        ulonglong2 x[NV];
#pragma unroll
        for (int v = 0; v < NV; ++v) x[v] = *reinterpret_cast<const ulonglong2*>(ring + slot * DIM + v * 128);
        slot = slot + 1 == KM_DEPTH ? 0 : slot + 1;
        float dk[KM];                                                             // this lane's share of every squared distance
#pragma unroll
        for (int kk = 0; kk < KM; ++kk) {
            dk[kk] = 0.f;
            if (kk < k) {                                                         // uniform
                f32x2 d2 = 0ull;
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    const ulonglong2 c = CREG ? creg[CREG ? kk : 0][CREG ? v : 0] : *reinterpret_cast<const ulonglong2*>(cs + kk * DIM + (v * 32 + lane) * 4);
                    const f32x2 a = f2_sub(x[v].x, c.x), b = f2_sub(x[v].y, c.y);
                    d2 = f2_fma(a, a, d2); d2 = f2_fma(b, b, d2);
                }
                dk[kk] = f2_hsum(d2);
            }
        }
        if (KM == 4) {
            // Four sums over the warp with ten shuffles instead of twenty: halves of the warp trade two of the four
            // values, quarters one of the two, three more steps finish one value per lane group, and the four totals
            // are read back from lanes 0, 8, 16 and 24 (every lane ends with the same four numbers).
            const bool hi16 = lane & 16, hi8 = lane & 8;
            float a = hi16 ? dk[KM == 4 ? 2 : 0] : dk[0], sa = hi16 ? dk[0] : dk[KM == 4 ? 2 : 0];
            float b = hi16 ? dk[KM == 4 ? 3 : 0] : dk[KM == 4 ? 1 : 0], sb = hi16 ? dk[KM == 4 ? 1 : 0] : dk[KM == 4 ? 3 : 0];
            a += __shfl_xor_sync(0xffffffffu, sa, 16);
            b += __shfl_xor_sync(0xffffffffu, sb, 16);
            float e = hi8 ? b : a;
            const float se = hi8 ? a : b;
            e += __shfl_xor_sync(0xffffffffu, se, 8);
            e += __shfl_xor_sync(0xffffffffu, e, 4);
            e += __shfl_xor_sync(0xffffffffu, e, 2);
            e += __shfl_xor_sync(0xffffffffu, e, 1);
            // lane group (bit 4, bit 3) holds cluster 2 * bit4 + bit3
            dk[0] = __shfl_sync(0xffffffffu, e, 0);
            if (KM == 4) { dk[KM == 4 ? 1 : 0] = __shfl_sync(0xffffffffu, e, 8); dk[KM == 4 ? 2 : 0] = __shfl_sync(0xffffffffu, e, 16); dk[KM == 4 ? 3 : 0] = __shfl_sync(0xffffffffu, e, 24); }
        } else {
#pragma unroll
            for (int kk = 0; kk < KM; ++kk)
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) dk[kk] += __shfl_xor_sync(0xffffffffu, dk[kk], o);      // every lane ends with the same sums
        }
        float best = INFINITY;
        int label = 0;
#pragma unroll
        for (int kk = 0; kk < KM; ++kk)
            if (kk < k && dk[kk] < best) { best = dk[kk]; label = kk; }            // a later centroid must be strictly closer
        if (lane == 0) labels[i] = label;
        inertia += (double)best;
#pragma unroll
        for (int kk = 0; kk < KM; ++kk) {
            if (kk == label) {                                                    // uniform
                cnt[kk] += 1;
#pragma unroll
                for (int v = 0; v < NV; ++v) { acc[kk][v].x = f2_add(acc[kk][v].x, x[v].x); acc[kk][v].y = f2_add(acc[kk][v].y, x[v].y); }
            }
        }
    }

    // the block's sums: its warps in warp order
    for (int w = 0; w < KM_WARPS; ++w) {
        if (warp == w) {
#pragma unroll
            for (int kk = 0; kk < KM; ++kk) {
                if (kk < k) {
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        ulonglong2* dst = reinterpret_cast<ulonglong2*>(acc_s + kk * DIM + (v * 32 + lane) * 4);
                        ulonglong2 s = w == 0 ? make_ulonglong2(0ull, 0ull) : *dst;
                        s.x = f2_add(s.x, acc[kk][v].x); s.y = f2_add(s.y, acc[kk][v].y);
                        *dst = s;
                    }
                    if (lane == 0) cnt_s[kk] = (w == 0 ? 0 : cnt_s[kk]) + (long long)cnt[kk];
                }
            }
            if (lane == 0) inertia_s = (w == 0 ? 0.0 : inertia_s) + inertia;
        }
        __syncthreads();
    }
    for (int i = threadIdx.x; i < k * DIM; i += blockDim.x) part_sums[(size_t)blockIdx.x * k * DIM + i] = acc_s[i];
    if (threadIdx.x < k) part_counts[(size_t)blockIdx.x * k + threadIdx.x] = cnt_s[threadIdx.x];
    if (threadIdx.x == 0) part_inertia[blockIdx.x] = inertia_s;
}

// New centroids = (sum over blocks) / count; a cluster without points keeps its centroid.  One CTA per (cluster, 32
// columns): eight threads per column each add a contiguous run of the blocks' partial sums in block order (independent
// loads, several in flight), and the eight runs are added in run order: a fixed order, in double.
__global__ void __launch_bounds__(256)
k_kmeans_reduce(const float* __restrict__ part_sums, const long long* __restrict__ part_counts,
                const double* __restrict__ part_inertia, int n_blocks, int k, int dim,
                const float* __restrict__ cent, float* __restrict__ cent_out, long long* __restrict__ counts_out,
                double* __restrict__ inertia_out) {
    __shared__ double run_sum[8][32];
    __shared__ long long run_cnt[8];
    __shared__ double run_in[8];
    const int kk = blockIdx.x, d = blockIdx.y * 32 + (threadIdx.x & 31), run = threadIdx.x >> 5;
    const int per = (n_blocks + 7) / 8, b0 = run * per, b1 = min(n_blocks, b0 + per);
    double s = 0.0;
    if (d < dim) {
#pragma unroll 8
        for (int b = b0; b < b1; ++b) s += (double)__ldcg(part_sums + ((size_t)b * k + kk) * dim + d);
    }
    run_sum[run][threadIdx.x & 31] = s;
    {   // the run's counts and inertia: a lane per block, then a fixed tree over the lanes
        long long c = 0;
        double in = 0.0;
        for (int b = b0 + (int)(threadIdx.x & 31); b < b1; b += 32) { c += part_counts[(size_t)b * k + kk]; in += part_inertia[b]; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { c += __shfl_xor_sync(0xffffffffu, c, o); in += __shfl_xor_sync(0xffffffffu, in, o); }
        if ((threadIdx.x & 31) == 0) { run_cnt[run] = c; run_in[run] = in; }
    }
    __syncthreads();
    if (run != 0) return;
    long long c = 0;
    double tot = 0.0, in = 0.0;
    for (int r = 0; r < 8; ++r) { c += run_cnt[r]; tot += run_sum[r][threadIdx.x]; in += run_in[r]; }
    if (d < dim && cent_out) cent_out[(size_t)kk * dim + d] = c > 0 ? (float)(tot / (double)c) : cent[(size_t)kk * dim + d];
    if (threadIdx.x == 0 && blockIdx.y == 0) {
        if (counts_out) counts_out[kk] = c;
        if (kk == 0 && inertia_out) *inertia_out = in;
    }
}

int km_blocks() {
    int dev = 0, n_sm = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    return 2 * n_sm;
}

size_t km_align(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace
}  // namespace sd

extern "C" size_t sd_kmeans_workspace(int dim, int k) {
    if (dim < 1 || k < 1) return 0;
    const size_t b = (size_t)sd::km_blocks();
    return sd::km_align(b * k * dim * sizeof(float)) + sd::km_align(b * k * sizeof(long long)) + sd::km_align(b * sizeof(double));
}

extern "C" sd_status sd_kmeans_step(const float* points, int64_t n, int dim, const float* centroids, int k, int32_t* labels,
                                    float* centroids_out, int64_t* counts_out, double* inertia_out, void* workspace,
                                    size_t workspace_bytes, void* cuda_stream) {
    using namespace sd;
    if (!centroids || n < 0 || k < 1 || dim < 1 || (n > 0 && (!points || !labels))) return SD_ERR_INVALID_ARG;
    if (k > KM_MAX_K || (dim % 128) || dim > 512) return SD_ERR_UNSUPPORTED;
    if (((uintptr_t)points & 15) || ((uintptr_t)centroids & 15)) return SD_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < sd_kmeans_workspace(dim, k)) return SD_ERR_CAPACITY;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int blocks = km_blocks();
    char* w = (char*)workspace;
    float* part_sums = (float*)w;              w += km_align((size_t)blocks * k * dim * sizeof(float));
    long long* part_counts = (long long*)w;    w += km_align((size_t)blocks * k * sizeof(long long));
    double* part_inertia = (double*)w;
    const int km = k <= 4 ? 4 : KM_MAX_K;
    const size_t smem = ((size_t)2 * km + (size_t)KM_WARPS * KM_DEPTH) * dim * sizeof(float);
    cudaError_t e = cudaSuccess;
#define KM_LAUNCH(NV, KM)                                                                                                        \
    do {                                                                                                                     \
        e = cudaFuncSetAttribute(k_kmeans_assign<NV, KM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);           \
        if (e == cudaSuccess) k_kmeans_assign<NV, KM><<<blocks, 32 * KM_WARPS, smem, st>>>(points, n, k, centroids, labels, part_sums, part_counts, part_inertia); \
    } while (0)
    switch (dim / 128) {
    case 1: if (km == 4) KM_LAUNCH(1, 4); else KM_LAUNCH(1, 8); break;
    case 2: if (km == 4) KM_LAUNCH(2, 4); else KM_LAUNCH(2, 8); break;
    case 3: if (km == 4) KM_LAUNCH(3, 4); else KM_LAUNCH(3, 8); break;
    default: if (km == 4) KM_LAUNCH(4, 4); else KM_LAUNCH(4, 8); break;
    }
#undef KM_LAUNCH
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return SD_ERR_CUDA;
    k_kmeans_reduce<<<dim3(k, (dim + 31) / 32), 256, 0, st>>>(part_sums, part_counts, part_inertia, blocks, k, dim, centroids, centroids_out,
                                       (long long*)counts_out, inertia_out);
    return cudaGetLastError() == cudaSuccess ? SD_OK : SD_ERR_CUDA;
}
