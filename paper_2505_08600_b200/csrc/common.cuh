// Shared device helpers of the CUDA library (not used by the CPU checker).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sd.h"

namespace sd {

typedef __nv_bfloat16 bf16;

struct SeqList {            // passed by value to kernels: which sequence slots a call covers
    int n;
    int ids[SD_MAX_BATCH];  // sequence slot of entry i
    int out[SD_MAX_BATCH];  // row of the caller's [n_seq][...] buffers that entry i reads and writes
};

// Per-sequence state, all on the device so that an iteration needs no host round trip.
struct SeqState {
    int32_t* len;           // tokens known so far (prompt + emitted)
    int32_t* tkv;           // positions held by the target cache
    int32_t* dkv;           // positions held by the routed draft's cache
    uint32_t* iter;         // iterations done; Philox counter word 0
    uint32_t* seq_id;       // Philox counter word 2
    int32_t* draft_id;      // which draft the sequence is routed to
    int32_t* n_prompt;      // prompt length (the classifier pools over the prompt only)
    int64_t* counters;      // [slot][4]: iterations, drafted, accepted, emitted
    double* alpha_sum;      // [slot]: sum over judged slots of sum_k min(p, q)
    int64_t* judged;        // [slot]: judged slots so far (slot s of an iteration is judged iff all before it were accepted)
    int32_t* tokens;        // [slot][tok_stride]
    int tok_stride;
    int max_ctx;
    uint32_t* status;       // device status word (SD_DEV_* bits)
};

// How the rows of one forward pass map to (sequence, position, token).
enum PlanKind { PLAN_PREFILL = 0, PLAN_VERIFY = 1, PLAN_DRAFT_FIRST = 2, PLAN_DRAFT_NEXT = 3, PLAN_TARGET_STEP = 4 };
struct RowPlan {
    int kind;
    int rows_per_seq;
    int pos0;               // PLAN_PREFILL: position of row 0
    int step;               // PLAN_DRAFT_NEXT: s >= 1
    int gamma;              // row stride of x
    const int32_t* x;       // [n_seq][gamma] draft tokens (device)
    int ctx_bound;          // host's upper bound on 1 + the largest position any row of the pass sees
};

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<bf16>(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Block-wide reductions for blocks of up to 1024 threads; `red` holds 32 floats of shared memory.
__device__ __forceinline__ float block_sum(float v, float* red) {
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    float r = (threadIdx.x < nw) ? red[threadIdx.x] : 0.f;
    if (w == 0) { r = warp_sum(r); if (lane == 0) red[0] = r; }
    __syncthreads();
    return red[0];
}
__device__ __forceinline__ float block_max(float v, float* red) {
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_max(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    float r = (threadIdx.x < nw) ? red[threadIdx.x] : -INFINITY;
    if (w == 0) { r = warp_max(r); if (lane == 0) red[0] = r; }
    __syncthreads();
    return red[0];
}

// Philox4x32-10 (Salmon et al., SC'11), ten rounds, key bumped by the Weyl constants.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

enum { DRAW_DRAFT = 0, DRAW_ACCEPT = 1, DRAW_RESAMPLE = 2 };

// 24-bit uniform as an integer in [1, 2^24]: counter (iter, slot, seq, purpose), key = seed.
__device__ __forceinline__ uint32_t uniform24(uint64_t seed, uint32_t iter, uint32_t slot, uint32_t seq, uint32_t purpose) {
    uint32_t o[4];
    philox4x32_10(iter, slot, seq, purpose, (uint32_t)seed, (uint32_t)(seed >> 32), o);
    return (o[0] >> 8) + 1u;
}

}  // namespace sd
