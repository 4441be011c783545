// Weight-streaming GEMM on the fifth-generation tensor cores (tcgen05 + TMEM + TMA), bf16.
//
//   P = X[m_tok][K] * W[n_out][K]^T          (fp32 accumulation)
//
// The weight matrix is the 128-row operand (A, K-major), the handful of token rows is the
// narrow one (B, N = m_pad = m_tok rounded up to 16), so one tcgen05.mma covers 128 weight
// rows x m_pad tokens x 16 reduction elements and the accumulator lives in TMEM as
// 128 lanes x m_pad fp32 columns.  The kernel is bound by the one pass over W from HBM:
//   - tiles of 128 rows x 64 k (16 KB, 128-byte swizzle) arrive by TMA into a ring of stages;
//   - work is cut stream-K style: the (row tile, k block) pairs are numbered row-tile-major
//     and split evenly over the grid, so that every SM streams the same number of bytes
//     whatever the matrix shape; a CTA whose range crosses a tile boundary produces one
//     partial accumulator ("segment") per tile it touches;
//   - segments are written to a workspace as fp32 [slot][token][128] and the CTA is done: the
//     kernel that follows (fused_step.cu) adds the segments of each tile in the fixed order of
//     their CTAs and applies the step that follows the GEMM in the decoder layer, while the
//     next GEMM's CTAs already occupy the SMs this one has left and stream their weights;
//   - the kernel is written for programmatic dependent launch: it lets its successor start at
//     once; the first part of its weight stream does not wait for the predecessor (the token rows
//     and the workspace do), so most of the ring is full when the consumers are released.
// Roles: warp 0 streams weights, warp 1 allocates TMEM and issues MMAs, warps 2..5 drain TMEM
// into the workspace, warp 6 loads the token rows.  Every mbarrier wait is bounded; on expiry
// the kernel flags SD_DEV_WAIT_EXPIRED and winds down.
#include <cuda.h>

#include "gemm_tc.h"
#include "tc_ptx.cuh"

namespace sd {

namespace {

constexpr int TILE_N = 128;                 // weight rows per tile (UMMA M)
constexpr int TILE_K = 64;                  // bf16 elements per k block = one 128-byte swizzle row
constexpr int A_BYTES = TILE_N * TILE_K * 2;
constexpr int NUM_THREADS = 224;
constexpr int MAX_STAGES = 12;
constexpr int RING_BYTES = 198 * 1024;          // stage ring of a CTA; the rest of the SM's shared memory is left to the fused-step CTAs
constexpr int GEMM_PREFILL_BYTES = 120 * 1024;  // bytes per SM requested while the previous kernel is still at work (see the weight producer)
constexpr int GEMM_PACED_PREFILL_STAGES = 4;    // ... or, with pacing: stages requested at once, the rest one by one
constexpr int GEMM_PACE_NS = 300;
constexpr int GEMM_STEADY_BYTES = 160 * 1024;   // bytes per SM kept in flight once the ring has been filled (measured best: 9 of 11 stages at 16 rows)

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }    // the four epilogue warps

constexpr int XR_MAX_TILES = 512;      // most tiles of token rows a GEMM tracks one by one (beyond: it waits for the kernel before)

struct Shared {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    int epi_abort;
    int dep_seen;            // the token-row producer is past its wait for the kernel before
    unsigned char xr_ready[XR_MAX_TILES];      // tiles of the token rows seen complete (token-row producer warp only)
};

// Ring bookkeeping.  The first `stages` loads of a CTA fill the whole ring (run-ahead while the
// consumers wait for the previous kernel); after that only the first `steady` stages are reused,
// which keeps somewhat fewer loads in flight: the same bandwidth with a shorter queue, so the last
// tile arrives sooner after it is requested.  use = how often the stage was used before this load.
struct RingPos {
    int stage; uint32_t use; int filled;
    __device__ __forceinline__ RingPos() : stage(0), use(0u), filled(0) {}
    __device__ __forceinline__ void next(int stages, int steady) {         // position of the following load (no divisions: the MMA
        ++stage;                                                           // thread's loop is bound by its own instruction latencies)
        if (!filled) { if (stage == stages) { stage = 0; use = 1u; filled = 1; } }
        else if (stage == steady) { stage = 0; ++use; }
    }
};

// The four epilogue warps of a CTA: drain each finished accumulator from TMEM into the workspace.
__device__ void epilogue_warps(const GemmGeom& g, float* __restrict__ partials, uint32_t* __restrict__ arrive, Shared& sh,
                               uint32_t tmem_base, int warp, int lane, uint32_t u0, uint32_t u1) {
    volatile int* abort_flag = &sh.abort_flag;
    pdl_wait();                                                        // the workspace may still be read by the previous kernel
    const uint32_t quarter = (uint32_t)(warp & 3);                    // TMEM lanes this warp may read
    const int et = quarter * 32 + lane;                                // weight row inside the tile
    uint32_t seg = 0;
    for (uint32_t u = u0; u < u1; ++seg) {
        const uint32_t kb0 = u % g.kb_per_tile;
        const uint32_t n_kb = min((uint32_t)g.kb_per_tile - kb0, u1 - u);
        const uint32_t buf = seg & 1u;
        if (!mbar_wait(smem_u32(&sh.tmem_full[buf]), (seg >> 1) & 1u, abort_flag)) sh.epi_abort = 1;
        epi_bar();
        if (sh.epi_abort) break;                                       // all four warps leave together
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        float* out = partials + ((size_t)blockIdx.x * g.max_seg + seg) * (size_t)g.m_pad * TILE_N;
        if (g.lo_off) {                                                // columns r (x_hi) and r + lo_off (x_lo) are one token row
            const uint32_t t0 = tmem_base + ((quarter * 32u) << 16) + buf * (uint32_t)g.m_pad;
            uint32_t r[16], r2[16];
            tmem_ld16(t0, r);
            if (g.lo_off == 16) tmem_ld16(t0 + 16u, r2);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float lo = g.lo_off == 16 ? __uint_as_float(r2[j]) : __uint_as_float(r[(j + 8) & 15]);
                if (j < g.m_real) __stcg(out + (size_t)j * TILE_N + et, __uint_as_float(r[j]) + lo);
            }
        } else
        for (int c0 = 0; c0 < g.m_pad; c0 += 16) {
            uint32_t r[16];
            tmem_ld16(tmem_base + ((quarter * 32u) << 16) + buf * (uint32_t)g.m_pad + (uint32_t)c0, r);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (c0 + j < g.m_tok) __stcg(out + (size_t)(c0 + j) * TILE_N + et, __uint_as_float(r[j]));
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh.tmem_empty[buf]));
        if (arrive) {
            // The barrier orders the four warps' stores before thread 0's release, which is cumulative: whoever
            // acquires the tile's word after the last arrival sees every piece of the tile.
            epi_bar();
            if (et == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(arrive + u / g.kb_per_tile) : "memory");
        }
        u += n_kb;
    }
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
k_gemm_streamk(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x,
               GemmGeom g, float* __restrict__ partials, uint32_t* __restrict__ arrive, uint32_t* status) {
    extern __shared__ uint8_t dyn_smem[];
    __shared__ Shared sh;
    pdl_launch_dependents();                 // the next kernel may be scheduled; it waits for this one where it must
    if (threadIdx.x == 0) stamp_first(g.stamp, ST_START);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tiles0 = (smem_u32(dyn_smem) + 1023u) & ~1023u;        // 1024-byte aligned stage ring
    const uint32_t x_bytes = (uint32_t)g.m_pad * 128u, stage_bytes = A_BYTES + x_bytes;
    volatile int* abort_flag = &sh.abort_flag;

    // this CTA's share of the (row tile, k block) pairs
    const uint32_t T = (uint32_t)g.n_tiles * (uint32_t)g.kb_per_tile;
    const uint32_t u0 = (blockIdx.x * T) / gridDim.x;
    const uint32_t u1 = ((blockIdx.x + 1) * T) / gridDim.x;
    const uint32_t n_units = u1 - u0;
    uint32_t tmem_cols = 32;
    while (tmem_cols < 2u * (uint32_t)g.m_pad) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(smem_u32(&sh.full[s]), 2);           // the weight tile and the token rows arrive from two producers
            mbar_init(smem_u32(&sh.empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&sh.tmem_full[b]), 1); mbar_init(smem_u32(&sh.tmem_empty[b]), 4); }
        sh.abort_flag = 0;
        sh.epi_abort = 0;
        sh.dep_seen = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = sh.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ weight producer
        // The first tiles do not wait for the previous kernel (weights do not depend on it): the stream
        // starts as soon as the CTA is resident, while the consumers wait on the previous kernel.
        if (lane == 0) {
            uint64_t pol_stream;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            RingPos rp;
            bool dep_ok = false;
            uint64_t t_last = 0;
            volatile int* dep_seen = &sh.dep_seen;
            int tile = u0 / g.kb_per_tile, kb = u0 % g.kb_per_tile;
            for (uint32_t it = 0; it < n_units; ++it, rp.next(g.stages, g.steady)) {
                const int s = rp.stage;
                // A full ring of requests at this point slowed the step down: they compete with the small,
                // latency-critical reads of the kernel that reduces the previous GEMM.  So the run-ahead stops
                // short of the ring's depth until that kernel has finished.
                if (it >= (uint32_t)g.prefill && !dep_ok) {
                    if (g.pace_ns <= 0) { pdl_wait(); dep_ok = true; }
                    else {          // paced: one more stage every pace_ns, so that requests stay in flight until the kernel before is done
                        const uint64_t t_next = t_last + (uint64_t)g.pace_ns;
                        while (!(dep_ok = *dep_seen != 0) && global_ns() < t_next) {}
                    }
                }
                if (rp.use > 0u && !mbar_wait(smem_u32(&sh.empty[s]), (rp.use & 1u) ^ 1u, abort_flag)) break;
                const uint32_t bar = smem_u32(&sh.full[s]);
                mbar_expect_tx(bar, A_BYTES);
                tma_load_2d(tiles0 + s * stage_bytes, &tm_w, kb * TILE_K, tile * TILE_N, bar, pol_stream);
                if (g.pace_ns > 0 && !dep_ok) t_last = global_ns();
                if (++kb == g.kb_per_tile) { kb = 0; ++tile; }
            }
        }
    } else if (warp == 6) {
        // ------------------------------------------------------------------ token-row producer
        const int n_src = g.xr ? ((g.kb_per_tile - 1) >> g.xr_shift) + 1 : 0;      // tiles the token rows were written in
        if (g.xr && n_src <= XR_MAX_TILES) {
            // The rows are handed over tile by tile: the step kernel before counts into a word per tile once a tile's rows
            // are written, and a k block is loaded as soon as its tile's word is there; the whole warp watches words (a
            // lane per tile, the tile needed next first), lane 0 issues the copies.
            volatile unsigned char* ready = sh.xr_ready;
            for (int t = lane; t < n_src; t += 32) ready[t] = 0;
            __syncwarp();
            uint64_t pol_keep;
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            RingPos rp;
            int kb = u0 % g.kb_per_tile;
            bool first = true, gave_up = false, stop = false;
            for (uint32_t it = 0; it < n_units && !stop; ++it, rp.next(g.stages, g.steady)) {
                const int tile = kb >> g.xr_shift;
                if (!gave_up && !ready[tile]) {                                   // uniform: every lane reads the same byte
                    const uint64_t t0 = global_ns();
                    for (uint32_t spin = 0;; ++spin) {
                        const int tl = tile + lane;
                        if (tl < n_src && !ready[tl]) {
                            uint32_t v;
                            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(g.xr + tl) : "memory");
                            if (v >= g.xr_need) ready[tl] = 1;
                        }
                        __syncwarp();
                        if (ready[tile]) break;
                        __nanosleep(40);
                        if ((spin & 63u) == 63u && global_ns() - t0 > 200000000ull) {      // 0.2 s: not expected; wait for the whole kernel instead, and say so
                            pdl_wait();
                            if (lane == 0 && status) atomicOr(status, SD_DEV_WAIT_EXPIRED);
                            gave_up = true;
                            break;
                        }
                    }
                    if (lane == 0) asm volatile("fence.proxy.async;" ::: "memory");      // rows written with ordinary stores, read by the bulk copy below
                    __syncwarp();
                }
                if (lane == 0) {
                    if (first) { *(volatile int*)&sh.dep_seen = 1; stamp_pair(g.stamp, ST_DEP_FIRST); }
                    const int s = rp.stage;
                    if (rp.use > 0u && !mbar_wait(smem_u32(&sh.empty[s]), (rp.use & 1u) ^ 1u, abort_flag)) stop = true;
                    else {
                        const uint32_t bar = smem_u32(&sh.full[s]);
                        mbar_expect_tx(bar, x_bytes);
                        tma_load_2d(tiles0 + s * stage_bytes + A_BYTES, &tm_x, kb * TILE_K, 0, bar, pol_keep);
                    }
                }
                first = false;
                stop = __shfl_sync(0xffffffffu, (int)stop, 0) != 0;
                if (++kb == g.kb_per_tile) kb = 0;
            }
        } else if (lane == 0) {
            uint64_t pol_keep;
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            pdl_wait();                                           // the token rows are the previous kernel's output
            *(volatile int*)&sh.dep_seen = 1;
            stamp_pair(g.stamp, ST_DEP_FIRST);
            RingPos rp;
            int kb = u0 % g.kb_per_tile;
            for (uint32_t it = 0; it < n_units; ++it, rp.next(g.stages, g.steady)) {
                const int s = rp.stage;
                if (rp.use > 0u && !mbar_wait(smem_u32(&sh.empty[s]), (rp.use & 1u) ^ 1u, abort_flag)) break;
                const uint32_t bar = smem_u32(&sh.full[s]);
                mbar_expect_tx(bar, x_bytes);
                tma_load_2d(tiles0 + s * stage_bytes + A_BYTES, &tm_x, kb * TILE_K, 0, bar, pol_keep);
                if (++kb == g.kb_per_tile) kb = 0;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(g.m_pad >> 3) << 17) | ((uint32_t)(TILE_N >> 4) << 24);
            uint32_t seg = 0;
            bool ok = true;
            RingPos rp;
            const uint64_t desc0 = umma_desc(tiles0);
            uint32_t kb0 = u0 % g.kb_per_tile;
            for (uint32_t u = u0; u < u1 && ok; ++seg, kb0 = 0) {
                const uint32_t n_kb = min((uint32_t)g.kb_per_tile - kb0, u1 - u);
                const uint32_t buf = seg & 1u;
                if (!mbar_wait(smem_u32(&sh.tmem_empty[buf]), ((seg >> 1) & 1u) ^ 1u, abort_flag)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + buf * (uint32_t)g.m_pad;
                for (uint32_t j = 0; j < n_kb; ++j, rp.next(g.stages, g.steady)) {
                    const int s = rp.stage;
                    if (!mbar_wait(smem_u32(&sh.full[s]), rp.use & 1u, abort_flag)) { ok = false; break; }
                    if (u == u0 && j == 0) stamp_pair(g.stamp, ST_DATA_FIRST);
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t da = desc0 + (uint64_t)((uint32_t)s * (stage_bytes >> 4)), db = da + (A_BYTES >> 4);   // start-address field counts 16 bytes
#pragma unroll
                    for (uint32_t k = 0; k < TILE_K / 16; ++k)     // 16 elements = 32 bytes further along the swizzled row
                        umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (j | k) != 0u);
                    umma_commit(smem_u32(&sh.empty[s]));           // frees the stage once these MMAs have read it
                }
                if (ok) umma_commit(smem_u32(&sh.tmem_full[buf]));
                u += n_kb;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: TMEM -> workspace
        epilogue_warps(g, partials, arrive, sh, tmem_base, warp, lane, u0, u1);
    }

    // ---------------------------------------------------------------------- wind-down
    __syncwarp();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0) stamp_pair(g.stamp, ST_DONE_FIRST);
    if (sh.abort_flag) {
        if (threadIdx.x == 0 && status) atomicOr(status, SD_DEV_WAIT_EXPIRED);
        const uint64_t t0 = global_ns();                   // let copies in flight land before the CTA goes away
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

}  // namespace

// bf16 matrix [rows][K] row-major as a 2-D tensor map with boxes of box_rows x 64 elements,
// 128-byte swizzle; reads outside the matrix return zeros.
bool make_tensor_map_bf16(TensorMap* out, const void* base, int rows, int K, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || ((uintptr_t)base & 15) || (K & 7) || box_rows < 1 || box_rows > 256) return false;
    static_assert(sizeof(TensorMap) == sizeof(CUtensorMap), "tensor map size");
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)TILE_K, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

GemmGeom gemm_geometry(int m_tok, int n_out, int K, int n_sm, int max_stages, bool prefill_all, int extra_tiles) {
    GemmGeom g;
    g.lo_off = 0; g.m_real = m_tok; g.stamp = nullptr; g.pace_ns = 0;
    g.xr = nullptr; g.xr_shift = 0; g.xr_need = 0;
    g.m_tok = m_tok;
    g.m_pad = (m_tok + 15) & ~15;
    g.n_out = n_out;
    g.K = K;
    g.n_tiles = (n_out + TILE_N - 1) / TILE_N + extra_tiles;
    g.kb_per_tile = (K + TILE_K - 1) / TILE_K;
    const long long T = (long long)g.n_tiles * g.kb_per_tile;
    g.grid = (int)std::min<long long>(n_sm, T);
    const int per_cta = (int)((T + g.grid - 1) / g.grid);
    g.max_seg = (per_cta + g.kb_per_tile - 2) / g.kb_per_tile + 1;
    if ((T + 1) * (g.grid + 1) >= (1ll << 32)) g.grid = 0;   // the kernels split the work in 32-bit arithmetic
    const int stage_bytes = A_BYTES + g.m_pad * 128;
    g.stages = std::max(2, std::min(MAX_STAGES, RING_BYTES / stage_bytes));
    if (max_stages >= 2) g.stages = std::min(g.stages, max_stages);
    g.steady = std::min(g.stages, std::max(2, (GEMM_STEADY_BYTES + stage_bytes - 1) / stage_bytes));
    // (measured: with more than 16 token rows the reduction kernel is bound by throughput, not latency, and the full run-ahead wins)
    g.prefill = g.m_pad > 16 ? g.stages : std::min(g.stages, std::max(2, (GEMM_PREFILL_BYTES + stage_bytes - 1) / stage_bytes));
    if (g.m_pad <= 16) {            // few rows: four stages at once, then one more every 300 ns until the kernel before has finished
        g.prefill = std::min(g.stages, GEMM_PACED_PREFILL_STAGES);      // (measured against 7 stages at once and none after: -0.7 % at 7B, -1 % at 1B)
        g.pace_ns = GEMM_PACE_NS;
    }
    if (prefill_all) { g.prefill = g.stages; g.pace_ns = 0; }
    return g;
}

size_t gemm_partials_bytes(const GemmGeom& g) { return sizeof(float) * (size_t)g.grid * g.max_seg * g.m_pad * TILE_N; }

bool gemm_tc_supported(int m_tok, int n_out, int K) {
    return m_tok >= 1 && m_tok <= 256 && n_out >= 1 && K >= 8 && (K & 7) == 0 && (long long)((n_out + 127) / 128) * ((K + 63) / 64) < (1ll << 24);
}

cudaError_t launch_gemm_streamk(const TensorMap& tm_w, const TensorMap& tm_x, const GemmGeom& g, float* partials, uint32_t* arrive,
                                uint32_t* status, int dependent, cudaStream_t st) {
    const size_t smem = (size_t)g.stages * (A_BYTES + g.m_pad * 128) + 1024;
    {   // the attribute belongs to the current device: set it on every launch (a host-side table lookup)
        cudaError_t e = cudaFuncSetAttribute(k_gemm_streamk, cudaFuncAttributeMaxDynamicSharedMemorySize, RING_BYTES + 2048);
        if (e != cudaSuccess) return e;
    }
    if (g.grid < 1 || g.stages < 2 || g.steady < 1 || g.steady > g.stages || g.m_tok > SD_MAX_ROWS || smem > RING_BYTES + 2048) return cudaErrorInvalidValue;
    return launch_pdl(k_gemm_streamk, dim3(g.grid), dim3(NUM_THREADS), smem, st, dependent,
                      *(const CUtensorMap*)&tm_w, *(const CUtensorMap*)&tm_x, g, partials, arrive, status);
}

}  // namespace sd
