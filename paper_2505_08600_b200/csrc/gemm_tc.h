// Interface of the tensor-core weight-streaming GEMM (gemm_tc.cu) and of the fused step that follows it (fused_step.cu).
#pragma once
#include <algorithm>
#include <utility>

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
    int steady;             // stages reused once the ring has been filled (<= stages)
    int prefill;            // weight tiles requested before the previous kernel has finished
    unsigned long long* stamp;   // optional time stamps of this launch (see LaunchStamp); nullptr: none
    // Per-tile readiness of the token rows (nullptr: wait for the whole kernel before).  The step kernel that writes the
    // rows counts one into xr[t] when its CTA for 128-row tile t (64 features of the activation: xr_shift 0; 128 columns
    // of the normed residual: xr_shift 1) has written everything it writes; k block kb of this GEMM is loaded once
    // xr[kb >> xr_shift] has reached xr_need (the step's row batches per tile).
    const uint32_t* xr; int xr_shift; uint32_t xr_need;
    int pace_ns;            // > 0: past `prefill`, one more stage is requested every pace_ns until the kernel before has finished
    int lo_off, m_real;     // two-part input rows (see Epilogue::lo_off): the epilogue adds accumulator columns r and r + lo_off
                            // and leaves m_real merged rows in each piece; 0: every column is a row of its own
};

// RMSNorm folded around a GEMM: the GEMM's input rows are h * gain (no 1/rms factor), the
// factor rsqrt(mean(h^2) + eps) of each row multiplies the GEMM's output instead.  The sum of
// squares of a row arrives in n_parts pieces (one per 128-wide tile of the kernel that wrote h).
struct RowScale {
    const float* ssq;       // [row][SSQ_STRIDE]; nullptr: no scaling
    int n_parts;
    float inv_d, eps;
};
constexpr int SSQ_STRIDE = 64;

// What happens to a 128-row output tile once its pieces are summed (the step that follows the
// GEMM in the decoder layer), so that no fp32 intermediate matrix goes through memory.
enum { EPI_PLAIN = 0, EPI_QKV_ROPE = 1, EPI_RESIDUAL = 2, EPI_SWIGLU = 3 };
struct Epilogue {
    int mode;
    // Activations in two bf16 parts: when lo_off > 0 the GEMM's input rows were [x_hi rows][x_lo rows at +lo_off] with
    // x_hi = bf16(x), x_lo = bf16(x - x_hi), so that accumulator rows r and r + lo_off are added (the activation enters the
    // product almost unrounded, at no extra weight traffic: both parts sit in the 16 columns the MMA covers anyway), and
    // the rows this step writes for the next GEMM are split the same way.  m_real = token rows (the GEMM saw lo_off + m_real).
    int lo_off, m_real;
    unsigned long long* stamp;       // optional time stamps of the step's launch (see LaunchStamp)
    // Low-rank adapters (nullptr: none).  The GEMM's last output tile holds x A^T for every adapter (adapter a in its
    // columns a * r ... a * r + r - 1); row i uses the adapter of its sequence, lora_task[i], and the step adds
    // lora_scale * sum_j t[i][j] * lora_b[adapter][n][j] to output feature n before anything else.
    const bf16* lora_b;              // [adapters][n_out][r], rows in the order of the GEMM's output features
    const int32_t* lora_task;        // [row], written with the row plan by the pass's first kernel
    int lora_r, lora_n;              // rank, adapters
    float lora_scale;
    uint32_t* xready;                // non-null: words [tile] the step counts into when a CTA's outputs are written (see GemmGeom::xr)
    int many_rows_cb;                // many-row form of the step: 4 = request up to four pieces per round when a tile has more than two (default: two)
    int ring_stages, prefill_all;    // GEMM before this step: cap on its stage ring (0: none) / request the whole ring before the dependency
    unsigned long long poll_ns;      // how long a tile's CTA watches its arrival word before it falls back to the grid dependency (0: 0.2 s)
    RowScale rs;                     // PLAIN, QKV_ROPE, SWIGLU: 1/rms factor of each token row
    // EPI_PLAIN: y[i][n] = scale * acc[token i*row_stride + row_offset][n], i < n_out_rows
    float* y; int n_out_rows, row_stride, row_offset;
    // EPI_QKV_ROPE: rotary embedding, then query buffer / KV-cache append (bf16)
    bf16* q_out; bf16* kc; bf16* vc; const int32_t* row_slot; const int32_t* row_pos;
    int H, Hkv, hd, max_ctx; const float* rcos; const float* rsin;     // rcos/rsin: [token row][hd/2], the row's position applied
    // EPI_RESIDUAL: h += acc; xn = bf16(h * gain_next); ssq_out[row][tile] = sum over the tile of h^2
    float* h; const float* gain_next; bf16* xn; float* ssq_out;
    // EPI_SWIGLU: rows of the weight matrix interleaved per tile (64 gate rows, then the 64 up
    // rows of the same features): act[row][tile*64 + f] = silu(gate_f) * up_f
    bf16* act; int F;
};

bool gemm_tc_supported(int m_tok, int n_out, int K);
// max_stages > 0 caps the ring (a smaller ring leaves shared memory for CTAs of the kernel before, e.g. attention, so that
// this GEMM's CTAs are resident and streaming while that kernel still runs); prefill_all: request the whole ring early.
// extra_tiles: 128-row tiles appended after the matrix's own (rounded up to whole tiles): rows of a low-rank adapter.
GemmGeom gemm_geometry(int m_tok, int n_out, int K, int n_sm, int max_stages = 0, bool prefill_all = false, int extra_tiles = 0);
size_t gemm_partials_bytes(const GemmGeom& g);
bool make_tensor_map_bf16(TensorMap* out, const void* base, int rows, int K, int box_rows);
// The GEMM proper: leaves the split accumulators in `partials` (gemm_partials_bytes()).
// dependent != 0: launched with programmatic stream serialisation (may start while the previous
// kernel on the stream drains; the kernel itself waits before it touches that kernel's results).
// arrive (nullable): one word per output tile, zero before the launch; every CTA adds one to a tile's
// word when its piece of the tile is in the workspace, so that the step after the GEMM can start on a
// tile as soon as the tile is complete instead of when the whole grid has retired.  Kernels of several
// consecutive GEMMs can be resident at once (each only needs its predecessor to have started), so
// every GEMM between two ordinary (fully ordered) launches needs words of its own.
cudaError_t launch_gemm_streamk(const TensorMap& tm_w, const TensorMap& tm_x, const GemmGeom& g, float* partials, uint32_t* arrive,
                                uint32_t* status, int dependent, cudaStream_t st);
// The step after the GEMM (fused_step.cu): reduces `partials` and applies `ep`.  With `arrive` (the
// words the GEMM counts in; left at zero again) and a single batch of rows, a tile's CTA polls its word
// (bounded; on expiry it falls back to waiting for the GEMM's grid and flags SD_DEV_WAIT_EXPIRED).
cudaError_t launch_fused_step(const GemmGeom& g, const Epilogue& ep, const float* partials, uint32_t* arrive, uint32_t* status,
                              int dependent, cudaStream_t st);
// Whether launch_fused_step polls (and clears) the arrival words for this step; the GEMM must count exactly then.
bool fused_step_polls(const GemmGeom& g, const Epilogue& ep);
int fused_step_row_batches(const GemmGeom& g, const Epilogue& ep);      // CTAs of the step per output tile

// Launch with the programmatic-dependent-launch attribute (or plainly when dependent == 0).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int dependent, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Device side of the same protocol: let the next kernel on the stream start its prologue, and
// wait until everything the previous kernel wrote is visible.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Nanoseconds of the GPU's global timer: the clock of every bounded wait.
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Optional time stamps of one launch: eight 64-bit words that start as all ones and are kept with atomicMin, so a word
// named "first" holds the earliest time any CTA reported and a word named "last" the bitwise complement of the latest.
enum LaunchStamp { ST_START = 0,        // a CTA began
                   ST_DEP_FIRST = 1, ST_DEP_LAST = 2,       // what the CTA waits for (the kernel before it, its tile's pieces) was there
                   ST_DATA_FIRST = 3, ST_DATA_LAST = 4,     // GEMM: the first stage of a CTA was complete and its first MMA issued
                   ST_DONE_FIRST = 5, ST_DONE_LAST = 6,     // a CTA had written its results
                   ST_WORDS = 8 };
__device__ __forceinline__ void stamp_first(unsigned long long* rec, int i) { if (rec) atomicMin(rec + i, (unsigned long long)global_ns()); }
__device__ __forceinline__ void stamp_pair(unsigned long long* rec, int i_first) {
    if (rec) { const unsigned long long t = global_ns(); atomicMin(rec + i_first, t); atomicMin(rec + i_first + 1, ~t); }
}


}  // namespace sd
