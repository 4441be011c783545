// Persistent streaming kernel: one launch runs every decoder layer and the lm_head of a forward pass over a
// handful of query rows (the verify rows of Fig. 1(b), or one decoding row), one CTA per SM.
//
// The pass is bound by one read of every weight matrix from HBM, and between two matrices of a layer lies a
// chain of small dependent steps (sum the split accumulators, normalise / rotate / gate, publish the next
// matrix's input rows).  With a kernel per matrix that chain is paid at every boundary while HBM idles.  Here
//   - every CTA streams its share of ALL matrices, layer after layer, through one ring of shared-memory stages
//     (tcgen05.mma, bf16 in, fp32 accumulators in TMEM; weights by TMA, input rows by bulk copies);
//   - a matrix is cut into tile waves x K chunks (pass_program.h): four spare warps per CTA sum the pieces of
//     finished tiles and apply the step after the GEMM while later waves stream, and the next matrix starts on
//     the chunk of its input that the first wave produced;
//   - attention over the cache runs on the same spare warps, head by head, as soon as a head's query / key /
//     value tiles are reduced; its output feeds the Wo GEMM chunk by chunk.
// What one CTA hands to another travels as tagged 64-bit words (pass_stream.h): a reader polls the data itself, so no
// flag, fence or atomic sits between a producer and its consumers, and a consumer starts on a k block of its input
// the moment that block exists.  Every wait is bounded: the first one that gives up raises a flag that winds the
// whole grid down, and the host sees SD_DEV_WAIT_EXPIRED.
// Warps: 0 weight producer, 1 MMA issuer, 2..3 input-row producers, 4..7 TMEM -> workspace, 8..11 tasks (sum finished tiles, attention).
#include <cuda.h>

#include "pass_stream.h"
#include "tc_ptx.cuh"

namespace sd {

namespace {

constexpr int TILE_N = 128, TILE_K = 64, A_BYTES = TILE_N * TILE_K * 2;
constexpr int NUM_THREADS = 384;
constexpr int MAX_STAGES = 10;
constexpr int MAX_ACC = 16;                      // accumulators in tensor memory (a CTA returns to a tile in the wave's next chunk)
constexpr int PROG_BYTES = 8 * 1024;             // the CTA's section of the program
constexpr int RING_BUDGET = 148 * 1024;
constexpr int ATTN_BYTES = 64 * 1024;            // key / value chunks and merge buffers of the attention tasks
constexpr int NQ = 16;                           // query vectors of one attention item (one MMA row tile)
constexpr int AW = 4;                            // warps of the task group
constexpr uint64_t WAIT_NS = 500000000ull;       // every wait gives up after half a second

struct PassShared {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], tmem_full[MAX_ACC], tmem_empty[MAX_ACC];
    uint32_t tmem_base;
    int abort_flag, epi_abort, aux_flag;
    float scale[8];
    float val[8][TILE_N];
    float wsum[8][4];
    float wgt[NQ * 32];
};

struct Abort { volatile int* local; volatile uint32_t* global; };
__device__ __forceinline__ bool aborted(const Abort& a) { return *a.local != 0 || *a.global != 0u; }
__device__ __forceinline__ void give_up(const Abort& a) {
    *a.local = 1; *a.global = 1u;
}

__device__ __forceinline__ bool mbar_wait_b(uint32_t bar, uint32_t parity, const Abort& ab) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    for (uint32_t i = 1;; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 0u) {
            if (aborted(ab)) return false;
            if (global_ns() - t0 > WAIT_NS) { give_up(ab); return false; }
        }
    }
}
enum { USE_A = 1, USE_B = 2 };                   // uses of a buffer within one iteration (part of the tag)

// A load from L2, where every SM's stores land.  An ordinary load as far as the compiler is concerned, so that a batch of them is
// issued back to back; loops that look again put a compiler barrier between two looks (Retry::again).
__device__ __forceinline__ tagged_t ldq(const tagged_t* p) { return __ldcg(p); }
__device__ __forceinline__ void stq(tagged_t* p, uint32_t payload, uint32_t tag) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(((tagged_t)tag << 32) | payload) : "memory");
}
__device__ __forceinline__ bool has_tag(tagged_t v, uint32_t tag) { return (uint32_t)(v >> 32) == tag; }
// Bookkeeping of a retry loop: true while the caller should look again.
struct Retry {
    uint64_t t0; uint32_t n;
    __device__ __forceinline__ Retry() : t0(0), n(0) {}
    __device__ __forceinline__ bool again(const Abort& ab) {
        if (n == 0) t0 = global_ns();
        if ((++n & 15u) == 0u) {
            if (aborted(ab)) return false;
            if (global_ns() - t0 > WAIT_NS) { give_up(ab); return false; }
        }
        __nanosleep(40);
        asm volatile("" ::: "memory");               // the next look really loads again
        return true;
    }
};
// One word, looked at until it carries the tag.
__device__ __forceinline__ bool ldq_wait(const tagged_t* p, uint32_t tag, uint32_t& payload, const Abort& ab) {
    Retry r;
    for (;;) {
        const tagged_t v = ldq(p);
        if (has_tag(v, tag)) { payload = (uint32_t)v; return true; }
        if (!r.again(ab)) { payload = 0u; return false; }
    }
}

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }    // warps 4..7
__device__ __forceinline__ void aux_bar() { asm volatile("bar.sync 2, 128;" ::: "memory"); }    // warps 8..11

// Barrier of the task group that also tells whether `ok` held for all 128 threads.
__device__ __forceinline__ int __syncthreads_and_aux(int ok) {
    int r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %1, 0;\n\tbar.red.and.pred q, 2, 128, p;\n\tselp.s32 %0, 1, 0, q;\n\t}" : "=r"(r) : "r"(ok) : "memory");
    return r;
}
// One value from the task group's first thread to all 128 of them (the flag may be rewritten right after).
template <class SH> __device__ __forceinline__ int aux_broadcast(SH& sh, int t, int v) {
    if (t == 0) sh.aux_flag = v;
    aux_bar();
    const int r = sh.aux_flag;
    aux_bar();
    return r;
}

__device__ __forceinline__ void ring_next(int& stage, uint32_t& use, int stages) { if (++stage == stages) { stage = 0; ++use; } }

struct Program {
    const PassSeg* segs[2]; const PassTask* tasks[2]; const uint16_t* pieces;
    int n_seg[2], n_task[2];
};

// ------------------------------------------------------------------------------------------ reduce task
// Sums the pieces of one 128-row output tile in the program's fixed order and applies the step that follows
// the GEMM in the decoder layer: QKV -> 1/rms, rotary embedding, queries / KV append; Wo and down -> residual
// add, next norm's operand h * gain (bf16) and the tile's share of sum h^2; gate/up -> 1/rms, SwiGLU;
// lm_head -> 1/rms, fp32 logits.  128 threads, one per row of the tile.  Inputs and outputs that other CTAs of
// this launch write or read are tagged words: the task starts by watching one word of each piece, then loads
// everything and looks again at whatever does not carry the tag yet.
__device__ void reduce_task(const PassParams& P, PassShared& sh, const PassTask& tk, const uint16_t* pl, int it, uint32_t epoch,
                            const Abort& ab, int et) {
    const int mat = tk.mat, tile = (int)tk.item, lane = et & 31, warp = et >> 5;
    enum { ROPE, RESID, SWIGLU, PLAIN };
    const int mode = mat == MAT_QKV ? ROPE : mat == MAT_GU ? SWIGLU : mat == MAT_LM ? PLAIN : RESID;
    const int n_out = P.n_out[mat], n = tile * TILE_N + et;
    const bool live = n < n_out;
    const tagged_t* __restrict__ partials = P.partials[mat & 1];
    const size_t piece_elems = (size_t)P.m_tok * TILE_N;
    // tags: of the pieces, of what the step reads (residual stream, sums of squares) and of what it writes
    const uint32_t tag_piece = pass_tag(epoch, it, (mat == MAT_GU || mat == MAT_DN) ? USE_B : USE_A);
    const uint32_t tag_in = pass_tag(epoch, it, (mat == MAT_GU || mat == MAT_DN) ? USE_B : USE_A);      // h / ssq as the matrix's input saw them
    const uint32_t tag_out = mat == MAT_WO ? pass_tag(epoch, it, USE_B) : mat == MAT_DN ? pass_tag(epoch, it + 1, USE_A) : pass_tag(epoch, it, USE_A);
    const int n_parts = (mat == MAT_QKV && it == 0) ? 1 : (P.d + 127) / 128;
    const float inv_d = 1.f / (float)P.d;
    const float* gain_next = nullptr;
    if (mode == RESID)
        gain_next = mat == MAT_WO ? P.norm2 + (size_t)it * P.norm_stride
                                  : (it + 1 < P.n_layers ? P.norm1 + (size_t)(it + 1) * P.norm_stride : (P.has_tail ? P.final_norm : nullptr));
    const float gain = (gain_next && live) ? gain_next[n] : 0.f;
    const int n_rows = mode == PLAIN ? P.logits_rows : P.m_tok;
    const int hd = P.hd, half = hd >> 1, head = n / hd, e = n % hd;
    const bool rot = head < P.H + P.Hkv;
    bf16* kc = P.kc + (size_t)it * P.kv_layer_elems;
    bf16* vc = P.vc + (size_t)it * P.kv_layer_elems;
    // ---- watch one word of every piece (the last row's last column) until all of them are there
    {
        int ok = 1;
        if (et < (int)tk.n_pieces) {
            uint32_t dummy;
            ok = ldq_wait(partials + (size_t)pl[et] * piece_elems + (size_t)(P.m_tok - 1) * TILE_N + (TILE_N - 1), tag_piece, dummy, ab) ? 1 : 0;
        }
        ok = __syncthreads_and_aux(ok);
        if (!ok) return;
    }
    for (int m0 = 0; m0 < n_rows; m0 += 8) {
        int rows[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = m0 + i;
            rows[i] = r < n_rows ? (mode == PLAIN ? r * P.row_stride + P.row_offset : r) : -1;
        }
        float cs[8], sn[8];
        int pos[8], slot[8];
        if (mode == ROPE) {
            const bool lower = live && e < half;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const bool ok = lower && rows[i] >= 0;
                pos[i] = ok ? __ldg(P.row_pos + rows[i]) : -1;
                slot[i] = (ok && head >= P.H) ? __ldg(P.row_slot + rows[i]) : 0;
                cs[i] = (ok && rot) ? __ldg(P.rcos + (size_t)rows[i] * half + e) : 1.f;
                sn[i] = (ok && rot) ? __ldg(P.rsin + (size_t)rows[i] * half + e) : 0.f;
            }
        }
        bool good = true;
        float ssa[2] = {0.f, 0.f}, ssb[2] = {0.f, 0.f};
        float hv[8];
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) { v[i] = 0.f; hv[i] = 0.f; }
        Retry retry;
        for (;;) {
            bool all = true;
            if (mode != RESID) {                  // one warp per token row, one lane per piece of its sum of squares
#pragma unroll
                for (int ii = 0; ii < 2; ++ii) {
                    const int r = m0 + warp + 4 * ii;
                    const bool ok = r < n_rows;
                    const tagged_t* ps = P.ssq + (size_t)(ok ? (mode == PLAIN ? r * P.row_stride + P.row_offset : r) : 0) * SSQ_STRIDE;
                    const tagged_t wa = (ok && lane < n_parts) ? ldq(ps + lane) : 0ull;
                    const tagged_t wb = (ok && lane + 32 < n_parts) ? ldq(ps + lane + 32) : 0ull;
                    all = all && (!(ok && lane < n_parts) || has_tag(wa, tag_in)) && (!(ok && lane + 32 < n_parts) || has_tag(wb, tag_in));
                    ssa[ii] = (ok && lane < n_parts) ? __uint_as_float((uint32_t)wa) : 0.f;
                    ssb[ii] = (ok && lane + 32 < n_parts) ? __uint_as_float((uint32_t)wb) : 0.f;
                }
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const bool ok = live && rows[i] >= 0;
                    const tagged_t w = ok ? ldq(P.h + (size_t)rows[i] * n_out + n) : 0ull;
                    all = all && (!ok || has_tag(w, tag_in));
                    hv[i] = ok ? __uint_as_float((uint32_t)w) : 0.f;
                }
            }
            if (all) break;
            if (!retry.again(ab)) { good = false; break; }
        }
        if (live) {
            for (int c0 = 0; c0 < (int)tk.n_pieces && good; c0 += 4) {
                float tmp[4][8];
                Retry rp;
                for (;;) {
                    bool all = true;
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        const bool okc = c0 + cc < (int)tk.n_pieces;
                        const tagged_t* base = partials + (size_t)(okc ? pl[c0 + cc] : 0) * piece_elems + et;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const bool ok = okc && rows[i] >= 0;
                            const tagged_t w = ok ? ldq(base + (size_t)rows[i] * TILE_N) : 0ull;
                            all = all && (!ok || has_tag(w, tag_piece));
                            tmp[cc][i] = ok ? __uint_as_float((uint32_t)w) : 0.f;
                        }
                    }
                    if (all) break;
                    if (!rp.again(ab)) { good = false; break; }
                }
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)                                   // the pieces are added in the program's order
#pragma unroll
                    for (int i = 0; i < 8; ++i) v[i] += tmp[cc][i];
            }
        }
        if (!__syncthreads_and_aux(good ? 1 : 0)) return;          // a wait gave up somewhere: nobody goes on
        if (mode != RESID) {
#pragma unroll
            for (int ii = 0; ii < 2; ++ii) {
                const float ss = warp_sum(ssa[ii] + ssb[ii]);
                if (lane == 0) sh.scale[warp + 4 * ii] = rsqrtf(ss * inv_d + P.rms_eps);
            }
            aux_bar();
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] *= sh.scale[i];
        }
        if (mode == PLAIN) {
            if (live) {
#pragma unroll
                for (int i = 0; i < 8; ++i) if (rows[i] >= 0) P.logits[(size_t)(m0 + i) * n_out + n] = v[i];
            }
        } else if (mode == ROPE) {
#pragma unroll
            for (int i = 0; i < 8; ++i) sh.val[i][et] = v[i];
            aux_bar();
            // the thread of element e < hd/2 rotates the pair (e, e + hd/2); even e then writes two words: (e, e+1) and (e+hd/2, e+1+hd/2)
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float a = v[i], b = (e < half) ? sh.val[i][et + half] : 0.f;
                const float ra = a * cs[i] - b * sn[i], rb = a * sn[i] + b * cs[i];
                const uint32_t bits = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(ra)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(rb)) << 16);
                const uint32_t next = __shfl_down_sync(0xffffffffu, bits, 1);      // element e + 1 (same half: hd/2 is even)
                if (!(live && e < half) || rows[i] < 0 || (e & 1)) continue;
                // (a row without a position - the slot of a token the draft did not miss - still gets its tagged words: others wait for them)
                const uint32_t w_lo = (bits & 0xFFFFu) | (next << 16), w_hi = (bits >> 16) | (next & 0xFFFF0000u);
                if (head < P.H) {
                    tagged_t* dst = P.q + ((size_t)rows[i] * P.H + head) * half;          // hd / 2 words per head
                    stq(dst + (e >> 1), w_lo, tag_out);
                    stq(dst + ((e + half) >> 1), w_hi, tag_out);
                } else {
                    const int kvh = (head - P.H) % P.Hkv, part = rot ? 0 : 1;
                    if (pos[i] >= 0) {
                        bf16* cdst = (rot ? kc : vc) + (((size_t)slot[i] * P.Hkv + kvh) * P.max_ctx + pos[i]) * hd;
                        *reinterpret_cast<uint32_t*>(cdst + e) = w_lo;                     // the cache itself: read by later passes
                        *reinterpret_cast<uint32_t*>(cdst + e + half) = w_hi;
                    }
                    tagged_t* dst = P.newkv + (((size_t)rows[i] * 2 + part) * P.Hkv + kvh) * half;   // ... and a tagged copy for this pass
                    stq(dst + (e >> 1), w_lo, tag_out);
                    stq(dst + ((e + half) >> 1), w_hi, tag_out);
                }
            }
        } else if (mode == RESID) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                hv[i] += v[i];
                const uint32_t xb = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hv[i] * gain));
                const uint32_t nb = __shfl_down_sync(0xffffffffu, xb, 1);                  // column n + 1
                if (live && rows[i] >= 0) {
                    stq(P.h + (size_t)rows[i] * n_out + n, __float_as_uint(hv[i]), tag_out);
                    if (gain_next && !(et & 1)) stq(P.xn + xtagged_index(rows[i], n, P.m_pad), xb | (nb << 16), tag_out);
                }
            }
            if (gain_next) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float ss = warp_sum(hv[i] * hv[i]);
                    if (lane == 0) sh.wsum[i][warp] = ss;
                }
                aux_bar();
                if (et < 8 && m0 + et < n_rows) {
                    const float* w = sh.wsum[et];
                    stq(P.ssq + (size_t)(m0 + et) * SSQ_STRIDE + tile, __float_as_uint((w[0] + w[1]) + (w[2] + w[3])), tag_out);
                }
            }
        } else {                                  // SWIGLU: 64 gate rows then the 64 up rows of the same features
            const int f = tile * 64 + et;
#pragma unroll
            for (int i = 0; i < 8; ++i) sh.val[i][et] = v[i];
            aux_bar();
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float gt = v[i], up = et < 64 ? sh.val[i][et + 64] : 0.f;
                const uint32_t ab16 = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(gt / (1.f + expf(-gt)) * up));
                const uint32_t nb = __shfl_down_sync(0xffffffffu, ab16, 1);
                if (et < 64 && !(et & 1) && f < P.F && rows[i] >= 0) stq(P.act + xtagged_index(rows[i], f, P.m_pad), ab16 | (nb << 16), tag_out);
            }
        }
        if (m0 + 8 < n_rows) aux_bar();           // the exchange buffers are reused by the next batch of rows
    }
}

// ------------------------------------------------------------------------------------------ attention task
__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// One slice of one KV head's cache x the query rows of one block (times the query heads that share the KV
// head) as a 16-row tensor-core tile (mma.sync m16n8k16, bf16 in, fp32 accumulate).  The slice is walked in
// chunks of 64 keys, double-buffered in shared memory (16-byte asynchronous copies into an XOR-swizzled layout
// that ldmatrix reads without bank conflicts); each warp owns 16 keys of a chunk and keeps its own running
// max / sum / output (online softmax, exp2 domain).  The positions that earlier passes wrote are requested at
// once; the queries and the keys / values this pass appends come as tagged words from the tasks that reduce the
// QKV tiles.  With one slice the normalised output is written directly (as input rows of the Wo GEMM); with
// several, every slice leaves a tagged partial result and the task of slice 0 merges them in slice order.
template <int HD>
__device__ void attention_task(const PassParams& P, PassShared& sh, uint8_t* sm_raw, const PassTask& tk, int it, uint32_t epoch,
                               const Abort& ab, int t) {
    constexpr int NT = 32 * AW, CK = 16 * AW;
    constexpr int ROWB = HD * 2, CPR = HD / 8, KS = HD / 16, NV = HD / 8, BUF = CK * ROWB, OLD = HD + 8, HALF = HD / 2;
    const uint32_t tag = pass_tag(epoch, it, USE_A);
    const int ns = P.n_splits;
    const int split = (int)(tk.item % (uint32_t)ns), rest = (int)(tk.item / (uint32_t)ns);
    const int kvh = rest % P.Hkv, blk = rest / P.Hkv;
    const int group = P.H / P.Hkv;
    const int bps = (P.rows_per_seq + P.rows_per_block - 1) / P.rows_per_block;
    const int seq_first = (blk / bps) * P.rows_per_seq;
    const int r0 = seq_first + (blk % bps) * P.rows_per_block;
    const int nr = min(P.rows_per_block, P.rows_per_seq - (blk % bps) * P.rows_per_block);
    const int nq = nr * group;
    const int lane = t & 31, warp = t >> 5, gid = lane >> 2, tig = lane & 3;
    const uint32_t smem0 = smem_u32(sm_raw);
    const bf16* kcl = P.kc + (size_t)it * P.kv_layer_elems;
    const bf16* vcl = P.vc + (size_t)it * P.kv_layer_elems;

    // The row plan (positions, slots) was written by the kernel before this one.
    int mp = lane < nr ? __ldg(P.row_pos + r0 + lane) : -1;
    const int slot = __ldg(P.row_slot + r0);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mp = max(mp, __shfl_xor_sync(0xffffffffu, mp, o));
    const int len = mp + 1;
    const int slice = (((len + ns - 1) / ns) + 15) & ~15;
    const int p_begin = split * slice;
    const int np = max(0, min(p_begin + slice, len) - p_begin);
    int new_begin;                                           // first position this pass appends for the block's sequence
    {
        const int fp = lane < min(P.rows_per_seq, 32) ? __ldg(P.row_pos + seq_first + lane) : -1;
        int nb = fp >= 0 ? fp : 0x7fffffff;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) nb = min(nb, __shfl_xor_sync(0xffffffffu, nb, o));
        new_begin = nb == 0x7fffffff ? 0 : nb;
    }
    // row of the pass that holds position p >= new_begin of this sequence (rows of a sequence hold consecutive positions;
    // rows without a position come first)
    int first_live = 0;
    {
        const int fp = lane < min(P.rows_per_seq, 32) ? __ldg(P.row_pos + seq_first + lane) : 0;
        first_live = __popc(__ballot_sync(0xffffffffu, lane < min(P.rows_per_seq, 32) && fp < 0));
    }

    const int j_lo = gid, j_hi = gid + 8;
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
    float O[NV][4];
#pragma unroll
    for (int i = 0; i < NV; ++i) { O[i][0] = O[i][1] = O[i][2] = O[i][3] = 0.f; }

    const bf16* K = kcl + (((size_t)slot * P.Hkv + kvh) * P.max_ctx + p_begin) * HD;
    const bf16* V = vcl + (((size_t)slot * P.Hkv + kvh) * P.max_ctx + p_begin) * HD;
    int good = 1;
    // Chunk c -> buffer c & 1: [K][V].  do_old: the positions in front of new_begin, from the cache by asynchronous copies (one
    // copy group); do_new: the others, from this pass's tagged copy (looked at until they are there), and the padding rows.
    auto issue_part = [&](int c, bool do_old, bool do_new) {
        const int nk = min(CK, np - c * CK);
        const int k_lo = 0, k_hi = nk;
        const uint32_t kb = smem0 + (uint32_t)(c & 1) * 2u * BUF, vb = kb + BUF;
        const bf16* ks = K + (size_t)c * CK * HD;
        const bf16* vs = V + (size_t)c * CK * HD;
        const int old_hi = max(k_lo, min(k_hi, new_begin - (p_begin + c * CK)));      // keys [k_lo, old_hi) are old
        for (int i = k_lo * CPR + t; do_old && i < old_hi * CPR; i += NT) {
            const int key = i / CPR, ch = i % CPR;
            const uint32_t off = (uint32_t)key * ROWB + (uint32_t)((ch ^ (key & 7)) << 4);
            cp_async16(kb + off, ks + (size_t)i * 8);
            cp_async16(vb + off, vs + (size_t)i * 8);
        }
        if (do_old) asm volatile("cp.async.commit_group;" ::: "memory");
        for (int i = old_hi * CPR + t; do_new && i < k_hi * CPR; i += NT) {        // appended by this pass: four tagged words per 16 bytes
            const int key = i / CPR, ch = i % CPR;
            const int row = seq_first + first_live + (p_begin + c * CK + key - new_begin);
            const uint32_t off = (uint32_t)key * ROWB + (uint32_t)((ch ^ (key & 7)) << 4);
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                const tagged_t* src = P.newkv + (((size_t)row * 2 + part) * P.Hkv + kvh) * HALF + 4 * ch;
                uint32_t w[4];
                Retry r;
                for (;;) {
                    bool all = true;
#pragma unroll
                    for (int k = 0; k < 4; ++k) { const tagged_t v = ldq(src + k); all = all && has_tag(v, tag); w[k] = (uint32_t)v; }
                    if (all) break;
                    if (!r.again(ab)) { good = 0; break; }
                }
                *reinterpret_cast<uint4*>(sm_raw + (size_t)(c & 1) * 2 * BUF + (size_t)part * BUF + off) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
        const int nk16 = (nk + 15) & ~15;         // value rows past the slice inside a warp's 16-key group must be finite
        for (int i = nk * CPR + t; do_new && i < nk16 * CPR; i += NT) {
            const int key = i / CPR, ch = i % CPR;
            *reinterpret_cast<uint4*>(sm_raw + (size_t)(c & 1) * 2 * BUF + BUF + (size_t)key * ROWB + ((ch ^ (key & 7)) << 4)) = make_uint4(0, 0, 0, 0);
        }
    };
    const int n_chunks = (np + CK - 1) / CK;
#pragma unroll
    for (int c = 0; c < 2; ++c)
        if (c < n_chunks) issue_part(c, true, false);            // what earlier passes wrote is requested at once
    // The queries and the keys / values this pass appends exist once the tasks that reduce the QKV tiles have written them.
    // While they are not there, one thread watches one word (the last query's last one); then everything is loaded and
    // whatever does not carry the tag yet is looked at again.  A slice without positions waits too: nothing else keeps its
    // task from running ahead of the merge of the layer before.
    {
        uint32_t dummy;
        const int jl = nq - 1;
        const tagged_t* q_last = P.q + ((size_t)(r0 + jl / group) * P.H + kvh * group + jl % group) * HALF + (HALF - 1);
        if (!aux_broadcast(sh, t, t == 0 && ldq_wait(q_last, tag, dummy, ab) ? 1 : 0)) {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            return;
        }
    }
#pragma unroll
    for (int c = 0; c < 2; ++c)
        if (c < n_chunks) issue_part(c, false, true);
    // query fragments in the MMA's register layout: each is one tagged word (two bf16)
    uint32_t a[KS][4];
    {
        const tagged_t* q_lo = P.q + ((size_t)(r0 + j_lo / group) * P.H + kvh * group + j_lo % group) * HALF;
        const tagged_t* q_hi = P.q + ((size_t)(r0 + j_hi / group) * P.H + kvh * group + j_hi % group) * HALF;
        Retry r;
        for (;;) {
            bool all = true;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                const tagged_t w0 = j_lo < nq ? ldq(q_lo + 8 * ks + tig) : 0ull, w1 = j_hi < nq ? ldq(q_hi + 8 * ks + tig) : 0ull;
                const tagged_t w2 = j_lo < nq ? ldq(q_lo + 8 * ks + 4 + tig) : 0ull, w3 = j_hi < nq ? ldq(q_hi + 8 * ks + 4 + tig) : 0ull;
                all = all && (j_lo >= nq || (has_tag(w0, tag) && has_tag(w2, tag))) && (j_hi >= nq || (has_tag(w1, tag) && has_tag(w3, tag)));
                a[ks][0] = (uint32_t)w0; a[ks][1] = (uint32_t)w1; a[ks][2] = (uint32_t)w2; a[ks][3] = (uint32_t)w3;
            }
            if (all) break;
            if (!r.again(ab)) { good = 0; break; }
        }
    }
    if (np > 0) {
        const int pos_lo = j_lo < nq ? __ldg(P.row_pos + r0 + j_lo / group) : -1;
        const int pos_hi = j_hi < nq ? __ldg(P.row_pos + r0 + j_hi / group) : -1;
        const float sl2 = rsqrtf((float)HD) * 1.4426950408889634f;
        for (int c = 0; c < n_chunks; ++c) {
            // chunks c and c + 1 are in flight, one copy group each
            if (c + 1 < n_chunks) asm volatile("cp.async.wait_group 1;" ::: "memory");
            else asm volatile("cp.async.wait_group 0;" ::: "memory");
            aux_bar();
            const int nk = min(CK, np - c * CK);
            if (16 * warp < nk) {
                const uint32_t kb = smem0 + (uint32_t)(c & 1) * 2u * BUF, vb = kb + BUF;
                float S[2][4];
#pragma unroll
                for (int i = 0; i < 2; ++i) { S[i][0] = S[i][1] = S[i][2] = S[i][3] = 0.f; }
                {
                    const int mi = lane >> 3, r = lane & 7;
                    const int key = 16 * warp + 8 * (mi >> 1) + r;
                    const uint32_t rowaddr = kb + (uint32_t)key * ROWB;
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        uint32_t b[4];
                        ldmatrix_x4(rowaddr + (uint32_t)(((2 * ks + (mi & 1)) ^ (key & 7)) << 4), b);
                        mma_bf16(S[0], a[ks], b[0], b[1]);
                        mma_bf16(S[1], a[ks], b[2], b[3]);
                    }
                }
                const int pbase = p_begin + c * CK + 16 * warp + 2 * tig;
                float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int p = pbase + 8 * nt + (e & 1);
                        const bool ok = (p - p_begin) < np && p <= ((e < 2) ? pos_lo : pos_hi);
                        const float v = ok ? S[nt][e] * sl2 : -INFINITY;
                        S[nt][e] = v;
                        if (e < 2) mx_lo = fmaxf(mx_lo, v); else mx_hi = fmaxf(mx_hi, v);
                    }
                mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1)); mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
                mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1)); mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
                const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
                const float c_lo = (mn_lo == -INFINITY) ? 1.f : exp2f(m_lo - mn_lo);
                const float c_hi = (mn_hi == -INFINITY) ? 1.f : exp2f(m_hi - mn_hi);
                m_lo = mn_lo; m_hi = mn_hi;
                float s_lo = 0.f, s_hi = 0.f;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float mn = (e < 2) ? mn_lo : mn_hi;
                        const float pr = (mn == -INFINITY) ? 0.f : exp2f(S[nt][e] - mn);
                        S[nt][e] = pr;
                        if (e < 2) s_lo += pr; else s_hi += pr;
                    }
                l_lo = l_lo * c_lo + s_lo; l_hi = l_hi * c_hi + s_hi;
                uint32_t pa[4];
                pa[0] = pack_bf16(S[0][0], S[0][1]); pa[1] = pack_bf16(S[0][2], S[0][3]);
                pa[2] = pack_bf16(S[1][0], S[1][1]); pa[3] = pack_bf16(S[1][2], S[1][3]);
                {
                    const int mi = lane >> 3, r = lane & 7;
                    const int key = 16 * warp + 8 * (mi & 1) + r;
                    const uint32_t rowaddr = vb + (uint32_t)key * ROWB;
#pragma unroll
                    for (int nv = 0; nv < NV; nv += 2) {
                        O[nv][0] *= c_lo; O[nv][1] *= c_lo; O[nv][2] *= c_hi; O[nv][3] *= c_hi;
                        O[nv + 1][0] *= c_lo; O[nv + 1][1] *= c_lo; O[nv + 1][2] *= c_hi; O[nv + 1][3] *= c_hi;
                        uint32_t v[4];
                        ldmatrix_x4_trans(rowaddr + (uint32_t)(((nv + (mi >> 1)) ^ (key & 7)) << 4), v);
                        mma_bf16(O[nv], pa, v[0], v[1]);
                        mma_bf16(O[nv + 1], pa, v[2], v[3]);
                    }
                }
            }
            aux_bar();
            if (c + 2 < n_chunks) issue_part(c + 2, true, true);      // the buffer just read is free again
        }
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    }

    // ---- merge of the warps (each saw different keys)
    float* Ow = reinterpret_cast<float*>(sm_raw);           // [warps][16][OLD]
    float* mw = Ow + AW * NQ * OLD;                         // [warps][16]
    float* lw = mw + AW * NQ;
    if (np > 0) {
#pragma unroll
        for (int nv = 0; nv < NV; ++nv) {
            *reinterpret_cast<float2*>(Ow + ((size_t)warp * NQ + gid) * OLD + 8 * nv + 2 * tig) = make_float2(O[nv][0], O[nv][1]);
            *reinterpret_cast<float2*>(Ow + ((size_t)warp * NQ + gid + 8) * OLD + 8 * nv + 2 * tig) = make_float2(O[nv][2], O[nv][3]);
        }
        if (tig == 0) {
            mw[warp * NQ + gid] = m_lo; mw[warp * NQ + gid + 8] = m_hi;
            lw[warp * NQ + gid] = l_lo; lw[warp * NQ + gid + 8] = l_hi;
        }
    }
    good = __syncthreads_and_aux(good);
    constexpr int TPR = NT / NQ, CPT = HD / TPR;            // threads per query row, columns per thread
    const int j = t / TPR, c0 = (t % TPR) * CPT;
    float M = -INFINITY, L = 0.f;
    float acc[CPT];
#pragma unroll
    for (int cc = 0; cc < CPT; ++cc) acc[cc] = 0.f;
    if (np > 0) {
#pragma unroll
        for (int w = 0; w < AW; ++w) M = fmaxf(M, mw[w * NQ + j]);
#pragma unroll
        for (int w = 0; w < AW; ++w) {
            const float m = mw[w * NQ + j];
            const float wt = (m == -INFINITY) ? 0.f : exp2f(m - M);
            L += wt * lw[w * NQ + j];
            if (wt != 0.f) {
#pragma unroll
                for (int cc = 0; cc < CPT; ++cc) acc[cc] = fmaf(wt, Ow[((size_t)w * NQ + j) * OLD + c0 + cc], acc[cc]);
            }
        }
    }
    const int r = r0 + j / group, h = kvh * group + j % group;       // this thread's query (valid when j < nq)
    if (!good) return;                                                   // a wait gave up: leave nothing behind that looks complete
    if (ns > 1 && split != 0) {
        // a slice other than the first leaves its partial result, tagged, for the first one's task
        if (j < nq) {
            tagged_t* po = P.part_o + (((size_t)r * P.H + h) * ns + split) * HD + c0;
            tagged_t* ml = P.part_ml + (((size_t)r * P.H + h) * ns + split) * 2;
#pragma unroll
            for (int cc = 0; cc < CPT; ++cc) stq(po + cc, __float_as_uint(acc[cc]), tag);
            if ((t % TPR) == 0) { stq(ml, __float_as_uint(M), tag); stq(ml + 1, __float_as_uint(L), tag); }
        }
        return;
    }
    if (ns > 1) {
        // ---- slice 0 merges: out = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s, always in slice order
        {   // while the other slices' results are not there, one thread per slice watches one word of it
            const int jl = nq - 1, rl = r0 + jl / group, hl = kvh * group + jl % group;
            int ok = 1;
            uint32_t dummy;
            if (t >= 1 && t < ns) ok = ldq_wait(P.part_o + (((size_t)rl * P.H + hl) * ns + t) * HD + (HD - 1), tag, dummy, ab) ? 1 : 0;
            if (!__syncthreads_and_aux(ok)) return;
        }
        if (j < nq) {
            float Mt = M, ms[32], ls[32];
            ms[0] = M; ls[0] = L;
            {
                const tagged_t* mlg = P.part_ml + ((size_t)r * P.H + h) * ns * 2;
                Retry rt;
                for (;;) {
                    bool all = true;
                    for (int s2 = 1; s2 < ns; ++s2) {
                        const tagged_t a0 = ldq(mlg + 2 * s2), a1 = ldq(mlg + 2 * s2 + 1);
                        all = all && has_tag(a0, tag) && has_tag(a1, tag);
                        ms[s2] = __uint_as_float((uint32_t)a0); ls[s2] = __uint_as_float((uint32_t)a1);
                    }
                    if (all) break;
                    if (!rt.again(ab)) {
                        good = 0; break; }
                }
            }
            for (int s2 = 1; s2 < ns; ++s2) Mt = fmaxf(Mt, ms[s2]);
            float den = 0.f;
            for (int s2 = 0; s2 < ns; ++s2) den += (ms[s2] == -INFINITY ? 0.f : exp2f(ms[s2] - Mt)) * ls[s2];
            const float w0 = ms[0] == -INFINITY ? 0.f : exp2f(ms[0] - Mt);
#pragma unroll
            for (int cc = 0; cc < CPT; ++cc) acc[cc] *= w0;
            for (int s2 = 1; s2 < ns && good; ++s2) {
                const float w = ms[s2] == -INFINITY ? 0.f : exp2f(ms[s2] - Mt);
                const tagged_t* po = P.part_o + (((size_t)r * P.H + h) * ns + s2) * HD + c0;
                float o[CPT];
                Retry rt;
                for (;;) {
                    bool all = true;
#pragma unroll
                    for (int cc = 0; cc < CPT; ++cc) { const tagged_t v = ldq(po + cc); all = all && has_tag(v, tag); o[cc] = __uint_as_float((uint32_t)v); }
                    if (all) break;
                    if (!rt.again(ab)) { good = 0; break; }
                }
                if (w != 0.f) {
#pragma unroll
                    for (int cc = 0; cc < CPT; ++cc) acc[cc] = fmaf(w, o[cc], acc[cc]);
                }
            }
            L = den;
        }
    }
    if (j < nq && good) {                        // normalised output as input rows of the Wo GEMM (two bf16 per tagged word)
        const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
        for (int cc = 0; cc < CPT; cc += 2) {
            const __nv_bfloat162 v2 = __floats2bfloat162_rn(acc[cc] * inv, acc[cc + 1] * inv);
            stq(P.attn + xtagged_index(r, h * HD + c0 + cc, P.m_pad), *reinterpret_cast<const uint32_t*>(&v2), tag);
        }
    }
}

// ------------------------------------------------------------------------------------------ input rows of the segments
struct RingState { int stage; uint32_t use; };

// The batches of k blocks (KB at most, never across a segment) that the input-row warp walks through, in ring order.
struct RowBatches {
    const PassParams* Pp; const Program* pgp; uint32_t epoch;
    int n_it, it, si, j0, kb_step;
    __device__ RowBatches(const PassParams& p, const Program& g, uint32_t e, int nit, int step) : Pp(&p), pgp(&g), epoch(e), n_it(nit), it(0), si(0), j0(0), kb_step(step) { skip(); }
    __device__ void skip() { const PassParams& P = *Pp; const Program& pg = *pgp; while (it < n_it && si >= pg.n_seg[it == P.n_layers ? 1 : 0]) { ++it; si = 0; j0 = 0; } }
    __device__ bool done() const { return it >= n_it; }
    __device__ void get(const tagged_t*& src, int& nb, uint32_t& tag) const {
        const PassParams& P = *Pp; const Program& pg = *pgp;
        const PassSeg sg = pg.segs[it == P.n_layers ? 1 : 0][si];
        src = P.x[sg.mat] + ((size_t)sg.kb0 + j0) * P.m_pad * 32;
        nb = min(kb_step, (int)sg.n_kb - j0);
        tag = pass_tag(epoch, it, sg.mat == MAT_GU ? USE_B : USE_A);
    }
    __device__ void next() {
        const PassParams& P = *Pp; const Program& pg = *pgp;
        const PassSeg sg = pg.segs[it == P.n_layers ? 1 : 0][si];
        j0 += kb_step;
        if (j0 >= (int)sg.n_kb) { ++si; j0 = 0; skip(); }
    }
};

// Two warps bring the input rows of every segment from their tagged words in global memory into the stages' operand
// layout (128-byte rows, 16-byte pieces XOR-swizzled by row), KB k blocks of at most R rows at a time, taking turns
// batch by batch: lane l owns word l (two bf16) of every row.  A warp requests the words of its next batch while its
// current one goes into the stages, so that several batches are on their way at any time.  A batch whose words do not
// all carry the tag yet is where a matrix waits for the rows that the step before it produces: one lane then watches
// one word, and the batch is loaded again.
template <int KB, int R>
__device__ void produce_rows(const PassParams& P, PassShared& sh, const Program& pg, uint32_t epoch, int n_it, uint8_t* ring, uint32_t stage_bytes,
                             const Abort& ab, int lane, int which, int n_warps) {
    RowBatches cur(P, pg, epoch, n_it, KB);
    uint32_t unit = 0;                                       // k blocks of all batches before `cur`: fixes its stages
    auto advance = [&](RowBatches& b, uint32_t& u, int steps) {
        for (int i = 0; i < steps && !b.done(); ++i) { const tagged_t* s0; int nb; uint32_t tag; b.get(s0, nb, tag); u += (uint32_t)nb; b.next(); }
    };
    advance(cur, unit, which);
    if (cur.done()) return;
    tagged_t w[KB][R];
    auto load = [&](const tagged_t* s0, int nb, tagged_t (&dst)[KB][R]) {
#pragma unroll
        for (int k = 0; k < KB; ++k)
#pragma unroll
            for (int r = 0; r < R; ++r) dst[k][r] = (k < nb && r < P.m_tok) ? ldq(s0 + ((size_t)k * P.m_pad + r) * 32 + lane) : 0ull;
    };
    auto valid = [&](int nb, uint32_t tag, const tagged_t (&src)[KB][R]) {
        bool all = true;
#pragma unroll
        for (int k = 0; k < KB; ++k)
#pragma unroll
            for (int r = 0; r < R; ++r) all = all && (!(k < nb && r < P.m_tok) || has_tag(src[k][r], tag));
        return __all_sync(0xffffffffu, all) != 0;
    };
    {
        const tagged_t* s0; int nb; uint32_t tag;
        cur.get(s0, nb, tag);
        load(s0, nb, w);
    }
    for (;;) {
        const tagged_t* s0; int nb; uint32_t tag;
        cur.get(s0, nb, tag);
        if (!valid(nb, tag, w)) {
            // not there yet: watch the batch's last word, then load the batch again (and once more, should a straggler remain)
            Retry retry;
            for (;;) {
                int ok0 = 1;
                uint32_t dummy;
                if (lane == 0) ok0 = ldq_wait(s0 + ((size_t)(nb - 1) * P.m_pad + (P.m_tok - 1)) * 32 + 31, tag, dummy, ab) ? 1 : 0;
                if (!__shfl_sync(0xffffffffu, ok0, 0)) return;
                load(s0, nb, w);
                if (valid(nb, tag, w)) break;
                const bool cont = retry.again(ab);
                if (!__all_sync(0xffffffffu, cont)) return;
            }
        }
        RowBatches nxt = cur;
        uint32_t unit_next = unit;
        advance(nxt, unit_next, n_warps);
        tagged_t wn[KB][R];
        if (!nxt.done()) {                                   // request this warp's next batch now; it is looked at in the next round
            const tagged_t* s1; int nb1; uint32_t tag1;
            nxt.get(s1, nb1, tag1);
            load(s1, nb1, wn);
        }
#pragma unroll
        for (int k = 0; k < KB; ++k) {
            if (k >= nb) break;
            const uint32_t u = unit + (uint32_t)k;
            const int stage = (int)(u % (uint32_t)P.stages);
            const uint32_t use = u / (uint32_t)P.stages;
            int free_ok = 1;
            if (lane == 0 && use > 0u) free_ok = mbar_wait_b(smem_u32(&sh.empty[stage]), (use & 1u) ^ 1u, ab) ? 1 : 0;
            if (!__shfl_sync(0xffffffffu, free_ok, 0)) return;
            uint8_t* xs = ring + (size_t)stage * stage_bytes + A_BYTES;
#pragma unroll
            for (int r = 0; r < R; ++r)
                if (r < P.m_tok) *reinterpret_cast<uint32_t*>(xs + r * 128 + (((lane >> 2) ^ (r & 7)) << 4) + (lane & 3) * 4) = (uint32_t)w[k][r];
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // ordinary stores, read by the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.full[stage]));
        }
        if (nxt.done()) return;
#pragma unroll
        for (int k = 0; k < KB; ++k)
#pragma unroll
            for (int r = 0; r < R; ++r) w[k][r] = wn[k][r];
        cur = nxt; unit = unit_next;
    }
}

// ------------------------------------------------------------------------------------------ the kernel
__global__ void __launch_bounds__(NUM_THREADS, 1)
k_pass_stream(const __grid_constant__ PassMaps maps, const __grid_constant__ PassParams P) {
    extern __shared__ __align__(1024) uint8_t dyn[];
    __shared__ PassShared sh;
    pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_it = P.n_layers + P.has_tail;
    const uint32_t x_bytes = (uint32_t)P.m_pad * 128u, stage_bytes = A_BYTES + x_bytes;
    const uint32_t ring0 = (smem_u32(dyn) + PROG_BYTES + 1023u) & ~1023u;
    uint8_t* attn_smem = dyn + (ring0 - smem_u32(dyn)) + (size_t)P.stages * stage_bytes;
    const Abort ab{&sh.abort_flag, P.abort_word};

    // the CTA's section of the program (uploaded long before the launch) -> shared memory
    {
        const uint32_t* table = reinterpret_cast<const uint32_t*>(P.program);
        const uint32_t o0 = table[blockIdx.x], o1 = table[blockIdx.x + 1];
        const uint4* src = reinterpret_cast<const uint4*>(P.program + o0);
        uint4* dst = reinterpret_cast<uint4*>(dyn);
        for (uint32_t i = threadIdx.x; i < (o1 - o0) / 16u && i < PROG_BYTES / 16u; i += NUM_THREADS) dst[i] = src[i];
    }
    // rows of the narrow operand beyond the pass's rows stay zero for the whole launch
    for (uint32_t i = threadIdx.x; i < (uint32_t)P.stages * (x_bytes / 16u); i += NUM_THREADS) {
        const uint32_t s = i / (x_bytes / 16u), o = i % (x_bytes / 16u);
        *reinterpret_cast<uint4*>(dyn + (ring0 - smem_u32(dyn)) + (size_t)s * stage_bytes + A_BYTES + (size_t)o * 16) = make_uint4(0, 0, 0, 0);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    const int n_acc = max(2, min(MAX_ACC, 512 / P.m_pad));
    uint32_t tmem_cols = 32;
    while (tmem_cols < (uint32_t)(n_acc * P.m_pad)) tmem_cols <<= 1;
    if (threadIdx.x == 0) {
        for (int s = 0; s < P.stages; ++s) {
            mbar_init(smem_u32(&sh.full[s]), 2);           // the weight block and the input rows arrive from two producers
            mbar_init(smem_u32(&sh.empty[s]), 1);
        }
        for (int b = 0; b < n_acc; ++b) { mbar_init(smem_u32(&sh.tmem_full[b]), 1); mbar_init(smem_u32(&sh.tmem_empty[b]), 4); }
        sh.abort_flag = 0; sh.epi_abort = 0; sh.aux_flag = 0;
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
    Program pg;
    {
        const PassCtaHeader* h = reinterpret_cast<const PassCtaHeader*>(dyn);
        for (int k = 0; k < 2; ++k) {
            pg.segs[k] = reinterpret_cast<const PassSeg*>(dyn + h->seg_off[k]);
            pg.tasks[k] = reinterpret_cast<const PassTask*>(dyn + h->task_off[k]);
            pg.n_seg[k] = (int)h->n_seg[k]; pg.n_task[k] = (int)h->n_task[k];
        }
        pg.pieces = reinterpret_cast<const uint16_t*>(dyn + h->piece_off);
    }

    if (warp == 0) {
        // ------------------------------------------------------------------ weight producer: never waits for anything but a free stage
        if (lane == 0) {
            uint64_t pol_stream;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            int stage = 0; uint32_t use = 0; bool ok = true;
            for (int it = 0; it < n_it && ok; ++it) {
                const int k = it == P.n_layers ? 1 : 0, z = k ? 0 : it;
                for (int si = 0; si < pg.n_seg[k] && ok; ++si) {
                    const PassSeg sg = pg.segs[k][si];
                    const CUtensorMap* map = reinterpret_cast<const CUtensorMap*>(&maps.m[sg.mat]);
                    for (int j = 0; j < (int)sg.n_kb; ++j) {
                        if (use > 0u && !mbar_wait_b(smem_u32(&sh.empty[stage]), (use & 1u) ^ 1u, ab)) { ok = false; break; }
                        const uint32_t bar = smem_u32(&sh.full[stage]);
                        mbar_expect_tx(bar, A_BYTES);
                        tma_load_3d(ring0 + stage * stage_bytes, map, ((int)sg.kb0 + j) * TILE_K, (int)sg.tile * TILE_N, z, bar, pol_stream);
                        ring_next(stage, use, P.stages);
                    }
                }
            }
        }
    } else if (warp == 2 || warp == 3) {
        // ------------------------------------------------------------------ input-row producers: tagged words -> operand rows of the stages
        pdl_wait();                                           // the first rows (and the epoch) come from the kernels before this one
        const uint32_t epoch = *reinterpret_cast<const volatile uint32_t*>(P.epoch);
        uint8_t* ring = dyn + (ring0 - smem_u32(dyn));
        if (P.m_tok <= 8) produce_rows<4, 8>(P, sh, pg, epoch, n_it, ring, stage_bytes, ab, lane, warp - 2, 2);
        else if (P.m_tok <= 16) produce_rows<2, 16>(P, sh, pg, epoch, n_it, ring, stage_bytes, ab, lane, warp - 2, 2);
        else produce_rows<1, 32>(P, sh, pg, epoch, n_it, ring, stage_bytes, ab, lane, warp - 2, 2);
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(P.m_pad >> 3) << 17) | ((uint32_t)(TILE_N >> 4) << 24);
            const uint64_t desc0 = umma_desc(ring0);
            int stage = 0; uint32_t use = 0, acc_phase = 0; bool ok = true;       // acc_phase: bit a = parity of accumulator a's uses so far
            for (int it = 0; it < n_it && ok; ++it) {
                const int k = it == P.n_layers ? 1 : 0;
                for (int si = 0; si < pg.n_seg[k] && ok; ++si) {
                    const PassSeg sg = pg.segs[k][si];
                    const int n_kb = (int)sg.n_kb;
                    const uint32_t acc = (uint32_t)sg.flags >> 4;
                    const uint32_t cont = (sg.flags & SEG_FIRST) ? 0u : 1u;           // 0: the segment starts a fresh accumulator
                    unsigned long long* stamp = P.stamps ? P.stamps + (((size_t)blockIdx.x * n_it + it) * P.stamp_segs + si) * 2 : nullptr;
                    if (!cont) {                                                       // ... once the epilogue has drained its last use
                        if (!mbar_wait_b(smem_u32(&sh.tmem_empty[acc]), ((acc_phase >> acc) & 1u) ^ 1u, ab)) { ok = false; break; }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    }
                    if (stamp) stamp[0] = global_ns();
                    const uint32_t d_tmem = tmem_base + acc * (uint32_t)P.m_pad;
                    for (int j = 0; j < n_kb; ++j) {
                        if (!mbar_wait_b(smem_u32(&sh.full[stage]), use & 1u, ab)) { ok = false; break; }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint64_t da = desc0 + (uint64_t)((uint32_t)stage * (stage_bytes >> 4)), db = da + (A_BYTES >> 4);
#pragma unroll
                        for (uint32_t kk = 0; kk < TILE_K / 16; ++kk)
                            umma_bf16(d_tmem, da + 2 * kk, db + 2 * kk, idesc, cont | (uint32_t)j | kk);
                        umma_commit(smem_u32(&sh.empty[stage]));
                        ring_next(stage, use, P.stages);
                    }
                    if (ok && (sg.flags & SEG_LAST)) { umma_commit(smem_u32(&sh.tmem_full[acc])); acc_phase ^= 1u << acc; }
                    if (stamp) stamp[1] = global_ns();
                }
            }
        }
    } else if (warp >= 4 && warp < 8) {
        // ------------------------------------------------------------------ TMEM -> workspace: the CTA's piece of a tile, as tagged words
        const uint32_t quarter = (uint32_t)(warp & 3);
        const int et = quarter * 32 + lane;
        pdl_wait();
        const uint32_t epoch = *reinterpret_cast<const volatile uint32_t*>(P.epoch);
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int it = 0; it < n_it && ok; ++it) {
            const int k = it == P.n_layers ? 1 : 0;
            for (int si = 0; si < pg.n_seg[k]; ++si) {
                const PassSeg sg = pg.segs[k][si];
                if (!(sg.flags & SEG_LAST)) continue;             // the accumulator goes on in a later segment
                const uint32_t acc = (uint32_t)sg.flags >> 4;
                const uint32_t tag = pass_tag(epoch, it, (sg.mat == MAT_GU || sg.mat == MAT_DN) ? USE_B : USE_A);
                if (!mbar_wait_b(smem_u32(&sh.tmem_full[acc]), (acc_phase >> acc) & 1u, ab)) sh.epi_abort = 1;
                acc_phase ^= 1u << acc;
                epi_bar();
                if (sh.epi_abort) { ok = false; break; }      // all four warps leave together
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                tagged_t* out = P.partials[sg.mat & 1] + (size_t)sg.slot * P.m_tok * TILE_N;
                for (int c0 = 0; c0 < P.m_pad; c0 += 16) {
                    uint32_t r[16];
                    tmem_ld16(tmem_base + ((quarter * 32u) << 16) + acc * (uint32_t)P.m_pad + (uint32_t)c0, r);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (c0 + j < P.m_tok) stq(out + (size_t)(c0 + j) * TILE_N + et, r[j], tag);
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.tmem_empty[acc]));
            }
        }
    } else if (warp >= 8) {
        // ------------------------------------------------------------------ tasks: sum finished tiles, attention
        const int t = threadIdx.x - 256;
        pdl_wait();
        const uint32_t epoch = *reinterpret_cast<const volatile uint32_t*>(P.epoch);
        for (int it = 0; it < n_it; ++it) {
            const int k = it == P.n_layers ? 1 : 0;
            for (int ti = 0; ti < pg.n_task[k]; ++ti) {
                const PassTask tk = pg.tasks[k][ti];
                unsigned long long* ts = (P.task_stamps && ti < P.stamp_tasks) ? P.task_stamps + (((size_t)blockIdx.x * n_it + it) * P.stamp_tasks + ti) * 2 : nullptr;
                if (ts && t == 0) ts[0] = global_ns();
                // (after a wait has given up, the remaining tasks return at their own waits: every branch here is taken by all 128 threads)
                if (tk.kind == TASK_REDUCE) reduce_task(P, sh, tk, pg.pieces + tk.piece0, it, epoch, ab, t);
                else if (P.hd == 128) attention_task<128>(P, sh, attn_smem, tk, it, epoch, ab, t);
                else attention_task<64>(P, sh, attn_smem, tk, it, epoch, ab, t);
                if (ts && t == 0) ts[1] = global_ns();
            }
        }
    }

    // ---------------------------------------------------------------------- wind-down
    __syncwarp();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0) sh.aux_flag = (sh.abort_flag != 0 || *ab.global != 0u) ? 1 : 0;
    __syncthreads();
    if (sh.aux_flag) {
        if (threadIdx.x == 0 && P.status) atomicOr(P.status, SD_DEV_WAIT_EXPIRED);
        const uint64_t t0 = global_ns();                       // let copies in flight land before the CTA goes away
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
EncodeTiledFn encode_fn3() {
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

// bf16 matrices [n_layers][rows][K], consecutive layers layer_stride_bytes apart, as a 3-D tensor map with
// boxes of 128 rows x 64 elements, 128-byte swizzle; reads outside a matrix return zeros.
bool make_tensor_map_layers(TensorMap* out, const void* base, int rows, int K, int n_layers, size_t layer_stride_bytes) {
    EncodeTiledFn fn = encode_fn3();
    if (!fn || ((uintptr_t)base & 15) || (K & 7) || n_layers < 1 || (layer_stride_bytes & 15)) return false;
    if (n_layers == 1) layer_stride_bytes = ((size_t)rows * K * 2 + 15) & ~(size_t)15;
    cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)n_layers};
    cuuint64_t strides[2] = {(cuuint64_t)K * 2, (cuuint64_t)layer_stride_bytes};
    cuuint32_t box[3] = {(cuuint32_t)TILE_K, (cuuint32_t)TILE_N, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {
__global__ void k_pass_begin(uint32_t* epoch, uint32_t* abort_word) { *epoch = *epoch + 1u; *abort_word = 0u; }
}  // namespace

cudaError_t launch_pass_begin(uint32_t* epoch, uint32_t* abort_word, cudaStream_t st) {
    k_pass_begin<<<1, 1, 0, st>>>(epoch, abort_word);
    return cudaGetLastError();
}

size_t pass_stream_smem(int m_pad, int* stages_out) {
    const int stage_bytes = A_BYTES + m_pad * 128;
    const int stages = std::max(2, std::min(MAX_STAGES, RING_BUDGET / stage_bytes));
    if (stages_out) *stages_out = stages;
    return (size_t)PROG_BYTES + 1024 + (size_t)stages * stage_bytes + ATTN_BYTES;
}

cudaError_t launch_pass_stream(const PassMaps& maps, const PassParams& p, int grid, int dependent, cudaStream_t st) {
    int stages = 0;
    const size_t smem = pass_stream_smem(p.m_pad, &stages);
    if (p.stages < 2 || p.stages > stages || p.m_pad < 16 || p.m_pad > 256 || (p.m_pad & 15) || p.m_tok > p.m_pad || grid < 1) return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(k_pass_stream, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_pdl(k_pass_stream, dim3(grid), dim3(NUM_THREADS), smem, st, dependent, maps, p);
}

}  // namespace sd
