// The step that follows each weight GEMM of a decoder layer, fused with the reduction of the
// GEMM's split accumulators: one small CTA per (128-row output tile, batch of token rows) adds
// the pieces of the tile in the fixed order of the CTAs that produced them (run-to-run identical
// results) and applies, in the same pass,
//   QKV      -> 1/rms factor -> rotary embedding -> query buffer / KV-cache append (bf16),
//   Wo, down -> residual add -> next norm's operand h * gain in bf16 + the tile's share of sum h^2,
//   gate/up  -> 1/rms factor -> SwiGLU (gate and up rows of a feature sit in one tile),
//   lm_head  -> 1/rms factor -> fp32 logits,
// so that no fp32 intermediate matrix goes through memory.  It runs as a programmatic dependent
// of the GEMM: its CTAs are resident (and hold only a few KB) while the GEMM streams, the GEMM's
// CTAs leave their SMs as soon as their pieces are written, and the next GEMM's CTAs take those
// SMs and start streaming weights while this kernel is still working.  Everything a CTA needs
// is requested in one round of loads.
#include "gemm_tc.h"

namespace sd {

namespace {

constexpr int TILE_N = 128;


template <int MB>
struct StepShared {
    float scale[MB];                // 1/rms factor of the CTA's token rows
    float val[MB][TILE_N];          // exchange between the rows of the tile (rotary pairs, gate/up pairs)
    float wsum[MB][4];              // per-warp sums of squares
    float lora_t[MB][32];           // x A^T of the CTA's token rows for their own adapters
};

// MB token rows x CB pieces are in flight together: (8, 8) for the verify rows, (2, 32) for one or
// two rows (draft steps), where a tile of a small matrix is cut into many pieces, (16, 4) or (16, 2)
// for many rows on few pieces.  MODE < 0: the step is read from ep.mode; with many row batches one
// instantiation per step is used instead, whose lower register count lets more CTAs be resident.
// LORA: the matrix carries low-rank adapters.  XR: the CTA counts into a word of its tile when its outputs are written
// (tile-by-tile hand-off of token rows to the next GEMM: an opt-in measurement path, compiled for the eight-row form only).
template <int MODE, int MB, int CB, bool HL = false, bool LORA = false, bool XR = false>
__global__ void __launch_bounds__(128) k_fused_step(GemmGeom g, Epilogue ep, const float* __restrict__ partials,
                                                    uint32_t* __restrict__ arrive, uint32_t* status) {
    __shared__ StepShared<MB> sh;
    const int mode = MODE < 0 ? ep.mode : MODE;
    pdl_launch_dependents();
    const int et = threadIdx.x, lane = et & 31, warp = et >> 5;
    if (et == 0) stamp_first(ep.stamp, ST_START);
    const uint32_t tile = blockIdx.x;
    const int m0 = blockIdx.y * MB;
    const int n = (int)tile * TILE_N + et;
    const bool live = n < g.n_out;
    // first and last CTA of the GEMM that hold a piece of this tile, and which of its pieces the first one gave
    const uint32_t KB = (uint32_t)g.kb_per_tile, T = (uint32_t)g.n_tiles * KB, G = (uint32_t)g.grid;
    const uint32_t ua = tile * KB, ub = ua + KB - 1;
    const uint32_t i_first = ((ua + 1) * G + T - 1) / T - 1;      // T * G < 2^32 (checked on the host)
    const uint32_t i_last = ((ub + 1) * G + T - 1) / T - 1;
    const uint32_t j_first = tile - ((i_first * T) / G) / KB;
    const int n_rows = mode == EPI_PLAIN ? ep.n_out_rows : (HL ? ep.m_real : g.m_tok);
    int rows[MB];
#pragma unroll
    for (int i = 0; i < MB; ++i) {
        const int r = m0 + i;
        rows[i] = r < n_rows ? (mode == EPI_PLAIN ? r * ep.row_stride + ep.row_offset : r) : -1;
    }
    const float gain = (mode == EPI_RESIDUAL && ep.gain_next && live) ? ep.gain_next[n] : 0.f;   // a weight: needs no wait
    // The row plan and the rows' rotary factors were written by the pass's first kernel, an ordinary launch that every
    // later kernel of the pass started after: they need no wait either.
    float cs[MB], sn[MB];
    int pos[MB], slot[MB];
    if (mode == EPI_QKV_ROPE) {
        const int half = ep.hd >> 1, e = n % ep.hd, head = n / ep.hd;
        const bool lower = live && e < half, rot = head < ep.H + ep.Hkv;
#pragma unroll
        for (int i = 0; i < MB; ++i) {
            const bool ok = lower && rows[i] >= 0;
            pos[i] = ok ? __ldcg(ep.row_pos + rows[i]) : -1;
            slot[i] = (ok && head >= ep.H) ? __ldcg(ep.row_slot + rows[i]) : 0;
            cs[i] = (ok && rot) ? __ldcg(ep.rcos + (size_t)rows[i] * half + e) : 1.f;     // per-row rotary factors (the row's position applied)
            sn[i] = (ok && rot) ? __ldcg(ep.rsin + (size_t)rows[i] * half + e) : 0.f;
        }
    }
    int task[MB];                                 // the rows' adapters (part of the row plan: no wait needed)
    uint4 braw[MB <= 2 ? MB : 1][MB <= 2 ? 4 : 1];  // one or two rows: their rows of B are requested before the wait as well
    if (LORA) {
#pragma unroll
        for (int i = 0; i < MB; ++i) {
            task[i] = rows[i] >= 0 ? __ldcg(ep.lora_task + rows[i]) : -1;
            if (task[i] >= ep.lora_n) task[i] = -1;
            if (MB <= 2 && live && task[i] >= 0) {
                const bf16* b = ep.lora_b + ((size_t)task[i] * g.n_out + n) * ep.lora_r;
#pragma unroll
                for (int jj = 0; jj < 4; ++jj)
                    if (jj * 8 < ep.lora_r) braw[MB <= 2 ? i : 0][MB <= 2 ? jj : 0] = __ldg(reinterpret_cast<const uint4*>(b + jj * 8));
            }
        }
    }
    // The pieces come from the GEMM before (the rows' sums of squares from kernels further back, long finished).
    // With arrival words the CTA starts as soon as its own tile is complete; otherwise when the GEMM's grid has retired.
    if (arrive) {
        // every warp watches the tile's word for itself (one request per warp and poll): no barrier between the arrival
        // of the last piece and the loads below
        const uint32_t need = i_last - i_first + 1u;
        uint32_t seen = 0;
        const uint64_t t0 = global_ns(), limit = ep.poll_ns ? ep.poll_ns : 200000000ull;
        for (uint32_t spin = 0;; ++spin) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(arrive + tile) : "memory");
            if (seen >= need) break;
            if ((spin & 63u) == 63u && global_ns() - t0 > limit) break;      // (0.2 s unless told otherwise): give up polling
        }
        if (seen < need) {                         // not expected: wait for the whole grid instead, and say so
            pdl_wait();
            if (lane == 0 && status) atomicOr(status, SD_DEV_WAIT_EXPIRED);
        }
    } else {
        pdl_wait();
    }

    if (et == 0) stamp_pair(ep.stamp, ST_DEP_FIRST);

    // ---- one round of loads: (adapters: the pieces of x A^T,) sums of squares, residual / row plan / rotary factors, the pieces
    // t = x A^T sits in the GEMM's last tile; its pieces are summed like any tile's, by MB * r threads.  The first four
    // pieces of every sum are requested here, ahead of the tile's own pieces, so that both come back in the same round.
    // (one or two rows only: with more rows per CTA the extra registers cost more than the round trip saves)
    constexpr bool LPRE = LORA && MB <= 2;
    constexpr int LNP = LPRE ? (MB * 32 + 127) / 128 : 1;
    float tl[LNP][4];
    uint32_t x_first = 0, x_last = 0, xj_first = 0;
    auto lora_tile = [&]() {                      // which CTAs of the GEMM hold pieces of its last tile
        const uint32_t tx = (uint32_t)g.n_tiles - 1u, xa = tx * KB, xb = xa + KB - 1;
        x_first = ((xa + 1) * G + T - 1) / T - 1; x_last = ((xb + 1) * G + T - 1) / T - 1;
        xj_first = tx - ((x_first * T) / G) / KB;
    };
    if (LPRE) {
        lora_tile();
        const int r = ep.lora_r;
#pragma unroll
        for (int pp = 0; pp < LNP; ++pp) {
            const int p = et + pp * 128, i = p / r, j = p % r, row = m0 + i;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) tl[pp][cc] = 0.f;
            if (LPRE && p < MB * r && row < n_rows) {
                const int tk = __ldcg(ep.lora_task + row);
                if (tk >= 0 && tk < ep.lora_n) {
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        const uint32_t c = x_first + cc, jj = cc == 0 ? xj_first : 0u;
                        if (c <= x_last) tl[pp][cc] = __ldcg(partials + ((size_t)c * g.max_seg + jj) * g.m_pad * TILE_N + (size_t)row * TILE_N + tk * r + j);
                    }
                }
            }
        }
    }
    float ssa[(MB + 3) / 4], ssb[(MB + 3) / 4];
    if (ep.rs.ssq) {                              // one warp per token row, one lane per piece of its sum of squares
#pragma unroll
        for (int ii = 0; ii < (MB + 3) / 4; ++ii) {
            const int i = warp + 4 * ii, r = m0 + i;
            const bool ok = i < MB && r < n_rows;
            const float* ps = ep.rs.ssq + (size_t)(ok ? (mode == EPI_PLAIN ? r * ep.row_stride + ep.row_offset : r) : 0) * SSQ_STRIDE;
            ssa[ii] = (ok && lane < ep.rs.n_parts) ? __ldcg(ps + lane) : 0.f;
            ssb[ii] = (ok && lane + 32 < ep.rs.n_parts) ? __ldcg(ps + lane + 32) : 0.f;
        }
    }
    float hv[MB];
    if (mode == EPI_RESIDUAL) {
#pragma unroll
        for (int i = 0; i < MB; ++i) hv[i] = (live && rows[i] >= 0) ? __ldcg(ep.h + (size_t)rows[i] * g.n_out + n) : 0.f;
    }
    float v[MB];
#pragma unroll
    for (int i = 0; i < MB; ++i) v[i] = 0.f;
    if (live) {
        for (uint32_t c0 = i_first; c0 <= i_last; c0 += CB) {
            float tmp[CB][MB];
#pragma unroll
            for (int cc = 0; cc < CB; ++cc) {
                const uint32_t c = c0 + cc;
                const bool ok = c <= i_last;
                const uint32_t j = c == i_first ? j_first : 0u;              // later CTAs start inside the tile: their first piece
                const float* base = partials + ((size_t)c * g.max_seg + j) * g.m_pad * TILE_N + et;
#pragma unroll
                for (int i = 0; i < MB; ++i) {
                    tmp[cc][i] = (ok && rows[i] >= 0) ? __ldcg(base + (size_t)rows[i] * TILE_N) : 0.f;
                }
            }
#pragma unroll
            for (int cc = 0; cc < CB; ++cc)                                   // the pieces are added in the order of their CTAs
#pragma unroll
                for (int i = 0; i < MB; ++i) v[i] += tmp[cc][i];
        }
    }
    if (LORA) {                                   // the low-rank update of this matrix
        const int r = ep.lora_r;
        if (!LPRE) {
            lora_tile();
            for (int p = et; p < MB * r; p += 128) {
                const int i = p / r, j = p % r, row = m0 + i;
                float t = 0.f;
                if (row < n_rows) {
                    const int tk = __ldcg(ep.lora_task + row);
                    if (tk >= 0 && tk < ep.lora_n) {
                        for (uint32_t c = x_first; c <= x_last; ++c) {
                            const uint32_t jj = c == x_first ? xj_first : 0u;
                            t += __ldcg(partials + ((size_t)c * g.max_seg + jj) * g.m_pad * TILE_N + (size_t)row * TILE_N + tk * r + j);
                        }
                    }
                }
                sh.lora_t[i][j] = t;
            }
        }
#pragma unroll
        for (int pp = 0; pp < LNP; ++pp) {
            const int p = et + pp * 128, i = p / r, j = p % r, row = m0 + i;
            if (LPRE && p < MB * r) {
                float t = (tl[pp][0] + tl[pp][1]) + (tl[pp][2] + tl[pp][3]);
                if (x_last > x_first + 3u && row < n_rows) {      // a tile cut into more than four pieces (small matrices on many SMs)
                    const int tk = __ldcg(ep.lora_task + row);
                    if (tk >= 0 && tk < ep.lora_n)
                        for (uint32_t c = x_first + 4u; c <= x_last; ++c)
                            t += __ldcg(partials + ((size_t)c * g.max_seg) * g.m_pad * TILE_N + (size_t)row * TILE_N + tk * r + j);
                }
                sh.lora_t[i][j] = t;
            }
        }
        __syncthreads();
        if (live) {
#pragma unroll
            for (int i = 0; i < MB; ++i) {
                if (rows[i] < 0 || task[i] < 0) continue;
                const bf16* b = ep.lora_b + ((size_t)task[i] * g.n_out + n) * r;
                float acc = 0.f;
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {                 // r is a multiple of 8, at most 32: 16-byte pieces of the row of B
                    const int j = jj * 8;
                    if (j >= r) break;
                    const uint4 raw = MB <= 2 ? braw[MB <= 2 ? i : 0][MB <= 2 ? jj : 0] : __ldg(reinterpret_cast<const uint4*>(b + j));
                    const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __bfloat1622float2(h2[e]);
                        acc = fmaf(sh.lora_t[i][j + 2 * e], f.x, acc);
                        acc = fmaf(sh.lora_t[i][j + 2 * e + 1], f.y, acc);
                    }
                }
                v[i] = fmaf(ep.lora_scale, acc, v[i]);
            }
        }
    }
    if (ep.rs.ssq) {
#pragma unroll
        for (int ii = 0; ii < (MB + 3) / 4; ++ii) {
            const int i = warp + 4 * ii;
            const float ss = warp_sum(ssa[ii] + ssb[ii]);
            if (lane == 0 && i < MB) sh.scale[i] = rsqrtf(ss * ep.rs.inv_d + ep.rs.eps);
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < MB; ++i) v[i] *= sh.scale[i];
    }

    switch (mode) {
    case EPI_PLAIN: {
        if (live) {
#pragma unroll
            for (int i = 0; i < MB; ++i) if (rows[i] >= 0) ep.y[(size_t)(m0 + i) * g.n_out + n] = v[i];
        }
        break;
    }
    case EPI_QKV_ROPE: {
        const int hd = ep.hd, half = hd >> 1, head = n / hd, e = n % hd;
        const bool rot = head < ep.H + ep.Hkv;
#pragma unroll
        for (int i = 0; i < MB; ++i) sh.val[i][et] = v[i];
        __syncthreads();
#pragma unroll
        for (int i = 0; i < MB; ++i) {
            if (pos[i] < 0) continue;
            const float a = v[i], b = sh.val[i][et + half];
            const float ra = a * cs[i] - b * sn[i], rb = a * sn[i] + b * cs[i];
            bf16* dst;
            if (head < ep.H) dst = ep.q_out + ((size_t)rows[i] * ep.H + head) * hd;
            else {
                const int kvh = (head - ep.H) % ep.Hkv;
                bf16* base = rot ? ep.kc : ep.vc;
                dst = base + (((size_t)slot[i] * ep.Hkv + kvh) * ep.max_ctx + pos[i]) * hd;
            }
            dst[e] = __float2bfloat16_rn(ra);
            dst[e + half] = __float2bfloat16_rn(rb);
        }
        break;
    }
    case EPI_RESIDUAL: {
        const int d = g.n_out;
#pragma unroll
        for (int i = 0; i < MB; ++i) {
            hv[i] += v[i];
            if (live && rows[i] >= 0) {
                ep.h[(size_t)rows[i] * d + n] = hv[i];
                if (ep.gain_next) {
                    const float x = hv[i] * gain;
                    const bf16 hi = __float2bfloat16_rn(x);
                    ep.xn[(size_t)rows[i] * d + n] = hi;
                    if (HL) ep.xn[(size_t)(rows[i] + ep.lo_off) * d + n] = __float2bfloat16_rn(x - __bfloat162float(hi));
                }
            }
        }
        if (ep.gain_next) {
#pragma unroll
            for (int i = 0; i < MB; ++i) {
                const float ss = warp_sum(hv[i] * hv[i]);
                if (lane == 0) sh.wsum[i][warp] = ss;
            }
            __syncthreads();
            if (et < MB && m0 + et < n_rows) {
                const float* w = sh.wsum[et];
                ep.ssq_out[(size_t)(m0 + et) * SSQ_STRIDE + tile] = (w[0] + w[1]) + (w[2] + w[3]);
            }
        }
        break;
    }
    case EPI_SWIGLU: {
        const int f = (int)tile * 64 + et;
#pragma unroll
        for (int i = 0; i < MB; ++i) sh.val[i][et] = v[i];
        __syncthreads();
        if (et < 64 && f < ep.F) {
#pragma unroll
            for (int i = 0; i < MB; ++i) {
                if (rows[i] < 0) continue;
                const float gt = v[i], up = sh.val[i][et + 64];
                const float x = gt / (1.f + expf(-gt)) * up;
                const bf16 hi = __float2bfloat16_rn(x);
                ep.act[(size_t)rows[i] * ep.F + f] = hi;
                if (HL) ep.act[(size_t)(rows[i] + ep.lo_off) * ep.F + f] = __float2bfloat16_rn(x - __bfloat162float(hi));
            }
        }
        break;
    }
    default: break;
    }
    if (et == 0) stamp_pair(ep.stamp, ST_DONE_FIRST);
    if (arrive) {                                 // left at zero for the next pass (every warp is past its polls by now)
        __syncthreads();
        if (et == 0) arrive[tile] = 0u;
    }
    if (XR && ep.xready) {                        // everything this CTA writes is written: the next GEMM may load the tile's columns
        __syncthreads();                          // (orders the CTA's stores before thread 0's release, which is cumulative)
        if (et == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(ep.xready + tile) : "memory");
    }
}

template <int MODE, bool HL, bool LORA>
cudaError_t launch_many_rows(const GemmGeom& g, const Epilogue& ep, const float* partials, uint32_t* arrive, uint32_t* status, int n_rows,
                             int pieces, int dependent, cudaStream_t st) {
    const dim3 grid(g.n_tiles, (n_rows + 15) / 16);
    // Two pieces per round unless told otherwise: with three or four pieces that is one more round of loads, but the
    // kernel then needs 80-128 registers instead of 128-212, a whole step fits the SMs in one wave of CTAs, and the
    // batched configurations run 1.4-2.5 % faster.
    if (pieces <= 2 || ep.many_rows_cb != 4) return launch_pdl(k_fused_step<MODE, 16, 2, HL, LORA>, grid, dim3(128), 0, st, dependent, g, ep, partials, arrive, status);
    return launch_pdl(k_fused_step<MODE, 16, 4, HL, LORA>, grid, dim3(128), 0, st, dependent, g, ep, partials, arrive, status);
}

}  // namespace

namespace {

// Pieces per tile, at most: a tile's k blocks over the k blocks a CTA of the GEMM owns.
int pieces_bound(const GemmGeom& g) {
    const long long T = (long long)g.n_tiles * g.kb_per_tile;
    const int per_cta = (int)std::max<long long>(1, T / g.grid);
    return (g.kb_per_tile + per_cta - 1) / per_cta + 1;
}

// Token rows per CTA of the form launch_fused_step picks.
int rows_per_cta(int n_rows, int pieces) { return n_rows <= 2 ? 2 : (n_rows > 8 && pieces <= 4 ? 16 : 8); }

}  // namespace

int fused_step_row_batches(const GemmGeom& g, const Epilogue& ep) {
    const int n_rows = ep.mode == EPI_PLAIN ? ep.n_out_rows : (ep.lo_off ? ep.m_real : g.m_tok);
    if (n_rows <= 2) return 1;
    const int mb = (n_rows > 8 && pieces_bound(g) <= 4) ? 16 : 8;
    return (n_rows + mb - 1) / mb;
}

bool fused_step_polls(const GemmGeom& g, const Epilogue& ep) {
    // One batch of rows per tile (several would share a tile's word).  With one or two rows (draft and plain
    // decoding steps: small matrices, kernels of several GEMMs resident and polling at once) waiting for the
    // grid measured faster.
    const int n_rows = ep.mode == EPI_PLAIN ? ep.n_out_rows : (ep.lo_off ? ep.m_real : g.m_tok);
    return g.grid >= 1 && n_rows > 2 && n_rows <= rows_per_cta(n_rows, pieces_bound(g));
}

namespace {

template <bool HL, bool LORA>
cudaError_t launch_step(const GemmGeom& g, const Epilogue& ep, const float* partials, uint32_t* arrive, uint32_t* status, int n_rows, int pieces,
                        int dependent, cudaStream_t st) {
    if (n_rows <= 2) return launch_pdl(k_fused_step<-1, 2, 32, HL, LORA>, dim3(g.n_tiles, 1), dim3(128), 0, st, dependent, g, ep, partials, arrive, status);
    if (n_rows > 8 && pieces <= 4) {
        switch (ep.mode) {
        case EPI_PLAIN: return launch_many_rows<EPI_PLAIN, HL, LORA>(g, ep, partials, arrive, status, n_rows, pieces, dependent, st);
        case EPI_QKV_ROPE: return launch_many_rows<EPI_QKV_ROPE, HL, LORA>(g, ep, partials, arrive, status, n_rows, pieces, dependent, st);
        case EPI_RESIDUAL: return launch_many_rows<EPI_RESIDUAL, HL, LORA>(g, ep, partials, arrive, status, n_rows, pieces, dependent, st);
        case EPI_SWIGLU: return launch_many_rows<EPI_SWIGLU, HL, LORA>(g, ep, partials, arrive, status, n_rows, pieces, dependent, st);
        default: return cudaErrorInvalidValue;
        }
    }
    if (ep.xready && !LORA)
        return launch_pdl(k_fused_step<-1, 8, 8, HL, false, true>, dim3(g.n_tiles, (n_rows + 7) / 8), dim3(128), 0, st, dependent, g, ep, partials, arrive, status);
    return launch_pdl(k_fused_step<-1, 8, 8, HL, LORA>, dim3(g.n_tiles, (n_rows + 7) / 8), dim3(128), 0, st, dependent, g, ep, partials, arrive, status);
}

}  // namespace

cudaError_t launch_fused_step(const GemmGeom& g, const Epilogue& ep, const float* partials, uint32_t* arrive, uint32_t* status,
                              int dependent, cudaStream_t st) {
    if (g.grid < 1 || g.m_tok > SD_MAX_ROWS) return cudaErrorInvalidValue;
    if (!fused_step_polls(g, ep)) arrive = nullptr;
    if (ep.mode == EPI_QKV_ROPE && (128 % ep.hd)) return cudaErrorInvalidValue;            // a head must not straddle two tiles
    if (ep.mode == EPI_RESIDUAL && g.n_tiles > SSQ_STRIDE) return cudaErrorInvalidValue;
    if (ep.mode == EPI_SWIGLU && (ep.F % 64)) return cudaErrorInvalidValue;
    if (ep.rs.ssq && ep.rs.n_parts > 64) return cudaErrorInvalidValue;
    if (ep.lora_b) {                                   // the adapter's tile is complete only when the GEMM's grid is
        if (ep.lora_r < 8 || ep.lora_r > 32 || (ep.lora_r & 7) || ep.lora_n * ep.lora_r > TILE_N || !ep.lora_task ||
            ep.mode == EPI_PLAIN || g.n_out % TILE_N || g.n_tiles != g.n_out / TILE_N + 1)
            return cudaErrorInvalidValue;
        arrive = nullptr;
    }
    const int n_rows = ep.mode == EPI_PLAIN ? ep.n_out_rows : (ep.lo_off ? ep.m_real : g.m_tok);
    const int pieces = pieces_bound(g);
    if (ep.lo_off) {                                   // two-part activations: accumulator rows r and r + lo_off belong together
        // (the GEMM's epilogue has already added the two columns of a row: the pieces hold m_real merged rows)
        if (ep.m_real < 1 || ep.m_real > ep.lo_off || ep.m_real + ep.lo_off != g.m_tok || g.lo_off != ep.lo_off || g.m_real != ep.m_real) return cudaErrorInvalidValue;
        if (ep.lo_off != 8 && ep.lo_off != 16) return cudaErrorInvalidValue;
        return ep.lora_b ? launch_step<true, true>(g, ep, partials, arrive, status, n_rows, pieces, dependent, st)
                         : launch_step<true, false>(g, ep, partials, arrive, status, n_rows, pieces, dependent, st);
    }
    return ep.lora_b ? launch_step<false, true>(g, ep, partials, arrive, status, n_rows, pieces, dependent, st)
                     : launch_step<false, false>(g, ep, partials, arrive, status, n_rows, pieces, dependent, st);
}

}  // namespace sd
