// Split-KV attention for the verify / draft rows (bf16 cache, head_dim 64 or 128) on the
// warp-level tensor-core path (mma.sync m16n8k16, bf16 in, fp32 accumulate).
//
// A block of consecutive query rows of one sequence (the gamma+1 verify rows) times the query
// heads that share one KV head is scored against one slice of that head's cache; every slice
// is streamed from HBM once, whatever the number of rows.  Slices leave unnormalised partial
// outputs with their running max and sum; the CTA whose slice arrives last (an arrival
// counter, nothing spins) merges them.
// Cache layout of one layer: [slot][kv_head][position][head_dim].
#include <cooperative_groups.h>

#include "gemm_tc.h"
#include "kernels.h"

namespace sd {

namespace {

// Warps per CTA: eight when there are few CTAs (each finishes its slice sooner), four when there are several
// per SM (three of them fit an SM, and one's set-up and merge overlap the others' streaming).
constexpr int WARPS_FEW = 8, WARPS_MANY = 4;
constexpr int NQ = 16;              // query vectors per CTA (rows in the block x heads per KV head): one MMA row tile
constexpr int SLICE_KEYS = 1024;    // a slice of the cache per CTA: up to this many positions
constexpr int SLICE_KEYS_MANY = 2048; // ... when there are several CTAs per SM anyway (fewer set-ups and merges; 512...8192 swept)
constexpr size_t ATTN_COUNTER_BYTES = 65536;     // one arrival counter per (query block, kv head)

struct AttnParams {
    const bf16* q; const bf16* kc; const bf16* vc;
    const int32_t* row_slot; const int32_t* row_pos;
    float* part_o;      // [rows][H][n_splits][hd] unnormalised partial outputs
    float* part_ml;     // [rows][H][n_splits][2] running max (log2 domain) and sum
    uint32_t* counters; // [query block][kv head]: slices that have delivered; zero between launches
    bf16* out;          // [rows][H][hd]
    int n_rows, rows_per_seq, rows_per_block, H, Hkv, max_ctx, n_splits;
    int csize;          // CTAs of a thread-block cluster that share one slice (1, 2 or 4)
    int lo_off;         // > 0: the output is also written as a second bf16 part (x - bf16(x)) lo_off rows further down
    unsigned long long* stamp;   // optional time stamps of the launch (see LaunchStamp)
    int use_order;               // sequences are taken in seq_order (longest context first: CTAs are handed out in grid order,
    unsigned char seq_order[64]; // and the sequence that takes longest should not be the one that starts last)
};

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16x8 fp32) += A (16x16 bf16, row) * B (16x8 bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// One CTA = one slice of one KV head's cache x the query rows of one block (times the query
// heads that share the KV head), as a 16-row tensor-core tile.  The slice is walked in chunks
// of 64 keys, double-buffered in shared memory (16-byte asynchronous copies into an
// XOR-swizzled layout that ldmatrix reads without bank conflicts); each warp owns 16 keys of a
// chunk and keeps its own running max / sum / output (online softmax, exp2 domain), the warps
// are merged at the end.  When there are few (head, row block, slice) items, two or four CTAs of
// a thread-block cluster share a slice and hand their results to the first one through
// distributed shared memory.  A context of up to SLICE_KEYS positions is one slice, whose output
// is written directly; longer contexts are cut into slices whose partial results are merged by
// whichever slice arrives last.
template <int HD, int NW>
__global__ void __launch_bounds__(32 * NW) k_attn_mma(AttnParams P) {
    constexpr int NT = 32 * NW;              // threads; each warp takes 16 of the keys of a chunk
    constexpr int CK = 16 * NW;              // keys per chunk
    extern __shared__ __align__(128) uint8_t sm_raw[];
    constexpr int ROWB = HD * 2;             // bytes of one key / value row
    constexpr int CPR = HD / 8;              // 16-byte pieces per row
    constexpr int KS = HD / 16;              // reduction steps of Q K^T
    constexpr int NV = HD / 8;               // 8-wide column tiles of the output
    constexpr int BUF = CK * ROWB;           // one chunk of keys (or values)
    constexpr int OLD = HD + 8;              // padded row of the cross-warp merge buffer (floats)
    pdl_launch_dependents();
    if (threadIdx.x == 0) stamp_first(P.stamp, ST_START);
    const int CS = P.csize;
    const int split = blockIdx.x / CS, crank = blockIdx.x % CS, kvh = blockIdx.y;
    const int group = P.H / P.Hkv;
    const int bps = (P.rows_per_seq + P.rows_per_block - 1) / P.rows_per_block;     // query blocks per sequence
    const int zseq = P.use_order ? (int)P.seq_order[blockIdx.z / bps] : (int)(blockIdx.z / bps);
    const int zb = zseq * bps + (int)(blockIdx.z % bps);                             // query block this CTA works on
    const int r0 = zseq * P.rows_per_seq + (zb % bps) * P.rows_per_block;
    const int nr = min(P.rows_per_block, P.rows_per_seq - (zb % bps) * P.rows_per_block);
    const int nq = nr * group;
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5, gid = lane >> 2, tig = lane & 3;
    const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(sm_raw);
    __shared__ int last_sm;

    // The row plan (positions, slots) was written by the pass's first kernel, an ordinary launch that every later
    // kernel of the pass started after: it may be read before the wait below, and so may the cache positions in
    // front of the pass's first new one, which earlier passes wrote.
    // longest context among the block's rows (every warp works it out for itself), and the sequence slot
    int mp = lane < nr ? __ldcg(P.row_pos + r0 + lane) : -1;
    const int slot = __ldcg(P.row_slot + r0);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mp = max(mp, __shfl_xor_sync(0xffffffffu, mp, o));
    // the positions in use are cut evenly into the launched slices, whatever bound the grid was sized for
    const int len = mp + 1;
    const int slice = (((len + P.n_splits - 1) / P.n_splits) + 15) & ~15;
    const int s_begin = split * slice;
    const int s_np = max(0, min(s_begin + slice, len) - s_begin);    // positions of the slice, shared by the cluster's CTAs
    const int sub = (((s_np + CS - 1) / CS) + 15) & ~15;
    const int p_begin = s_begin + crank * sub;
    const int np = min(p_begin + sub, s_begin + s_np) - p_begin;     // positions of this CTA (<= 0: nothing to do)

    // this thread's two query rows of the tile (gid and gid + 8)
    const int j_lo = gid, j_hi = gid + 8;
    const bf16* q_lo = P.q + ((size_t)(r0 + j_lo / group) * P.H + kvh * group + j_lo % group) * HD;
    const bf16* q_hi = P.q + ((size_t)(r0 + j_hi / group) * P.H + kvh * group + j_hi % group) * HD;
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
    float O[NV][4];
#pragma unroll
    for (int i = 0; i < NV; ++i) { O[i][0] = O[i][1] = O[i][2] = O[i][3] = 0.f; }

    // first position this pass appends for the block's sequence (its rows' positions rise; inactive rows are -1)
    int new_begin;
    {
        const int seq_first = zseq * P.rows_per_seq;
        const int fp = lane < min(P.rows_per_seq, 32) ? __ldcg(P.row_pos + seq_first + lane) : -1;
        int nb = fp >= 0 ? fp : 0x7fffffff;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) nb = min(nb, __shfl_xor_sync(0xffffffffu, nb, o));
        new_begin = nb == 0x7fffffff ? 0 : nb;
    }
    const bf16* K = P.kc + (((size_t)slot * P.Hkv + kvh) * P.max_ctx + max(p_begin, 0)) * HD;
    const bf16* V = P.vc + (((size_t)slot * P.Hkv + kvh) * P.max_ctx + max(p_begin, 0)) * HD;
    // keys [k_lo, k_hi) of chunk c -> buffer c & 1: [K][V]; last: also clears the padding rows and closes the chunk
    auto issue_part = [&](int c, int k_lo, int k_hi, bool last) {
            const int nk = min(CK, np - c * CK);
            const uint32_t kb = smem0 + (uint32_t)(c & 1) * 2u * BUF, vb = kb + BUF;
            const bf16* ks = K + (size_t)c * CK * HD;
            const bf16* vs = V + (size_t)c * CK * HD;
            for (int i = k_lo * CPR + t; i < k_hi * CPR; i += NT) {
                const int key = i / CPR, ch = i % CPR;
                const uint32_t off = (uint32_t)key * ROWB + (uint32_t)((ch ^ (key & 7)) << 4);
                cp_async16(kb + off, ks + (size_t)i * 8);
                cp_async16(vb + off, vs + (size_t)i * 8);
            }
            // value rows past the end of the slice inside a warp's 16-key group must be finite (their weight is zero)
            const int nk16 = (nk + 15) & ~15;
            for (int i = nk * CPR + t; last && i < nk16 * CPR; i += NT) {
                const int key = i / CPR, ch = i % CPR;
                *reinterpret_cast<uint4*>(sm_raw + (size_t)(c & 1) * 2 * BUF + BUF + (size_t)key * ROWB + ((ch ^ (key & 7)) << 4)) = make_uint4(0, 0, 0, 0);
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
    };
    auto issue = [&](int c) { issue_part(c, 0, min(CK, np - c * CK), true); };
    // the part of the first chunk that earlier passes wrote is requested before the wait
    const int old0 = np > 0 ? max(0, min(min(CK, np), new_begin - p_begin)) : 0;
    if (np > 0) issue_part(0, 0, old0, false);
    pdl_wait();                                  // queries and the keys/values appended by this pass come from the kernels before
    if (threadIdx.x == 0) stamp_pair(P.stamp, ST_DEP_FIRST);
    if (np > 0) {
        const int n_chunks = (np + CK - 1) / CK;
        issue_part(0, old0, min(CK, np), true);
        // query fragments (bf16, straight from memory in the MMA's register layout) and the rows' positions
        uint32_t a[KS][4];
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            a[ks][0] = j_lo < nq ? __ldcg(reinterpret_cast<const uint32_t*>(q_lo + 16 * ks + 2 * tig)) : 0u;
            a[ks][1] = j_hi < nq ? __ldcg(reinterpret_cast<const uint32_t*>(q_hi + 16 * ks + 2 * tig)) : 0u;
            a[ks][2] = j_lo < nq ? __ldcg(reinterpret_cast<const uint32_t*>(q_lo + 16 * ks + 8 + 2 * tig)) : 0u;
            a[ks][3] = j_hi < nq ? __ldcg(reinterpret_cast<const uint32_t*>(q_hi + 16 * ks + 8 + 2 * tig)) : 0u;
        }
        const int pos_lo = j_lo < nq ? __ldcg(P.row_pos + r0 + j_lo / group) : -1;
        const int pos_hi = j_hi < nq ? __ldcg(P.row_pos + r0 + j_hi / group) : -1;
        const float sl2 = rsqrtf((float)HD) * 1.4426950408889634f;        // softmax scale in the exp2 domain

        for (int c = 0; c < n_chunks; ++c) {
            if (c + 1 < n_chunks) { issue(c + 1); asm volatile("cp.async.wait_group 1;" ::: "memory"); }
            else asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncthreads();
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
                // scale, mask (past the slice, or after the row's own position), online softmax
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
            __syncthreads();                     // the buffer may be refilled (or reused for the merge) from here on
        }
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    }

    // ---- merge of the warps (each saw different keys), then the slice's partial result
    float* Ow = reinterpret_cast<float*>(sm_raw);                // [warps][16][OLD]
    float* mw = Ow + NW * NQ * OLD;                       // [warps][16]
    float* lw = mw + NW * NQ;                             // [warps][16]
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
    __syncthreads();
    // this CTA's result: per query row the running max, the sum and the unnormalised output
    constexpr int TPR = NT / NQ;                                 // threads that span a query row
    constexpr int CPT = HD / TPR;                                // columns per thread
    float* Oc = reinterpret_cast<float*>(sm_raw) + NW * NQ * OLD + 2 * NW * NQ;   // [16][HD]
    float* Mc = Oc + NQ * HD;                                    // [16]
    float* Lc = Mc + NQ;                                         // [16]
    const int j = t / TPR, c0 = (t % TPR) * CPT;
    {
        float M = -INFINITY, L = 0.f;
        float4 acc[CPT / 4];
#pragma unroll
        for (int cc = 0; cc < CPT / 4; ++cc) acc[cc] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (np > 0) {
#pragma unroll
            for (int w = 0; w < NW; ++w) M = fmaxf(M, mw[w * NQ + j]);
            float wt[NW];
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const float m = mw[w * NQ + j];
                wt[w] = (m == -INFINITY) ? 0.f : exp2f(m - M);
                L += wt[w] * lw[w * NQ + j];
            }
#pragma unroll
            for (int cc = 0; cc < CPT / 4; ++cc)
#pragma unroll
                for (int w = 0; w < NW; ++w) {
                    if (wt[w] != 0.f) {                       // a warp without keys left nothing behind
                        const float4 o = *reinterpret_cast<const float4*>(Ow + ((size_t)w * NQ + j) * OLD + c0 + 4 * cc);
                        acc[cc].x = fmaf(wt[w], o.x, acc[cc].x); acc[cc].y = fmaf(wt[w], o.y, acc[cc].y);
                        acc[cc].z = fmaf(wt[w], o.z, acc[cc].z); acc[cc].w = fmaf(wt[w], o.w, acc[cc].w);
                    }
                }
        }
#pragma unroll
        for (int cc = 0; cc < CPT / 4; ++cc) *reinterpret_cast<float4*>(Oc + (size_t)j * HD + c0 + 4 * cc) = acc[cc];
        if ((t % TPR) == 0) { Mc[j] = M; Lc[j] = L; }
    }
    // the CTAs of the cluster hand their results to the first one through distributed shared memory
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    if (CS > 1) cluster.sync(); else __syncthreads();
    if (crank == 0 && j < nq) {
        float Mr[4], Lr[4];
        float M = -INFINITY, L = 0.f;
#pragma unroll
        for (int rc = 0; rc < 4; ++rc) {
            Mr[rc] = -INFINITY; Lr[rc] = 0.f;
            if (rc < CS) {
                const float* rm = CS > 1 ? cluster.map_shared_rank(Mc, rc) : Mc;
                const float* rl = CS > 1 ? cluster.map_shared_rank(Lc, rc) : Lc;
                Mr[rc] = rm[j]; Lr[rc] = rl[j];
            }
            M = fmaxf(M, Mr[rc]);
        }
        float4 acc[CPT / 4];
#pragma unroll
        for (int cc = 0; cc < CPT / 4; ++cc) acc[cc] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int rc = 0; rc < 4; ++rc) {
            const float w = (rc < CS && Mr[rc] != -INFINITY) ? exp2f(Mr[rc] - M) : 0.f;
            L += w * Lr[rc];
            if (w != 0.f) {
                const float* ro = CS > 1 ? cluster.map_shared_rank(Oc, rc) : Oc;
#pragma unroll
                for (int cc = 0; cc < CPT / 4; ++cc) {
                    const float4 o = *reinterpret_cast<const float4*>(ro + (size_t)j * HD + c0 + 4 * cc);
                    acc[cc].x = fmaf(w, o.x, acc[cc].x); acc[cc].y = fmaf(w, o.y, acc[cc].y);
                    acc[cc].z = fmaf(w, o.z, acc[cc].z); acc[cc].w = fmaf(w, o.w, acc[cc].w);
                }
            }
        }
        const int r = r0 + j / group, h = kvh * group + j % group;
        if (P.n_splits == 1) {                       // a single slice is final: normalise and write the output
            const float inv = L > 0.f ? 1.f / L : 0.f;
            bf16* dst = P.out + ((size_t)r * P.H + h) * HD + c0;
#pragma unroll
            for (int cc = 0; cc < CPT / 4; ++cc) {
                const float x[4] = {acc[cc].x * inv, acc[cc].y * inv, acc[cc].z * inv, acc[cc].w * inv};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const bf16 hi = __float2bfloat16_rn(x[k]);
                    dst[4 * cc + k] = hi;
                    if (P.lo_off) dst[(size_t)P.lo_off * P.H * HD + 4 * cc + k] = __float2bfloat16_rn(x[k] - __bfloat162float(hi));
                }
            }
        } else {
            float* po = P.part_o + (((size_t)r * P.H + h) * P.n_splits + split) * HD + c0;
            float* ml = P.part_ml + (((size_t)r * P.H + h) * P.n_splits + split) * 2;
#pragma unroll
            for (int cc = 0; cc < CPT / 4; ++cc) __stcg(reinterpret_cast<float4*>(po + 4 * cc), acc[cc]);
            if ((t % TPR) == 0) { __stcg(ml, M); __stcg(ml + 1, L); }
        }
    }
    if (CS > 1) cluster.sync();                      // nobody leaves while its shared memory may still be read
    if (crank != 0) return;
    if (P.n_splits == 1) { if (t == 0) stamp_pair(P.stamp, ST_DONE_FIRST); return; }      // nothing to merge

    // ---- the slice that delivers last merges all of them: out = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s,
    //      always in slice order, so the result does not depend on which slice that was
    __syncthreads();                                 // the block's writes are ordered before thread 0's release below
    if (t == 0) {
        uint32_t* ctr = P.counters + (size_t)zb * P.Hkv + kvh;
        uint32_t old;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(ctr) : "memory");
        const int last = old == (uint32_t)P.n_splits - 1u;
        if (last) *ctr = 0u;
        last_sm = last;
    }
    __syncthreads();
    if (!last_sm) { if (t == 0) stamp_pair(P.stamp, ST_DONE_FIRST); return; }
    // Everything the merge reads (every slice's max, sum and partial output for the block's
    // queries) is fetched into shared memory in one go, so the merge costs one memory round trip.
    const int ns = P.n_splits;
    float* o_all = reinterpret_cast<float*>(sm_raw);             // [nq][ns][HD]
    __shared__ float wgt[NQ * 32];                               // normalised weight of each (query, slice)
    const bool staged = (size_t)nq * ns * HD * sizeof(float) <= (size_t)4 * BUF;
    if (staged) {
        const int per_q = ns * (HD / 4);                         // 16-byte pieces of one query's partial outputs
        for (int j = 0; j < nq; ++j) {
            const int r = r0 + j / group, h = kvh * group + j % group;
            const float* src = P.part_o + ((size_t)r * P.H + h) * ns * HD;
            const uint32_t dst = smem0 + (uint32_t)j * (uint32_t)per_q * 16u;
            for (int c = t; c < per_q; c += NT) cp_async16(dst + (uint32_t)c * 16u, src + (size_t)c * 4);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    for (int j = warp; j < nq; j += NT / 32) {          // n_splits <= 32: one lane per slice
        const int r = r0 + j / group, h = kvh * group + j % group;
        const float* mlg = P.part_ml + ((size_t)r * P.H + h) * ns * 2;
        float m = -INFINITY, l = 0.f;
        if (lane < ns) { const float2 v = __ldcg(reinterpret_cast<const float2*>(mlg) + lane); m = v.x; l = v.y; }
        const float M = warp_max(m);
        const float w = (m == -INFINITY) ? 0.f : exp2f(m - M);
        const float den = warp_sum(w * l);
        if (lane < ns) wgt[j * 32 + lane] = den > 0.f ? w / den : 0.f;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    // each thread owns one output column of up to NQ queries: independent sums, slices in order
    constexpr int TPQ = NT / HD;                        // queries handled side by side (1 or 2)
    const int e = t % HD, jq0 = t / HD;
    float acc[NQ / TPQ];
#pragma unroll
    for (int i = 0; i < NQ / TPQ; ++i) acc[i] = 0.f;
    if (staged) {                    // branch-free: rows past nq re-read the last valid row and are dropped below
        for (int sidx = 0; sidx < ns; ++sidx) {
#pragma unroll
            for (int i = 0; i < NQ / TPQ; ++i) {
                const int j = min(jq0 + i * TPQ, nq - 1);
                const float w = wgt[j * 32 + sidx];
                const float o = o_all[((size_t)j * ns + sidx) * HD + e];
                acc[i] = fmaf(w, w != 0.f ? o : 0.f, acc[i]);    // an empty slice left no output behind
            }
        }
    } else {
        for (int sidx = 0; sidx < ns; ++sidx) {
#pragma unroll
            for (int i = 0; i < NQ / TPQ; ++i) {
                const int j = min(jq0 + i * TPQ, nq - 1);
                const int r = r0 + j / group, h = kvh * group + j % group;
                const float w = wgt[j * 32 + sidx];
                const float o = __ldcg(P.part_o + (((size_t)r * P.H + h) * ns + sidx) * HD + e);
                acc[i] = fmaf(w, w != 0.f ? o : 0.f, acc[i]);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < NQ / TPQ; ++i) {
        const int j = jq0 + i * TPQ;
        if (j < nq) {
            const int r = r0 + j / group, h = kvh * group + j % group;
            const bf16 hi = __float2bfloat16_rn(acc[i]);
            P.out[((size_t)r * P.H + h) * HD + e] = hi;
            if (P.lo_off) P.out[((size_t)(r + P.lo_off) * P.H + h) * HD + e] = __float2bfloat16_rn(acc[i] - __bfloat162float(hi));
        }
    }
    if (t == 0) stamp_pair(P.stamp, ST_DONE_FIRST);
}

}  // namespace

bool attention_split_supported(int dtype, int H, int Hkv, int hd) {
    return dtype == SD_BF16 && (hd == 64 || hd == 128) && H / Hkv <= NQ;
}

size_t attention_split_workspace(int rows, int H, int hd, int max_ctx) {
    const int n_splits = std::min(32, (max_ctx + SLICE_KEYS - 1) / SLICE_KEYS);
    return ATTN_COUNTER_BYTES + sizeof(float) * (size_t)rows * H * n_splits * (hd + 2);
}

// Rows come in runs of rows_per_seq consecutive rows of one sequence (n_rows is a multiple of it);
// ctx_bound: no row sees a position >= ctx_bound (bounds the number of slices launched).
// The first ATTN_COUNTER_BYTES of the workspace are arrival counters: zero before the first
// launch, left at zero by every launch.
cudaError_t launch_attention_split(const void* q, const void* kc, const void* vc, void* out, const int32_t* row_slot,
                                   const int32_t* row_pos, int n_rows, int rows_per_seq, int H, int Hkv, int hd,
                                   int max_ctx, int ctx_bound, void* workspace, size_t workspace_bytes, int dependent,
                                   cudaStream_t st, int lo_off, unsigned long long* stamp, int force_warps, int max_cluster, const int* seq_len_hint) {
    if (n_rows <= 0) return cudaSuccess;
    ctx_bound = std::max(1, std::min(ctx_bound, max_ctx));
    AttnParams P;
    P.q = (const bf16*)q; P.kc = (const bf16*)kc; P.vc = (const bf16*)vc; P.out = (bf16*)out;
    P.row_slot = row_slot; P.row_pos = row_pos; P.lo_off = lo_off; P.stamp = stamp;
    P.use_order = 0;
    if (seq_len_hint && rows_per_seq >= 1 && n_rows / rows_per_seq > 1 && n_rows / rows_per_seq <= 64) {      // longest first
        const int ns = n_rows / rows_per_seq;
        int idx[64];
        for (int i = 0; i < ns; ++i) idx[i] = i;
        std::stable_sort(idx, idx + ns, [&](int a, int b) { return seq_len_hint[a] > seq_len_hint[b]; });
        for (int i = 0; i < ns; ++i) P.seq_order[i] = (unsigned char)idx[i];
        P.use_order = 1;
    }
    if (rows_per_seq < 1 || n_rows % rows_per_seq || H / Hkv > NQ) return cudaErrorInvalidValue;
    P.n_rows = n_rows; P.rows_per_seq = rows_per_seq; P.H = H; P.Hkv = Hkv; P.max_ctx = max_ctx;
    P.rows_per_block = std::max(1, std::min(rows_per_seq, NQ / (H / Hkv)));
    const int bps = (rows_per_seq + P.rows_per_block - 1) / P.rows_per_block;
    const int n_blocks = (n_rows / rows_per_seq) * bps;
    // one slice while the context is short (no cross-CTA merge at all), SLICE_KEYS positions per slice beyond
    P.n_splits = std::max(1, std::min(32, (ctx_bound + SLICE_KEYS - 1) / SLICE_KEYS));
    int sm = 148;
    { int dev = 0; if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev); }
    if (P.n_splits * Hkv * n_blocks > 2 * sm) {
        P.n_splits = std::max(1, std::min(32, (ctx_bound + SLICE_KEYS_MANY - 1) / SLICE_KEYS_MANY));
    }
    const size_t need = ATTN_COUNTER_BYTES + sizeof(float) * (size_t)n_rows * H * P.n_splits * (hd + 2);
    if (need > workspace_bytes || (size_t)n_blocks * Hkv * sizeof(uint32_t) > ATTN_COUNTER_BYTES) return cudaErrorInvalidValue;
    P.counters = (uint32_t*)workspace;
    P.part_o = (float*)((char*)workspace + ATTN_COUNTER_BYTES);
    P.part_ml = P.part_o + (size_t)n_rows * H * P.n_splits * hd;
    // few (head, row block, slice) items: two or four CTAs of a cluster share each of them
    const int items = P.n_splits * Hkv * n_blocks;
    P.csize = items * 4 <= sm ? 4 : (items * 2 <= sm ? 2 : 1);
    if (max_cluster == 1 || max_cluster == 2) P.csize = std::min(P.csize, max_cluster);
    const int nw = force_warps == WARPS_MANY || force_warps == WARPS_FEW ? force_warps : (items > 2 * sm ? WARPS_MANY : WARPS_FEW);
    const size_t smem = std::max((size_t)4 * 16 * nw * hd * 2, sizeof(float) * ((size_t)nw * NQ * (hd + 8) + 2 * nw * NQ + (size_t)NQ * hd + 2 * NQ));
    dim3 grid(P.n_splits * P.csize, Hkv, n_blocks);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = dim3(32 * nw); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (P.csize > 1) { attr[na].id = cudaLaunchAttributeClusterDimension; attr[na].val.clusterDim.x = P.csize; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1; ++na; }
    if (dependent) { attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization; attr[na].val.programmaticStreamSerializationAllowed = 1; ++na; }
    cfg.attrs = attr; cfg.numAttrs = na;
    void (*kern)(AttnParams) = hd == 128 ? (nw == WARPS_MANY ? k_attn_mma<128, WARPS_MANY> : k_attn_mma<128, WARPS_FEW>)
                                         : (nw == WARPS_MANY ? k_attn_mma<64, WARPS_MANY> : k_attn_mma<64, WARPS_FEW>);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return cudaLaunchKernelEx(&cfg, kern, P);
}

}  // namespace sd
