// Host-side launchers of the library's kernels.  Every launcher enqueues on `st` and returns
// the launch error, if any; none synchronises.
#pragma once
#include "common.cuh"

namespace sd {

// ---- elementwise.cu
cudaError_t launch_embed(const SeqState& S, const SeqList& list, const RowPlan& plan, int n_rows,
                         const void* embed, int dtype, int d, int vocab,
                         float* h, int32_t* row_slot, int32_t* row_pos,
                         const float* gain /*nullable: also writes xn = bf16(h * gain) and ssq[row][0] = sum h^2*/,
                         void* xn, float* ssq,
                         const float* rope_cos, const float* rope_sin, int half,      // position tables [max_ctx][half]
                         float* row_cos, float* row_sin /*nullable: [row][half] factors of each row's position*/,
                         int tagged_m_pad /*0: plain h, xn [row][d], ssq; else all three as tagged 64-bit words for the streaming kernel (m_pad rows)*/,
                         const uint32_t* epoch /*device word the tags derive from (tagged mode)*/, cudaStream_t st,
                         int lo_off = 0 /*> 0 (plain mode): xn's second bf16 part, bf16(x - bf16(x)), goes lo_off rows further down*/);
// xn[i] = rmsnorm(h[src_row(i)]) * gain; src_row(i) = i * row_stride + row_offset
cudaError_t launch_rmsnorm(const float* h, const float* gain, void* xn, int dtype, int n_rows, int d, float eps,
                           int row_stride, int row_offset, cudaStream_t st);
cudaError_t launch_rope_kv(const float* qkv, void* q_out, void* kcache_layer, void* vcache_layer, int dtype,
                           const int32_t* row_slot, const int32_t* row_pos, int n_rows,
                           int n_heads, int n_kv_heads, int head_dim, int max_ctx,
                           const float* rope_cos, const float* rope_sin, uint32_t* status, cudaStream_t st);
cudaError_t launch_residual_add(float* h, const float* y, size_t n, cudaStream_t st);
// act[r][f] = silu(gate_f) * up_f; gu[r] holds the gate values then the up values, or, when
// interleaved, 128-wide groups of 64 gate values followed by the 64 up values of the same features
cudaError_t launch_swiglu(const float* gu, void* act, int dtype, int n_rows, int F, int interleaved, cudaStream_t st);
cudaError_t launch_set_state(const SeqState& S, int slot, int len, int tkv, int dkv, uint32_t iter, uint32_t seq_id,
                             int reset_counters, cudaStream_t st);
cudaError_t launch_rollback(const SeqState& S, const SeqList& list, int gamma, const int32_t* n_acc,
                            const int32_t* out_tok, const float* alpha_terms /*nullable: [n_seq][gamma]*/, cudaStream_t st);

// ---- linear_simt.cu : y[rows][n_out] fp32 = x[rows][n_in] * W[n_out][n_in]^T on CUDA cores
cudaError_t launch_linear_simt(const void* x, const void* w, float* y, int rows, int n_out, int n_in, int dtype,
                               cudaStream_t st);

// ---- attention.cu
size_t attention_workspace_bytes(int rows, int n_heads, int head_dim, int max_ctx);
cudaError_t launch_attention(const void* q, const void* kcache_layer, const void* vcache_layer, void* out, int dtype,
                             const int32_t* row_slot, const int32_t* row_pos, int n_rows,
                             int n_heads, int n_kv_heads, int head_dim, int max_ctx,
                             void* workspace, size_t workspace_bytes, cudaStream_t st);

// ---- attention_split.cu : split-KV kernel for bf16 caches with head_dim 64 / 128
bool attention_split_supported(int dtype, int H, int Hkv, int hd);
size_t attention_split_workspace(int rows, int H, int hd, int max_ctx);
cudaError_t launch_attention_split(const void* q, const void* kc, const void* vc, void* out, const int32_t* row_slot,
                                   const int32_t* row_pos, int n_rows, int rows_per_seq, int H, int Hkv, int hd,
                                   int max_ctx, int ctx_bound, void* workspace, size_t workspace_bytes, int dependent,
                                   cudaStream_t st, int lo_off = 0 /*> 0: also write out's second bf16 part, lo_off rows further down*/,
                                   unsigned long long* stamp = nullptr /*optional time stamps of the launch*/,
                                   int force_warps = 0 /*4 or 8: warps per CTA; 0: chosen from the number of work items*/,
                                   int max_cluster = 0 /*1 or 2: at most this many CTAs share a slice; 0: up to 4*/,
                                   const int* seq_len_hint = nullptr /*host, one per sequence: context lengths (bounds will do); longest sequences are started first*/);

// ---- sampling.cu
cudaError_t launch_philox(const uint32_t* ctr, int n, uint32_t k0, uint32_t k1, uint32_t* out, cudaStream_t st);
// probs[r] = softmax(logits[r] / T); tok[r] drawn with u_int[r] (explicit) ...
cudaError_t launch_softmax_sample_explicit(const float* logits, int rows, int V, float T, const uint32_t* u_int,
                                           float* probs, int32_t* tok, cudaStream_t st);
// ... or with the draft draw of (iter, slot = step, seq_id) of each listed sequence; outputs strided by gamma
cudaError_t launch_draft_sample(const float* logits, const SeqState& S, const SeqList& list, int V, float T,
                                uint64_t seed, int step, int gamma, float* q_out, int32_t* x_out, cudaStream_t st);
struct AcceptParams {
    const float* target; int target_is_logits; const float* q; const int32_t* x;
    int B, gamma, V; float T; uint64_t seed;
    const uint32_t* iter; const uint32_t* seq_id;   // indexed through `list` when use_list
    int use_list; SeqList list;
    int32_t* n_acc; int32_t* out_tok;
    float* alpha_terms;          // nullable: [B][gamma] receives sum_k min(p_s(k), q_s(k)) of every slot (the estimate of Eq. 1's alpha)
};
cudaError_t launch_accept(const AcceptParams& p, int dependent, cudaStream_t st);

// ---- classifier.cu
cudaError_t launch_classifier(const SeqState& S, const SeqList& list, const SeqList& forced /*ids[i] >= 0: given task*/,
                              const void* embed, int dtype, int d, int vocab,
                              const float* w1, const float* b1, int d_hidden, const float* w2, const float* b2,
                              int n_classes, cudaStream_t st);

}  // namespace sd
