/*
 * sd.h - C ABI of the speculative-decoding hot path for one B200 (sm_100a).
 *
 * The library runs the online half of task-routed heterogeneous speculative
 * decoding: route a prompt to one of several draft models, let that draft
 * propose gamma tokens one after the other, score them with one parallel pass
 * of the target model, accept or reject them, and forget the rejected part of
 * both KV caches.  Notation follows the paper: gamma = tokens drafted per
 * iteration, alpha = draft/target agreement, c = cost of one draft pass over
 * one target pass (Eq. 1), tau = tokens emitted per target pass (Sec. 3.1).
 *
 * Conventions that hold for every call:
 *  - the return value is an sd_status; argument and capacity errors are found
 *    on the host before anything is launched;
 *  - work is enqueued on the CUDA stream given at sd_create and the call
 *    returns without waiting, unless its comment says "synchronises";
 *  - "device" pointers are CUDA device addresses valid on the current device,
 *    "host" pointers are ordinary memory; the caller owns every buffer it
 *    passes and the library keeps no pointer past the call, except the arena
 *    and the stream handed to sd_create;
 *  - the library owns its weight copies, KV caches and per-sequence state, all
 *    carved out of the caller's arena; it never allocates device memory;
 *  - nothing traps: a kernel that meets an impossible value (a token id out of
 *    range, a position past the cache) skips the access and sets a bit in a
 *    status word that sd_device_status returns.
 */
#ifndef SD_H
#define SD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sd_ctx sd_ctx;

typedef enum {
    SD_OK = 0,
    SD_ERR_INVALID_ARG = 1,
    SD_ERR_STATE = 2,        /* call out of order for that sequence */
    SD_ERR_CAPACITY = 3,     /* KV cache, batch or row limit would be exceeded */
    SD_ERR_OOM = 4,          /* arena too small */
    SD_ERR_CUDA = 5,
    SD_ERR_TIMEOUT = 6,
    SD_ERR_UNSUPPORTED = 7
} sd_status;

enum { SD_F32 = 0, SD_BF16 = 1 };

#define SD_MAX_BATCH 64      /* sequences per call */
#define SD_MAX_ROWS 256      /* query rows per forward pass: n_seq * (gamma + 1) */
#define SD_MAX_GAMMA 15

/* bits of the device status word */
#define SD_DEV_BAD_TOKEN 1u      /* token id outside [0, vocab) */
#define SD_DEV_BAD_POS 2u        /* position outside the KV cache */
#define SD_DEV_BAD_NACC 4u       /* n_acc outside [0, gamma] at rollback */
#define SD_DEV_WAIT_EXPIRED 8u   /* a bounded wait inside a kernel gave up */

/* Decoder-only transformer of the LLaMA family (the paper's target and drafts,
 * Sec. 3.1): RMSNorm, rotary position embedding (pairs (i, i + head_dim/2)),
 * grouped-query attention, SwiGLU feed-forward, no biases, untied lm_head. */
typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
    int32_t dtype;           /* SD_F32 or SD_BF16: storage of weights, activations, KV */
    float rms_eps;
    float rope_base;
} sd_model_desc;

typedef struct {
    int32_t max_seqs;        /* sequence slots, <= SD_MAX_BATCH */
    int32_t max_ctx;         /* KV positions per sequence */
    int32_t max_gamma;       /* <= SD_MAX_GAMMA */
    int32_t n_drafts;        /* K heterogeneous drafts; models[0] is the target, models[1..K] the drafts */
    float temperature;       /* same for draft and target; 0 = greedy */
    uint64_t seed;           /* Philox4x32-10 key */
    int32_t clf_d_hidden;    /* prompt classifier d_model(target) -> clf_d_hidden -> n_drafts; 0 = none */
    int32_t lora_adapters;   /* 0: models[1..K] are K separate drafts.  K (= n_drafts): the drafts are ONE base model,
                                models[1], plus one low-rank adapter per task (Section 2.3: every draft is the same base
                                draft fine-tuned with LoRA); sequences of different tasks then share each draft pass */
    int32_t lora_rank;       /* r: a multiple of 8, lora_adapters * r <= 128 */
    float lora_scale;        /* alpha / r of the LoRA paper: W' = W + lora_scale * B A */
} sd_config;

typedef struct {
    int64_t iterations, drafted, accepted, emitted;   /* Eq. 2: accepted / drafted; tau = emitted / iterations */
} sd_counters;

/* tensor kinds for sd_load_tensor; matrices are row-major [out_features][in_features] */
enum {
    SD_T_EMBED = 0, SD_T_LM_HEAD = 1, SD_T_FINAL_NORM = 2,
    SD_T_WQ = 3, SD_T_WK = 4, SD_T_WV = 5, SD_T_WO = 6, SD_T_WG = 7, SD_T_WU = 8, SD_T_WD = 9,
    SD_T_NORM1 = 10, SD_T_NORM2 = 11
};

/* matrices of a layer that carry an adapter (sd_load_lora) */
enum { SD_LORA_QKV = 0, SD_LORA_WO = 1, SD_LORA_GU = 2, SD_LORA_WD = 3 };

/* ---------------------------------------------------------------- lifecycle */

/* Bytes of device memory sd_create needs for this configuration (weights, KV
 * caches, state, scratch).  models: 1 + n_drafts descriptors.  0 on bad input. */
size_t sd_arena_bytes(const sd_config* cfg, const sd_model_desc* models);

/* Creates a context on the current device.  arena: device memory of at least
 * sd_arena_bytes, 256-byte aligned, owned by the caller and left alone by it
 * until sd_destroy.  cuda_stream: a cudaStream_t (NULL = legacy default).
 * Zeroes the state; weights are undefined until loaded.  Synchronises. */
sd_status sd_create(const sd_config* cfg, const sd_model_desc* models, void* cuda_stream,
                    void* arena_device, size_t arena_bytes, sd_ctx** out);
sd_status sd_destroy(sd_ctx* ctx);

/* Copies one tensor into the library's own layout.  model_id 0 = target,
 * 1..K = drafts.  layer is ignored for SD_T_EMBED / LM_HEAD / FINAL_NORM.
 * Matrices are in the model's dtype (bf16 as raw 16-bit patterns), norm gains
 * are fp32.  src may be host (src_on_device = 0) or device memory. */
sd_status sd_load_tensor(sd_ctx* ctx, int model_id, int kind, int layer, const void* src, int src_on_device);

/* One low-rank adapter of the shared base draft (contexts created with lora_adapters > 0): for matrix `mat` of `layer`,
 * task `adapter` uses W' = W + lora_scale * B A (the LoRA paper's definition; Section 2.3 fine-tunes every draft this
 * way).  a: [lora_rank][in_features], b: [out_features][lora_rank], both bf16 bit patterns, row-major, host or device.
 * out_features follow the fused matrices: SD_LORA_QKV (H + 2 Hkv) * head_dim rows (query, key, value rows in that
 * order), SD_LORA_GU 2 * d_ffn rows (gate rows, then up rows), SD_LORA_WO / SD_LORA_WD d_model rows.  Adapters that
 * were never loaded are zero: the task runs the base draft.  The embedding and the lm_head carry no adapter.
 * The product x A^T rides along in the matrix's own GEMM (A's rows are appended to W as one more output tile) and
 * B is applied by the step kernel after the GEMM: no extra launch, no extra pass over the weights. */
sd_status sd_load_lora(sd_ctx* ctx, int adapter, int layer, int mat, const void* a, const void* b, int src_on_device);

/* Prompt classifier, MLP variant of Sec. 3.3.3: fp32 w1 [h][d], b1 [h], w2 [K][h], b2 [K]. */
sd_status sd_load_classifier(sd_ctx* ctx, const float* w1, const float* b1, const float* w2, const float* b2,
                             int src_on_device);

/* Starts sequence slot `seq` with a prompt (host, n_prompt >= 2 token ids) and
 * a Philox stream id; resets its lengths, iteration counter and counters. */
sd_status sd_seq_begin(sd_ctx* ctx, int seq, const int32_t* prompt_host, int n_prompt, uint32_t seq_id);

/* Runs prompt tokens [0, n_prompt - 1) of each listed sequence through the
 * target and through the sequence's routed draft so that both KV caches hold
 * everything but the last prompt token.  Needs sd_route_prompt first. */
sd_status sd_prefill(sd_ctx* ctx, const int32_t* seqs_host, int n_seq);

/* ------------------------------------------------------- the five hot calls */

/* Sec. 2.1 / 2.4: picks the draft model for each listed sequence.  A
 * forced_task_host[i] >= 0 (task type given by the user) is taken as is; -1 (or
 * a NULL array) runs the classifier on the prompt: mean of the target's
 * embedding rows over the prompt -> FC + ReLU -> FC -> argmax (lowest index
 * on ties).  draft_id_out_host may be NULL.  Synchronises (the draft id selects
 * which weights later calls launch on). */
sd_status sd_route_prompt(sd_ctx* ctx, const int32_t* seqs_host, int n_seq, const int32_t* forced_task_host,
                          int32_t* draft_id_out_host);

/* Fig. 1(a): the routed draft proposes gamma tokens for each listed sequence,
 * one autoregressive step after the other.  x_dev [n_seq][gamma] receives the
 * tokens, q_dev [n_seq][gamma][vocab] the fp32 distributions they were drawn
 * from (softmax(logits / T); one-hot when T = 0).  Sequences are grouped by
 * draft internally; the first step also feeds the token the draft missed after
 * a fully accepted iteration. */
sd_status sd_draft_steps(sd_ctx* ctx, const int32_t* seqs_host, int n_seq, int gamma,
                         int32_t* x_dev, float* q_dev);

/* The same, but step s > 0 feeds x_forced_dev[.][s-1] instead of the token the draft drew
 * at step s-1 (x_sampled_dev still receives the draws).  It lets a caller replay a recorded
 * run step by step; sd_draft_steps is this call with both arrays the same. */
sd_status sd_draft_steps_replay(sd_ctx* ctx, const int32_t* seqs_host, int n_seq, int gamma,
                                const int32_t* x_forced_dev, int32_t* x_sampled_dev, float* q_dev);

/* Fig. 1(b): one pass of the target over [last token, x_0 .. x_{gamma-1}] of
 * every listed sequence against its KV cache (keys/values of the gamma+1 rows
 * are appended).  logits_dev [n_seq][gamma+1][vocab] fp32: row j is the
 * target's prediction for the token after row j's input. */
sd_status sd_verify(sd_ctx* ctx, const int32_t* seqs_host, int n_seq, int gamma,
                    const int32_t* x_dev, float* logits_dev);

/* Sec. 3.1 (the stochastic verification rule of Leviathan et al. that the paper
 * adopts): with p_j the target distribution of row j and q_s the draft's, slot s
 * is accepted iff u_s * q_s(x_s) <= p_s(x_s) (one rounded fp32 multiply, u_s in
 * (0,1] from Philox); n = number of leading accepted slots; the next token y is
 * drawn from norm(max(0, p_n - q_n)) when n < gamma, from p_gamma otherwise,
 * by an exact integer inverse CDF.  A pure function of its buffers. */
typedef struct {
    const float* target;     /* device [B][gamma+1][V]: logits (target_is_logits) or probabilities */
    int32_t target_is_logits;/* 1: p = softmax(target / temperature) is computed inside the kernel */
    const float* q;          /* device [B][gamma][V] draft probabilities */
    const int32_t* x;        /* device [B][gamma] draft tokens */
    int32_t B, gamma, V;
    float temperature;       /* used with logits only; 0 = one-hot argmax */
    uint64_t seed;           /* Philox key */
    const uint32_t* iter;    /* device [B]: Philox counter word 0 of each row */
    const uint32_t* seq_id;  /* device [B]: Philox counter word 2 of each row */
    int32_t* n_acc;          /* device [B] out */
    int32_t* out_tok;        /* device [B][gamma+1] out: x_0..x_{n-1}, y, then -1 */
    void* cuda_stream;
} sd_accept_args;
sd_status sd_accept(const sd_accept_args* args);

/* The same rule for sequences of a context: temperature, seed, iteration and
 * stream ids come from the context's per-sequence state on the device. */
sd_status sd_accept_seqs(sd_ctx* ctx, const int32_t* seqs_host, int n_seq, int gamma,
                         const float* target_logits_dev, const float* q_dev, const int32_t* x_dev,
                         int32_t* n_acc_dev, int32_t* out_tok_dev);

/* Commits an iteration: appends out_tok[0..n_acc] to each sequence, sets the
 * target cache length to L + n_acc and the draft cache length to
 * min(L + n_acc, L + gamma - 1) (L = length before the iteration), advances the
 * iteration counter and the counters of Eq. 2.  No KV data moves: rejected
 * positions stay where they are and the next append overwrites them. */
sd_status sd_kv_rollback(sd_ctx* ctx, const int32_t* seqs_host, int n_seq, int gamma,
                         const int32_t* n_acc_dev, const int32_t* out_tok_dev);

/* sd_verify + sd_accept_seqs + sd_kv_rollback as one call (one captured launch sequence):
 * logits_dev [n_seq][gamma+1][vocab] is scratch owned by the caller and holds the target's
 * logits afterwards. */
sd_status sd_verify_accept(sd_ctx* ctx, const int32_t* seqs_host, int n_seq, int gamma,
                           const int32_t* x_dev, const float* q_dev, float* logits_dev,
                           int32_t* n_acc_dev, int32_t* out_tok_dev);

/* One verify step for a caller whose drafts live in host memory: copies x_host [n_seq][gamma]
 * and q_host [n_seq][gamma][vocab] to the device, runs sd_verify, sd_accept_seqs and
 * sd_kv_rollback on them and copies n_acc [n_seq] and out_tok [n_seq][gamma+1] back.
 * Pinned host memory makes the copies asynchronous.  Synchronises before returning. */
sd_status sd_verify_accept_host(sd_ctx* ctx, const int32_t* seqs_host, int n_seq, int gamma,
                                const int32_t* x_host, const float* q_host,
                                int32_t* n_acc_host, int32_t* out_tok_host);

/* ------------------------------------------------------ choice of gamma (host) */

/* Eq. 1: expected speedup over plain autoregressive decoding when the draft agrees with the
 * target with probability alpha per token, gamma tokens are drafted per iteration and one draft
 * pass costs c target passes: (1 - alpha^(gamma+1)) / ((1 - alpha) (gamma c + 1)).
 * alpha in [0, 1], gamma >= 0, c >= 0; alpha = 1 gives (gamma + 1) / (gamma c + 1).  Pure host arithmetic. */
double sd_eq1_speedup(double alpha, int gamma, double c);

/* The gamma in [1, gamma_max] that maximises Eq. 1 for a measured alpha and c (the paper tunes gamma
 * per task by sweeping it, Sec. 3.2); ties go to the smaller gamma.  Returns 0 when no gamma beats
 * plain decoding (speedup <= 1) or on bad arguments.  speedup_out may be NULL. */
int sd_best_gamma(double alpha, double c, int gamma_max, double* speedup_out);

/* Time stamps of the launches of a forward pass, taken inside the kernels (the device's nanosecond timer) while the
 * pass runs the way it always runs (captured graph, programmatic dependent launches): what a profiler's serialised
 * per-kernel times cannot show.  While enabled, every weight GEMM, the step kernel after it and every attention launch
 * of the most recent forward pass on the kernel-per-matrix path (bf16 models) fill one record of SD_STAMP_WORDS 64-bit
 * words; sd_launch_stamps_read synchronises and copies the first `cap` records (launch order) to the host:
 *   [0] first CTA began                    [1],[2] first / last CTA saw what it waits for (the kernel before it; its
 *   tile's pieces)                         [3],[4] GEMM only: first / last CTA had its first stage complete
 *   [5],[6] first / last CTA finished      [7] 0.            A word is 0 when nothing reported it.
 * kinds_host[i] = SD_STAMP_GEMM / _STEP / _ATTENTION | (step after the GEMM: 0 plain, 1 QKV+rotary, 2 residual,
 * 3 SwiGLU) << 8; *n_out = records of the pass (may exceed cap).  Enabling changes the captured graphs' keys: the
 * first call afterwards captures anew.  A few atomics per CTA: for measurement, off by default. */
/* Sequences routed to different draft models run their draft passes side by side (default, when the context has two or
 * more separate draft models): every group after the first is enqueued on a stream of its own, forked from and joined
 * back to the context's stream, with its own scratch memory from the arena.  on = 0: group after group on the
 * context's stream. */
sd_status sd_use_draft_streams(sd_ctx* ctx, int on);

/* Measurement knobs of the kernel-per-matrix path (0 = the library's own choice).  Setting one drops the captured graphs.
 *   SD_TUNE_WO_STAGES       cap on the stage ring of the Wo GEMM (16 KB weight block + token rows per stage): with a
 *                           smaller ring its CTAs fit beside the attention kernel's and stream weights while it runs
 *   SD_TUNE_WO_PREFILL_ALL  1: the Wo GEMM requests its whole ring before attention has finished
 *   SD_TUNE_ATTN_WARPS      4 or 8 warps per attention CTA (64 or 128 KB of shared memory at head_dim 128)
 *   SD_TUNE_PREFILL_STAGES  stages a weight GEMM requests at once before the kernel before it has finished (default 4 for
 *                           passes of up to 16 rows)
 *   SD_TUNE_PACE_NS         after those, one more stage every so many nanoseconds until that kernel has finished
 *                           (default 300); 1 = no pacing: seven stages at once, the rest when that kernel has finished
 *   SD_TUNE_TILE_HANDOFF    1: a weight GEMM loads each k block of token rows as soon as the step kernel's CTA for that
 *                           tile has written it (a word per tile, release / acquire) instead of waiting for the whole step
 *                           kernel (passes of 3..8 rows).  Measured slower (+4 % on the 7B verify step): off by default
 *   SD_TUNE_STEADY_STAGES   stages of the ring a weight GEMM keeps in use once the ring has been filled (default: 160 KB worth)
 *   SD_TUNE_MANY_ROWS_CB    4: the sixteen-row form of the step kernel requests up to four pieces of a tile per round
 *                           (one round of loads, but 128-212 registers: two waves of CTAs); default: two per round
 *   SD_TUNE_ATTN_CLUSTER    1 or 2: at most this many CTAs of a cluster share one slice of a head's cache (default up to 4) */
#define SD_TUNE_WO_STAGES 0
#define SD_TUNE_WO_PREFILL_ALL 1
#define SD_TUNE_ATTN_WARPS 2
#define SD_TUNE_ATTN_CLUSTER 3
#define SD_TUNE_PACE_NS 4
#define SD_TUNE_PREFILL_STAGES 5
#define SD_TUNE_MANY_ROWS_CB 6
#define SD_TUNE_STEADY_STAGES 7
#define SD_TUNE_TILE_HANDOFF 8
#define SD_TUNE_COUNT 9
sd_status sd_tuning(sd_ctx* ctx, int knob, int value);

#define SD_STAMP_WORDS 8
#define SD_STAMP_GEMM 0
#define SD_STAMP_STEP 1
#define SD_STAMP_ATTENTION 2
sd_status sd_launch_stamps(sd_ctx* ctx, int enable);
sd_status sd_launch_stamps_read(sd_ctx* ctx, uint64_t* stamps_host, int32_t* kinds_host, int cap, int32_t* n_out);

/* The gamma that maximises Eq. 1 for what the library itself has measured: alpha = (sum over judged slots of
 * sum_k min(p_s(k), q_s(k))) / judged slots of sequence `seq` (accumulated by sd_accept_seqs + sd_kv_rollback), c from
 * sd_cost_timing / sd_cost_read.  Returns 0 when nothing has been measured yet or no gamma beats plain decoding.
 * alpha_out, c_out and speedup_out may be NULL.  Synchronises. */
int sd_best_gamma_measured(sd_ctx* ctx, int seq, int gamma_max, double* alpha_out, double* c_out, double* speedup_out);

/* Estimate of Eq. 1's alpha for a sequence since sd_seq_begin: for the stochastic rule a draft token drawn from q_s is kept
 * with probability sum_k min(p_s(k), q_s(k)); sd_accept_seqs computes that sum for every slot, sd_kv_rollback (called with the
 * same sequence list) adds the judged slots' sums (slot s is judged iff all slots before it were accepted) to alpha_sum
 * and their number to judged.  alpha = alpha_sum / judged.  Synchronises. */
sd_status sd_seq_alpha(sd_ctx* ctx, int seq, double* alpha_sum_out, int64_t* judged_out);

/* The cost ratio c of Eq. 1 from the library's own clock: while enabled, sd_draft_steps, sd_verify / sd_verify_accept
 * and sd_target_step are bracketed by CUDA events on the context's stream.  sd_cost_read synchronises and returns the
 * mean time of one draft pass (one token), of one verify pass and of one single-row target pass, and
 * c = draft pass / target pass (the verify pass stands in for the target pass when no sd_target_step was timed: Eq. 1
 * takes them to cost the same).  reset != 0 clears the sums. */
typedef struct {
    double draft_pass_ms, verify_pass_ms, target_pass_ms, c;
    int64_t draft_passes, verify_passes, target_passes;
} sd_cost;
sd_status sd_cost_timing(sd_ctx* ctx, int enable);
sd_status sd_cost_read(sd_ctx* ctx, sd_cost* out, int reset);

/* -------------------------------------------------------------- observation */

/* Repeated calls replay captured CUDA graphs by default (keyed by sequences, gamma, buffers
 * and a 256-token bucket of the context length); on == 0 launches kernel by kernel. */
sd_status sd_use_graphs(sd_ctx* ctx, int on);

/* bf16 models run on the tensor-core kernels by default; on != 0 makes the context use the
 * plain CUDA-core kernels instead (the two paths check each other in the tests). */
sd_status sd_force_plain_path(sd_ctx* ctx, int on);

/* Forward passes over few query rows (the verify rows of Fig. 1(b), a decoding row) run by default as ONE launch of a
 * persistent kernel that streams every weight matrix of every layer through the SMs without stopping at matrix
 * boundaries; passes with more rows run one kernel per matrix.  target_on / drafts_on switch that kernel on or off
 * for the target and for the draft models (defaults: on, off); max_rows > 0 sets the largest pass it takes (default
 * 16, at most 32).  The two paths check each other in the tests. */
sd_status sd_use_pass_kernel(sd_ctx* ctx, int target_on, int drafts_on, int max_rows);

/* Schedule of that kernel, for measurements: waves[5] = tile waves of the QKV, Wo, gate/up, down and lm_head matrices
 * (1..8), chunk_major[5] = order of a matrix's (wave, chunk) blocks (0: wave after wave).  NULL waves restores the
 * defaults.  stages > 0 caps the ring of shared-memory stages (0: as many as fit).  Drops cached programs and graphs.
 * Synchronises. */
sd_status sd_pass_tuning(sd_ctx* ctx, const int32_t* waves, const int32_t* chunk_major, int stages);

/* Time stamps of the persistent kernel's passes from now on (NULL: none): stamps_dev is a device buffer of n_words
 * 64-bit words; CTA b writes, for segment s of iteration it (layers, then the lm_head), the global-timer nanoseconds
 * at which its MMA thread turned to the segment and at which the segment was committed, at
 * ((b * n_iterations + it) * max_segments + s) * 2; after all of those, at ((b * n_iterations + it) * 16 + k) * 2, the
 * times at which the CTA's task warps turned to their k-th task of the iteration (k < 16) and finished it.  Passes whose
 * stamps would not fit write none.  Synchronises. */
sd_status sd_pass_stamps(sd_ctx* ctx, unsigned long long* stamps_dev, size_t n_words);

/* Builds and replays on the host the schedule of that kernel for a shape (no GPU needed): shape12 = n_layers, d_model,
 * n_heads, n_kv_heads, head_dim, d_ffn, vocab, rows, rows_per_seq, cache slices, want_logits, CTAs.  info8 receives
 * words per layer, total words, workspace slots of the two regions, most segments of a CTA per layer, largest CTA
 * section in bytes, program bytes, 16 KB weight blocks per layer.  SD_ERR_UNSUPPORTED with a message in err when the
 * shape does not fit or the replay finds a wait that could never be satisfied. */
sd_status sd_pass_schedule_check(const int32_t* shape12, const int32_t* waves, const int32_t* chunk_major, int32_t* info8,
                                 char* err, size_t err_cap);

/* The program itself (same arguments): copies it to out when cap suffices and returns its size in bytes (0 on failure).
 * Layout: uint32 offset of each CTA's section (CTAs + 1 entries), then per CTA a header (segments and tasks per layer
 * and for the lm_head, byte offsets of the four arrays and of the piece list), 16-byte segment records (tile, first k
 * block, k blocks, matrix, flags, wait word, wait count, arrival word, workspace slot) and 20-byte task records. */
size_t sd_pass_schedule_blob(const int32_t* shape12, const int32_t* waves, const int32_t* chunk_major, void* out, size_t cap);

/* With 3..16 query rows (the verify rows of one sequence) the tensor-core path feeds every GEMM its input rows in two
 * bf16 parts, bf16(x) and bf16(x - bf16(x)), in the columns that the 16- or 32-wide MMA covers anyway: the weights stream
 * once all the same, and the activations enter the products with 16 bits of mantissa instead of 8.  on = 0 switches
 * that off (one bf16 part, as with other row counts); the tests measure both.  Synchronises, drops cached graphs. */
sd_status sd_use_two_part_activations(sd_ctx* ctx, int on);

/* Number of kernels this context has launched since sd_create. */
sd_status sd_launch_count(sd_ctx* ctx, uint64_t* out);

/* Per-kernel timing for measurements: while enabled, a CUDA event is recorded in front of
 * every launch.  sd_profile_read synchronises, adds the time between consecutive events to
 * the category of the launch that followed the first one, and clears the record.
 * Categories: 0 weight GEMMs, 1 attention, 2 norm/rotary/elementwise, 3 sampling and
 * accept, 4 state updates, 5 the fused steps that follow the tensor-core GEMMs. */
#define SD_PROF_NCAT 6
sd_status sd_profile(sd_ctx* ctx, int enable);
sd_status sd_profile_read(sd_ctx* ctx, float* ms_by_cat, uint32_t* launches_by_cat);


/* Copies the sequence's tokens (up to cap) and counters to the host; also
 * refreshes the host's capacity bookkeeping with the true length.  Synchronises. */
sd_status sd_seq_read(sd_ctx* ctx, int seq, int32_t* tokens_host, int cap, int32_t* len_out, sd_counters* counters_out);

/* Overrides a sequence's token history (host) so that a test can replay another
 * run's iterations: keeps the KV caches, sets length to n_tokens, target cache
 * length to n_tokens - 1 and the draft cache length to draft_kv_len. */
sd_status sd_seq_force(sd_ctx* ctx, int seq, const int32_t* tokens_host, int n_tokens, int draft_kv_len, uint32_t iter);

/* Reads and clears the device status word.  Synchronises.  Returns SD_ERR_TIMEOUT (with the flags still written) when
 * SD_DEV_WAIT_EXPIRED is among them: a bounded wait inside a kernel gave up, results of that call are not to be trusted. */
sd_status sd_device_status(sd_ctx* ctx, uint32_t* flags_out);

/* Plain autoregressive pass of the target over the last token of each listed
 * sequence (the baseline that defines c in Eq. 1): logits_dev [n_seq][vocab].
 * Appends one KV position but does not commit a token. */
sd_status sd_target_step(sd_ctx* ctx, const int32_t* seqs_host, int n_seq, float* logits_dev);

/* ------------------------------------------- single operators (for testing) */

/* y[rows][n_out] (fp32) = x[rows][n_in] * W[n_out][n_in]^T; x and W in `dtype`.
 * impl: 0 = automatic, 1 = plain CUDA-core kernel, 2 = tensor-core kernel
 * (SD_ERR_UNSUPPORTED if the shape does not fit it).  All pointers device. */
sd_status sd_op_linear(const void* x, const void* w, float* y, int rows, int n_out, int n_in, int dtype,
                       int impl, void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t sd_op_linear_workspace(int rows, int n_out, int n_in, int dtype, int impl);

/* sd_op_linear's tensor-core form (3..8 rows) with the bounded wait of the step after the GEMM made to run out, for
 * tests: the step's CTAs watch arrival words (arrive_dev, at least ceil(n_out / 128) of them) that the GEMM is not told to
 * count into, for wait_ns nanoseconds; then they fall back to waiting for the GEMM's grid, finish the job and set
 * SD_DEV_WAIT_EXPIRED in *status_dev.  y must equal sd_op_linear's.  Nothing hangs and nothing faults. */
sd_status sd_op_linear_wait_expiry(const void* x, const void* w, float* y, int rows, int n_out, int n_in,
                                   void* workspace, size_t workspace_bytes, uint32_t* arrive_dev, size_t arrive_words,
                                   unsigned long long wait_ns, uint32_t* status_dev, void* cuda_stream);

/* The bf16 tensor-core form of sd_op_linear for callers that cannot allocate device memory
 * (the paper has no counterpart; this serves embedders).  A host that runs this library
 * inside its own serving loop, under a memory pool that already owns the whole device or in
 * a section where cudaMalloc is forbidden, has only the buffers it was handed: x
 * [rows][n_in] and w [n_out][n_in] as bf16 bit patterns, y [rows][n_out] fp32, all device
 * pointers owned by the caller.  The split accumulators that sd_op_linear keeps in a
 * caller-supplied workspace live here in an array of SD_STATIC_SCRATCH_BYTES that is part of
 * the library image on every GPU that loads it, for the life of the process.  The call
 * allocates and frees nothing.
 *  - Shapes whose accumulators do not fit (roughly rows > 32 at 148 SMs) return
 *    SD_ERR_CAPACITY; shapes the tensor-core kernel cannot take return SD_ERR_UNSUPPORTED.
 *  - The first call on a device looks up the array's device address (with that device
 *    current); make that first call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps whatever the last call left:
 *    the kernel overwrites every word it later reads, so nothing needs clearing, but two
 *    calls whose kernels overlap on the GPU (different streams, no ordering) race. */
#define SD_STATIC_SCRATCH_BYTES (8 * 1024 * 1024)
sd_status sd_op_linear_static(const void* x, const void* w, float* y, int rows, int n_out, int n_in, void* cuda_stream);

/* Attention of `rows` query rows against a cache laid out as the library lays
 * it out: k_cache/v_cache [n_slots][n_kv_heads][max_ctx][head_dim], q
 * [rows][n_heads][head_dim], row r belongs to slot row_slot[r] and sees
 * positions 0..row_pos[r]; out [rows][n_heads][head_dim].  dtype as above. */
sd_status sd_op_attention(const void* q, const void* k_cache, const void* v_cache, void* out,
                          const int32_t* row_slot, const int32_t* row_pos, int rows,
                          int n_heads, int n_kv_heads, int head_dim, int max_ctx, int dtype,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);
/* The same with the rows in runs of rows_per_seq consecutive rows of one sequence at consecutive positions (the
 * gamma + 1 rows of a verify step): the rows of a run share one pass over their sequence's cache, which is how the
 * verify step launches attention.  rows must be a multiple of rows_per_seq; the caller guarantees that the rows of a
 * run have one slot and positions p, p + 1, ... */
sd_status sd_op_attention_runs(const void* q, const void* k_cache, const void* v_cache, void* out,
                               const int32_t* row_slot, const int32_t* row_pos, int rows, int rows_per_seq,
                               int n_heads, int n_kv_heads, int head_dim, int max_ctx, int dtype,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t sd_op_attention_workspace(int rows, int n_heads, int head_dim, int max_ctx);

/* The Mamba-based prompt classifier of Section 2.4 / Section 3.3.3: embedding layer -> one Mamba (selective state-space)
 * layer -> average pooling over the prompt -> fully connected layer -> argmax.  The paper names the parts and cites the
 * Mamba paper for the layer; the layer is that paper's block: input projection to (u, z), causal depthwise convolution
 * (d_conv taps, zeros before the prompt) + SiLU, input-dependent (dt, B, C) with dt = softplus(W_dt r + b_dt),
 * h_t = exp(dt_t A) h_{t-1} + dt_t v_t B_t with A = -exp(a_log), y_t = h_t C_t + d_skip v_t, gate silu(z_t), output
 * projection; no residual connection, no normalisation.  All weights fp32, row-major, DEVICE pointers owned by the
 * caller (read during the call only):
 *   embed [vocab][d_model]   w_in [2*Di][d_model] (u rows first, then z), Di = expand * d_model
 *   w_conv [Di][d_conv]  b_conv [Di]   w_x [dt_rank + 2*d_state][Di] (r, B, C rows)   w_dt [Di][dt_rank]  b_dt [Di]
 *   a_log [Di][d_state]  d_skip [Di]   w_out [d_model][Di]   w_fc [n_classes][d_model]  b_fc [n_classes]
 * sd_mamba_classify scores n_prompts prompts in one go: prompt i is tokens_dev[starts_host[i] .. + lens_host[i]) (device
 * tokens, host offsets and lengths >= 1; token ids are clamped to the vocabulary); scores_dev [n_prompts][n_classes]
 * fp32 and labels_dev [n_prompts] int32 (argmax, lowest index on ties) are device buffers, either may be NULL.
 * workspace_dev: sd_mamba_workspace(desc, sum of lengths, n_prompts) bytes of device memory.  Long prompts are scanned
 * in chunks side by side.  Limits: d_state <= 16, d_conv <= 8, d_model <= 512, Di <= 1024 (else SD_ERR_UNSUPPORTED).
 * Copies small host tables to the device and synchronises the stream once before launching; the launches are
 * asynchronous on cuda_stream. */
typedef struct { int32_t vocab, d_model, d_state, d_conv, expand, n_classes, dt_rank; } sd_mamba_desc;
typedef struct {
    const float *embed, *w_in, *w_conv, *b_conv, *w_x, *w_dt, *b_dt, *a_log, *d_skip, *w_out, *w_fc, *b_fc;
} sd_mamba_weights;
size_t sd_mamba_workspace(const sd_mamba_desc* desc, int64_t total_tokens, int n_prompts);
sd_status sd_mamba_classify(const sd_mamba_desc* desc, const sd_mamba_weights* weights_dev, const int32_t* tokens_dev,
                            const int64_t* starts_host, const int32_t* lens_host, int n_prompts, float* scores_dev,
                            int32_t* labels_dev, void* workspace_dev, size_t workspace_bytes, void* cuda_stream);
/* Routes sequences with that classifier instead of the MLP: classifies the prompts of `seqs` (begun with sd_seq_begin)
 * and records class k as draft k, exactly as sd_route_prompt does with forced tasks.  n_classes must equal the
 * context's number of drafts.  draft_id_out (host, nullable) receives the ids.  Synchronises. */
sd_status sd_route_prompt_mamba(sd_ctx* ctx, const sd_mamba_desc* desc, const sd_mamba_weights* weights_dev,
                                const int32_t* seqs, int n_seq, void* workspace_dev, size_t workspace_bytes,
                                int32_t* draft_id_out);

/* One iteration of the K-means algorithm (Lloyd) over dense fp32 vectors: the offline task-partitioning step of
 * Section 3.2, which clusters 384-dimensional sentence vectors into one subset per task.
 *   labels[i]       = argmin_k sum_d (points[i][d] - centroids[k][d])^2, distances summed in fp32, lowest k on ties
 *   centroids_out   = mean of the points of each cluster (a cluster without points keeps its centroid); nullable
 *   counts_out[k]   = points per cluster (int64); nullable      inertia_out = sum of the chosen squared distances
 *                     under the INPUT centroids (double); nullable
 * points [n][dim] and centroids [k][dim] are device pointers, row-major, 16-byte aligned; dim a multiple of 128 up
 * to 512, 1 <= k <= 8 (else SD_ERR_UNSUPPORTED); labels int32 [n] on the device.  The caller owns every buffer; the
 * workspace (device, sd_kmeans_workspace bytes) holds per-block partial sums.  Sums are formed in a fixed order:
 * results are identical from run to run.  Asynchronous on cuda_stream.  Bound by the one pass over the points. */
sd_status sd_kmeans_step(const float* points_dev, int64_t n, int dim, const float* centroids_dev, int k,
                         int32_t* labels_dev, float* centroids_out_dev, int64_t* counts_out_dev, double* inertia_out_dev,
                         void* workspace_dev, size_t workspace_bytes, void* cuda_stream);
size_t sd_kmeans_workspace(int dim, int k);

/* Philox4x32-10 on the device: out[i][0..3] for ctr[i][0..3], one key.  For tests. */
sd_status sd_op_philox(const uint32_t* ctr_dev, int n, uint32_t key0, uint32_t key1, uint32_t* out_dev, void* cuda_stream);

/* softmax(logits / T) and one draw per row by the integer inverse CDF:
 * probs_dev [rows][V] out, tok_dev [rows] out, u_int in [1, 2^24] per row (device). */
sd_status sd_op_softmax_sample(const float* logits_dev, int rows, int V, float temperature,
                               const uint32_t* u_int_dev, float* probs_dev, int32_t* tok_dev, void* cuda_stream);

const char* sd_status_str(sd_status s);

#ifdef __cplusplus
}
#endif
#endif /* SD_H */
