// Host runtime behind the C ABI: arena layout, model tables, per-sequence bookkeeping and
// the launch sequences of the five hot calls.  Nothing here allocates device memory; all of
// it is carved out of the arena handed to sd_create.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <vector>

#include "gemm_tc.h"
#include "kernels.h"
#include "pass_stream.h"

using namespace sd;

namespace {

struct Bump {                       // bump allocator over the arena; base == nullptr just measures
    char* base;
    size_t off;
    void* take(size_t bytes) {
        off = (off + 255) & ~(size_t)255;
        void* p = base ? base + off : nullptr;
        off += bytes;
        return p;
    }
};

struct Layer {
    void* wqkv;                     // [(H + 2 Hkv) hd][d]: query rows, then key rows, then value rows
    void* wo;                       // [d][H hd]
    void* wgu;                      // [2F][d]: gate rows, then up rows
    void* wd;                       // [d][F]
    float* norm1;
    float* norm2;
    TensorMap tm_qkv, tm_wo, tm_gu, tm_wd;   // TMA descriptors of the four matrices (bf16 models)
    bf16* lora_b[4];                // low-rank adapters: [adapter][out feature][r] per matrix (QKV, Wo, gate/up, down); nullptr: none
};

struct Model {
    sd_model_desc d;
    size_t esz;
    void* embed;
    void* lm_head;
    float* final_norm;
    std::vector<Layer> layers;
    char* kcache;                   // [layer][slot][kv_head][position][head_dim]
    char* vcache;
    size_t kv_layer_bytes;
    float* rope_cos;                // [max_ctx][head_dim / 2]
    float* rope_sin;
    TensorMap tm_lm;
    bool tc;                        // the tensor-core path applies (bf16, shapes fit)
    PassMaps pmaps;                 // the layers' matrices as [layer][row][k] tensor maps (persistent streaming kernel)
    bool pass_ok;                   // ... which applies to this model
    bool lora;                      // the matrices carry one more 128-row tile: the adapters' A rows
    int n_qkv() const { return (d.n_heads + 2 * d.n_kv_heads) * d.head_dim; }
};

enum Phase { PH_FREE = 0, PH_BEGUN = 1, PH_ROUTED = 2, PH_READY = 3 };

}  // namespace

constexpr int STAMP_CAP = 1024;                 // launches of one pass whose time stamps can be kept
constexpr size_t XREADY_WORDS = 32768;          // readiness words of one pass (one per step kernel that feeds a GEMM and tile)
constexpr size_t ARRIVE_WORDS = 65536;          // arrival words of one pass (the 13B target needs about 17,000)
constexpr int PASS_ROWS_CAP = 32;               // most query rows of a pass on the persistent streaming kernel
constexpr size_t PASS_REGION_BYTES = (size_t)64 << 20;      // each of the two workspace regions of that kernel
constexpr size_t PASS_PROG_BYTES = (size_t)768 << 10;       // one cached program
constexpr int PASS_PROG_SLOTS = 8;

struct sd_ctx {
    sd_config cfg;
    std::vector<Model> models;
    cudaStream_t st;
    SeqState S;
    // scratch of one forward pass
    float* h; void* xn; void* q; void* attn; void* act; float* lin; float* draft_logits;
    int32_t* row_slot; int32_t* row_pos;
    void* attn_ws; size_t attn_ws_bytes;
    float* partials; size_t partials_bytes;     // split accumulators of the tensor-core GEMM
    float* ssq;                                 // [row][SSQ_STRIDE] pieces of sum h^2 for the folded RMSNorm
    uint32_t* gemm_arrive;                      // per GEMM of a pass and output tile: pieces that have arrived (zero between passes)
    size_t arrive_used;                         // words handed out to the GEMMs of the pass being enqueued
    // per-tile readiness of token rows between a step kernel and the GEMM after it (zeroed at the start of a pass that uses them)
    uint32_t* xready; size_t xready_used; bool xready_on;
    struct XReady { uint32_t* words; int n_tiles; int shift; uint32_t need; };
    XReady x_from;                              // what the most recent step kernel counts into (words == nullptr: nothing)
    float* rope_row_cos; float* rope_row_sin;   // [row][head_dim/2] rotary factors of the pass's rows (their positions applied)
    // Draft groups side by side: sequences routed to different draft models run their draft passes on streams of their own,
    // each with a scratch set of its own (set 0 is the fields above; sets 1... are sized for the draft models only).
    struct ScratchSet {
        float* h; void* xn; void* q; void* attn; void* act; float* lin; float* draft_logits; int32_t* row_slot; int32_t* row_pos;
        void* attn_ws; size_t attn_ws_bytes; float* partials; size_t partials_bytes; float* ssq; uint32_t* gemm_arrive; uint32_t* xready;
        float* rope_row_cos; float* rope_row_sin;
    };
    std::vector<ScratchSet> sets;
    std::vector<cudaStream_t> group_streams;    // streams of groups 1...
    std::vector<cudaEvent_t> ev_join;
    cudaEvent_t ev_fork;
    bool groups_concurrent;
    // persistent streaming kernel (pass_stream.cu): packed input rows, workspace, programs
    // (everything CTAs of that kernel hand to one another is tagged 64-bit words; the whole block is cleared when tags are about to repeat)
    tagged_t* tg_h; tagged_t* tg_xn; tagged_t* tg_attn; tagged_t* tg_act; tagged_t* tg_q; tagged_t* tg_newkv; tagged_t* tg_ssq;
    tagged_t* tg_partials[2];
    tagged_t* tg_part_o; tagged_t* tg_part_ml;
    char* tg_begin; char* tg_end;               // extent of the tagged buffers
    uint32_t* pass_epoch;                       // device: number of the pass; pass_epoch + 1: the abort word
    uint64_t pass_count;                        // host: passes enqueued so far (mirrors the device word)
    bool tags_due_clear;                        // the tagged buffers are to be cleared before the next launch sequence
    uint8_t* pass_prog;
    bool pass_on, pass_drafts; int pass_max_rows;
    PassTuning pass_tuning; bool pass_tuned; int pass_stages;
    struct CachedProgram { int model, m_tok, rows_per_seq, n_splits, want_logits, slot; PassProgram meta; uint64_t last_use; };
    std::vector<CachedProgram> programs;
    unsigned long long* stamps; size_t stamps_words;          // optional time stamps of the next passes (caller's buffer)
    bool two_part;                              // feed the verify rows' activations to the GEMMs in two bf16 parts (see Epilogue::lo_off)
    bool force_plain;                           // run the CUDA-core kernels even where the tensor-core path applies
    bool graphs_on;                             // replay captured CUDA graphs for repeated calls
    struct CachedGraph { std::vector<uint8_t> key; cudaGraphExec_t exec; uint64_t launches; uint64_t last_use; uint64_t passes; std::vector<int32_t> stamp_kinds; };
    std::vector<CachedGraph> graphs;
    uint64_t graph_clock;
    // classifier
    float* clf_w1; float* clf_b1; float* clf_w2; float* clf_b2; bool clf_loaded;
    // host bookkeeping
    std::vector<int> phase, len_ub, n_prompt, draft_id;
    size_t arena_used;
    // staging for the host-buffer entry point
    int32_t* st_x; float* st_q; float* st_logits; int32_t* st_nacc; int32_t* st_out;
    float* alpha_terms;                         // [seq of the call][gamma]: sum_k min(p, q) of the last sd_accept_seqs, consumed by sd_kv_rollback
    // optional timing of the draft and target passes (the cost ratio c of Eq. 1 from the library's own clock)
    bool cost_on; int cost_depth;
    // optional time stamps of the launches of a forward pass on the kernel-per-matrix path
    int tune[SD_TUNE_COUNT];                    // measurement knobs (sd_tuning)
    bool stamps_on; unsigned long long* stamp_buf; std::vector<int32_t> stamp_kinds;
    struct CostMark { cudaEvent_t e0, e1; int kind; int units; };
    std::vector<CostMark> cost_pending;
    std::vector<cudaEvent_t> cost_free;
    double cost_ms[3]; uint64_t cost_units[3];  // 0 draft passes, 1 verify passes, 2 single-row target passes
    // launch accounting and optional per-category timing
    uint64_t launches;
    bool prof_on;
    std::vector<cudaEvent_t> prof_ev;
    std::vector<int> prof_cat;
    size_t prof_used;
};

namespace {

size_t esize(int dtype) { return dtype == SD_BF16 ? 2 : 4; }

int sm_count() {                               // of the current device
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) return v;
    return 148;
}

bool valid_desc(const sd_model_desc& m) {
    if (m.n_layers < 1 || m.d_model < 8 || m.n_heads < 1 || m.n_kv_heads < 1 || m.d_ffn < 8 || m.vocab < 2) return false;
    if (m.n_heads % m.n_kv_heads) return false;
    if (m.head_dim < 8 || m.head_dim > 256 || (m.head_dim & 7)) return false;
    if (m.dtype != SD_F32 && m.dtype != SD_BF16) return false;
    if ((m.d_model & 7) || (m.d_ffn & 7)) return false;
    return true;
}

// Contexts with low-rank adapters hold ONE draft model (models[1]) shared by all tasks.
int n_models(const sd_config& cfg) { return 1 + (cfg.lora_adapters > 0 ? 1 : cfg.n_drafts); }
int draft_model_index(const sd_config& cfg, int task) { return cfg.lora_adapters > 0 ? 1 : 1 + task; }
size_t tile_rows(size_t n) { return (n + 127) / 128 * 128; }

bool valid_cfg(const sd_config* c, const sd_model_desc* ms) {
    if (!c || !ms) return false;
    if (c->max_seqs < 1 || c->max_seqs > SD_MAX_BATCH || c->max_ctx < 4 || c->max_gamma < 0 || c->max_gamma > SD_MAX_GAMMA) return false;
    if (c->n_drafts < 0 || c->n_drafts > 16 || !(c->temperature >= 0.f) || c->clf_d_hidden < 0) return false;
    if (c->lora_adapters < 0) return false;
    if (c->lora_adapters > 0) {
        if (c->lora_adapters != c->n_drafts || c->lora_rank < 8 || c->lora_rank > 32 || (c->lora_rank & 7) ||
            c->lora_adapters * c->lora_rank > 128 || !(c->lora_scale == c->lora_scale))
            return false;
    }
    for (int i = 0; i < n_models(*c); ++i) {
        if (!valid_desc(ms[i])) return false;
        if (ms[i].vocab != ms[0].vocab) return false;        // draft and target share the vocabulary
    }
    if (c->lora_adapters > 0) {                              // adapters ride on the tensor-core path: whole tiles of bf16
        const sd_model_desc& m = ms[1];
        if (m.dtype != SD_BF16 || ((m.n_heads + 2 * m.n_kv_heads) * m.head_dim) % 128 || m.d_model % 128 || (2 * m.d_ffn) % 128) return false;
    }
    return true;
}

// The single place that decides where everything lives.  Run once with a null base to size
// the arena, once more with the real base to place the pointers.
void layout(sd_ctx* c, const sd_model_desc* ms, Bump& B) {
    const sd_config& cfg = c->cfg;
    const int S = cfg.max_seqs, nm = n_models(cfg);
    c->models.resize(nm);
    int d_max = 0, f_max = 0, qkv_max = 0, dq_max = 0, lin_max = 0;
    for (int i = 0; i < nm; ++i) {
        Model& M = c->models[i];
        M.d = ms[i];
        M.esz = esize(ms[i].dtype);
        const sd_model_desc& m = M.d;
        const size_t dq = (size_t)m.n_heads * m.head_dim, dkv = (size_t)m.n_kv_heads * m.head_dim;
        M.embed = B.take((size_t)m.vocab * m.d_model * M.esz);
        M.lm_head = B.take((size_t)m.vocab * m.d_model * M.esz);
        M.final_norm = (float*)B.take(sizeof(float) * m.d_model);
        M.layers.resize(m.n_layers);
        M.lora = cfg.lora_adapters > 0 && i == 1;
        const size_t extra = M.lora ? 128 : 0;               // one more tile of rows per matrix: A of every adapter
        const size_t n_lb = M.lora ? (size_t)cfg.lora_adapters * cfg.lora_rank : 0;
        for (int l = 0; l < m.n_layers; ++l) {
            Layer& L = M.layers[l];
            L.wqkv = B.take((dq + 2 * dkv + extra) * m.d_model * M.esz);
            L.wo = B.take(((size_t)m.d_model + extra) * dq * M.esz);
            L.wgu = B.take(((size_t)2 * m.d_ffn + extra) * m.d_model * M.esz);
            L.wd = B.take(((size_t)m.d_model + extra) * m.d_ffn * M.esz);
            L.norm1 = (float*)B.take(sizeof(float) * m.d_model);
            L.norm2 = (float*)B.take(sizeof(float) * m.d_model);
            const size_t outs[4] = {dq + 2 * dkv, (size_t)m.d_model, (size_t)2 * m.d_ffn, (size_t)m.d_model};
            for (int k = 0; k < 4; ++k) L.lora_b[k] = M.lora ? (bf16*)B.take(n_lb * outs[k] * sizeof(bf16)) : nullptr;
        }
        M.kv_layer_bytes = (size_t)S * dkv * cfg.max_ctx * M.esz;
        M.kcache = (char*)B.take(M.kv_layer_bytes * m.n_layers);
        M.vcache = (char*)B.take(M.kv_layer_bytes * m.n_layers);
        M.rope_cos = (float*)B.take(sizeof(float) * (size_t)cfg.max_ctx * (m.head_dim / 2));
        M.rope_sin = (float*)B.take(sizeof(float) * (size_t)cfg.max_ctx * (m.head_dim / 2));
        d_max = std::max(d_max, m.d_model);
        f_max = std::max(f_max, m.d_ffn);
        qkv_max = std::max(qkv_max, M.n_qkv());
        dq_max = std::max(dq_max, (int)dq);
        lin_max = std::max(lin_max, std::max(std::max(M.n_qkv(), 2 * m.d_ffn), m.d_model));
    }
    const size_t R = SD_MAX_ROWS;
    c->S.len = (int32_t*)B.take(sizeof(int32_t) * S);
    c->S.tkv = (int32_t*)B.take(sizeof(int32_t) * S);
    c->S.dkv = (int32_t*)B.take(sizeof(int32_t) * S);
    c->S.iter = (uint32_t*)B.take(sizeof(uint32_t) * S);
    c->S.seq_id = (uint32_t*)B.take(sizeof(uint32_t) * S);
    c->S.draft_id = (int32_t*)B.take(sizeof(int32_t) * S);
    c->S.n_prompt = (int32_t*)B.take(sizeof(int32_t) * S);
    c->S.counters = (int64_t*)B.take(sizeof(int64_t) * 4 * S);
    c->S.alpha_sum = (double*)B.take(sizeof(double) * S);
    c->S.judged = (int64_t*)B.take(sizeof(int64_t) * S);
    c->S.tok_stride = cfg.max_ctx + 1;
    c->S.max_ctx = cfg.max_ctx;
    c->S.tokens = (int32_t*)B.take(sizeof(int32_t) * (size_t)S * c->S.tok_stride);
    c->S.status = (uint32_t*)B.take(sizeof(uint32_t));
    c->h = (float*)B.take(sizeof(float) * R * d_max);
    c->xn = B.take(4 * R * d_max);
    c->q = B.take(4 * R * dq_max);
    c->attn = B.take(4 * R * dq_max);
    c->act = B.take(4 * R * f_max);
    c->lin = (float*)B.take(sizeof(float) * R * lin_max);
    c->draft_logits = (float*)B.take(sizeof(float) * (size_t)SD_MAX_BATCH * ms[0].vocab);
    c->row_slot = (int32_t*)B.take(sizeof(int32_t) * 2 * R);          // [row] slot, then [row] task of the slot (draft / adapter id)
    c->row_pos = (int32_t*)B.take(sizeof(int32_t) * R);
    c->attn_ws_bytes = 0;
    for (int i = 0; i < nm; ++i)
        c->attn_ws_bytes = std::max(c->attn_ws_bytes, attention_split_supported(ms[i].dtype, ms[i].n_heads, ms[i].n_kv_heads, ms[i].head_dim)
                                        ? attention_split_workspace((int)R, ms[i].n_heads, ms[i].head_dim, cfg.max_ctx)
                                        : attention_workspace_bytes((int)R, ms[i].n_heads, ms[i].head_dim, cfg.max_ctx));
    c->attn_ws = B.take(c->attn_ws_bytes);
    c->partials_bytes = 0;
    for (int i = 0; i < nm; ++i) {
        const sd_model_desc& m = ms[i];
        if (m.dtype != SD_BF16) continue;
        const int shapes[5][2] = {{(m.n_heads + 2 * m.n_kv_heads) * m.head_dim, m.d_model}, {m.d_model, m.n_heads * m.head_dim},
                                  {2 * m.d_ffn, m.d_model}, {m.d_model, m.d_ffn}, {m.vocab, m.d_model}};
        for (auto& s : shapes)
            c->partials_bytes = std::max(c->partials_bytes, gemm_partials_bytes(gemm_geometry(SD_MAX_ROWS, s[0], s[1], sm_count(), 0, false, 1)));
    }
    c->partials = (float*)B.take(c->partials_bytes);
    c->ssq = (float*)B.take(sizeof(float) * SD_MAX_ROWS * SSQ_STRIDE);
    c->gemm_arrive = (uint32_t*)B.take(sizeof(uint32_t) * ARRIVE_WORDS);
    c->arrive_used = 0;
    size_t half_max = 1;
    for (int i = 0; i < nm; ++i) half_max = std::max(half_max, (size_t)ms[i].head_dim / 2);
    c->rope_row_cos = (float*)B.take(sizeof(float) * SD_MAX_ROWS * half_max);
    c->rope_row_sin = (float*)B.take(sizeof(float) * SD_MAX_ROWS * half_max);
    c->xready = (uint32_t*)B.take(sizeof(uint32_t) * XREADY_WORDS);
    c->xready_used = 0;
    c->sets.clear();
    c->sets.push_back(sd_ctx::ScratchSet{c->h, c->xn, c->q, c->attn, c->act, c->lin, c->draft_logits, c->row_slot, c->row_pos, c->attn_ws,
                                         c->attn_ws_bytes, c->partials, c->partials_bytes, c->ssq, c->gemm_arrive, c->xready, c->rope_row_cos,
                                         c->rope_row_sin});
    if (cfg.n_drafts >= 2 && cfg.lora_adapters == 0) {       // one more scratch set per further draft group, sized for the drafts
        int dd = 0, df = 0, dqm = 0, dlin = 0;
        size_t dhalf = 1, d_ws = 0, d_part = 0;
        for (int i = 1; i < nm; ++i) {
            const sd_model_desc& m = ms[i];
            const int dq = m.n_heads * m.head_dim, nqkv = (m.n_heads + 2 * m.n_kv_heads) * m.head_dim;
            dd = std::max(dd, (int)m.d_model); df = std::max(df, (int)m.d_ffn); dqm = std::max(dqm, dq);
            dlin = std::max(dlin, std::max(std::max(nqkv, 2 * (int)m.d_ffn), (int)m.d_model));
            dhalf = std::max(dhalf, (size_t)m.head_dim / 2);
            d_ws = std::max(d_ws, attention_split_supported(m.dtype, m.n_heads, m.n_kv_heads, m.head_dim)
                                      ? attention_split_workspace((int)R, m.n_heads, m.head_dim, cfg.max_ctx)
                                      : attention_workspace_bytes((int)R, m.n_heads, m.head_dim, cfg.max_ctx));
            if (m.dtype == SD_BF16) {
                const int shapes[5][2] = {{nqkv, m.d_model}, {m.d_model, dq}, {2 * m.d_ffn, m.d_model}, {m.d_model, m.d_ffn}, {m.vocab, m.d_model}};
                for (auto& sh : shapes) d_part = std::max(d_part, gemm_partials_bytes(gemm_geometry(SD_MAX_ROWS, sh[0], sh[1], sm_count(), 0, false, 1)));
            }
        }
        for (int k = 1; k < cfg.n_drafts; ++k) {
            sd_ctx::ScratchSet s;
            s.h = (float*)B.take(sizeof(float) * R * dd);
            s.xn = B.take(4 * R * dd); s.q = B.take(4 * R * dqm); s.attn = B.take(4 * R * dqm); s.act = B.take(4 * R * df);
            s.lin = (float*)B.take(sizeof(float) * R * dlin);
            s.draft_logits = (float*)B.take(sizeof(float) * (size_t)SD_MAX_BATCH * ms[0].vocab);
            s.row_slot = (int32_t*)B.take(sizeof(int32_t) * 2 * R); s.row_pos = (int32_t*)B.take(sizeof(int32_t) * R);
            s.attn_ws_bytes = d_ws; s.attn_ws = B.take(d_ws);
            s.partials_bytes = d_part; s.partials = (float*)B.take(d_part);
            s.ssq = (float*)B.take(sizeof(float) * SD_MAX_ROWS * SSQ_STRIDE);
            s.gemm_arrive = (uint32_t*)B.take(sizeof(uint32_t) * ARRIVE_WORDS);
            s.xready = (uint32_t*)B.take(sizeof(uint32_t) * XREADY_WORDS);
            s.rope_row_cos = (float*)B.take(sizeof(float) * SD_MAX_ROWS * dhalf);
            s.rope_row_sin = (float*)B.take(sizeof(float) * SD_MAX_ROWS * dhalf);
            c->sets.push_back(s);
        }
    }
    {   // persistent streaming kernel: tagged 64-bit words for up to PASS_ROWS_CAP rows (padded to a multiple of 16)
        const size_t rows_pad = (PASS_ROWS_CAP + 15) & ~15;
        int h_max = 1, hd_max = 8, kvd_max = 8;
        for (int i = 0; i < nm; ++i) {
            h_max = std::max(h_max, (int)ms[i].n_heads); hd_max = std::max(hd_max, (int)ms[i].head_dim);
            kvd_max = std::max(kvd_max, (int)(ms[i].n_kv_heads * ms[i].head_dim));
        }
        c->tg_begin = (char*)B.take(0);
        c->tg_h = (tagged_t*)B.take(sizeof(tagged_t) * rows_pad * d_max);
        c->tg_xn = (tagged_t*)B.take(sizeof(tagged_t) * (size_t)((d_max + 63) / 64) * rows_pad * 32);
        c->tg_attn = (tagged_t*)B.take(sizeof(tagged_t) * (size_t)((dq_max + 63) / 64) * rows_pad * 32);
        c->tg_act = (tagged_t*)B.take(sizeof(tagged_t) * (size_t)((f_max + 63) / 64) * rows_pad * 32);
        c->tg_q = (tagged_t*)B.take(sizeof(tagged_t) * rows_pad * (dq_max / 2));
        c->tg_newkv = (tagged_t*)B.take(sizeof(tagged_t) * rows_pad * 2 * (kvd_max / 2));
        c->tg_ssq = (tagged_t*)B.take(sizeof(tagged_t) * rows_pad * SSQ_STRIDE);
        c->tg_partials[0] = (tagged_t*)B.take(PASS_REGION_BYTES);
        c->tg_partials[1] = (tagged_t*)B.take(PASS_REGION_BYTES);
        c->tg_part_o = (tagged_t*)B.take(sizeof(tagged_t) * (size_t)PASS_ROWS_CAP * h_max * 32 * hd_max);
        c->tg_part_ml = (tagged_t*)B.take(sizeof(tagged_t) * (size_t)PASS_ROWS_CAP * h_max * 32 * 2);
        c->tg_end = (char*)B.take(0);
        c->pass_epoch = (uint32_t*)B.take(sizeof(uint32_t) * 2);
        c->pass_prog = (uint8_t*)B.take(PASS_PROG_BYTES * PASS_PROG_SLOTS);
    }
    const size_t V0 = ms[0].vocab, g_max = std::max(cfg.max_gamma, 1);
    c->st_x = (int32_t*)B.take(sizeof(int32_t) * S * g_max);
    c->st_q = (float*)B.take(sizeof(float) * S * g_max * V0);
    c->st_logits = (float*)B.take(sizeof(float) * std::min((size_t)SD_MAX_ROWS, (size_t)S * (cfg.max_gamma + 1)) * V0);
    c->alpha_terms = (float*)B.take(sizeof(float) * S * g_max);
    c->stamp_buf = (unsigned long long*)B.take(sizeof(unsigned long long) * ST_WORDS * STAMP_CAP);
    c->st_nacc = (int32_t*)B.take(sizeof(int32_t) * S);
    c->st_out = (int32_t*)B.take(sizeof(int32_t) * S * (cfg.max_gamma + 1));
    if (cfg.clf_d_hidden > 0 && cfg.n_drafts > 0) {
        c->clf_w1 = (float*)B.take(sizeof(float) * (size_t)cfg.clf_d_hidden * ms[0].d_model);
        c->clf_b1 = (float*)B.take(sizeof(float) * cfg.clf_d_hidden);
        c->clf_w2 = (float*)B.take(sizeof(float) * (size_t)cfg.n_drafts * cfg.clf_d_hidden);
        c->clf_b2 = (float*)B.take(sizeof(float) * cfg.n_drafts);
    } else {
        c->clf_w1 = c->clf_b1 = c->clf_w2 = c->clf_b2 = nullptr;
    }
}

#define CUDA_TRY(expr)                                                                     \
    do {                                                                                   \
        cudaError_t e__ = (expr);                                                          \
        if (e__ != cudaSuccess) {                                                          \
            fprintf(stderr, "[sd] CUDA error %s at %s:%d\n", cudaGetErrorString(e__), __FILE__, __LINE__); \
            return SD_ERR_CUDA;                                                            \
        }                                                                                  \
    } while (0)
#define SD_TRY(expr)                      \
    do {                                  \
        sd_status s__ = (expr);           \
        if (s__ != SD_OK) return s__;     \
    } while (0)

// Categories of the optional per-kernel timing (sd_profile).
enum { CAT_LINEAR = 0, CAT_ATTENTION = 1, CAT_ELEMENTWISE = 2, CAT_SAMPLING = 3, CAT_STATE = 4, CAT_FUSED_STEP = 5, CAT_NONE = 6 };

// When profiling is on, an event is recorded in front of every launch and tagged with the
// category of that launch; sd_profile_read adds up the gaps between consecutive events.
cudaError_t prof_mark(sd_ctx* c, int cat) {
    if (!c->prof_on) return cudaSuccess;
    if (c->prof_used == c->prof_ev.size()) {
        cudaEvent_t e;
        cudaError_t err = cudaEventCreate(&e);
        if (err != cudaSuccess) return err;
        c->prof_ev.push_back(e);
        c->prof_cat.push_back(CAT_NONE);
    }
    c->prof_cat[c->prof_used] = cat;
    return cudaEventRecord(c->prof_ev[c->prof_used++], c->st);
}

#define LAUNCH(cat, expr)                 \
    do {                                  \
        CUDA_TRY(prof_mark(c, cat));      \
        CUDA_TRY(expr);                   \
        c->launches += 1;                 \
    } while (0)

sd_status linear(sd_ctx* c, const void* x, const void* w, float* y, int rows, int n_out, int n_in, int dtype) {
    LAUNCH(CAT_LINEAR, launch_linear_simt(x, w, y, rows, n_out, n_in, dtype, c->st));
    return SD_OK;
}

enum LogitsMode { LOGITS_NONE = 0, LOGITS_ALL = 1, LOGITS_LAST = 2 };

// One pass of a model over n_rows query rows described by `plan`.
sd_status forward_tc(sd_ctx* c, Model& M, const SeqList& list, const RowPlan& plan, int n_rows, int mode, float* logits_out);

// The tags of a pass derive from its number (a device word that every pass bumps).  Well before numbers repeat, every tagged
// word is cleared: note_passes counts, clear_tags_if_due runs between launch sequences (never inside a capture).
void note_passes(sd_ctx* c, uint64_t n) {
    const uint64_t period = PASS_EPOCH_WRAP / 2;
    if ((c->pass_count + n) / period != c->pass_count / period) c->tags_due_clear = true;
    c->pass_count += n;
}

cudaError_t clear_tags_if_due(sd_ctx* c) {
    if (!c->tags_due_clear) return cudaSuccess;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(c->st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return cudaSuccess;
    c->tags_due_clear = false;
    return cudaMemsetAsync(c->tg_begin, 0, c->tg_end - c->tg_begin, c->st);
}

sd_ctx::CachedProgram* find_program(sd_ctx* c, int model, int m_tok, int rows_per_seq, int n_splits, int want_logits) {
    for (auto& p : c->programs)
        if (p.model == model && p.m_tok == m_tok && p.rows_per_seq == rows_per_seq && p.n_splits == n_splits && p.want_logits == want_logits) return &p;
    return nullptr;
}

// Slices of the cache per (query block, kv head) on the persistent kernel: about one attention item per SM, slices
// of at most 2048 positions.
int pass_splits(const sd_model_desc& m, int n_rows, int rows_per_seq, int ctx_bound) {
    const int grp = m.n_heads / m.n_kv_heads;
    const int rpb = std::max(1, std::min(rows_per_seq, 16 / std::max(1, grp)));
    const int n_blocks = (n_rows / rows_per_seq) * ((rows_per_seq + rpb - 1) / rpb);
    int ns = std::max(1, sm_count() / std::max(1, n_blocks * m.n_kv_heads));
    ns = std::min(ns, std::max(1, ctx_bound / 64));                        // a slice is worth at least one chunk of keys
    ns = std::max(ns, (ctx_bound + 2047) / 2048);
    return std::max(1, std::min(32, ns));
}

bool pass_wanted(sd_ctx* c, const Model& M, const RowPlan& plan, int n_rows) {
    return c->pass_on && (&M == &c->models[0] || c->pass_drafts) && M.tc && M.pass_ok && !c->force_plain && n_rows <= c->pass_max_rows && n_rows <= PASS_ROWS_CAP &&
           plan.rows_per_seq >= 1 && n_rows % plan.rows_per_seq == 0;
}

// Makes sure the program of a pass is built and in device memory.  Called by the entry points before anything is
// captured into a graph (the upload is an ordinary copy followed by a synchronisation).
sd_status prepare_pass(sd_ctx* c, int model, const RowPlan& plan, int n_rows, int mode) {
    Model& M = c->models[model];
    if (!pass_wanted(c, M, plan, n_rows)) return SD_OK;
    const sd_model_desc& m = M.d;
    const int ns = pass_splits(m, n_rows, plan.rows_per_seq, plan.ctx_bound), want = mode != 0 ? 1 : 0;
    c->graph_clock += 1;
    if (sd_ctx::CachedProgram* p = find_program(c, model, n_rows, plan.rows_per_seq, ns, want)) { p->last_use = c->graph_clock; return SD_OK; }
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(c->st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return SD_ERR_STATE;
    PassShape sh{m.n_layers, m.d_model, m.n_heads, m.n_kv_heads, m.head_dim, m.d_ffn, m.vocab, n_rows, plan.rows_per_seq, ns, want, sm_count()};
    sd_ctx::CachedProgram cp;
    cp.model = model; cp.m_tok = n_rows; cp.rows_per_seq = plan.rows_per_seq; cp.n_splits = ns; cp.want_logits = want; cp.last_use = c->graph_clock;
    cp.meta = build_pass_program(sh, c->pass_tuned ? c->pass_tuning : default_pass_tuning(sh));
    const bool fits = cp.meta.error.empty() && cp.meta.blob.size() <= PASS_PROG_BYTES && cp.meta.max_section <= 8192 &&
                      (size_t)std::max(cp.meta.slots[0], cp.meta.slots[1]) * n_rows * 128 * sizeof(tagged_t) <= PASS_REGION_BYTES &&
                      m.n_layers < 255;
    if (!fits) {                                      // remembered, so that the pass quietly takes the kernel-per-matrix path
        cp.slot = -1; cp.meta.blob.clear();
        c->programs.push_back(cp);
        return SD_OK;
    }
    int slot = -1;
    std::vector<bool> used(PASS_PROG_SLOTS, false);
    for (auto& p : c->programs) if (p.slot >= 0) used[p.slot] = true;
    for (int i = 0; i < PASS_PROG_SLOTS; ++i) if (!used[i]) { slot = i; break; }
    if (slot < 0) {
        // every slot is taken: drop the least recently used program, and the graphs that may have captured its address
        size_t victim = c->programs.size();
        for (size_t i = 0; i < c->programs.size(); ++i)
            if (c->programs[i].slot >= 0 && (victim == c->programs.size() || c->programs[i].last_use < c->programs[victim].last_use)) victim = i;
        CUDA_TRY(cudaStreamSynchronize(c->st));
        for (auto& g : c->graphs) cudaGraphExecDestroy(g.exec);
        c->graphs.clear();
        slot = c->programs[victim].slot;
        c->programs.erase(c->programs.begin() + victim);
    }
    cp.slot = slot;
    CUDA_TRY(cudaMemcpyAsync(c->pass_prog + (size_t)slot * PASS_PROG_BYTES, cp.meta.blob.data(), cp.meta.blob.size(), cudaMemcpyHostToDevice, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
    cp.meta.blob.clear(); cp.meta.blob.shrink_to_fit();
    c->programs.push_back(cp);
    return SD_OK;
}

sd_status forward_pass(sd_ctx* c, Model& M, const sd_ctx::CachedProgram& cp, const SeqList& list, const RowPlan& plan, int n_rows, int mode,
                       float* logits_out);

sd_status forward(sd_ctx* c, Model& M, const SeqList& list, const RowPlan& plan, int n_rows, int mode, float* logits_out) {
    if (pass_wanted(c, M, plan, n_rows)) {
        const int model = (int)(&M - &c->models[0]);
        SD_TRY(prepare_pass(c, model, plan, n_rows, mode));
        const sd_ctx::CachedProgram* cp = find_program(c, model, n_rows, plan.rows_per_seq, pass_splits(M.d, n_rows, plan.rows_per_seq, plan.ctx_bound), mode != 0 ? 1 : 0);
        if (cp && cp->slot >= 0) return forward_pass(c, M, *cp, list, plan, n_rows, mode, logits_out);
    }
    if (M.tc && !c->force_plain) return forward_tc(c, M, list, plan, n_rows, mode, logits_out);
    const sd_model_desc& m = M.d;
    const int d = m.d_model, H = m.n_heads, Hkv = m.n_kv_heads, hd = m.head_dim, F = m.d_ffn, dt = m.dtype;
    cudaStream_t st = c->st;
    LAUNCH(CAT_ELEMENTWISE, launch_embed(c->S, list, plan, n_rows, M.embed, dt, d, m.vocab, c->h, c->row_slot, c->row_pos,
                                         nullptr, nullptr, nullptr, nullptr, nullptr, 0, nullptr, nullptr, 0, nullptr, st));
    for (int l = 0; l < m.n_layers; ++l) {
        const Layer& L = M.layers[l];
        void* kc = M.kcache + M.kv_layer_bytes * l;
        void* vc = M.vcache + M.kv_layer_bytes * l;
        LAUNCH(CAT_ELEMENTWISE, launch_rmsnorm(c->h, L.norm1, c->xn, dt, n_rows, d, m.rms_eps, 1, 0, st));
        SD_TRY(linear(c, c->xn, L.wqkv, c->lin, n_rows, M.n_qkv(), d, dt));
        LAUNCH(CAT_ELEMENTWISE, launch_rope_kv(c->lin, c->q, kc, vc, dt, c->row_slot, c->row_pos, n_rows, H, Hkv, hd, c->cfg.max_ctx,
                                M.rope_cos, M.rope_sin, c->S.status, st));
        LAUNCH(CAT_ATTENTION, launch_attention(c->q, kc, vc, c->attn, dt, c->row_slot, c->row_pos, n_rows, H, Hkv, hd, c->cfg.max_ctx,
                                  c->attn_ws, c->attn_ws_bytes, st));
        SD_TRY(linear(c, c->attn, L.wo, c->lin, n_rows, d, H * hd, dt));
        LAUNCH(CAT_ELEMENTWISE, launch_residual_add(c->h, c->lin, (size_t)n_rows * d, st));
        LAUNCH(CAT_ELEMENTWISE, launch_rmsnorm(c->h, L.norm2, c->xn, dt, n_rows, d, m.rms_eps, 1, 0, st));
        SD_TRY(linear(c, c->xn, L.wgu, c->lin, n_rows, 2 * F, d, dt));
        LAUNCH(CAT_ELEMENTWISE, launch_swiglu(c->lin, c->act, dt, n_rows, F, M.tc ? 1 : 0, st));
        SD_TRY(linear(c, c->act, L.wd, c->lin, n_rows, d, F, dt));
        LAUNCH(CAT_ELEMENTWISE, launch_residual_add(c->h, c->lin, (size_t)n_rows * d, st));
    }
    if (mode == LOGITS_ALL) {
        LAUNCH(CAT_ELEMENTWISE, launch_rmsnorm(c->h, M.final_norm, c->xn, dt, n_rows, d, m.rms_eps, 1, 0, st));
        SD_TRY(linear(c, c->xn, M.lm_head, logits_out, n_rows, m.vocab, d, dt));
    } else if (mode == LOGITS_LAST) {
        const int R = plan.rows_per_seq;
        LAUNCH(CAT_ELEMENTWISE, launch_rmsnorm(c->h, M.final_norm, c->xn, dt, list.n, d, m.rms_eps, R, R - 1, st));
        SD_TRY(linear(c, c->xn, M.lm_head, logits_out, list.n, m.vocab, d, dt));
    }
    CUDA_TRY(prof_mark(c, CAT_NONE));
    return SD_OK;
}

// Makes scratch set k the one the forward pass uses (pointers are read when a launch is enqueued).
void use_set(sd_ctx* c, size_t k) {
    const sd_ctx::ScratchSet& s = c->sets[k];
    c->h = s.h; c->xn = s.xn; c->q = s.q; c->attn = s.attn; c->act = s.act; c->lin = s.lin; c->draft_logits = s.draft_logits;
    c->row_slot = s.row_slot; c->row_pos = s.row_pos; c->attn_ws = s.attn_ws; c->attn_ws_bytes = s.attn_ws_bytes;
    c->partials = s.partials; c->partials_bytes = s.partials_bytes; c->ssq = s.ssq; c->gemm_arrive = s.gemm_arrive; c->xready = s.xready;
    c->rope_row_cos = s.rope_row_cos; c->rope_row_sin = s.rope_row_sin;
}

// The next record of the stamp buffer (nullptr when stamps are off or the buffer is full); kind: SD_STAMP_* | detail << 8.
unsigned long long* next_stamp(sd_ctx* c, int kind) {
    if (!c->stamps_on || (int)c->stamp_kinds.size() >= STAMP_CAP) return nullptr;
    c->stamp_kinds.push_back(kind);
    return c->stamp_buf + (size_t)ST_WORDS * (c->stamp_kinds.size() - 1);
}

// One weight GEMM and the step that follows it.
sd_status gemm_tc(sd_ctx* c, const TensorMap& tw, const void* x, int rows, int n_out, int K, const Epilogue& ep) {
    if (ep.lo_off) rows += ep.lo_off;           // the input rows come in two bf16 parts: [x_hi rows][x_lo rows at + lo_off]
    GemmGeom g = gemm_geometry(rows, n_out, K, sm_count(), ep.ring_stages, ep.prefill_all != 0, ep.lora_b ? 1 : 0);
    if (ep.lo_off) { g.lo_off = ep.lo_off; g.m_real = ep.m_real; }
    if (c->tune[SD_TUNE_PACE_NS] == 1) { g.pace_ns = 0; g.prefill = g.m_pad > 16 ? g.stages : std::min(g.stages, 7); }
    else if (c->tune[SD_TUNE_PACE_NS] > 1) g.pace_ns = c->tune[SD_TUNE_PACE_NS];
    if (c->tune[SD_TUNE_PREFILL_STAGES] >= 2) g.prefill = std::min(g.stages, c->tune[SD_TUNE_PREFILL_STAGES]);
    if (c->tune[SD_TUNE_STEADY_STAGES] >= 2) g.steady = std::min(g.stages, c->tune[SD_TUNE_STEADY_STAGES]);
    Epilogue eps = ep;
    eps.many_rows_cb = c->tune[SD_TUNE_MANY_ROWS_CB];
    // token rows tile by tile: this GEMM watches the words the step kernel before it counts into (if that kernel wrote
    // these rows), and its own step kernel gets words of its own when what it writes feeds the next GEMM
    if (c->x_from.words && c->x_from.n_tiles >= ((g.kb_per_tile - 1) >> c->x_from.shift) + 1) {
        g.xr = c->x_from.words; g.xr_shift = c->x_from.shift; g.xr_need = c->x_from.need;
    }
    c->x_from.words = nullptr;
    const bool feeds_gemm = ep.mode == EPI_SWIGLU || (ep.mode == EPI_RESIDUAL && ep.gain_next != nullptr);
    const int step_tiles = (n_out + 127) / 128;
    if (c->xready_on && feeds_gemm && !ep.lora_b && c->xready_used + (size_t)step_tiles <= XREADY_WORDS) {
        eps.xready = c->xready + c->xready_used;
        c->xready_used += (size_t)step_tiles;
        c->x_from = sd_ctx::XReady{eps.xready, step_tiles, ep.mode == EPI_SWIGLU ? 0 : 1, (uint32_t)fused_step_row_batches(g, ep)};
    }
    g.stamp = next_stamp(c, SD_STAMP_GEMM | (ep.mode << 8));
    eps.stamp = next_stamp(c, SD_STAMP_STEP | (ep.mode << 8));
    if (gemm_partials_bytes(g) > c->partials_bytes) return SD_ERR_CAPACITY;
    TensorMap tx;
    if (!make_tensor_map_bf16(&tx, x, rows, K, g.m_pad)) return SD_ERR_CUDA;
    uint32_t* arrive = nullptr;                 // words of this GEMM alone; when they run out the step waits for the GEMM's grid
    if (!ep.lora_b && fused_step_polls(g, ep) && c->arrive_used + (size_t)g.n_tiles <= ARRIVE_WORDS) {
        arrive = c->gemm_arrive + c->arrive_used;
        c->arrive_used += (size_t)g.n_tiles;
    }
    LAUNCH(CAT_LINEAR, launch_gemm_streamk(tw, tx, g, c->partials, arrive, c->S.status, 1, c->st));
    LAUNCH(CAT_FUSED_STEP, launch_fused_step(g, eps, c->partials, arrive, c->S.status, 1, c->st));
    return SD_OK;
}

// The same pass on the tensor-core path (bf16 models): per layer the QKV GEMM, attention, the Wo,
// gate/up and down GEMMs, each GEMM followed by a small kernel that sums its split accumulators
// and applies the step after it; every kernel is a programmatic dependent of the one before.
sd_status forward_tc(sd_ctx* c, Model& M, const SeqList& list, const RowPlan& plan, int n_rows, int mode, float* logits_out) {
    const sd_model_desc& m = M.d;
    const int d = m.d_model, H = m.n_heads, Hkv = m.n_kv_heads, hd = m.head_dim, F = m.d_ffn, dt = m.dtype;
    cudaStream_t st = c->st;
    c->arrive_used = 0;                          // the embedding kernel below is an ordinary launch: everything before it has finished
    c->xready_used = 0;
    c->x_from.words = nullptr;
    // Off unless asked for: measured on the 7B verify step it loses 4 % (3.05 -> 3.18 ms).  The release / acquire / proxy
    // fence chain from a step CTA to the copy of its tile costs more than the end of the step kernel and the release of its
    // dependent do, and a CTA whose first k block belongs to a late tile stalls the loads queued behind it.
    c->xready_on = c->tune[SD_TUNE_TILE_HANDOFF] == 1 && n_rows >= 3 && n_rows <= 8;
    if (c->xready_on) CUDA_TRY(cudaMemsetAsync(c->xready, 0, sizeof(uint32_t) * XREADY_WORDS, st));
    // With 3..16 rows (the verify rows of one sequence) the 16 (or 32) columns of the MMA hold every activation twice over:
    // as bf16(x) and as bf16(x - bf16(x)), 8 (or 16) rows apart.  The weights stream once all the same, and the GEMMs'
    // inputs are no longer rounded to 8 bits of mantissa.
    const int lo = !c->two_part ? 0 : (n_rows >= 3 && n_rows <= 8) ? 8 : (n_rows >= 9 && n_rows <= 16) ? 16 : 0;
    if (c->stamps_on) {                                                     // the stamps of this pass replace the previous pass's
        c->stamp_kinds.clear();
        CUDA_TRY(cudaMemsetAsync(c->stamp_buf, 0xFF, sizeof(unsigned long long) * ST_WORDS * STAMP_CAP, st));
    }
    auto with_lora = [&](Epilogue& e, const Layer& L, int mat) {            // the adapters of this matrix, if the model has any
        if (!M.lora) return;
        e.lora_b = L.lora_b[mat]; e.lora_task = c->row_slot + SD_MAX_ROWS; e.lora_r = c->cfg.lora_rank; e.lora_n = c->cfg.lora_adapters;
        e.lora_scale = c->cfg.lora_scale; e.row_slot = c->row_slot;
    };
    int len_hint[SD_MAX_BATCH];                                             // context bounds of the pass's sequences, for attention's launch order
    for (int i = 0; i < list.n && i < SD_MAX_BATCH; ++i) len_hint[i] = c->len_ub[list.ids[i]];
    const RowScale first{c->ssq, 1, 1.f / d, m.rms_eps};                    // sum of squares in one piece (after the embedding)
    const RowScale tiled{c->ssq, (d + 127) / 128, 1.f / d, m.rms_eps};      // ... in one piece per 128-wide tile of h
    LAUNCH(CAT_ELEMENTWISE, launch_embed(c->S, list, plan, n_rows, M.embed, dt, d, m.vocab, c->h, c->row_slot, c->row_pos,
                                         M.layers[0].norm1, c->xn, c->ssq, M.rope_cos, M.rope_sin, hd / 2, c->rope_row_cos, c->rope_row_sin, 0, nullptr, st, lo));
    for (int l = 0; l < m.n_layers; ++l) {
        const Layer& L = M.layers[l];
        void* kc = M.kcache + M.kv_layer_bytes * l;
        void* vc = M.vcache + M.kv_layer_bytes * l;
        Epilogue e;
        memset(&e, 0, sizeof(e));
        e.lo_off = lo; e.m_real = n_rows;
        e.mode = EPI_QKV_ROPE; e.rs = l == 0 ? first : tiled;
        e.q_out = (bf16*)c->q; e.kc = (bf16*)kc; e.vc = (bf16*)vc; e.row_slot = c->row_slot; e.row_pos = c->row_pos;
        e.H = H; e.Hkv = Hkv; e.hd = hd; e.max_ctx = c->cfg.max_ctx; e.rcos = c->rope_row_cos; e.rsin = c->rope_row_sin;
        with_lora(e, L, SD_LORA_QKV);
        SD_TRY(gemm_tc(c, L.tm_qkv, c->xn, n_rows, M.n_qkv(), d, e));
        LAUNCH(CAT_ATTENTION, launch_attention_split(c->q, kc, vc, c->attn, c->row_slot, c->row_pos, n_rows, plan.rows_per_seq, H, Hkv,
                                                     hd, c->cfg.max_ctx, plan.ctx_bound, c->attn_ws, c->attn_ws_bytes, 1, st, lo,
                                                     next_stamp(c, SD_STAMP_ATTENTION), c->tune[SD_TUNE_ATTN_WARPS], c->tune[SD_TUNE_ATTN_CLUSTER],
                                                     list.n > 1 ? len_hint : nullptr));
        memset(&e, 0, sizeof(e));
        e.lo_off = lo; e.m_real = n_rows;
        e.ring_stages = c->tune[SD_TUNE_WO_STAGES]; e.prefill_all = c->tune[SD_TUNE_WO_PREFILL_ALL];
        e.mode = EPI_RESIDUAL; e.h = c->h; e.gain_next = L.norm2; e.xn = (bf16*)c->xn; e.ssq_out = c->ssq;
        with_lora(e, L, SD_LORA_WO);
        SD_TRY(gemm_tc(c, L.tm_wo, c->attn, n_rows, d, H * hd, e));
        memset(&e, 0, sizeof(e));
        e.lo_off = lo; e.m_real = n_rows;
        e.mode = EPI_SWIGLU; e.rs = tiled; e.act = (bf16*)c->act; e.F = F;
        with_lora(e, L, SD_LORA_GU);
        SD_TRY(gemm_tc(c, L.tm_gu, c->xn, n_rows, 2 * F, d, e));
        memset(&e, 0, sizeof(e));
        e.lo_off = lo; e.m_real = n_rows;
        e.mode = EPI_RESIDUAL; e.h = c->h; e.xn = (bf16*)c->xn; e.ssq_out = c->ssq;
        e.gain_next = l + 1 < m.n_layers ? M.layers[l + 1].norm1 : (mode != LOGITS_NONE ? M.final_norm : nullptr);
        with_lora(e, L, SD_LORA_WD);
        SD_TRY(gemm_tc(c, L.tm_wd, c->act, n_rows, d, F, e));
    }
    if (mode != LOGITS_NONE) {
        // the lm_head GEMM runs over all rows (they share the one pass over the weights); only the wanted rows are written
        const int R = plan.rows_per_seq;
        Epilogue e;
        memset(&e, 0, sizeof(e));
        e.lo_off = lo; e.m_real = n_rows;
        e.mode = EPI_PLAIN; e.rs = tiled; e.y = logits_out;
        if (mode == LOGITS_ALL) { e.n_out_rows = n_rows; e.row_stride = 1; e.row_offset = 0; }
        else { e.n_out_rows = list.n; e.row_stride = R; e.row_offset = R - 1; }
        SD_TRY(gemm_tc(c, M.tm_lm, c->xn, n_rows, m.vocab, d, e));
    }
    CUDA_TRY(prof_mark(c, CAT_NONE));
    return SD_OK;
}

// The same pass as one launch of the persistent streaming kernel (few query rows): the embedding kernel writes the first
// input rows in the packed layout, then every layer and the lm_head run inside k_pass_stream.
sd_status forward_pass(sd_ctx* c, Model& M, const sd_ctx::CachedProgram& cp, const SeqList& list, const RowPlan& plan, int n_rows, int mode,
                       float* logits_out) {
    const sd_model_desc& m = M.d;
    const int d = m.d_model, hd = m.head_dim;
    cudaStream_t st = c->st;
    PassParams P;
    memset(&P, 0, sizeof(P));
    P.m_tok = n_rows; P.m_pad = (n_rows + 15) & ~15; P.n_layers = m.n_layers; P.has_tail = mode != LOGITS_NONE ? 1 : 0;
    P.d = d; P.H = m.n_heads; P.Hkv = m.n_kv_heads; P.hd = hd; P.F = m.d_ffn; P.V = m.vocab; P.max_ctx = c->cfg.max_ctx;
    P.n_out[MAT_QKV] = M.n_qkv(); P.n_out[MAT_WO] = d; P.n_out[MAT_GU] = 2 * m.d_ffn; P.n_out[MAT_DN] = d; P.n_out[MAT_LM] = m.vocab;
    (void)pass_stream_smem(P.m_pad, &P.stages);
    if (c->pass_stages >= 2 && c->pass_stages < P.stages) P.stages = c->pass_stages;
    P.epoch = c->pass_epoch;
    P.h = c->tg_h; P.xn = c->tg_xn; P.attn = c->tg_attn; P.act = c->tg_act;
    P.x[MAT_QKV] = c->tg_xn; P.x[MAT_WO] = c->tg_attn; P.x[MAT_GU] = c->tg_xn; P.x[MAT_DN] = c->tg_act; P.x[MAT_LM] = c->tg_xn;
    P.q = c->tg_q; P.newkv = c->tg_newkv;
    P.kc = (bf16*)M.kcache; P.vc = (bf16*)M.vcache; P.kv_layer_elems = M.kv_layer_bytes / sizeof(bf16);
    P.row_slot = c->row_slot; P.row_pos = c->row_pos; P.rcos = c->rope_row_cos; P.rsin = c->rope_row_sin; P.ssq = c->tg_ssq;
    P.norm1 = M.layers[0].norm1; P.norm2 = M.layers[0].norm2;
    P.norm_stride = m.n_layers > 1 ? (size_t)(M.layers[1].norm1 - M.layers[0].norm1) : 0;
    P.final_norm = M.final_norm; P.rms_eps = m.rms_eps;
    P.logits = logits_out;
    const int R = plan.rows_per_seq;
    if (mode == LOGITS_LAST) { P.logits_rows = list.n; P.row_stride = R; P.row_offset = R - 1; }
    else { P.logits_rows = n_rows; P.row_stride = 1; P.row_offset = 0; }
    P.partials[0] = c->tg_partials[0]; P.partials[1] = c->tg_partials[1];
    P.abort_word = c->pass_epoch + 1; P.status = c->S.status;
    P.program = c->pass_prog + (size_t)cp.slot * PASS_PROG_BYTES;
    P.rows_per_seq = R; P.rows_per_block = cp.meta.rows_per_block; P.n_splits = cp.n_splits;
    P.part_o = c->tg_part_o; P.part_ml = c->tg_part_ml;
    const int n_it = m.n_layers + P.has_tail;
    const size_t seg_words = (size_t)sm_count() * n_it * cp.meta.max_seg * 2, task_words = (size_t)sm_count() * n_it * 16 * 2;
    if (c->stamps && seg_words + task_words <= c->stamps_words) {
        P.stamps = c->stamps; P.stamp_segs = cp.meta.max_seg;
        P.task_stamps = c->stamps + seg_words; P.stamp_tasks = 16;
    }
    CUDA_TRY(prof_mark(c, CAT_STATE));
    // The tags of a pass derive from its number; well before numbers repeat, every tagged word is cleared.
    CUDA_TRY(clear_tags_if_due(c));
    note_passes(c, 1);
    LAUNCH(CAT_STATE, launch_pass_begin(c->pass_epoch, c->pass_epoch + 1, st));
    LAUNCH(CAT_ELEMENTWISE, launch_embed(c->S, list, plan, n_rows, M.embed, m.dtype, d, m.vocab, (float*)c->tg_h, c->row_slot, c->row_pos,
                                         M.layers[0].norm1, c->tg_xn, (float*)c->tg_ssq, M.rope_cos, M.rope_sin, hd / 2, c->rope_row_cos, c->rope_row_sin,
                                         P.m_pad, c->pass_epoch, st));
    LAUNCH(CAT_LINEAR, launch_pass_stream(M.pmaps, P, sm_count(), 1, st));
    CUDA_TRY(prof_mark(c, CAT_NONE));
    return SD_OK;
}

// Calls of the hot path repeat with the same shapes and buffers, and all state they depend on
// lives on the device, so the launch sequence of a call is captured once into a CUDA graph
// and replayed: one host call instead of hundreds of launches.  The key holds everything that
// shapes the launches (sequences, gamma, buffers, context-length bucket).
struct KeyBuilder {
    std::vector<uint8_t> bytes;
    template <typename T> KeyBuilder& add(const T& v) {
        const uint8_t* p = reinterpret_cast<const uint8_t*>(&v);
        bytes.insert(bytes.end(), p, p + sizeof(T));
        return *this;
    }
    KeyBuilder& add_list(const int32_t* seqs, int n) { add(n); for (int i = 0; i < n; ++i) add(seqs[i]); return *this; }
};

int bound_bucket(int bound) { return (bound + 255) & ~255; }

template <class Body>
sd_status run_graphed(sd_ctx* c, const KeyBuilder& key, Body body) {
    CUDA_TRY(clear_tags_if_due(c));
    if (!c->graphs_on || c->prof_on) return body();
    c->graph_clock += 1;
    for (auto& g : c->graphs)
        if (g.key == key.bytes) {
            CUDA_TRY(cudaGraphLaunch(g.exec, c->st));
            c->launches += g.launches;
            note_passes(c, g.passes);
            if (c->stamps_on) c->stamp_kinds = g.stamp_kinds;       // the records this graph's launches fill
            g.last_use = c->graph_clock;
            return SD_OK;
        }
    const uint64_t l0 = c->launches, p0 = c->pass_count;
    if (cudaStreamBeginCapture(c->st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        (void)cudaGetLastError();                       // e.g. the legacy default stream cannot capture:
        c->graphs_on = false;                           // launch kernel by kernel from now on
        return body();
    }
    const sd_status s = body();
    cudaGraph_t graph = nullptr;
    const cudaError_t e = cudaStreamEndCapture(c->st, &graph);
    if (s != SD_OK || e != cudaSuccess) {
        if (graph) cudaGraphDestroy(graph);
        c->launches = l0;
        return s != SD_OK ? s : SD_ERR_CUDA;
    }
    cudaGraphExec_t exec = nullptr;
    const cudaError_t ei = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ei != cudaSuccess) { c->launches = l0; return SD_ERR_CUDA; }
    if (c->graphs.size() >= 24) {                       // drop the least recently used entry
        size_t victim = 0;
        for (size_t i = 1; i < c->graphs.size(); ++i) if (c->graphs[i].last_use < c->graphs[victim].last_use) victim = i;
        cudaGraphExecDestroy(c->graphs[victim].exec);
        c->graphs.erase(c->graphs.begin() + victim);
    }
    c->graphs.push_back({key.bytes, exec, c->launches - l0, c->graph_clock, c->pass_count - p0, c->stamp_kinds});
    CUDA_TRY(cudaGraphLaunch(exec, c->st));
    return SD_OK;
}

// Optional timing of whole calls with CUDA events on the context's stream (around the graph launch or the launches).
struct CostScope {
    sd_ctx* c; int idx;
    CostScope(sd_ctx* ctx, int kind, int units) : c(ctx), idx(-1) {
        ++c->cost_depth;
        if (!c->cost_on || c->cost_depth > 1 || c->cost_pending.size() >= 8192) return;      // only the outermost call is timed; sd_cost_read drains the list
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(c->st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return;      // inside another call's capture
        sd_ctx::CostMark m;
        for (cudaEvent_t* e : {&m.e0, &m.e1}) {
            if (!c->cost_free.empty()) { *e = c->cost_free.back(); c->cost_free.pop_back(); }
            else if (cudaEventCreate(e) != cudaSuccess) return;
        }
        m.kind = kind; m.units = units;
        if (cudaEventRecord(m.e0, c->st) != cudaSuccess) return;
        c->cost_pending.push_back(m);
        idx = (int)c->cost_pending.size() - 1;
    }
    ~CostScope() { --c->cost_depth; if (idx >= 0) cudaEventRecord(c->cost_pending[idx].e1, c->st); }
};

sd_status make_list(sd_ctx* c, const int32_t* seqs, int n_seq, int min_phase, SeqList& list) {
    if (!c || !seqs || n_seq < 1 || n_seq > SD_MAX_BATCH) return SD_ERR_INVALID_ARG;
    list.n = n_seq;
    for (int i = 0; i < n_seq; ++i) {
        const int s = seqs[i];
        if (s < 0 || s >= c->cfg.max_seqs) return SD_ERR_INVALID_ARG;
        for (int j = 0; j < i; ++j) if (seqs[j] == s) return SD_ERR_INVALID_ARG;
        if (c->phase[s] < min_phase) return SD_ERR_STATE;
        list.ids[i] = s;
        list.out[i] = i;
    }
    for (int i = n_seq; i < SD_MAX_BATCH; ++i) { list.ids[i] = 0; list.out[i] = 0; }
    return SD_OK;
}

}  // namespace

extern "C" {

const char* sd_status_str(sd_status s) {
    switch (s) {
        case SD_OK: return "ok";
        case SD_ERR_INVALID_ARG: return "invalid argument";
        case SD_ERR_STATE: return "call out of order for this sequence";
        case SD_ERR_CAPACITY: return "capacity exceeded";
        case SD_ERR_OOM: return "arena too small";
        case SD_ERR_CUDA: return "CUDA error";
        case SD_ERR_TIMEOUT: return "timeout";
        case SD_ERR_UNSUPPORTED: return "unsupported";
    }
    return "unknown";
}

size_t sd_arena_bytes(const sd_config* cfg, const sd_model_desc* models) {
    if (!valid_cfg(cfg, models)) return 0;
    sd_ctx tmp;
    tmp.cfg = *cfg;
    Bump B{nullptr, 0};
    layout(&tmp, models, B);
    return B.off + 256;
}

sd_status sd_create(const sd_config* cfg, const sd_model_desc* models, void* cuda_stream, void* arena, size_t arena_bytes,
                    sd_ctx** out) {
    if (!out) return SD_ERR_INVALID_ARG;
    *out = nullptr;
    if (!valid_cfg(cfg, models) || !arena || ((uintptr_t)arena & 255)) return SD_ERR_INVALID_ARG;
    if (cfg->clf_d_hidden > 0 && cfg->n_drafts < 1) return SD_ERR_INVALID_ARG;
    const size_t need = sd_arena_bytes(cfg, models);
    if (arena_bytes < need) return SD_ERR_OOM;
    sd_ctx* c = new sd_ctx();
    c->cfg = *cfg;
    c->st = (cudaStream_t)cuda_stream;
    Bump B{(char*)arena, 0};
    layout(c, models, B);
    c->arena_used = B.off;
    c->clf_loaded = false;
    c->launches = 0; c->prof_on = false; c->prof_used = 0;
    c->phase.assign(cfg->max_seqs, PH_FREE);
    c->len_ub.assign(cfg->max_seqs, 0);
    c->n_prompt.assign(cfg->max_seqs, 0);
    c->draft_id.assign(cfg->max_seqs, -1);
    cudaStream_t st = c->st;
    auto fail = [&](sd_status s) {
        for (cudaStream_t gs : c->group_streams) cudaStreamDestroy(gs);
        for (cudaEvent_t e : c->ev_join) cudaEventDestroy(e);
        if (c->ev_fork) cudaEventDestroy(c->ev_fork);
        delete c;
        return s;
    };
    c->ev_fork = nullptr;
    // state starts at zero; rotary tables are computed here in double and stored as fp32
    if (cudaMemsetAsync(c->S.len, 0, (char*)c->S.status + sizeof(uint32_t) - (char*)c->S.len, st) != cudaSuccess) return fail(SD_ERR_CUDA);
    for (size_t i = 0; i < c->models.size(); ++i) {
        Model& M = c->models[i];
        const int half = M.d.head_dim / 2;
        std::vector<float> cs((size_t)cfg->max_ctx * half), sn((size_t)cfg->max_ctx * half);
        for (int i2 = 0; i2 < half; ++i2) {
            const double inv_freq = pow((double)M.d.rope_base, -2.0 * i2 / M.d.head_dim);
            for (int p = 0; p < cfg->max_ctx; ++p) {
                cs[(size_t)p * half + i2] = (float)cos(p * inv_freq);
                sn[(size_t)p * half + i2] = (float)sin(p * inv_freq);
            }
        }
        if (cudaMemcpyAsync(M.rope_cos, cs.data(), cs.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(M.rope_sin, sn.data(), sn.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess)
            return fail(SD_ERR_CUDA);
    }
    if (cudaMemsetAsync(c->attn_ws, 0, std::min(c->attn_ws_bytes, (size_t)65536), st) != cudaSuccess ||
        cudaMemsetAsync(c->gemm_arrive, 0, sizeof(uint32_t) * ARRIVE_WORDS, st) != cudaSuccess)
        return fail(SD_ERR_CUDA);
    for (size_t k = 1; k < c->sets.size(); ++k)
        if (cudaMemsetAsync(c->sets[k].attn_ws, 0, std::min(c->sets[k].attn_ws_bytes, (size_t)65536), st) != cudaSuccess ||
            cudaMemsetAsync(c->sets[k].gemm_arrive, 0, sizeof(uint32_t) * ARRIVE_WORDS, st) != cudaSuccess)
            return fail(SD_ERR_CUDA);
    if (cudaStreamSynchronize(st) != cudaSuccess) return fail(SD_ERR_CUDA);
    c->groups_concurrent = c->sets.size() > 1;
    c->ev_fork = nullptr;
    if (c->sets.size() > 1) {
        if (cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess) return fail(SD_ERR_CUDA);
        for (size_t k = 1; k < c->sets.size(); ++k) {
            cudaStream_t gs = nullptr; cudaEvent_t ge = nullptr;
            if (cudaStreamCreateWithFlags(&gs, cudaStreamNonBlocking) != cudaSuccess || cudaEventCreateWithFlags(&ge, cudaEventDisableTiming) != cudaSuccess)
                return fail(SD_ERR_CUDA);
            c->group_streams.push_back(gs); c->ev_join.push_back(ge);
        }
    }
    if (cudaMemsetAsync(c->tg_begin, 0, c->tg_end - c->tg_begin, st) != cudaSuccess ||          // no word carries a tag a pass could expect
        cudaMemsetAsync(c->pass_epoch, 0, 2 * sizeof(uint32_t), st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return fail(SD_ERR_CUDA);
    c->pass_count = 0; c->tags_due_clear = false;
    c->pass_on = false; c->pass_drafts = false; c->pass_max_rows = 16; c->pass_tuned = false; c->pass_stages = 0; c->stamps = nullptr; c->stamps_words = 0;
    c->two_part = true;
    c->cost_on = false; c->cost_depth = 0;
    c->stamps_on = false;
    c->xready_on = false; c->x_from.words = nullptr;
    for (int i = 0; i < SD_TUNE_COUNT; ++i) c->tune[i] = 0;
    for (int i = 0; i < 3; ++i) { c->cost_ms[i] = 0.0; c->cost_units[i] = 0; }
    c->force_plain = false;
    c->graphs_on = true;
    c->graph_clock = 0;
    for (Model& M : c->models) {
        const sd_model_desc& m = M.d;
        M.pass_ok = false;
        M.tc = m.dtype == SD_BF16 && (m.head_dim == 64 || m.head_dim == 128) && m.d_model <= 128 * SSQ_STRIDE && m.d_ffn % 64 == 0 &&
               attention_split_supported(m.dtype, m.n_heads, m.n_kv_heads, m.head_dim);
        if (!M.tc && M.lora) return fail(SD_ERR_UNSUPPORTED);
        if (!M.tc) continue;
        const int dq = m.n_heads * m.head_dim;
        const int extra = M.lora ? 128 : 0;
        bool ok = make_tensor_map_bf16(&M.tm_lm, M.lm_head, m.vocab, m.d_model, 128);
        for (Layer& L : M.layers) {
            ok = ok && make_tensor_map_bf16(&L.tm_qkv, L.wqkv, M.n_qkv() + extra, m.d_model, 128);
            ok = ok && make_tensor_map_bf16(&L.tm_wo, L.wo, m.d_model + extra, dq, 128);
            ok = ok && make_tensor_map_bf16(&L.tm_gu, L.wgu, 2 * m.d_ffn + extra, m.d_model, 128);
            ok = ok && make_tensor_map_bf16(&L.tm_wd, L.wd, m.d_model + extra, m.d_ffn, 128);
            if (M.lora) {                                    // adapters start at zero: the base draft
                const size_t n_lb = (size_t)cfg->lora_adapters * cfg->lora_rank * sizeof(bf16);
                const size_t outs[4] = {(size_t)M.n_qkv(), (size_t)m.d_model, (size_t)2 * m.d_ffn, (size_t)m.d_model};
                const size_t ins[4] = {(size_t)m.d_model, (size_t)dq, (size_t)m.d_model, (size_t)m.d_ffn};
                void* mats[4] = {L.wqkv, L.wo, L.wgu, L.wd};
                for (int k = 0; k < 4; ++k) {
                    ok = ok && cudaMemsetAsync(L.lora_b[k], 0, n_lb * outs[k], st) == cudaSuccess;
                    ok = ok && cudaMemsetAsync((char*)mats[k] + outs[k] * ins[k] * M.esz, 0, 128 * ins[k] * M.esz, st) == cudaSuccess;
                }
            }
        }
        if (!ok || cudaStreamSynchronize(st) != cudaSuccess) return fail(SD_ERR_CUDA);
        // the persistent streaming kernel sees the layers of a matrix as one [layer][row][k] tensor
        const size_t stride = m.n_layers > 1 ? (size_t)((char*)M.layers[1].wqkv - (char*)M.layers[0].wqkv) : 0;
        M.pass_ok = !M.lora && m.d_model % 64 == 0 && dq % 64 == 0 && m.d_ffn % 64 == 0 &&
                    make_tensor_map_layers(&M.pmaps.m[MAT_QKV], M.layers[0].wqkv, M.n_qkv(), m.d_model, m.n_layers, stride) &&
                    make_tensor_map_layers(&M.pmaps.m[MAT_WO], M.layers[0].wo, m.d_model, dq, m.n_layers, stride) &&
                    make_tensor_map_layers(&M.pmaps.m[MAT_GU], M.layers[0].wgu, 2 * m.d_ffn, m.d_model, m.n_layers, stride) &&
                    make_tensor_map_layers(&M.pmaps.m[MAT_DN], M.layers[0].wd, m.d_model, m.d_ffn, m.n_layers, stride) &&
                    make_tensor_map_layers(&M.pmaps.m[MAT_LM], M.lm_head, m.vocab, m.d_model, 1, 0);
        for (int l = 1; l < m.n_layers && M.pass_ok; ++l)         // every layer at the same distance from the one before
            M.pass_ok = (size_t)((char*)M.layers[l].wqkv - (char*)M.layers[l - 1].wqkv) == stride &&
                        (size_t)((char*)M.layers[l].norm1 - (char*)M.layers[l - 1].norm1) == stride;
    }
    *out = c;
    return SD_OK;
}

sd_status sd_destroy(sd_ctx* c) {
    if (!c) return SD_ERR_INVALID_ARG;
    cudaStreamSynchronize(c->st);
    for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
    for (cudaStream_t gs : c->group_streams) cudaStreamDestroy(gs);
    for (cudaEvent_t e : c->ev_join) cudaEventDestroy(e);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    for (auto& m : c->cost_pending) { cudaEventDestroy(m.e0); cudaEventDestroy(m.e1); }
    for (cudaEvent_t e : c->cost_free) cudaEventDestroy(e);
    for (auto& g : c->graphs) cudaGraphExecDestroy(g.exec);
    delete c;
    return SD_OK;
}

sd_status sd_load_tensor(sd_ctx* c, int model_id, int kind, int layer, const void* src, int on_dev) {
    if (!c || !src || model_id < 0 || model_id >= (int)c->models.size()) return SD_ERR_INVALID_ARG;
    Model& M = c->models[model_id];
    const sd_model_desc& m = M.d;
    const size_t dq = (size_t)m.n_heads * m.head_dim, dkv = (size_t)m.n_kv_heads * m.head_dim, d = m.d_model, F = m.d_ffn;
    const bool per_layer = kind >= SD_T_WQ;
    if (per_layer && (layer < 0 || layer >= m.n_layers)) return SD_ERR_INVALID_ARG;
    void* dst = nullptr;
    size_t bytes = 0;
    Layer* L = per_layer ? &M.layers[layer] : nullptr;
    switch (kind) {
        case SD_T_EMBED: dst = M.embed; bytes = (size_t)m.vocab * d * M.esz; break;
        case SD_T_LM_HEAD: dst = M.lm_head; bytes = (size_t)m.vocab * d * M.esz; break;
        case SD_T_FINAL_NORM: dst = M.final_norm; bytes = d * 4; break;
        case SD_T_WQ: dst = L->wqkv; bytes = dq * d * M.esz; break;
        case SD_T_WK: dst = (char*)L->wqkv + dq * d * M.esz; bytes = dkv * d * M.esz; break;
        case SD_T_WV: dst = (char*)L->wqkv + (dq + dkv) * d * M.esz; bytes = dkv * d * M.esz; break;
        case SD_T_WO: dst = L->wo; bytes = d * dq * M.esz; break;
        case SD_T_WG:
        case SD_T_WU:
            if (M.tc) {
                // tensor-core layout: 128-row tiles of 64 gate rows followed by the 64 up rows of the same features,
                // so that the CTA finishing a tile holds both halves of SwiGLU
                const size_t chunk = 64 * d * M.esz;
                CUDA_TRY(cudaMemcpy2DAsync((char*)L->wgu + (kind == SD_T_WU ? chunk : 0), 2 * chunk, src, chunk, chunk, F / 64,
                                           on_dev ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, c->st));
                if (!on_dev) CUDA_TRY(cudaStreamSynchronize(c->st));
                return SD_OK;
            }
            dst = kind == SD_T_WG ? (char*)L->wgu : (char*)L->wgu + F * d * M.esz; bytes = F * d * M.esz; break;
        case SD_T_WD: dst = L->wd; bytes = d * F * M.esz; break;
        case SD_T_NORM1: dst = L->norm1; bytes = d * 4; break;
        case SD_T_NORM2: dst = L->norm2; bytes = d * 4; break;
        default: return SD_ERR_INVALID_ARG;
    }
    CUDA_TRY(cudaMemcpyAsync(dst, src, bytes, on_dev ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, c->st));
    if (!on_dev) CUDA_TRY(cudaStreamSynchronize(c->st));     // the host buffer may go away after the call
    return SD_OK;
}

sd_status sd_load_lora(sd_ctx* c, int adapter, int layer, int mat, const void* a, const void* b, int on_dev) {
    if (!c || !a || !b || mat < 0 || mat > 3) return SD_ERR_INVALID_ARG;
    if (c->cfg.lora_adapters < 1) return SD_ERR_STATE;
    Model& M = c->models[1];
    const sd_model_desc& m = M.d;
    if (adapter < 0 || adapter >= c->cfg.lora_adapters || layer < 0 || layer >= m.n_layers) return SD_ERR_INVALID_ARG;
    Layer& L = M.layers[layer];
    const size_t dq = (size_t)m.n_heads * m.head_dim, r = c->cfg.lora_rank, F = m.d_ffn;
    const size_t outs[4] = {(size_t)M.n_qkv(), (size_t)m.d_model, 2 * F, (size_t)m.d_model};
    const size_t ins[4] = {(size_t)m.d_model, dq, (size_t)m.d_model, F};
    void* mats[4] = {L.wqkv, L.wo, L.wgu, L.wd};
    const cudaMemcpyKind kd = on_dev ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
    // A: rows adapter * r ... of the tile that follows the matrix's own rows
    char* a_dst = (char*)mats[mat] + (outs[mat] + (size_t)adapter * r) * ins[mat] * sizeof(bf16);
    CUDA_TRY(cudaMemcpyAsync(a_dst, a, r * ins[mat] * sizeof(bf16), kd, c->st));
    // B: in the order of the GEMM's output features (gate / up rows interleaved in 64-row halves of a tile, as the weights are)
    bf16* b_dst = L.lora_b[mat] + (size_t)adapter * outs[mat] * r;
    if (mat == SD_LORA_GU) {
        const size_t chunk = 64 * r * sizeof(bf16);
        CUDA_TRY(cudaMemcpy2DAsync(b_dst, 2 * chunk, b, chunk, chunk, F / 64, kd, c->st));                                   // gate rows
        CUDA_TRY(cudaMemcpy2DAsync((char*)b_dst + chunk, 2 * chunk, (const char*)b + F * r * sizeof(bf16), chunk, chunk, F / 64, kd, c->st));   // up rows
    } else {
        CUDA_TRY(cudaMemcpyAsync(b_dst, b, outs[mat] * r * sizeof(bf16), kd, c->st));
    }
    CUDA_TRY(cudaStreamSynchronize(c->st));
    return SD_OK;
}

sd_status sd_load_classifier(sd_ctx* c, const float* w1, const float* b1, const float* w2, const float* b2, int on_dev) {
    if (!c || !w1 || !b1 || !w2 || !b2) return SD_ERR_INVALID_ARG;
    if (!c->clf_w1) return SD_ERR_STATE;
    const size_t dh = c->cfg.clf_d_hidden, d = c->models[0].d.d_model, K = c->cfg.n_drafts;
    cudaMemcpyKind kd = on_dev ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
    CUDA_TRY(cudaMemcpyAsync(c->clf_w1, w1, dh * d * 4, kd, c->st));
    CUDA_TRY(cudaMemcpyAsync(c->clf_b1, b1, dh * 4, kd, c->st));
    CUDA_TRY(cudaMemcpyAsync(c->clf_w2, w2, K * dh * 4, kd, c->st));
    CUDA_TRY(cudaMemcpyAsync(c->clf_b2, b2, K * 4, kd, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
    c->clf_loaded = true;
    return SD_OK;
}

sd_status sd_seq_begin(sd_ctx* c, int seq, const int32_t* prompt, int n_prompt, uint32_t seq_id) {
    if (!c || !prompt || seq < 0 || seq >= c->cfg.max_seqs || n_prompt < 2) return SD_ERR_INVALID_ARG;
    if (n_prompt > c->cfg.max_ctx) return SD_ERR_CAPACITY;
    const int V = c->models[0].d.vocab;
    for (int i = 0; i < n_prompt; ++i) if (prompt[i] < 0 || prompt[i] >= V) return SD_ERR_INVALID_ARG;
    CUDA_TRY(cudaMemcpyAsync(c->S.tokens + (size_t)seq * c->S.tok_stride, prompt, sizeof(int32_t) * n_prompt,
                             cudaMemcpyHostToDevice, c->st));
    LAUNCH(CAT_STATE, launch_set_state(c->S, seq, n_prompt, 0, 0, 0u, seq_id, 1, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
    c->phase[seq] = PH_BEGUN;
    c->len_ub[seq] = n_prompt;
    c->n_prompt[seq] = n_prompt;
    c->draft_id[seq] = -1;
    return SD_OK;
}

sd_status sd_route_prompt(sd_ctx* c, const int32_t* seqs, int n_seq, const int32_t* forced, int32_t* draft_out) {
    SeqList list, fl;
    SD_TRY(make_list(c, seqs, n_seq, PH_BEGUN, list));
    const int K = c->cfg.n_drafts;
    if (K < 1) return SD_ERR_STATE;
    fl = list;
    bool need_clf = false;
    for (int i = 0; i < n_seq; ++i) {
        int f = forced ? forced[i] : -1;
        if (f >= K) return SD_ERR_INVALID_ARG;
        fl.ids[i] = f < 0 ? -1 : f;
        need_clf |= f < 0;
    }
    if (need_clf && !c->clf_loaded) return SD_ERR_STATE;
    Model& T = c->models[0];
    LAUNCH(CAT_ELEMENTWISE, launch_classifier(c->S, list, fl, T.embed, T.d.dtype, T.d.d_model, T.d.vocab, c->clf_w1, c->clf_b1,
                               c->cfg.clf_d_hidden, c->clf_w2, c->clf_b2, K, c->st));
    std::vector<int32_t> ids(c->cfg.max_seqs);
    CUDA_TRY(cudaMemcpyAsync(ids.data(), c->S.draft_id, sizeof(int32_t) * ids.size(), cudaMemcpyDeviceToHost, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
    for (int i = 0; i < n_seq; ++i) {
        const int s = seqs[i];
        c->draft_id[s] = ids[s];
        if (c->phase[s] == PH_BEGUN) c->phase[s] = PH_ROUTED;
        if (draft_out) draft_out[i] = ids[s];
    }
    return SD_OK;
}

sd_status sd_route_prompt_mamba(sd_ctx* c, const sd_mamba_desc* desc, const sd_mamba_weights* w, const int32_t* seqs, int n_seq,
                                void* ws, size_t ws_bytes, int32_t* draft_out) {
    if (!c || !desc || !w || !seqs || n_seq < 1 || n_seq > c->cfg.max_seqs) return SD_ERR_INVALID_ARG;
    if (desc->n_classes != c->cfg.n_drafts) return SD_ERR_INVALID_ARG;
    std::vector<int64_t> starts(n_seq);
    std::vector<int32_t> lens(n_seq), labels(n_seq);
    for (int i = 0; i < n_seq; ++i) {
        const int s = seqs[i];
        if (s < 0 || s >= c->cfg.max_seqs) return SD_ERR_INVALID_ARG;
        if (c->phase[s] < PH_BEGUN) return SD_ERR_STATE;
        starts[i] = (int64_t)s * c->S.tok_stride;
        lens[i] = c->n_prompt[s];
    }
    // labels land in the scratch words the accept path uses for its counts (n_seq <= max_seqs of them)
    SD_TRY(sd_mamba_classify(desc, w, c->S.tokens, starts.data(), lens.data(), n_seq, nullptr, c->st_nacc, ws, ws_bytes, c->st));
    c->launches += 6;
    CUDA_TRY(cudaMemcpyAsync(labels.data(), c->st_nacc, sizeof(int32_t) * n_seq, cudaMemcpyDeviceToHost, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
    return sd_route_prompt(c, seqs, n_seq, labels.data(), draft_out);
}

sd_status sd_prefill(sd_ctx* c, const int32_t* seqs, int n_seq) {
    SeqList all;
    SD_TRY(make_list(c, seqs, n_seq, c->cfg.n_drafts > 0 ? PH_ROUTED : PH_BEGUN, all));
    for (int i = 0; i < n_seq; ++i) {
        const int s = seqs[i], n = c->n_prompt[s] - 1;
        SeqList one = all;
        one.n = 1; one.ids[0] = s; one.out[0] = 0;
        for (int pass = 0; pass < 2; ++pass) {
            if (pass == 1 && c->cfg.n_drafts < 1) break;
            Model& M = c->models[pass == 0 ? 0 : draft_model_index(c->cfg, c->draft_id[s])];
            for (int p0 = 0; p0 < n; p0 += SD_MAX_ROWS) {
                const int rows = std::min(SD_MAX_ROWS, n - p0);
                RowPlan plan{PLAN_PREFILL, rows, p0, 0, 0, nullptr, p0 + rows};
                SD_TRY(forward(c, M, one, plan, rows, LOGITS_NONE, nullptr));
            }
        }
        LAUNCH(CAT_STATE, launch_set_state(c->S, s, n + 1, n, n, 0u, 0u, 0, c->st));
        c->phase[s] = PH_READY;
    }
    return SD_OK;
}

sd_status sd_draft_steps(sd_ctx* c, const int32_t* seqs, int n_seq, int gamma, int32_t* x_dev, float* q_dev) {
    return sd_draft_steps_replay(c, seqs, n_seq, gamma, x_dev, x_dev, q_dev);
}

sd_status sd_draft_steps_replay(sd_ctx* c, const int32_t* seqs, int n_seq, int gamma, const int32_t* x_in,
                                int32_t* x_dev, float* q_dev) {
    SeqList all;
    SD_TRY(make_list(c, seqs, n_seq, PH_READY, all));
    if (gamma < 1 || gamma > c->cfg.max_gamma || !x_dev || !q_dev || !x_in) return SD_ERR_INVALID_ARG;
    if (c->cfg.n_drafts < 1) return SD_ERR_STATE;
    for (int i = 0; i < n_seq; ++i)
        if (c->len_ub[seqs[i]] + gamma - 1 > c->cfg.max_ctx) return SD_ERR_CAPACITY;
    const int V = c->models[0].d.vocab;
    int bound = 0;
    for (int i = 0; i < n_seq; ++i) bound = std::max(bound, c->len_ub[seqs[i]]);
    KeyBuilder key;
    key.add(1).add_list(seqs, n_seq).add(gamma).add(x_in).add(x_dev).add(q_dev).add(bound_bucket(bound + gamma)).add(c->force_plain).add(c->stamps_on).add(c->pass_on).add(c->pass_drafts).add(c->pass_max_rows).add(c->groups_concurrent);
    for (int i = 0; i < n_seq; ++i) key.add(c->draft_id[seqs[i]]);
    bound = bound_bucket(bound + gamma) - gamma;
    CostScope cost(c, 0, gamma);
    // with low-rank adapters every task runs on the one base draft: a single group, adapters picked row by row
    const bool shared = c->cfg.lora_adapters > 0;
    const int n_groups = shared ? 1 : c->cfg.n_drafts;
    for (int k = 0; k < n_groups; ++k) {                    // programs of the persistent kernel exist before anything is captured
        int n = 0;
        for (int i = 0; i < n_seq; ++i) n += shared || c->draft_id[seqs[i]] == k;
        if (n == 0) continue;
        for (int s = 0; s < gamma; ++s) {
            if (s == 0) { RowPlan plan{PLAN_DRAFT_FIRST, 2, 0, 0, gamma, x_in, bound}; SD_TRY(prepare_pass(c, 1 + k, plan, 2 * n, LOGITS_LAST)); }
            else { RowPlan plan{PLAN_DRAFT_NEXT, 1, 0, s, gamma, x_in, bound + s}; SD_TRY(prepare_pass(c, 1 + k, plan, n, LOGITS_ALL)); }
        }
    }
    return run_graphed(c, key, [&]() -> sd_status {
    // Groups of different draft models run side by side: every group after the first gets a stream and a scratch set of
    // its own, forked from and joined back to the context's stream (inside a capture these become parallel branches).
    int n_active = 0;
    for (int k = 0; k < n_groups; ++k) {
        bool any = false;
        for (int i = 0; i < n_seq; ++i) any |= shared || c->draft_id[seqs[i]] == k;
        n_active += any;
    }
    const bool side_by_side = c->groups_concurrent && n_active > 1 && !c->prof_on && !(c->pass_on && c->pass_drafts) &&
                              (int)c->sets.size() >= n_active;
    cudaStream_t main_st = c->st;
    struct Restore {                                       // whatever happens below, the context ends on its own stream and scratch set
        sd_ctx* c; cudaStream_t st;
        ~Restore() { c->st = st; use_set(c, 0); }
    } restore{c, main_st};
    if (side_by_side) CUDA_TRY(cudaEventRecord(c->ev_fork, main_st));
    int a = 0;                                             // index among the active groups
    for (int k = 0; k < n_groups; ++k) {                    // sequences grouped per routed draft
        SeqList g = all;
        g.n = 0;
        for (int i = 0; i < n_seq; ++i)
            if (shared || c->draft_id[seqs[i]] == k) { g.ids[g.n] = seqs[i]; g.out[g.n] = i; ++g.n; }
        if (g.n == 0) continue;
        if (side_by_side && a > 0) {
            use_set(c, (size_t)a);
            c->st = c->group_streams[a - 1];
            CUDA_TRY(cudaStreamWaitEvent(c->st, c->ev_fork, 0));
        }
        Model& M = c->models[1 + k];
        for (int s = 0; s < gamma; ++s) {
            if (s == 0) {
                RowPlan plan{PLAN_DRAFT_FIRST, 2, 0, 0, gamma, x_in, bound};
                SD_TRY(forward(c, M, g, plan, 2 * g.n, LOGITS_LAST, c->draft_logits));
            } else {
                RowPlan plan{PLAN_DRAFT_NEXT, 1, 0, s, gamma, x_in, bound + s};
                SD_TRY(forward(c, M, g, plan, g.n, LOGITS_ALL, c->draft_logits));
            }
            LAUNCH(CAT_SAMPLING, launch_draft_sample(c->draft_logits, c->S, g, V, c->cfg.temperature, c->cfg.seed, s, gamma, q_dev, x_dev, c->st));
        }
        if (side_by_side && a > 0) {
            CUDA_TRY(cudaEventRecord(c->ev_join[a - 1], c->st));
            c->st = main_st;
            use_set(c, 0);
        }
        ++a;
    }
    if (side_by_side)
        for (int j = 1; j < a; ++j) CUDA_TRY(cudaStreamWaitEvent(main_st, c->ev_join[j - 1], 0));
    return SD_OK;
    });
}

sd_status sd_verify(sd_ctx* c, const int32_t* seqs, int n_seq, int gamma, const int32_t* x_dev, float* logits_dev) {
    SeqList list;
    SD_TRY(make_list(c, seqs, n_seq, PH_READY, list));
    if (gamma < 0 || gamma > c->cfg.max_gamma || !logits_dev || (gamma > 0 && !x_dev)) return SD_ERR_INVALID_ARG;
    if (n_seq * (gamma + 1) > SD_MAX_ROWS) return SD_ERR_CAPACITY;
    for (int i = 0; i < n_seq; ++i)
        if (c->len_ub[seqs[i]] + gamma > c->cfg.max_ctx) return SD_ERR_CAPACITY;
    int bound = 0;
    for (int i = 0; i < n_seq; ++i) bound = std::max(bound, c->len_ub[seqs[i]] + gamma);
    RowPlan plan{PLAN_VERIFY, gamma + 1, 0, 0, gamma, x_dev, bound_bucket(bound)};
    KeyBuilder key;
    key.add(2).add_list(seqs, n_seq).add(gamma).add(x_dev).add(logits_dev).add(plan.ctx_bound).add(c->force_plain).add(c->stamps_on).add(c->pass_on).add(c->pass_max_rows);
    SD_TRY(prepare_pass(c, 0, plan, n_seq * (gamma + 1), LOGITS_ALL));
    CostScope cost(c, 1, 1);
    return run_graphed(c, key, [&]() { return forward(c, c->models[0], list, plan, n_seq * (gamma + 1), LOGITS_ALL, logits_dev); });
}

sd_status sd_target_step(sd_ctx* c, const int32_t* seqs, int n_seq, float* logits_dev) {
    SeqList list;
    SD_TRY(make_list(c, seqs, n_seq, PH_READY, list));
    if (!logits_dev) return SD_ERR_INVALID_ARG;
    for (int i = 0; i < n_seq; ++i)
        if (c->len_ub[seqs[i]] > c->cfg.max_ctx) return SD_ERR_CAPACITY;
    int bound = 0;
    for (int i = 0; i < n_seq; ++i) bound = std::max(bound, c->len_ub[seqs[i]]);
    RowPlan plan{PLAN_TARGET_STEP, 1, 0, 0, 0, nullptr, bound_bucket(bound)};
    KeyBuilder key;
    key.add(3).add_list(seqs, n_seq).add(logits_dev).add(plan.ctx_bound).add(c->force_plain).add(c->stamps_on).add(c->pass_on).add(c->pass_max_rows);
    SD_TRY(prepare_pass(c, 0, plan, n_seq, LOGITS_ALL));
    CostScope cost(c, 2, 1);
    return run_graphed(c, key, [&]() { return forward(c, c->models[0], list, plan, n_seq, LOGITS_ALL, logits_dev); });
}

sd_status sd_accept(const sd_accept_args* a) {
    if (!a || !a->target || !a->n_acc || !a->out_tok || !a->iter || !a->seq_id) return SD_ERR_INVALID_ARG;
    if (a->B < 1 || a->gamma < 0 || a->gamma > SD_MAX_GAMMA || a->V < 2 || !(a->temperature >= 0.f)) return SD_ERR_INVALID_ARG;
    if (a->gamma > 0 && (!a->q || !a->x)) return SD_ERR_INVALID_ARG;
    AcceptParams p;
    memset(&p, 0, sizeof(p));
    p.target = a->target; p.target_is_logits = a->target_is_logits; p.q = a->q; p.x = a->x;
    p.B = a->B; p.gamma = a->gamma; p.V = a->V; p.T = a->temperature; p.seed = a->seed;
    p.iter = a->iter; p.seq_id = a->seq_id; p.use_list = 0; p.n_acc = a->n_acc; p.out_tok = a->out_tok;
    CUDA_TRY(launch_accept(p, 0, (cudaStream_t)a->cuda_stream));
    return SD_OK;
}

sd_status sd_accept_seqs(sd_ctx* c, const int32_t* seqs, int n_seq, int gamma, const float* logits_dev, const float* q_dev,
                         const int32_t* x_dev, int32_t* n_acc_dev, int32_t* out_tok_dev) {
    AcceptParams p;
    memset(&p, 0, sizeof(p));
    SD_TRY(make_list(c, seqs, n_seq, PH_READY, p.list));
    if (gamma < 0 || gamma > c->cfg.max_gamma || !logits_dev || !n_acc_dev || !out_tok_dev) return SD_ERR_INVALID_ARG;
    if (gamma > 0 && (!q_dev || !x_dev)) return SD_ERR_INVALID_ARG;
    p.target = logits_dev; p.target_is_logits = 1; p.q = q_dev; p.x = x_dev;
    p.B = n_seq; p.gamma = gamma; p.V = c->models[0].d.vocab; p.T = c->cfg.temperature; p.seed = c->cfg.seed;
    p.iter = c->S.iter; p.seq_id = c->S.seq_id; p.use_list = 1; p.n_acc = n_acc_dev; p.out_tok = out_tok_dev;
    p.alpha_terms = gamma > 0 ? c->alpha_terms : nullptr;
    LAUNCH(CAT_SAMPLING, launch_accept(p, 1, c->st));
    CUDA_TRY(prof_mark(c, CAT_NONE));
    return SD_OK;
}

sd_status sd_kv_rollback(sd_ctx* c, const int32_t* seqs, int n_seq, int gamma, const int32_t* n_acc_dev, const int32_t* out_tok_dev) {
    SeqList list;
    SD_TRY(make_list(c, seqs, n_seq, PH_READY, list));
    if (gamma < 0 || gamma > c->cfg.max_gamma || !n_acc_dev || !out_tok_dev) return SD_ERR_INVALID_ARG;
    for (int i = 0; i < n_seq; ++i)
        if (c->len_ub[seqs[i]] + gamma + 1 > c->S.tok_stride) return SD_ERR_CAPACITY;
    LAUNCH(CAT_STATE, launch_rollback(c->S, list, gamma, n_acc_dev, out_tok_dev, gamma > 0 ? c->alpha_terms : nullptr, c->st));
    CUDA_TRY(prof_mark(c, CAT_NONE));
    for (int i = 0; i < n_seq; ++i) c->len_ub[seqs[i]] += gamma + 1;
    return SD_OK;
}

sd_status sd_seq_read(sd_ctx* c, int seq, int32_t* tokens, int cap, int32_t* len_out, sd_counters* cnt) {
    if (!c || seq < 0 || seq >= c->cfg.max_seqs || cap < 0 || (cap > 0 && !tokens)) return SD_ERR_INVALID_ARG;
    if (c->phase[seq] == PH_FREE) return SD_ERR_STATE;
    int32_t len = 0;
    CUDA_TRY(cudaMemcpyAsync(&len, c->S.len + seq, sizeof(int32_t), cudaMemcpyDeviceToHost, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
    const int n = std::min(cap, (int)len);
    if (n > 0) CUDA_TRY(cudaMemcpyAsync(tokens, c->S.tokens + (size_t)seq * c->S.tok_stride, sizeof(int32_t) * n, cudaMemcpyDeviceToHost, c->st));
    if (cnt) CUDA_TRY(cudaMemcpyAsync(cnt, c->S.counters + 4 * seq, sizeof(int64_t) * 4, cudaMemcpyDeviceToHost, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
    if (len_out) *len_out = len;
    c->len_ub[seq] = len;
    return SD_OK;
}

sd_status sd_seq_force(sd_ctx* c, int seq, const int32_t* tokens, int n_tokens, int draft_kv_len, uint32_t iter) {
    if (!c || !tokens || seq < 0 || seq >= c->cfg.max_seqs || n_tokens < 2 || draft_kv_len < 0 || draft_kv_len >= n_tokens) return SD_ERR_INVALID_ARG;
    if (c->phase[seq] < PH_READY) return SD_ERR_STATE;
    if (n_tokens > c->cfg.max_ctx) return SD_ERR_CAPACITY;
    CUDA_TRY(cudaMemcpyAsync(c->S.tokens + (size_t)seq * c->S.tok_stride, tokens, sizeof(int32_t) * n_tokens, cudaMemcpyHostToDevice, c->st));
    LAUNCH(CAT_STATE, launch_set_state(c->S, seq, n_tokens, n_tokens - 1, draft_kv_len, iter, 0u, 0, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
    c->len_ub[seq] = n_tokens;
    return SD_OK;
}

sd_status sd_device_status(sd_ctx* c, uint32_t* flags) {
    if (!c || !flags) return SD_ERR_INVALID_ARG;
    CUDA_TRY(cudaMemcpyAsync(flags, c->S.status, sizeof(uint32_t), cudaMemcpyDeviceToHost, c->st));
    CUDA_TRY(cudaMemsetAsync(c->S.status, 0, sizeof(uint32_t), c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
    return (*flags & SD_DEV_WAIT_EXPIRED) ? SD_ERR_TIMEOUT : SD_OK;      // a bounded wait inside a kernel gave up (flags say what else happened)
}

sd_status sd_verify_accept(sd_ctx* c, const int32_t* seqs, int n_seq, int gamma, const int32_t* x_dev, const float* q_dev,
                           float* logits_dev, int32_t* n_acc_dev, int32_t* out_tok_dev) {
    if (!c || !seqs || !logits_dev || !n_acc_dev || !out_tok_dev) return SD_ERR_INVALID_ARG;
    const bool saved = c->graphs_on;
    KeyBuilder key;
    // argument and capacity checks run on every call, captured or replayed, and before anything reads the lists
    if (n_seq < 1 || n_seq > SD_MAX_BATCH || gamma < 0 || gamma > c->cfg.max_gamma || n_seq * (gamma + 1) > SD_MAX_ROWS) return SD_ERR_INVALID_ARG;
    for (int i = 0; i < n_seq; ++i) {
        const int s = seqs[i];
        if (s < 0 || s >= c->cfg.max_seqs) return SD_ERR_INVALID_ARG;
        if (c->phase[s] < PH_READY) return SD_ERR_STATE;
        if (c->len_ub[s] + gamma + 1 > c->S.tok_stride || c->len_ub[s] + gamma > c->cfg.max_ctx) return SD_ERR_CAPACITY;
    }
    key.add(4).add_list(seqs, n_seq).add(gamma).add(x_dev).add(q_dev).add(logits_dev).add(n_acc_dev).add(out_tok_dev).add(c->force_plain).add(c->stamps_on).add(c->pass_on).add(c->pass_max_rows);
    int bound = 0;
    for (int i = 0; i < n_seq; ++i) bound = std::max(bound, c->len_ub[seqs[i]] + gamma);
    key.add(bound_bucket(bound));
    {
        RowPlan plan{PLAN_VERIFY, gamma + 1, 0, 0, gamma, x_dev, bound_bucket(bound)};
        SD_TRY(prepare_pass(c, 0, plan, n_seq * (gamma + 1), LOGITS_ALL));
    }
    std::vector<int> ub(c->len_ub);
    auto body = [&]() -> sd_status {
        c->graphs_on = false;                    // the three calls below must launch into this capture, not replay their own graphs
        sd_status s = sd_verify(c, seqs, n_seq, gamma, x_dev, logits_dev);
        if (s == SD_OK) s = sd_accept_seqs(c, seqs, n_seq, gamma, logits_dev, q_dev, x_dev, n_acc_dev, out_tok_dev);
        if (s == SD_OK) s = sd_kv_rollback(c, seqs, n_seq, gamma, n_acc_dev, out_tok_dev);
        c->graphs_on = saved;
        return s;
    };
    CostScope cost(c, 1, 1);                     // (sd_verify inside runs in this call's capture and does not time itself)
    const bool replay = saved && !c->prof_on;
    bool cached = false;
    if (replay) for (auto& g : c->graphs) cached |= g.key == key.bytes;
    const sd_status s = run_graphed(c, key, body);
    if (s == SD_OK && cached)                    // a replay does not run the host bookkeeping of sd_kv_rollback
        for (int i = 0; i < n_seq; ++i) c->len_ub[seqs[i]] += gamma + 1;
    if (s != SD_OK) c->len_ub = ub;
    return s;
}

sd_status sd_verify_accept_host(sd_ctx* c, const int32_t* seqs, int n_seq, int gamma, const int32_t* x_host,
                                const float* q_host, int32_t* n_acc_host, int32_t* out_tok_host) {
    if (!c || !seqs || n_seq < 1 || n_seq > c->cfg.max_seqs || gamma < 0 || gamma > c->cfg.max_gamma) return SD_ERR_INVALID_ARG;
    if (!n_acc_host || !out_tok_host || (gamma > 0 && (!x_host || !q_host))) return SD_ERR_INVALID_ARG;
    if (n_seq * (gamma + 1) > SD_MAX_ROWS) return SD_ERR_CAPACITY;
    const size_t V = c->models[0].d.vocab;
    if (gamma > 0) {
        CUDA_TRY(cudaMemcpyAsync(c->st_x, x_host, sizeof(int32_t) * n_seq * gamma, cudaMemcpyHostToDevice, c->st));
        CUDA_TRY(cudaMemcpyAsync(c->st_q, q_host, sizeof(float) * n_seq * gamma * V, cudaMemcpyHostToDevice, c->st));
    }
    SD_TRY(sd_verify_accept(c, seqs, n_seq, gamma, c->st_x, c->st_q, c->st_logits, c->st_nacc, c->st_out));
    CUDA_TRY(cudaMemcpyAsync(n_acc_host, c->st_nacc, sizeof(int32_t) * n_seq, cudaMemcpyDeviceToHost, c->st));
    CUDA_TRY(cudaMemcpyAsync(out_tok_host, c->st_out, sizeof(int32_t) * n_seq * (gamma + 1), cudaMemcpyDeviceToHost, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
    return SD_OK;
}

double sd_eq1_speedup(double alpha, int gamma, double c) {
    if (!(alpha >= 0.0) || alpha > 1.0 || gamma < 0 || !(c >= 0.0)) return 0.0;
    const double tokens = alpha == 1.0 ? (double)(gamma + 1) : (1.0 - pow(alpha, gamma + 1)) / (1.0 - alpha);
    return tokens / (gamma * c + 1.0);
}

int sd_best_gamma(double alpha, double c, int gamma_max, double* speedup_out) {
    int best = 0;
    double best_s = 1.0;
    if (alpha >= 0.0 && alpha <= 1.0 && c >= 0.0)
        for (int g = 1; g <= gamma_max; ++g) {
            const double s = sd_eq1_speedup(alpha, g, c);
            if (s > best_s) { best_s = s; best = g; }
        }
    if (speedup_out) *speedup_out = best_s;
    return best;
}

sd_status sd_use_pass_kernel(sd_ctx* c, int target_on, int drafts_on, int max_rows) {
    if (!c || max_rows < 0 || max_rows > PASS_ROWS_CAP) return SD_ERR_INVALID_ARG;
    c->pass_on = target_on != 0 || drafts_on != 0;
    c->pass_drafts = drafts_on != 0;
    if (max_rows > 0) c->pass_max_rows = max_rows;
    return SD_OK;
}

sd_status sd_pass_tuning(sd_ctx* c, const int32_t* waves, const int32_t* chunk_major, int stages) {
    if (!c || stages < 0) return SD_ERR_INVALID_ARG;
    c->pass_stages = stages;
    CUDA_TRY(cudaStreamSynchronize(c->st));
    for (auto& g : c->graphs) cudaGraphExecDestroy(g.exec);        // programs and the graphs that captured them are rebuilt
    c->graphs.clear();
    c->programs.clear();
    c->pass_tuned = waves != nullptr;
    for (int m = 0; m < N_MAT && waves; ++m) {
        if (waves[m] < 1 || waves[m] > PASS_MAX_WAVES) return SD_ERR_INVALID_ARG;
        c->pass_tuning.waves[m] = waves[m];
        c->pass_tuning.chunk_major[m] = chunk_major ? (chunk_major[m] != 0) : 0;
    }
    return SD_OK;
}

sd_status sd_pass_stamps(sd_ctx* c, unsigned long long* stamps_dev, size_t n_words) {
    if (!c) return SD_ERR_INVALID_ARG;
    CUDA_TRY(cudaStreamSynchronize(c->st));
    for (auto& g : c->graphs) cudaGraphExecDestroy(g.exec);        // the buffer's address is a kernel argument
    c->graphs.clear();
    c->stamps = stamps_dev; c->stamps_words = stamps_dev ? n_words : 0;
    return SD_OK;
}

sd_status sd_pass_schedule_check(const int32_t* shape12, const int32_t* waves, const int32_t* chunk_major, int32_t* info8, char* err, size_t err_cap) {
    if (!shape12 || !info8) return SD_ERR_INVALID_ARG;
    PassShape sh{shape12[0], shape12[1], shape12[2], shape12[3], shape12[4], shape12[5], shape12[6], shape12[7], shape12[8], shape12[9], shape12[10], shape12[11]};
    PassTuning t = default_pass_tuning(sh);
    for (int m = 0; m < N_MAT && waves; ++m) { t.waves[m] = waves[m]; t.chunk_major[m] = chunk_major ? chunk_major[m] : 0; }
    const PassProgram p = build_pass_program(sh, t);
    info8[0] = p.words_per_layer; info8[1] = p.total_words; info8[2] = p.slots[0]; info8[3] = p.slots[1];
    info8[4] = p.max_seg; info8[5] = p.max_section; info8[6] = (int32_t)p.blob.size(); info8[7] = (int32_t)p.units_per_layer;
    if (err && err_cap) { strncpy(err, p.error.c_str(), err_cap - 1); err[err_cap - 1] = 0; }
    return p.error.empty() ? SD_OK : SD_ERR_UNSUPPORTED;
}

size_t sd_pass_schedule_blob(const int32_t* shape12, const int32_t* waves, const int32_t* chunk_major, void* out, size_t cap) {
    if (!shape12) return 0;
    PassShape sh{shape12[0], shape12[1], shape12[2], shape12[3], shape12[4], shape12[5], shape12[6], shape12[7], shape12[8], shape12[9], shape12[10], shape12[11]};
    PassTuning t = default_pass_tuning(sh);
    for (int m = 0; m < N_MAT && waves; ++m) { t.waves[m] = waves[m]; t.chunk_major[m] = chunk_major ? chunk_major[m] : 0; }
    const PassProgram p = build_pass_program(sh, t);
    if (!p.error.empty()) return 0;
    if (out && cap >= p.blob.size()) memcpy(out, p.blob.data(), p.blob.size());
    return p.blob.size();
}

sd_status sd_seq_alpha(sd_ctx* c, int seq, double* alpha_sum_out, int64_t* judged_out) {
    if (!c || seq < 0 || seq >= c->cfg.max_seqs || !alpha_sum_out || !judged_out) return SD_ERR_INVALID_ARG;
    if (c->phase[seq] == PH_FREE) return SD_ERR_STATE;
    CUDA_TRY(cudaMemcpyAsync(alpha_sum_out, c->S.alpha_sum + seq, sizeof(double), cudaMemcpyDeviceToHost, c->st));
    CUDA_TRY(cudaMemcpyAsync(judged_out, c->S.judged + seq, sizeof(int64_t), cudaMemcpyDeviceToHost, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
    return SD_OK;
}

sd_status sd_use_draft_streams(sd_ctx* c, int on) {
    if (!c) return SD_ERR_INVALID_ARG;
    c->groups_concurrent = on != 0 && c->sets.size() > 1;
    return SD_OK;
}

sd_status sd_tuning(sd_ctx* c, int knob, int value) {
    if (!c || knob < 0 || knob >= SD_TUNE_COUNT || value < 0) return SD_ERR_INVALID_ARG;
    CUDA_TRY(cudaStreamSynchronize(c->st));
    for (auto& g : c->graphs) cudaGraphExecDestroy(g.exec);        // the captured launches were shaped by the old value
    c->graphs.clear();
    c->tune[knob] = value;
    return SD_OK;
}

sd_status sd_launch_stamps(sd_ctx* c, int enable) {
    if (!c) return SD_ERR_INVALID_ARG;
    c->stamps_on = enable != 0;
    c->stamp_kinds.clear();
    return SD_OK;
}

sd_status sd_launch_stamps_read(sd_ctx* c, uint64_t* stamps_host, int32_t* kinds_host, int cap, int32_t* n_out) {
    if (!c || !stamps_host || !kinds_host || !n_out || cap < 0) return SD_ERR_INVALID_ARG;
    CUDA_TRY(cudaStreamSynchronize(c->st));
    const int n = std::min<int>(cap, (int)c->stamp_kinds.size());
    *n_out = (int32_t)c->stamp_kinds.size();
    if (n == 0) return SD_OK;
    CUDA_TRY(cudaMemcpy(stamps_host, c->stamp_buf, sizeof(uint64_t) * ST_WORDS * n, cudaMemcpyDeviceToHost));
    for (int i = 0; i < n; ++i) {
        kinds_host[i] = c->stamp_kinds[i];
        uint64_t* r = stamps_host + (size_t)ST_WORDS * i;
        for (int w : {ST_DEP_LAST, ST_DATA_LAST, ST_DONE_LAST}) r[w] = r[w] == ~0ull ? 0ull : ~r[w];        // "last" words hold complements
        for (int w : {ST_START, ST_DEP_FIRST, ST_DATA_FIRST, ST_DONE_FIRST}) if (r[w] == ~0ull) r[w] = 0ull;   // never reported
        r[7] = 0;
    }
    return SD_OK;
}

sd_status sd_cost_timing(sd_ctx* c, int enable) {
    if (!c) return SD_ERR_INVALID_ARG;
    c->cost_on = enable != 0;
    return SD_OK;
}

sd_status sd_cost_read(sd_ctx* c, sd_cost* out, int reset) {
    if (!c || !out) return SD_ERR_INVALID_ARG;
    CUDA_TRY(cudaStreamSynchronize(c->st));
    for (auto& m : c->cost_pending) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, m.e0, m.e1) == cudaSuccess) { c->cost_ms[m.kind] += ms; c->cost_units[m.kind] += (uint64_t)m.units; }
        else (void)cudaGetLastError();
        c->cost_free.push_back(m.e0); c->cost_free.push_back(m.e1);
    }
    c->cost_pending.clear();
    memset(out, 0, sizeof(*out));
    out->draft_passes = (int64_t)c->cost_units[0]; out->verify_passes = (int64_t)c->cost_units[1]; out->target_passes = (int64_t)c->cost_units[2];
    out->draft_pass_ms = c->cost_units[0] ? c->cost_ms[0] / c->cost_units[0] : 0.0;
    out->verify_pass_ms = c->cost_units[1] ? c->cost_ms[1] / c->cost_units[1] : 0.0;
    out->target_pass_ms = c->cost_units[2] ? c->cost_ms[2] / c->cost_units[2] : 0.0;
    const double denom = out->target_pass_ms > 0.0 ? out->target_pass_ms : out->verify_pass_ms;      // Eq. 1 takes a verify pass to cost one target pass
    out->c = (out->draft_pass_ms > 0.0 && denom > 0.0) ? out->draft_pass_ms / denom : 0.0;
    if (reset) for (int i = 0; i < 3; ++i) { c->cost_ms[i] = 0.0; c->cost_units[i] = 0; }
    return SD_OK;
}

int sd_best_gamma_measured(sd_ctx* c, int seq, int gamma_max, double* alpha_out, double* c_out, double* speedup_out) {
    if (!c || seq < 0 || seq >= c->cfg.max_seqs || gamma_max < 1) return 0;
    double a_sum = 0.0;
    int64_t judged = 0;
    sd_cost cost;
    if (sd_seq_alpha(c, seq, &a_sum, &judged) != SD_OK || judged <= 0 || sd_cost_read(c, &cost, 0) != SD_OK || cost.c <= 0.0) return 0;
    const double alpha = std::min(1.0, std::max(0.0, a_sum / (double)judged));
    if (alpha_out) *alpha_out = alpha;
    if (c_out) *c_out = cost.c;
    return sd_best_gamma(alpha, cost.c, gamma_max, speedup_out);
}

sd_status sd_use_graphs(sd_ctx* c, int on) {
    if (!c) return SD_ERR_INVALID_ARG;
    c->graphs_on = on != 0;
    return SD_OK;
}

sd_status sd_use_two_part_activations(sd_ctx* c, int on) {
    if (!c) return SD_ERR_INVALID_ARG;
    CUDA_TRY(cudaStreamSynchronize(c->st));
    for (auto& g : c->graphs) cudaGraphExecDestroy(g.exec);
    c->graphs.clear();
    c->two_part = on != 0;
    return SD_OK;
}

sd_status sd_force_plain_path(sd_ctx* c, int on) {
    if (!c) return SD_ERR_INVALID_ARG;
    c->force_plain = on != 0;
    return SD_OK;
}

sd_status sd_launch_count(sd_ctx* c, uint64_t* out) {
    if (!c || !out) return SD_ERR_INVALID_ARG;
    *out = c->launches;
    return SD_OK;
}

sd_status sd_profile(sd_ctx* c, int enable) {
    if (!c) return SD_ERR_INVALID_ARG;
    CUDA_TRY(cudaStreamSynchronize(c->st));
    c->prof_on = enable != 0;
    c->prof_used = 0;
    return SD_OK;
}

sd_status sd_profile_read(sd_ctx* c, float* ms_by_cat, uint32_t* launches_by_cat) {
    if (!c || !ms_by_cat || !launches_by_cat) return SD_ERR_INVALID_ARG;
    CUDA_TRY(cudaStreamSynchronize(c->st));
    for (int i = 0; i < SD_PROF_NCAT; ++i) { ms_by_cat[i] = 0.f; launches_by_cat[i] = 0; }
    for (size_t i = 0; i + 1 < c->prof_used; ++i) {
        const int cat = c->prof_cat[i];
        if (cat < 0 || cat >= SD_PROF_NCAT) continue;
        float ms = 0.f;
        CUDA_TRY(cudaEventElapsedTime(&ms, c->prof_ev[i], c->prof_ev[i + 1]));
        ms_by_cat[cat] += ms;
        launches_by_cat[cat] += 1;
    }
    c->prof_used = 0;
    return SD_OK;
}

// ------------------------------------------------------------------ single operators
size_t sd_op_linear_workspace(int rows, int n_out, int n_in, int dtype, int impl) {
    if (impl == 1 || dtype != SD_BF16 || !gemm_tc_supported(rows, n_out, n_in)) return 0;
    return gemm_partials_bytes(gemm_geometry(rows, n_out, n_in, sm_count()));
}

sd_status sd_op_linear(const void* x, const void* w, float* y, int rows, int n_out, int n_in, int dtype, int impl,
                       void* workspace, size_t workspace_bytes, void* stream) {
    if (!x || !w || !y || rows < 1 || n_out < 1 || n_in < 1 || (dtype != SD_F32 && dtype != SD_BF16)) return SD_ERR_INVALID_ARG;
    if (impl < 0 || impl > 2) return SD_ERR_INVALID_ARG;
    const bool tc_ok = dtype == SD_BF16 && gemm_tc_supported(rows, n_out, n_in);
    if (impl == 2 && !tc_ok) return SD_ERR_UNSUPPORTED;
    if (impl == 2 || (impl == 0 && tc_ok)) {
        const GemmGeom g = gemm_geometry(rows, n_out, n_in, sm_count());
        if (!workspace || workspace_bytes < gemm_partials_bytes(g)) return SD_ERR_OOM;
        TensorMap tw, tx;
        if (!make_tensor_map_bf16(&tw, w, n_out, n_in, 128) || !make_tensor_map_bf16(&tx, x, rows, n_in, g.m_pad)) return SD_ERR_CUDA;
        Epilogue e;
        memset(&e, 0, sizeof(e));
        e.mode = EPI_PLAIN; e.y = y; e.n_out_rows = rows; e.row_stride = 1; e.row_offset = 0;
        CUDA_TRY(launch_gemm_streamk(tw, tx, g, (float*)workspace, nullptr, nullptr, 0, (cudaStream_t)stream));
        CUDA_TRY(launch_fused_step(g, e, (const float*)workspace, nullptr, nullptr, 1, (cudaStream_t)stream));
        return SD_OK;
    }
    if (n_in % (dtype == SD_BF16 ? 8 : 4)) return SD_ERR_UNSUPPORTED;
    CUDA_TRY(launch_linear_simt(x, w, y, rows, n_out, n_in, dtype, (cudaStream_t)stream));
    return SD_OK;
}

sd_status sd_op_linear_wait_expiry(const void* x, const void* w, float* y, int rows, int n_out, int n_in, void* workspace, size_t workspace_bytes,
                                   uint32_t* arrive_dev, size_t arrive_words, unsigned long long wait_ns, uint32_t* status_dev, void* stream) {
    if (!x || !w || !y || !workspace || !arrive_dev || !status_dev || rows < 3 || rows > 8 || wait_ns == 0) return SD_ERR_INVALID_ARG;
    if (!gemm_tc_supported(rows, n_out, n_in)) return SD_ERR_UNSUPPORTED;
    const GemmGeom g = gemm_geometry(rows, n_out, n_in, sm_count());
    if (workspace_bytes < gemm_partials_bytes(g)) return SD_ERR_OOM;
    if (arrive_words < (size_t)g.n_tiles) return SD_ERR_CAPACITY;
    TensorMap tw, tx;
    if (!make_tensor_map_bf16(&tw, w, n_out, n_in, 128) || !make_tensor_map_bf16(&tx, x, rows, n_in, g.m_pad)) return SD_ERR_CUDA;
    Epilogue e;
    memset(&e, 0, sizeof(e));
    e.mode = EPI_PLAIN; e.y = y; e.n_out_rows = rows; e.row_stride = 1; e.row_offset = 0; e.poll_ns = wait_ns;
    if (!fused_step_polls(g, e)) return SD_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_TRY(cudaMemsetAsync(arrive_dev, 0, sizeof(uint32_t) * g.n_tiles, st));
    // the GEMM is NOT given the words, so nobody counts into them: every tile's wait runs out and takes the fallback
    CUDA_TRY(launch_gemm_streamk(tw, tx, g, (float*)workspace, nullptr, status_dev, 0, st));
    CUDA_TRY(launch_fused_step(g, e, (const float*)workspace, arrive_dev, status_dev, 1, st));
    return SD_OK;
}

size_t sd_op_attention_workspace(int rows, int n_heads, int head_dim, int max_ctx) {
    return std::max(attention_workspace_bytes(rows, n_heads, head_dim, max_ctx),
                    (head_dim == 64 || head_dim == 128) ? attention_split_workspace(rows, n_heads, head_dim, max_ctx) : (size_t)0);
}

sd_status sd_op_attention(const void* q, const void* kc, const void* vc, void* out, const int32_t* row_slot,
                          const int32_t* row_pos, int rows, int H, int Hkv, int hd, int max_ctx, int dtype,
                          void* ws, size_t ws_bytes, void* stream) {
    return sd_op_attention_runs(q, kc, vc, out, row_slot, row_pos, rows, 1, H, Hkv, hd, max_ctx, dtype, ws, ws_bytes, stream);
}

sd_status sd_op_attention_runs(const void* q, const void* kc, const void* vc, void* out, const int32_t* row_slot,
                               const int32_t* row_pos, int rows, int rows_per_seq, int H, int Hkv, int hd, int max_ctx, int dtype,
                               void* ws, size_t ws_bytes, void* stream) {
    if (rows_per_seq < 1 || rows % rows_per_seq) return SD_ERR_INVALID_ARG;
    if (!q || !kc || !vc || !out || !row_slot || !row_pos || rows < 1 || H < 1 || Hkv < 1 || H % Hkv) return SD_ERR_INVALID_ARG;
    if (hd < 8 || hd > 256 || (hd & 7) || max_ctx < 1 || (dtype != SD_F32 && dtype != SD_BF16)) return SD_ERR_INVALID_ARG;
    if (ws_bytes < sd_op_attention_workspace(rows, H, hd, max_ctx)) return SD_ERR_OOM;
    if (attention_split_supported(dtype, H, Hkv, hd)) {
        if (!ws) return SD_ERR_INVALID_ARG;
        CUDA_TRY(cudaMemsetAsync(ws, 0, 65536, (cudaStream_t)stream));                               // the arrival counters
        CUDA_TRY(launch_attention_split(q, kc, vc, out, row_slot, row_pos, rows, rows_per_seq, H, Hkv, hd, max_ctx, max_ctx, ws, ws_bytes, 0, (cudaStream_t)stream));
        return SD_OK;
    }
    CUDA_TRY(launch_attention(q, kc, vc, out, dtype, row_slot, row_pos, rows, H, Hkv, hd, max_ctx, ws, ws_bytes, (cudaStream_t)stream));
    return SD_OK;
}

sd_status sd_op_philox(const uint32_t* ctr, int n, uint32_t k0, uint32_t k1, uint32_t* out, void* stream) {
    if (!ctr || !out || n < 0) return SD_ERR_INVALID_ARG;
    CUDA_TRY(launch_philox(ctr, n, k0, k1, out, (cudaStream_t)stream));
    return SD_OK;
}

sd_status sd_op_softmax_sample(const float* logits, int rows, int V, float T, const uint32_t* u_int, float* probs,
                               int32_t* tok, void* stream) {
    if (!logits || !u_int || !probs || !tok || rows < 1 || V < 2 || !(T >= 0.f)) return SD_ERR_INVALID_ARG;
    CUDA_TRY(launch_softmax_sample_explicit(logits, rows, V, T, u_int, probs, tok, (cudaStream_t)stream));
    return SD_OK;
}

}  // extern "C"
