// Interface of the persistent streaming kernel: one launch runs every decoder layer (and the lm_head) of a forward
// pass, one CTA per SM, following a static program (pass_program.h).
//
// Everything the CTAs hand to one another inside the launch travels as TAGGED 64-bit words: the low half is the
// payload (one fp32, or two bf16), the high half a tag that names the pass, the layer and the use of the buffer.  A
// reader loads the words it needs and looks at their tags; a word whose tag is not the expected one has not been
// written yet, and the reader looks again.  A 64-bit store is a single access, so payload and tag arrive together:
// no flag, no fence and no atomic sits on the path between a producer and its consumers.
#pragma once
#include "gemm_tc.h"
#include "pass_program.h"

namespace sd {

typedef unsigned long long tagged_t;

// tag of (pass epoch, iteration = layer or n_layers for the lm_head, use of the buffer within the iteration)
__host__ __device__ __forceinline__ uint32_t pass_tag(uint32_t epoch, int it, int use) { return (epoch << 11) | ((uint32_t)it << 3) | (uint32_t)use; }
constexpr uint32_t PASS_EPOCH_WRAP = 1u << 21;          // epochs before tags repeat (the host clears the tagged buffers by then)

// Activation rows that feed a GEMM, as tagged words: [k block][row (m_pad of them)][32 words of two bf16 each].
__host__ __device__ __forceinline__ size_t xtagged_index(int row, int col, int m_pad) {          // in words
    return ((size_t)(col >> 6) * (size_t)m_pad + (size_t)row) * 32 + (size_t)((col & 63) >> 1);
}

struct PassMaps { TensorMap m[N_MAT]; };         // weights as [layer][row][k] tensor maps, boxes of 128 rows x 64 k

struct PassParams {
    int m_tok, m_pad, n_layers, has_tail;
    int d, H, Hkv, hd, F, V, max_ctx;
    int n_out[N_MAT];                            // output features of each matrix
    int stages;
    const uint32_t* epoch;                       // device word: number of this pass (all tags of the pass derive from it)
    // activations (tagged unless noted)
    tagged_t* h;                                 // [row][d] fp32 residual stream
    tagged_t* x[N_MAT];                          // input rows of each matrix (xn, attention output, xn, activation, xn)
    tagged_t* xn; tagged_t* attn; tagged_t* act;
    tagged_t* q;                                 // [row][H * hd / 2] two bf16 per word
    tagged_t* newkv;                             // [row][2][Hkv * hd / 2] keys and values this pass appends (a copy for this pass's attention)
    bf16* kc; bf16* vc; size_t kv_layer_elems;   // plain caches of layer 0; layers are kv_layer_elems apart
    const int32_t* row_slot; const int32_t* row_pos;      // plain, written by the kernel before this one
    const float* rcos; const float* rsin;        // plain [row][hd/2]
    tagged_t* ssq;                               // [row][SSQ_STRIDE] fp32
    const float* norm1; const float* norm2; size_t norm_stride;      // gains of layer 0; layers are norm_stride floats apart
    const float* final_norm;
    float rms_eps;
    float* logits; int logits_rows, row_stride, row_offset;          // plain: read by the next kernel
    // workspace
    tagged_t* partials[2];                       // [slot][row][128] fp32 pieces of output tiles
    uint32_t* abort_word;                        // set by the first wait that gives up; everybody else then winds down
    uint32_t* status;
    const uint8_t* program;
    // attention
    int rows_per_seq, rows_per_block, n_splits;
    tagged_t* part_o; tagged_t* part_ml;         // [row][H][slice][hd] and [row][H][slice][2] fp32
    // optional time stamps: [cta][iteration][segment][2] = (MMA thread turns to the segment, segment committed)
    unsigned long long* stamps; int stamp_segs;
    // ... and [cta][iteration][task][2] = (the task warps turn to the task, the task is done), for the first stamp_tasks tasks
    unsigned long long* task_stamps; int stamp_tasks;
};

bool make_tensor_map_layers(TensorMap* out, const void* base, int rows, int K, int n_layers, size_t layer_stride_bytes);
size_t pass_stream_smem(int m_pad, int* stages_out);
cudaError_t launch_pass_stream(const PassMaps& maps, const PassParams& p, int grid, int dependent, cudaStream_t st);
// Starts a pass: adds one to the epoch word and clears the abort word (one thread).
cudaError_t launch_pass_begin(uint32_t* epoch, uint32_t* abort_word, cudaStream_t st);

}  // namespace sd
