// Interface of the persistent streaming kernel: one launch runs every decoder layer (and the lm_head) of a forward
// pass, one CTA per SM, following a static program (pass_program.h).
#pragma once
#include "gemm_tc.h"
#include "pass_program.h"

namespace sd {

// Activation rows as the GEMM's narrow operand, stored the way a ring stage wants them so that a k block is one
// contiguous copy: [k block][m_pad rows][64 elements], 128-byte rows with the 16-byte pieces XOR-swizzled by row.
__host__ __device__ __forceinline__ size_t xpacked_offset(int row, int col, int m_pad) {      // in bytes
    return (size_t)(col >> 6) * ((size_t)m_pad * 128) + (size_t)row * 128 + (size_t)((((col & 63) >> 3) ^ (row & 7)) << 4) + (size_t)(col & 7) * 2;
}

struct PassMaps { TensorMap m[N_MAT]; };         // weights as [layer][row][k] tensor maps, boxes of 128 rows x 64 k

struct PassParams {
    int m_tok, m_pad, n_layers, has_tail;
    int d, H, Hkv, hd, F, V, max_ctx;
    int n_out[N_MAT];                            // output features of each matrix
    int stages, words_per_layer;
    // activations
    float* h;                                    // [row][d] residual stream
    uint8_t* x[N_MAT];                           // packed input rows of each matrix (xn, attention output, xn, activation, xn)
    uint8_t* xn; uint8_t* attn; uint8_t* act;
    bf16* q;                                     // [row][H][hd]
    bf16* kc; bf16* vc; size_t kv_layer_elems;   // caches of layer 0; layers are kv_layer_elems apart
    const int32_t* row_slot; const int32_t* row_pos;
    const float* rcos; const float* rsin;        // [row][hd/2]
    float* ssq;                                  // [row][SSQ_STRIDE]
    const float* norm1; const float* norm2; size_t norm_stride;      // gains of layer 0; layers are norm_stride floats apart
    const float* final_norm;
    float rms_eps;
    float* logits; int logits_rows, row_stride, row_offset;
    // workspace and synchronisation
    float* partials[2];
    uint32_t* sync;                              // arrival / completion words, zero when the kernel starts
    uint32_t* abort_word;                        // set by the first wait that gives up; everybody else then winds down
    uint32_t* status;
    const uint8_t* program;
    // attention
    int rows_per_seq, rows_per_block, n_splits;
    float* part_o; float* part_ml; uint32_t* att_counters;
    // optional time stamps: [cta][iteration][segment][2] = (MMA thread starts waiting for the segment, segment committed)
    unsigned long long* stamps; int stamp_segs;
    // ... and [cta][iteration][task][2] = (the task warps turn to the task, the task is done), for the first stamp_tasks tasks
    unsigned long long* task_stamps; int stamp_tasks;
};

bool make_tensor_map_layers(TensorMap* out, const void* base, int rows, int K, int n_layers, size_t layer_stride_bytes);
size_t pass_stream_smem(int m_pad, int* stages_out);
cudaError_t launch_pass_stream(const PassMaps& maps, const PassParams& p, int grid, int dependent, cudaStream_t st);

}  // namespace sd
