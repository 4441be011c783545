// Static schedule ("program") of one forward pass on the persistent streaming kernel (pass_stream.cu).
//
// One CTA per SM walks, layer after layer, a list of segments (runs of 128 x 64 weight blocks of one
// output tile) through one ring of shared-memory stages, so that the weight stream never stops at a
// matrix boundary.  Every weight matrix is cut into tile waves x K chunks:
//   - the tiles of a matrix are grouped into waves; a wave's tiles are complete (all their pieces in
//     the workspace) well before the matrix ends, and the small tasks that sum the pieces and apply
//     the step after the GEMM run on spare warps while later waves stream;
//   - the reduction dimension of the next matrix is cut into chunks that match those waves: a chunk
//     of its input rows exists as soon as the wave that produces it has been reduced, so the next
//     matrix starts on its first chunk while the tail of the previous one is still being reduced.
// Blocks (wave, chunk) of a matrix are split evenly over all CTAs (stream-K within the block).
// The program holds, per CTA: its segments in ring order, its reduce / attention tasks in the order
// they become ready, and for every reduce task the workspace slots of the tile's pieces in a fixed
// order (run-to-run identical sums).  Everything is host arithmetic on shapes; build_pass_program
// also replays the program on the host and refuses one whose waits could not all be satisfied.
#pragma once
#include <stdint.h>

#include <string>
#include <vector>

namespace sd {

enum { MAT_QKV = 0, MAT_WO = 1, MAT_GU = 2, MAT_DN = 3, MAT_LM = 4, N_MAT = 5, MAT_ATT = 5 };
// flags of a segment: waits for a word; the word belongs to the previous layer; first / last segment of its accumulator
// (bits 4..7: which accumulator in tensor memory)
enum { SEG_DEP = 1, SEG_DEP_PREV = 2, SEG_FIRST = 4, SEG_LAST = 8 };
enum { TASK_REDUCE = 0, TASK_ATTENTION = 1 };
constexpr uint16_t NO_WORD = 0xFFFFu;
constexpr int PASS_MAX_WAVES = 8;

// One run of k blocks of one output tile.  A CTA's segments of the same tile (one per chunk of the wave) accumulate
// into one TMEM accumulator; the last of them leaves the CTA's piece of the tile in the workspace.
struct PassSeg {
    uint16_t tile, kb0, n_kb;
    uint8_t mat, flags;
    uint16_t dep, dep_need;      // word (relative to the layer's words) that must reach dep_need before the input rows are loaded
    uint16_t arrive;             // word that counts the pieces of the tile
    uint16_t slot;               // SEG_LAST: workspace slot of the piece (per region: matrices alternate between two regions)
};
static_assert(sizeof(PassSeg) == 16, "segment record");

struct PassTask {
    uint32_t item;               // reduce: output tile; attention: (query block * Hkv + kv head) * n_splits + slice
    uint32_t piece0;             // reduce: first entry of the CTA's piece list
    uint16_t kind, mat;
    uint16_t wait_word, wait_need;
    uint16_t done_word;          // word to add one to when the task's output is in memory (NO_WORD: none)
    uint16_t n_pieces;
};
static_assert(sizeof(PassTask) == 20, "task record");

// Per-CTA section of the program blob (offsets in bytes from the section start).
struct PassCtaHeader {
    uint32_t n_seg[2], n_task[2];            // [0] per layer, [1] after the last layer (lm_head)
    uint32_t seg_off[2], task_off[2], piece_off;
    uint32_t bytes;
    uint32_t pad[2];                         // sections are copied in 16-byte pieces: every part starts on a multiple of 16
};
static_assert(sizeof(PassCtaHeader) % 16 == 0, "section header");

struct PassShape {
    int n_layers, d, H, Hkv, hd, F, V;
    int m_tok;                   // query rows of the pass
    int rows_per_seq;            // rows come in runs of this many consecutive rows of one sequence
    int n_splits;                // slices of the cache per (query block, kv head)
    int want_logits;             // the pass ends with the lm_head
    int grid;                    // CTAs (one per SM)
};

struct PassTuning {
    int waves[N_MAT];            // tile waves per matrix (QKV, Wo, gate/up, down, lm_head)
    int chunk_major[N_MAT];      // block order of a matrix: 0 = wave after wave, 1 = chunk after chunk
};
PassTuning default_pass_tuning(const PassShape& s);

struct PassProgram {
    std::vector<uint8_t> blob;   // uint32 cta_off[grid + 1], then the CTA sections
    int words_per_layer;         // arrival / completion words of one layer
    int total_words;             // all layers + lm_head
    int slots[2];                // workspace slots per region
    int max_seg;                 // most segments of a CTA in one layer (or in the tail)
    int max_section;             // largest CTA section in bytes
    int rows_per_block;          // query rows of one attention item
    int n_blocks;                // query blocks of the pass
    int64_t units_per_layer;     // 16 KB weight blocks of one layer
    std::string error;           // non-empty: the program could not be built
};

bool pass_shape_supported(const PassShape& s);
PassProgram build_pass_program(const PassShape& s, const PassTuning& t);
// Replays the program on the host: every CTA advances through its segments and tasks whenever their
// waits are satisfied.  Returns an empty string if everything completes, every (tile, k block) of every
// matrix is covered exactly once and the counts the waits expect are the counts delivered.
std::string check_pass_program(const PassShape& s, const PassProgram& p);

}  // namespace sd
