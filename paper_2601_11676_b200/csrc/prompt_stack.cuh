// Parameter block of the persistent prompt-stack kernel (internal).
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "stack_persistent.cuh"

namespace halo {

// Tensor maps of one run, in device memory: per block l the three maps [3 l + 0] gate/up rows (box 64 x NS rows),
// [3 l + 1] down rows as an MN-major operand (box 64 columns x 64 rows), [3 l + 2] predictor W1 (box 64 x 128 rows);
// then x[0], x[1] (box 64 x 128 tokens) and H[0], H[1] (box 64 x 128 tokens).
struct PromptParams {
    int L, T, d, S, G, r, act;
    int tiles_x;       // 256-token tiles
    int n_tn;          // 256-column tiles of the down projection
    int n_pn;          // 256-unit tiles of the predictor's hidden layer
    int z_cuts;        // K runs per down-projection output tile
    int subs;          // hidden tiles per group (S / NS)
    int ctl_stride;    // control words per block
    int r_pad;         // n_pn * 256
    int l2_ahead;      // K steps whose weight tiles are prefetched to L2 ahead of their load (0 = none)
    uint32_t step;     // arrival-draw counter of this prompt
    const CUtensorMap* maps;
    const __nv_bfloat16* const* W2;   // device table [L]
    float* h;                         // [T][d] residual stream, updated in place (holds h_0 at launch)
    __nv_bfloat16* x[2];              // block inputs by parity of the block
    __nv_bfloat16* H[2];              // hidden activations [T][h_cols] by parity of the block
    int h_cols;
    float* zpart;                     // [2][tiles_x * 8][r_pad] column sums of the predictor's hidden layer
    PersistSel* sel;                  // [L]; sel[0] = everything kept, written by the host
    unsigned* ctl;                    // control words, zero at launch
    uint32_t* status;
    // optional records of this prompt (may be null): x [L][T][d], scores [L][G], ...
    __nv_bfloat16* tap_x;
    float* tap_scores;
    int32_t* tap_dev_of_group;
    uint8_t* tap_arrived;
    int32_t* tap_keep_list;
    int32_t* tap_n_keep;
    // optional: [gridDim.x][16] words per thread block.  Nanoseconds seen by the first epilogue warp: 1 hidden tiles,
    // 2 predictor tiles and selection, 3 down tiles, 4 waiting for the next tile, 7 first to last time stamp.  SM
    // cycles: 5 loader waiting for hidden tiles of other CTAs, 6 for the block's selection, 8 for a free stage, 9 for
    // the rows of x; 10 / 11 MMA thread waiting for a filled stage (hidden and predictor / down tiles), 12 for the
    // accumulators to be drained, 13 / 14 MMA thread from a tile's start to its last commit
    unsigned long long* trace;
    int trace_items;                  // behind the [gridDim.x][16] words: per thread block this many records of
                                      // (queue entry + 1, start ns, end ns) of the first tiles it took
    PlanDev plan;
};

bool prompt_stack_supported(const halo_ffn_shape& ffn, const halo_pred_shape& pred, int n_layers, int n_tok);
int prompt_stack_ctl_stride(int tiles_x, int G);
size_t prompt_stack_ctl_bytes(int n_layers, int tiles_x, int G);
halo_status launch_prompt_stack(const PromptParams& P, cudaStream_t st);

// bf16 matrix [rows][cols] (cols contiguous, row_stride_elems apart), box = box_cols x box_rows, 128-byte swizzle,
// zero fill out of range (prefill_ffn.cu)
bool make_bf16_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t row_stride_elems,
                   uint32_t box_cols, uint32_t box_rows);

}  // namespace halo
