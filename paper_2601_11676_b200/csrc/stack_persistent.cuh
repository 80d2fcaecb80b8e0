// Parameter block of the persistent decode-stack kernel (internal).
#pragma once
#include "common.cuh"

namespace halo {

// One selection result in device memory (written by the selecting thread block, read by every producer).
struct PersistSel {
    int32_t n_keep;
    int32_t pad[3];
    int32_t keep_list[HALO_MAX_GROUPS];
    int32_t dev_of_group[HALO_MAX_GROUPS];
    uint8_t arrived[HALO_MAX_DEVICES];
};

struct PersistParams {
    int L, steps, d, S, G, r, act;
    uint32_t step0;
    const __nv_bfloat16* const* W;         // device tables [L]
    const __nv_bfloat16* const* W1;
    const __nv_bfloat16* const* W2;
    const float* h0;                       // [steps][d]
    float* h_out;                          // [steps][d]
    float* partials;                       // [3][2][d] rotating interleaved accumulation buffers, zero at launch
    float* z;                              // [2][r]: hidden values, by parity of the prediction
    PersistSel* sel;                       // [3]: two rotating + the static first-block selection
    unsigned* sync;                        // [64]: 0 barrier count, 1 abort, 2 hidden rows done, 3 selections
                                           //       published, 32..63 rotating batch counters; zero at launch
    uint32_t* status;
    // optional records (thread block 0 / the selecting thread block write them)
    __nv_bfloat16* tap_x;
    float* tap_scores;
    int32_t* tap_dev_of_group;
    uint8_t* tap_arrived;
    int32_t* tap_keep_list;
    int32_t* tap_n_keep;
    float* tap_y;
    // optional trace: [trace_blocks][gridDim.x][8] timestamps (ns, global timer) written by thread 0 of every
    // thread block for the first trace_blocks blocks of the run
    int cross_stages;                      // stages of the next block a producer may issue before its consumers
                                           // have passed the grid barrier of the current block
    int l2_ahead;                          // batches per thread block prefetched into L2 on entering a block
    int tmem_ring;                         // 1: stages pass through tensor memory (d_model 2048 / 4096 only)
    int i4;                                // 1: W holds int4 codes (uint8), Wsc their bf16 scales per 128 elements
    const __nv_bfloat16* const* Wsc;       // device table [L] (i4 only)
    int pred_serial;                       // 1: the predictor rows and the selection of block l run at the start of
                                           // block l itself (from the recorded x_{l-1}), not beside block l-1
    int deterministic;                     // 1: fixed batch assignment and fixed-order sums (bitwise repeatable)
    __nv_bfloat16* x_hist;                 // [2][d]: input of the previous block (pred_serial only)
    float* det_rows;                       // [2][gridDim.x][d]: per-thread-block column sums (deterministic only)
    unsigned long long* trace;
    int trace_blocks;
    PlanDev plan;
};

bool persistent_supported(const halo_ffn_shape& sh, int n_tok, int G);
bool persistent_supported_i4(const halo_ffn_shape& sh, int n_tok, int G);   // int4 codes + scales
halo_status launch_stack_persistent(PersistParams& P, cudaStream_t st);

}  // namespace halo
