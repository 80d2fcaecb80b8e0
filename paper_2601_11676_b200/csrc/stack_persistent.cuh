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
    int sel_cost;                          // batches the selecting thread block is spared per block
    const __nv_bfloat16* const* W;         // device tables [L]
    const __nv_bfloat16* const* W1;
    const __nv_bfloat16* const* W2;
    const float* h0;                       // [steps][d]
    float* h_out;                          // [steps][d]
    float* partials;                       // [3][n_dev+1][d], zero at launch
    float* z;                              // [r]
    PersistSel* sel;                       // [3]: two rotating + the static first-block selection
    unsigned* sync;                        // [4]: barrier count, abort, hidden rows done, selections published
    uint32_t* status;
    // optional records (thread block 0 / the selecting thread block write them)
    __nv_bfloat16* tap_x;
    float* tap_scores;
    int32_t* tap_dev_of_group;
    uint8_t* tap_arrived;
    int32_t* tap_keep_list;
    int32_t* tap_n_keep;
    float* tap_y;
    PlanDev plan;
};

bool persistent_supported(const halo_ffn_shape& sh, int n_tok, int G);
halo_status launch_stack_persistent(PersistParams& P, cudaStream_t st);

}  // namespace halo
