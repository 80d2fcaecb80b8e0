// Steps a2..a5 for one block of 1024 threads: rank by counting, critical choice, Algorithm-3 chunk lookup,
// arrival mask, ordered compaction.  Callable from any kernel whose block has 1024 threads.
#pragma once
#include "common.cuh"
#include "philox.cuh"

namespace halo {

struct SelectSmem {
    float score[HALO_MAX_GROUPS];
    int boundary[HALO_MAX_DEVICES + 1];
    int arrived[HALO_MAX_DEVICES];
    int warp_count[32];
    int flags;
};

// `scores` may point to global or shared memory.  All 1024 threads must call.
__device__ __forceinline__ void select_block(SelectSmem& sm, const PlanDev& plan, int G, const float* scores,
                                             uint32_t step, uint32_t layer, int force_all, int32_t* order,
                                             int32_t* dev_of_group, uint8_t* arrived, uint8_t* keep,
                                             int32_t* keep_list, int32_t* n_keep, uint32_t* dev_status) {
    const int tid = threadIdx.x;
    const bool valid = tid < G;
    float v = -INFINITY;
    bool nonfinite = false;
    if (valid) {
        v = scores[tid];
        if (isnan(v)) { v = -INFINITY; nonfinite = true; }
        else if (isinf(v)) nonfinite = true;
        if (v == 0.0f) v = 0.0f;  // -0 and +0 are one value
    }
    if (tid == 0) sm.flags = 0;
    __syncthreads();  // also orders any earlier use of sm by the caller
    if (valid) sm.score[tid] = v;
    if (nonfinite) atomicOr(&sm.flags, 1);
    __syncthreads();

    // a2: position in the priority order = number of groups that come before this one
    int rank = 0;
    if (valid) {
        for (int o = 0; o < G; ++o) {
            const float so = sm.score[o];
            rank += (so > v || (so == v && o < tid)) ? 1 : 0;
        }
    }
    // a3: number of critical groups
    int k = plan.k_critical;
    if (plan.mode == HALO_SEL_THRESHOLD) k = __syncthreads_count(valid && v >= plan.threshold);
    if (plan.n_dev == 0) k = G;
    const int M = G - k;

    // a4 tables: chunk boundaries for M less-critical groups; a5: arrival draws
    if (tid <= plan.n_dev) {
        int b = 0;
        if (tid == plan.n_dev) b = M;
        else if (tid > 0) {
            const unsigned long long total = plan.cum_weight[plan.n_dev - 1];
            b = static_cast<int>((2ull * static_cast<unsigned long long>(M) * plan.cum_weight[tid - 1] + total) /
                                 (2ull * total));
        }
        sm.boundary[tid] = b;
    }
    if (tid < plan.n_dev) {
        const bool a = force_all || device_arrives(plan.seed_lo, plan.seed_hi, step, layer,
                                                    static_cast<uint32_t>(tid), plan.loss_thresh[tid]);
        sm.arrived[tid] = a ? 1 : 0;
        if (arrived) arrived[tid] = a ? 1 : 0;
    }
    __syncthreads();

    int dev = -1;
    if (valid && rank >= k) {
        const int p = rank - k;
        for (int j = 0; j < plan.n_dev; ++j)
            if (sm.boundary[j] <= p && p < sm.boundary[j + 1]) { dev = plan.dev_order[j]; break; }
    }
    const bool kept = valid && (dev < 0 || sm.arrived[dev] != 0);

    // ordered compaction: kept group ids ascending
    const unsigned ballot = __ballot_sync(0xffffffffu, kept);
    const int lane = tid & 31, warp = tid >> 5;
    if (lane == 0) sm.warp_count[warp] = __popc(ballot);
    __syncthreads();
    int before = 0, total_kept = 0;
    for (int w = 0; w < 32; ++w) {
        const int c = sm.warp_count[w];
        if (w < warp) before += c;
        total_kept += c;
    }
    const int pos = before + __popc(ballot & ((1u << lane) - 1u));
    if (valid) {
        if (order) order[rank] = tid;
        if (dev_of_group) dev_of_group[tid] = dev;
        if (keep) keep[tid] = kept ? 1 : 0;
        if (kept) keep_list[pos] = tid;
        if (tid >= total_kept) keep_list[tid] = -1;  // padding behind the kept ids
    }
    if (tid == 0) {
        *n_keep = total_kept;
        if (sm.flags) flag_status(dev_status, HALO_DEV_NONFINITE_SCORE);
    }
}

}  // namespace halo
