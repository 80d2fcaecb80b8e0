// Steps a2..a5 for one cooperating set of NT threads: rank by counting, critical choice, Algorithm-3 chunk
// lookup, arrival mask, ordered compaction.  `sync` is a barrier over exactly those NT threads.
#pragma once
#include "common.cuh"
#include "philox.cuh"

namespace halo {

struct SelectSmem {
    float score[HALO_MAX_GROUPS];
    unsigned char kept[HALO_MAX_GROUPS];
    int boundary[HALO_MAX_DEVICES + 1];
    int arrived[HALO_MAX_DEVICES];
    int flags;
    int count;
};

// `scores` may point to global or shared memory.  All NT threads must call; tid in [0, NT).
template <int NT, typename Sync>
__device__ __forceinline__ void select_block(SelectSmem& sm, const PlanDev& plan, int G, const float* scores,
                                             uint32_t step, uint32_t layer, int force_all, int32_t* order,
                                             int32_t* dev_of_group, uint8_t* arrived, uint8_t* keep,
                                             int32_t* keep_list, int32_t* n_keep, uint32_t* dev_status, int tid,
                                             Sync sync) {
    constexpr int PER = (HALO_MAX_GROUPS + NT - 1) / NT;
    static_assert(NT > HALO_MAX_DEVICES, "one thread per boundary entry");
    float v[PER];
    if (tid == 0) { sm.flags = 0; sm.count = 0; }
    sync();  // also orders any earlier use of sm by the caller
    int above = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int g = tid + i * NT;
        v[i] = -INFINITY;
        if (g < G) {
            float s = scores[g];
            bool nonfinite = false;
            if (isnan(s)) { s = -INFINITY; nonfinite = true; }
            else if (isinf(s)) nonfinite = true;
            if (s == 0.0f) s = 0.0f;  // -0 and +0 are one value
            v[i] = s;
            sm.score[g] = s;
            if (nonfinite) atomicOr(&sm.flags, 1);
            if (s >= plan.threshold) ++above;
        }
    }
    if (plan.mode == HALO_SEL_THRESHOLD && above) atomicAdd(&sm.count, above);
    sync();

    // a2: position in the priority order = number of groups that come before this one
    int rank[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int g = tid + i * NT;
        rank[i] = 0;
        if (g < G) {
            int r = 0;
            for (int o = 0; o < G; ++o) {
                const float so = sm.score[o];
                r += (so > v[i] || (so == v[i] && o < g)) ? 1 : 0;
            }
            rank[i] = r;
        }
    }
    // a3: number of critical groups
    int k = (plan.mode == HALO_SEL_THRESHOLD) ? sm.count : plan.k_critical;
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
    sync();

    int dev[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int g = tid + i * NT;
        dev[i] = -1;
        if (g < G) {
            if (rank[i] >= k) {
                const int p = rank[i] - k;
                for (int j = 0; j < plan.n_dev; ++j)
                    if (sm.boundary[j] <= p && p < sm.boundary[j + 1]) { dev[i] = plan.dev_order[j]; break; }
            }
            sm.kept[g] = (dev[i] < 0 || sm.arrived[dev[i]] != 0) ? 1 : 0;
        }
    }
    sync();

    // ordered compaction: a kept group's position = number of kept groups with a smaller id
    int total_kept = 0;
    for (int o = 0; o < G; ++o) total_kept += sm.kept[o];
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int g = tid + i * NT;
        if (g < G) {
            const bool kept = sm.kept[g] != 0;
            if (order) order[rank[i]] = g;
            if (dev_of_group) dev_of_group[g] = dev[i];
            if (keep) keep[g] = kept ? 1 : 0;
            if (kept) {
                int pos = 0;
                for (int o = 0; o < g; ++o) pos += sm.kept[o];
                keep_list[pos] = g;
            }
            if (g >= total_kept) keep_list[g] = -1;  // padding behind the kept ids
        }
    }
    if (tid == 0) {
        *n_keep = total_kept;
        if (sm.flags) flag_status(dev_status, HALO_DEV_NONFINITE_SCORE);
    }
}

struct BlockSync {
    __device__ __forceinline__ void operator()() const { __syncthreads(); }
};

}  // namespace halo
