// halo_select_groups: steps a2..a5 as one 1024-thread block; and the fused
// "second predictor layer + selection" block used by the decode stack.
#include "select_device.cuh"

namespace halo {

__global__ void __launch_bounds__(1024)
select_kernel(const __grid_constant__ PlanDev plan, int G, const float* __restrict__ scores, uint32_t step,
              uint32_t layer, int force_all, int32_t* order, int32_t* dev_of_group, uint8_t* arrived,
              uint8_t* keep, int32_t* keep_list, int32_t* n_keep, uint32_t* dev_status) {
    __shared__ SelectSmem sm;
    select_block<1024>(sm, plan, G, scores, step, layer, force_all, order, dev_of_group, arrived, keep, keep_list,
                       n_keep, dev_status, threadIdx.x, BlockSync());
}

// s[g] = <W2[g], hidden> for every group (one warp per group, strided), then the selection on those scores.
template <typename T>
__global__ void __launch_bounds__(1024)
score_select_kernel(const __grid_constant__ PlanDev plan, int G, int rank, const T* __restrict__ W2,
                    const float* __restrict__ hidden, uint32_t step, uint32_t layer, int force_all,
                    float* scores, int32_t* order, int32_t* dev_of_group, uint8_t* arrived, uint8_t* keep,
                    int32_t* keep_list, int32_t* n_keep, uint32_t* dev_status) {
    __shared__ SelectSmem sm;
    __shared__ float s_local[HALO_MAX_GROUPS];
    extern __shared__ float z[];  // [rank]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int u = tid; u < rank; u += blockDim.x) z[u] = hidden[u];
    __syncthreads();
    constexpr int E = Elem<T>::kPerChunk;
    const int chunks = rank / E;
    for (int g = warp; g < G; g += 32) {
        const uint4* row = reinterpret_cast<const uint4*>(W2 + static_cast<size_t>(g) * rank);
        float acc = 0.0f;
        for (int c = lane; c < chunks; c += 32) {
            float w[E];
            Elem<T>::widen(__ldg(row + c), w);
#pragma unroll
            for (int e = 0; e < E; ++e) acc = fmaf(w[e], z[c * E + e], acc);
        }
        acc = warp_sum(acc);
        if (lane == 0) { s_local[g] = acc; if (scores) scores[g] = acc; }
    }
    __syncthreads();
    select_block<1024>(sm, plan, G, s_local, step, layer, force_all, order, dev_of_group, arrived, keep, keep_list,
                       n_keep, dev_status, threadIdx.x, BlockSync());
}

halo_status launch_select(const PlanDev& plan, int G, const float* scores, uint32_t step, uint32_t layer,
                          int force_all, int32_t* order, int32_t* dev_of_group, uint8_t* arrived, uint8_t* keep,
                          int32_t* keep_list, int32_t* n_keep, uint32_t* dev_status, cudaStream_t st) {
    select_kernel<<<1, 1024, 0, st>>>(plan, G, scores, step, layer, force_all, order, dev_of_group, arrived, keep,
                                      keep_list, n_keep, dev_status);
    HALO_CHECK_LAUNCH();
    return HALO_OK;
}

halo_status launch_score_select(const halo_pred_shape& sh, const void* W2, const float* hidden,
                                const PlanDev& plan, uint32_t step, uint32_t layer, int force_all, float* scores,
                                int32_t* order, int32_t* dev_of_group, uint8_t* arrived, uint8_t* keep,
                                int32_t* keep_list, int32_t* n_keep, uint32_t* dev_status, cudaStream_t st) {
    const size_t smem = sizeof(float) * static_cast<size_t>(sh.rank);
    if (sh.wdtype == HALO_BF16)
        score_select_kernel<__nv_bfloat16><<<1, 1024, smem, st>>>(
            plan, sh.n_groups, sh.rank, static_cast<const __nv_bfloat16*>(W2), hidden, step, layer, force_all,
            scores, order, dev_of_group, arrived, keep, keep_list, n_keep, dev_status);
    else
        score_select_kernel<float><<<1, 1024, smem, st>>>(plan, sh.n_groups, sh.rank, static_cast<const float*>(W2),
                                                          hidden, step, layer, force_all, scores, order,
                                                          dev_of_group, arrived, keep, keep_list, n_keep,
                                                          dev_status);
    HALO_CHECK_LAUNCH();
    return HALO_OK;
}

}  // namespace halo
