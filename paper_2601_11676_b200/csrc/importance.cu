// halo_group_importance: the "true" importance of every neuron group for one input vector, i.e. the L2 norm of
// the group's partial output p_g (Sec. II-B: the loss of an activation is measured by its L2 norm; groups with
// large norms dominate the merged features).  It is what a semantic-aware predictor is trained to regress.
// Implementation: the decode FFN with every group kept and one accumulation slot per group, then one norm per
// slot.  Diagnostic / calibration path, not part of the per-token hot loop.
#include "common.cuh"

namespace halo {

// keep_list = 0..G-1, n_keep = G, dev_of_group[g] = g - 1 (so that slot(g) = g)
__global__ void importance_setup_kernel(int G, int32_t* keep_list, int32_t* n_keep, int32_t* dev_of_group) {
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g < G) { keep_list[g] = g; dev_of_group[g] = g - 1; }
    if (g == 0) *n_keep = G;
}

__global__ void __launch_bounds__(256)
group_norm_kernel(int d, const float* __restrict__ group_partials /*[G][d]*/, float* __restrict__ norms) {
    __shared__ float part[8];
    const int g = blockIdx.x;
    float acc = 0.0f;
    for (int c = threadIdx.x; c < d; c += 256) {
        const float v = group_partials[static_cast<size_t>(g) * d + c];
        acc = fmaf(v, v, acc);
    }
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) tot += part[w];
        norms[g] = sqrtf(tot);
    }
}

}  // namespace halo

extern "C" size_t halo_group_importance_workspace_bytes(const halo_ffn_shape* shape) {
    if (!shape || shape->group_size <= 0 || shape->d_ffn <= 0 || shape->d_model <= 0) return 0;
    const size_t G = static_cast<size_t>(shape->d_ffn / shape->group_size);
    return sizeof(float) * G * shape->d_model + sizeof(int32_t) * (2 * G + 4);
}

extern "C" halo_status halo_group_importance(const halo_ffn_shape* shape, const void* W_packed, const void* x,
                                             float* norms, void* workspace, size_t workspace_bytes,
                                             uint32_t* dev_status, void* stream) {
    if (!shape || !W_packed || !x || !norms) return HALO_ERR_ARG;
    if (shape->wdtype != HALO_F32 && shape->wdtype != HALO_BF16) return HALO_ERR_DTYPE;
    if (shape->d_model <= 0 || shape->d_model % 8 != 0 || shape->group_size <= 0 || shape->d_ffn <= 0 ||
        shape->d_ffn % shape->group_size != 0 || shape->d_ffn / shape->group_size > HALO_MAX_GROUPS)
        return HALO_ERR_SHAPE;
    if (!halo::aligned16(W_packed) || !halo::aligned16(x) || !halo::aligned16(workspace)) return HALO_ERR_ALIGN;
    if (!workspace || workspace_bytes < halo_group_importance_workspace_bytes(shape)) return HALO_ERR_WORKSPACE;
    const int G = shape->d_ffn / shape->group_size, d = shape->d_model;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* pg = static_cast<float*>(workspace);                                  // [G][d]
    int32_t* keep_list = reinterpret_cast<int32_t*>(pg + static_cast<size_t>(G) * d);
    int32_t* dev_of_group = keep_list + G;
    int32_t* n_keep = dev_of_group + G;
    halo::importance_setup_kernel<<<(G + 127) / 128, 128, 0, st>>>(G, keep_list, n_keep, dev_of_group);
    if (cudaGetLastError() != cudaSuccess) return HALO_ERR_CUDA;
    // one slot per group: slot(g) = dev_of_group[g] + 1 = g, n_dev = G - 1 (zeroes the slots first)
    halo_status rc = halo::launch_group_ffn_decode(*shape, W_packed, x, 1, keep_list, n_keep, dev_of_group, G - 1, pg,
                                                   dev_status, st);
    if (rc != HALO_OK) return rc;
    halo::group_norm_kernel<<<G, 256, 0, st>>>(d, pg, norms);
    return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}
