// LM-head neuron groups (Sec. II-A: an up-projection only, a collection of groups of vocabulary rows;
// Sec. III-B.3: delivered reliably, so nothing is dropped): logits[t][v] = <W[v], x_t> for the rows of the listed
// groups.  Bandwidth-bound: the rows are streamed once, a warp takes two rows at a time with sixteen 16-byte loads
// per lane in flight; further tokens re-read the block's 32 rows while they are still cached.
#include "common.cuh"

namespace halo {

namespace {
constexpr int kLmRowsPerWarp = 4;                      // taken two at a time
constexpr int kLmRowsPerBlock = 8 * kLmRowsPerWarp;

template <typename T>
__global__ void __launch_bounds__(256)
lm_head_kernel(int d, int vocab, int S, int n_tok, const T* __restrict__ W, const T* __restrict__ x,
               const int32_t* __restrict__ keep_list, const int32_t* __restrict__ n_keep_ptr,
               float* __restrict__ logits, uint32_t* dev_status) {
    constexpr int E = Elem<T>::kPerChunk;
    extern __shared__ __align__(16) float xs[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_groups = (vocab + S - 1) / S;
    const int blocks_per_group = (S + kLmRowsPerBlock - 1) / kLmRowsPerBlock;
    const int ki = blockIdx.x / blocks_per_group, rb = blockIdx.x - ki * blocks_per_group;
    int g = ki;
    if (keep_list) {
        int nk = *n_keep_ptr;
        nk = max(0, min(nk, n_groups));
        if (ki >= nk) return;
        g = keep_list[ki];
        if (g < 0 || g >= n_groups) {
            if (threadIdx.x == 0 && rb == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
            return;
        }
    }
    const int v_end = min(vocab, (g + 1) * S);
    const int v_warp = g * S + rb * kLmRowsPerBlock + warp * kLmRowsPerWarp;   // this warp's first row
    const int chunks = d / E;
    for (int t = 0; t < n_tok; ++t) {
        if (t > 0) __syncthreads();                              // everybody is done with the previous x
        const uint4* x4 = reinterpret_cast<const uint4*>(x + static_cast<size_t>(t) * d);
        for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
            float xf[E];
            Elem<T>::widen(__ldg(x4 + c), xf);
#pragma unroll
            for (int e = 0; e < E; ++e) xs[c * E + e] = xf[e];
        }
        __syncthreads();
#pragma unroll 1
        for (int v0 = v_warp; v0 < min(v_end, v_warp + kLmRowsPerWarp); v0 += 2) {
            const bool two = v0 + 1 < v_end;
            const uint4* a4 = reinterpret_cast<const uint4*>(W + static_cast<size_t>(v0) * d);
            const uint4* b4 = two ? a4 + chunks : a4;            // a lone last row is read twice, used once
            float acc_a = 0.0f, acc_b = 0.0f;
            for (int c0 = lane; c0 < chunks; c0 += 256) {
                uint4 wa[8], wb[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int c = c0 + 32 * i;
                    wa[i] = c < chunks ? ldg_stream16(a4 + c) : make_uint4(0, 0, 0, 0);
                    wb[i] = c < chunks ? ldg_stream16(b4 + c) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int c = c0 + 32 * i;
                    if (c < chunks) {
                        float fa[E], fb[E];
                        Elem<T>::widen(wa[i], fa);
                        Elem<T>::widen(wb[i], fb);
#pragma unroll
                        for (int e = 0; e < E; ++e) {
                            const float xv = xs[c * E + e];
                            acc_a = fmaf(fa[e], xv, acc_a);
                            acc_b = fmaf(fb[e], xv, acc_b);
                        }
                    }
                }
            }
            acc_a = warp_sum(acc_a);
            acc_b = warp_sum(acc_b);
            float* out = logits + static_cast<size_t>(t) * vocab + v0;
            if (lane == 0) out[0] = acc_a;
            if (lane == 1 && two) out[1] = acc_b;
        }
    }
}
}  // namespace

}  // namespace halo

using namespace halo;

extern "C" halo_status halo_group_lm_head(const halo_lm_shape* shape, const void* W, const void* x, int n_tok,
                                          const int32_t* keep_list, const int32_t* n_keep, float* logits,
                                          uint32_t* dev_status, void* stream) {
    if (!shape || !W || !x || !logits || !dev_status) return HALO_ERR_ARG;
    if ((keep_list == nullptr) != (n_keep == nullptr)) return HALO_ERR_ARG;
    if (shape->wdtype != HALO_F32 && shape->wdtype != HALO_BF16) return HALO_ERR_DTYPE;
    if (shape->d_model <= 0 || shape->d_model % 8 != 0 || shape->d_model > 8192 || shape->vocab <= 0 ||
        shape->group_size <= 0 || n_tok <= 0)
        return HALO_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(W) & 15u) || (reinterpret_cast<uintptr_t>(x) & 15u)) return HALO_ERR_ALIGN;
    const int d = shape->d_model, S = shape->group_size;
    const long long n_groups = (static_cast<long long>(shape->vocab) + S - 1) / S;
    const long long blocks = n_groups * ((S + kLmRowsPerBlock - 1) / kLmRowsPerBlock);
    if (blocks > 0x7fffffffll) return HALO_ERR_SHAPE;
    const size_t smem = sizeof(float) * static_cast<size_t>(d);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (shape->wdtype == HALO_BF16)
        lm_head_kernel<__nv_bfloat16><<<static_cast<unsigned>(blocks), 256, smem, st>>>(
            d, shape->vocab, S, n_tok, static_cast<const __nv_bfloat16*>(W), static_cast<const __nv_bfloat16*>(x),
            keep_list, n_keep, logits, dev_status);
    else
        lm_head_kernel<float><<<static_cast<unsigned>(blocks), 256, smem, st>>>(
            d, shape->vocab, S, n_tok, static_cast<const float*>(W), static_cast<const float*>(x), keep_list, n_keep,
            logits, dev_status);
    return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}
