// halo_group_ffn, decode form (steps a6..a8): bandwidth-bound stream over the kept groups' weights.
//
// The FFN splits per neuron: h_j depends only on gate/up rows j, and the output is sum_j h_j * down_j.
// So the kept neurons (n_keep * S of them, addressed through keep_list) are cut into equal contiguous
// ranges, one per thread block.  A block walks its range in batches of 8 neurons:
//   phase 1  one warp per neuron: 16-byte coalesced loads of the gate and up rows against x held in
//            shared memory (fp32), warp-shuffle reduction, SiLU * up;
//   phase 2  the whole block streams the 8 down rows; each thread owns fixed 16-byte column chunks and
//            keeps their fp32 sums in registers across batches.
// When the holder (slot) of the groups changes, and at the end, the block adds its column sums into
// partials[slot] with vector fp32 reductions in L2.  Skipped groups are never addressed.
#include "common.cuh"

namespace halo {

constexpr int kFfnThreads = 256;
constexpr int kFfnWarps = kFfnThreads / 32;
constexpr int kBlocksPerSm = 2;

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

// x in shared memory as fp32.  For 8-element chunks the two halves of a chunk live in two planes so that
// a warp's 16-byte reads of consecutive chunks hit consecutive banks.
template <int E> struct XLayout;
template <> struct XLayout<4> {
    __device__ static __forceinline__ void load(const float* xs, int /*chunks*/, int c, float (&x)[4]) {
        const float4 v = *reinterpret_cast<const float4*>(xs + 4 * c);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
    __device__ static __forceinline__ int index(int /*chunks*/, int col) { return col; }
};
template <> struct XLayout<8> {
    __device__ static __forceinline__ void load(const float* xs, int chunks, int c, float (&x)[8]) {
        const float4 lo = *reinterpret_cast<const float4*>(xs + 4 * c);
        const float4 hi = *reinterpret_cast<const float4*>(xs + 4 * (chunks + c));
        x[0] = lo.x; x[1] = lo.y; x[2] = lo.z; x[3] = lo.w;
        x[4] = hi.x; x[5] = hi.y; x[6] = hi.z; x[7] = hi.w;
    }
    __device__ static __forceinline__ int index(int chunks, int col) {
        const int c = col >> 3, e = col & 7;
        return (e < 4) ? 4 * c + e : 4 * (chunks + c) + (e - 4);
    }
};

template <typename T, int ITERS>
__global__ void __launch_bounds__(kFfnThreads, kBlocksPerSm)
group_ffn_decode_kernel(int d, int S, int G, const T* __restrict__ W, const T* __restrict__ x_all,
                        const int32_t* __restrict__ keep_list, const int32_t* __restrict__ n_keep_ptr,
                        const int32_t* __restrict__ dev_of_group, int n_dev, int n_tok,
                        float* __restrict__ partials, uint32_t* dev_status) {
    constexpr int E = Elem<T>::kPerChunk;
    extern __shared__ __align__(16) float smem_f[];
    float* xs = smem_f;         // [d] (plane layout)
    float* hs = smem_f + d;     // [kFfnWarps]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tok = blockIdx.y;
    const int chunks = d / E;  // 16-byte chunks per row

    int nk = *n_keep_ptr;
    if (nk < 0 || nk > G) {
        if (tid == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
        nk = nk < 0 ? 0 : G;
    }
    const long long total = static_cast<long long>(nk) * S;  // kept neurons
    const int lo = static_cast<int>(total * blockIdx.x / gridDim.x);
    const int hi = static_cast<int>(total * (blockIdx.x + 1) / gridDim.x);
    if (lo >= hi) return;

    const T* x = x_all + static_cast<size_t>(tok) * d;
    for (int c = tid; c < d; c += kFfnThreads) xs[XLayout<E>::index(chunks, c)] = to_float(x[c]);
    __syncthreads();

    float acc[ITERS][E];
#pragma unroll
    for (int i = 0; i < ITERS; ++i)
#pragma unroll
        for (int e = 0; e < E; ++e) acc[i][e] = 0.0f;
    int cur_slot = -1;
    const size_t slot_stride = static_cast<size_t>(n_tok) * d;

    auto flush = [&](int slot) {
        float* dst = partials + static_cast<size_t>(slot) * slot_stride + static_cast<size_t>(tok) * d;
#pragma unroll
        for (int i = 0; i < ITERS; ++i) {
            const int c = tid + kFfnThreads * i;
            if (c < chunks) {
#pragma unroll
                for (int e = 0; e < E; e += 4)
                    red_add_v4(dst + c * E + e, acc[i][e], acc[i][e + 1], acc[i][e + 2], acc[i][e + 3]);
            }
#pragma unroll
            for (int e = 0; e < E; ++e) acc[i][e] = 0.0f;
        }
    };

    int n = lo;
    while (n < hi) {
        const int ki = n / S, j0 = n - ki * S;
        const int g = keep_list[ki];
        int cnt = min(kFfnWarps, min(hi - n, S - j0));
        int slot = 0;
        bool ok = (g >= 0 && g < G);
        if (ok && dev_of_group) {
            slot = dev_of_group[g] + 1;
            ok = (slot >= 0 && slot <= n_dev);
        }
        if (!ok) {  // block-uniform: skip the rest of this group
            if (tid == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
            n += S - j0;
            continue;
        }
        if (slot != cur_slot) {
            if (cur_slot >= 0) flush(cur_slot);
            cur_slot = slot;
        }
        const T* group = W + static_cast<size_t>(g) * 3 * S * d;

        // ---- phase 1: gate / up dot products, one neuron per warp -------------------------------
        if (warp < cnt) {
            const uint4* gate = reinterpret_cast<const uint4*>(group + static_cast<size_t>(j0 + warp) * d);
            const uint4* up = reinterpret_cast<const uint4*>(group + static_cast<size_t>(S + j0 + warp) * d);
            float a = 0.0f, b = 0.0f;
            for (int c0 = lane; c0 < chunks; c0 += 128) {
                uint4 wg[4], wu[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int c = c0 + 32 * u;
                    if (c < chunks) { wg[u] = ldg_stream16(gate + c); wu[u] = ldg_stream16(up + c); }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int c = c0 + 32 * u;
                    if (c < chunks) {
                        float xv[E], g8[E], u8[E];
                        XLayout<E>::load(xs, chunks, c, xv);
                        Elem<T>::widen(wg[u], g8);
                        Elem<T>::widen(wu[u], u8);
#pragma unroll
                        for (int e = 0; e < E; ++e) { a = fmaf(g8[e], xv[e], a); b = fmaf(u8[e], xv[e], b); }
                    }
                }
            }
            a = warp_sum(a);
            b = warp_sum(b);
            if (lane == 0) hs[warp] = a / (1.0f + __expf(-a)) * b;
        }
        __syncthreads();

        // ---- phase 2: down rows, block-wide, fixed columns per thread -----------------------------
        const T* down = group + static_cast<size_t>(2 * S + j0) * d;
        for (int jb = 0; jb < cnt; jb += 4) {
            uint4 wd[4][ITERS];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj)
#pragma unroll
                for (int i = 0; i < ITERS; ++i) {
                    const int c = tid + kFfnThreads * i;
                    if (jb + jj < cnt && c < chunks)
                        wd[jj][i] = ldg_stream16(reinterpret_cast<const uint4*>(down + static_cast<size_t>(jb + jj) * d) + c);
                }
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                if (jb + jj < cnt) {
                    const float h = hs[jb + jj];
#pragma unroll
                    for (int i = 0; i < ITERS; ++i) {
                        const int c = tid + kFfnThreads * i;
                        if (c < chunks) {
                            float w8[E];
                            Elem<T>::widen(wd[jj][i], w8);
#pragma unroll
                            for (int e = 0; e < E; ++e) acc[i][e] = fmaf(h, w8[e], acc[i][e]);
                        }
                    }
                }
            }
        }
        __syncthreads();  // hs is rewritten by the next batch
        n += cnt;
    }
    if (cur_slot >= 0) flush(cur_slot);
}

template <typename T>
static halo_status launch_typed(const halo_ffn_shape& sh, const void* W, const void* x, int n_tok,
                                const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group,
                                int n_dev, float* partials, uint32_t* dev_status, cudaStream_t st) {
    constexpr int E = Elem<T>::kPerChunk;
    const int d = sh.d_model, S = sh.group_size, G = sh.d_ffn / sh.group_size;
    const int chunks = d / E;
    const int iters = (chunks + kFfnThreads - 1) / kFfnThreads;
    if (iters > 4) return HALO_ERR_SHAPE;
    const long long max_batches = (static_cast<long long>(G) * S + kFfnWarps - 1) / kFfnWarps;
    const int gx = static_cast<int>(std::min<long long>(max_batches, static_cast<long long>(kSmCount) * kBlocksPerSm));
    dim3 grid(gx, n_tok);
    const size_t smem = sizeof(float) * (static_cast<size_t>(d) + kFfnWarps);
    const T* Wt = static_cast<const T*>(W);
    const T* xt = static_cast<const T*>(x);
#define HALO_FFN_CASE(I)                                                                                     \
    case I:                                                                                                  \
        group_ffn_decode_kernel<T, I><<<grid, kFfnThreads, smem, st>>>(d, S, G, Wt, xt, keep_list, n_keep,    \
                                                                        dev_of_group, n_dev, n_tok, partials, \
                                                                        dev_status);                          \
        break;
    switch (iters) {
        HALO_FFN_CASE(1)
        HALO_FFN_CASE(2)
        HALO_FFN_CASE(3)
        HALO_FFN_CASE(4)
    }
#undef HALO_FFN_CASE
    HALO_CHECK_LAUNCH();
    return HALO_OK;
}

halo_status launch_group_ffn_decode(const halo_ffn_shape& sh, const void* W, const void* x, int n_tok,
                                    const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group,
                                    int n_dev, float* partials, uint32_t* dev_status, cudaStream_t st, bool already_zero) {
    // bf16 shapes with a streaming configuration take the shared-memory ring kernel (which zeroes under its own stream)
    const halo_status fast = launch_group_ffn_stream(sh, W, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials,
                                                     dev_status, st, !already_zero);
    if (fast != HALO_ERR_UNIMPLEMENTED) return fast;
    const size_t bytes = sizeof(float) * static_cast<size_t>(n_dev + 1) * n_tok * sh.d_model;
    if (!already_zero && cudaMemsetAsync(partials, 0, bytes, st) != cudaSuccess) return HALO_ERR_CUDA;
    if (sh.wdtype == HALO_BF16)
        return launch_typed<__nv_bfloat16>(sh, W, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials,
                                           dev_status, st);
    return launch_typed<float>(sh, W, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials, dev_status, st);
}

}  // namespace halo
