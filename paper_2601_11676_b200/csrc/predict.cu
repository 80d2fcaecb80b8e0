// halo_predict_groups (step a1): z = act(W1 f), s = W2 z, optional mean over tokens.
#include <mutex>

#include "common.cuh"

namespace halo {

// One warp per hidden unit: dot product of a W1 row with the token's features (staged in shared memory).
template <typename T>
__global__ void __launch_bounds__(256)
predict_hidden_kernel(int d_in, int rank, int act, const T* __restrict__ W1, const T* __restrict__ feat,
                      float* __restrict__ hidden /*[n_tok][rank]*/) {
    extern __shared__ float f_s[];  // [d_in]
    const int tok = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T* f = feat + static_cast<size_t>(tok) * d_in;
    for (int c = tid; c < d_in; c += blockDim.x) f_s[c] = to_float(f[c]);
    __syncthreads();
    const int u = blockIdx.x * 8 + warp;
    if (u >= rank) return;
    constexpr int E = Elem<T>::kPerChunk;
    const int chunks = d_in / E;
    const uint4* row = reinterpret_cast<const uint4*>(W1 + static_cast<size_t>(u) * d_in);
    float acc = 0.0f;
    for (int c0 = lane; c0 < chunks; c0 += 128) {
        uint4 w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = c0 + 32 * i;
            w[i] = c < chunks ? __ldg(row + c) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = c0 + 32 * i;
            if (c < chunks) {
                float wf[E];
                Elem<T>::widen(w[i], wf);
#pragma unroll
                for (int e = 0; e < E; ++e) acc = fmaf(wf[e], f_s[c * E + e], acc);
            }
        }
    }
    acc = warp_sum(acc);
    if (act == HALO_ACT_RELU) acc = fmaxf(acc, 0.0f);
    if (lane == 0) hidden[static_cast<size_t>(tok) * rank + u] = acc;
}

// One block per token: s[tok][g] = <W2[g], z[tok]>.
template <typename T>
__global__ void __launch_bounds__(256)
predict_out_kernel(int rank, int G, const T* __restrict__ W2, const float* __restrict__ hidden,
                   float* __restrict__ out /*[n_tok][G]*/, uint32_t* dev_status) {
    extern __shared__ float z[];  // [rank]
    const int tok = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int u = tid; u < rank; u += blockDim.x) z[u] = hidden[static_cast<size_t>(tok) * rank + u];
    __syncthreads();
    constexpr int E = Elem<T>::kPerChunk;
    const int chunks = rank / E;
    for (int g = warp; g < G; g += 8) {
        const uint4* row = reinterpret_cast<const uint4*>(W2 + static_cast<size_t>(g) * rank);
        float acc = 0.0f;
        for (int c = lane; c < chunks; c += 32) {
            float w[E];
            Elem<T>::widen(__ldg(row + c), w);
#pragma unroll
            for (int e = 0; e < E; ++e) acc = fmaf(w[e], z[c * E + e], acc);
        }
        acc = warp_sum(acc);
        if (lane == 0) {
            out[static_cast<size_t>(tok) * G + g] = acc;
            if (!isfinite(acc)) flag_status(dev_status, HALO_DEV_NONFINITE_SCORE);
        }
    }
}

// Mean over tokens: one block per group, threads stride over the tokens, fixed-shape tree reduction (the result
// does not depend on scheduling).
__global__ void __launch_bounds__(256)
mean_pool_kernel(int n_tok, int G, const float* __restrict__ per_tok, float* __restrict__ scores) {
    __shared__ float part[8];
    const int g = blockIdx.x;
    float acc = 0.0f;
    for (int t = threadIdx.x; t < n_tok; t += 256) acc += per_tok[static_cast<size_t>(t) * G + g];
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) tot += part[w];
        scores[g] = tot / static_cast<float>(n_tok);
    }
}

halo_status launch_predict_hidden(const halo_pred_shape& sh, const void* W1, const void* feat, int n_tok,
                                  float* hidden, cudaStream_t st) {
    dim3 grid((sh.rank + 7) / 8, n_tok);
    const size_t smem = sizeof(float) * static_cast<size_t>(sh.d_in);
    if (sh.wdtype == HALO_BF16)
        predict_hidden_kernel<__nv_bfloat16><<<grid, 256, smem, st>>>(
            sh.d_in, sh.rank, sh.act, static_cast<const __nv_bfloat16*>(W1), static_cast<const __nv_bfloat16*>(feat),
            hidden);
    else
        predict_hidden_kernel<float><<<grid, 256, smem, st>>>(sh.d_in, sh.rank, sh.act, static_cast<const float*>(W1),
                                                              static_cast<const float*>(feat), hidden);
    HALO_CHECK_LAUNCH();
    return HALO_OK;
}

halo_status launch_predict(const halo_pred_shape& sh, const void* W1, const void* W2, const void* feat, int n_tok,
                           int mean_pool, float* scores, float* workspace, uint32_t* dev_status, cudaStream_t st) {
    float* hidden = workspace;                                        // [n_tok][rank]
    float* per_tok = workspace + static_cast<size_t>(n_tok) * sh.rank;  // [n_tok][G], pooled case only
    // many tokens: the hidden layer is a dense contraction -> tensor cores; few tokens: one warp per hidden unit
    halo_status rc = pred_gemm_supported(sh, n_tok) ? launch_pred_hidden_gemm(sh, W1, feat, n_tok, hidden, dev_status, st)
                                                    : launch_predict_hidden(sh, W1, feat, n_tok, hidden, st);
    if (rc != HALO_OK) return rc;
    const bool pool = mean_pool && n_tok > 1;
    float* out = pool ? per_tok : scores;
    const size_t smem = sizeof(float) * static_cast<size_t>(sh.rank);
    if (sh.wdtype == HALO_BF16)
        predict_out_kernel<__nv_bfloat16><<<n_tok, 256, smem, st>>>(sh.rank, sh.n_groups,
                                                                     static_cast<const __nv_bfloat16*>(W2), hidden, out,
                                                                     dev_status);
    else
        predict_out_kernel<float><<<n_tok, 256, smem, st>>>(sh.rank, sh.n_groups, static_cast<const float*>(W2),
                                                            hidden, out, dev_status);
    HALO_CHECK_LAUNCH();
    if (pool) {
        mean_pool_kernel<<<sh.n_groups, 256, 0, st>>>(n_tok, sh.n_groups, per_tok, scores);
        HALO_CHECK_LAUNCH();
    }
    return HALO_OK;
}

}  // namespace halo

// ---- predictor without any caller-provided or allocated scratch --------------------------------------------
//
// Some programs that want to call the predictor cannot hand it a workspace because they cannot allocate one
// at that point: a serving process that gave all device memory to its own pool when it started, a plug-in
// running inside someone else's memory budget, or a latency-critical loop in which a call into the CUDA
// allocator (which may synchronise the whole device) is not acceptable.  For them the two intermediate
// arrays of the predictor live in the fixed array below, which is part of the library image: every GPU on
// which the library is loaded holds these 2 MiB from load to exit.
//
// The name `g_predict_scratch` is only meaningful to device code.  On the host it is a stand-in symbol, not
// a device address, so the entry point asks the runtime for the real address once per device
// (cudaGetSymbolAddress, with that device current) and passes it to the kernels like any other pointer.
static __device__ __align__(256) float g_predict_scratch[HALO_STATIC_SCRATCH_FLOATS];

namespace {
constexpr int kMaxDevices = 64;
float* g_scratch_addr[kMaxDevices] = {};  // device address of g_predict_scratch, per device ordinal
std::mutex g_scratch_mutex;
}  // namespace

extern "C" halo_status halo_predict_groups_static(const halo_pred_shape* shape, const void* W1, const void* W2,
                                                  const void* feat, int n_tok, int mean_pool, float* scores,
                                                  uint32_t* dev_status, void* stream) {
    // same argument rules as halo_predict_groups
    const halo_status rc = halo::check_pred_shape(shape);
    if (rc != HALO_OK) return rc;
    if (n_tok <= 0) return HALO_ERR_SHAPE;
    if (!W1 || !W2 || !feat || !scores) return HALO_ERR_ARG;
    if (!halo::aligned16(W1) || !halo::aligned16(W2) || !halo::aligned16(feat)) return HALO_ERR_ALIGN;
    // the fixed array bounds what fits: hidden values [n_tok][rank] + per-token scores [n_tok][n_groups]
    const unsigned long long need =
        static_cast<unsigned long long>(n_tok) * (static_cast<unsigned long long>(shape->rank) + shape->n_groups);
    if (need > HALO_STATIC_SCRATCH_FLOATS) return HALO_ERR_WORKSPACE;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return HALO_ERR_CUDA;
    float* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_scratch_mutex);
        if (!g_scratch_addr[dev]) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_predict_scratch) != cudaSuccess || !p) return HALO_ERR_CUDA;
            g_scratch_addr[dev] = static_cast<float*>(p);
        }
        scratch = g_scratch_addr[dev];
    }
    // Nothing in the array has to start at zero: every word a call reads it has written first, so whatever
    // the previous call left behind is harmless.
    return halo::launch_predict(*shape, W1, W2, feat, n_tok, mean_pool, scores, scratch, dev_status,
                                static_cast<cudaStream_t>(stream));
}

