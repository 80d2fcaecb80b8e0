// halo_merge_partials (step a9), halo_glue (residual + RMS normalisation between blocks), their fusion
// for the stack, and halo_pack_weights.
#include <initializer_list>

#include "common.cuh"

namespace halo {

__device__ __forceinline__ float merged_value(const float* __restrict__ partials, const uint8_t* __restrict__ arrived,
                                              int n_dev, size_t slot_stride, size_t idx) {
    float v = partials[idx];  // the master's own part is never lost
    for (int i = 0; i < n_dev; ++i)
        if (!arrived || arrived[i]) v += partials[static_cast<size_t>(i + 1) * slot_stride + idx];
    return v;
}

__global__ void merge_kernel(const float* __restrict__ partials, const uint8_t* __restrict__ arrived, int n_dev,
                             size_t slot_stride, float* __restrict__ y) {
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx < slot_stride) y[idx] = merged_value(partials, arrived, n_dev, slot_stride, idx);
}

__device__ __forceinline__ float block_sum_1024(float v, float* scratch /*[32]*/) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = (threadIdx.x < (blockDim.x >> 5)) ? scratch[threadIdx.x] : 0.0f;
    if (warp == 0) {
        t = warp_sum(t);
        if (lane == 0) scratch[0] = t;
    }
    __syncthreads();
    const float r = scratch[0];
    __syncthreads();
    return r;
}

__device__ __forceinline__ void store4(float* p, float a, float b, float c, float d) {
    *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
__device__ __forceinline__ void store4(__nv_bfloat16* p, float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
}

// One block per token.  MERGE: y is taken from the partial slots, else from y_in (may be NULL = 0).
template <typename T, bool MERGE>
__global__ void __launch_bounds__(1024)
glue_kernel(int d, const float* __restrict__ h, const float* __restrict__ y_in, const float* partials,
            const uint8_t* __restrict__ arrived, int n_dev, size_t slot_stride, float* h_out, T* __restrict__ x_out,
            float* __restrict__ y_tap, int vec, float* zero_slots) {
    __shared__ float scratch[32];
    extern __shared__ __align__(16) float hv[];  // [d]
    const int tok = blockIdx.x;
    const size_t base = static_cast<size_t>(tok) * d;
    float ss = 0.0f;
    if (vec) {
        // four columns per thread and access (every row starts 16-byte aligned)
        const int d4 = d >> 2;
        const float4* h4 = reinterpret_cast<const float4*>(h + base);
        // The arrival flags as one mask per warp (lane i reads flag i; the loads below do not wait for it): the slots of
        // a batch of devices are fetched unconditionally and masked afterwards, so a merge is one round trip to memory
        // instead of one per device.
        uint8_t my_flag = 1;
        if (MERGE && arrived && (threadIdx.x & 31) < n_dev) my_flag = arrived[threadIdx.x & 31];
        unsigned mask = 0u;
        bool have_mask = false;
        for (int c0 = 0; c0 < d4; c0 += blockDim.x) {   // same trip count for every thread: the vote below is warp-wide
            const int c = c0 + threadIdx.x;
            const bool on = c < d4;
            float4 y = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (MERGE) {
                if (on) y = reinterpret_cast<const float4*>(partials + base)[c];
                for (int i0 = 0; i0 < n_dev; i0 += 8) {
                    float4 p[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (on && i0 + k < n_dev)
                            p[k] = reinterpret_cast<const float4*>(partials + static_cast<size_t>(i0 + k + 1) * slot_stride + base)[c];
                    if (!have_mask) {
                        mask = __ballot_sync(0xffffffffu, my_flag != 0);
                        have_mask = true;
                    }
                    const unsigned m = mask >> i0;
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (on && i0 + k < n_dev && ((m >> k) & 1u)) { y.x += p[k].x; y.y += p[k].y; y.z += p[k].z; y.w += p[k].w; }
                }
                if (on && y_tap) reinterpret_cast<float4*>(y_tap + base)[c] = y;
                if (on && zero_slots)   // the slots are left zeroed for the next kernel that adds into them
                    for (int i = 0; i <= n_dev; ++i)
                        reinterpret_cast<float4*>(zero_slots + static_cast<size_t>(i) * slot_stride + base)[c] =
                            make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            } else if (y_in && on) {
                y = reinterpret_cast<const float4*>(y_in + base)[c];
            }
            if (on) {
                const float4 hh = h4[c];
                const float4 v = make_float4(hh.x + y.x, hh.y + y.y, hh.z + y.z, hh.w + y.w);
                reinterpret_cast<float4*>(hv)[c] = v;
                ss = fmaf(v.x, v.x, fmaf(v.y, v.y, fmaf(v.z, v.z, fmaf(v.w, v.w, ss))));
            }
        }
    } else {
        for (int c = threadIdx.x; c < d; c += blockDim.x) {
            float y = 0.0f;
            if (MERGE) {
                y = merged_value(partials, arrived, n_dev, slot_stride, base + c);
                if (y_tap) y_tap[base + c] = y;
                if (zero_slots)
                    for (int i = 0; i <= n_dev; ++i) zero_slots[static_cast<size_t>(i) * slot_stride + base + c] = 0.0f;
            } else if (y_in) {
                y = y_in[base + c];
            }
            const float v = h[base + c] + y;
            hv[c] = v;
            ss = fmaf(v, v, ss);
        }
    }
    ss = block_sum_1024(ss, scratch);
    const float scale = 1.0f / sqrtf(ss / static_cast<float>(d) + 1e-5f);
    if (vec) {
        const int d4 = d >> 2;
        for (int c = threadIdx.x; c < d4; c += blockDim.x) {
            const float4 v = reinterpret_cast<const float4*>(hv)[c];
            reinterpret_cast<float4*>(h_out + base)[c] = v;
            store4(x_out + base + 4 * c, v.x * scale, v.y * scale, v.z * scale, v.w * scale);
        }
    } else {
        for (int c = threadIdx.x; c < d; c += blockDim.x) {
            const float v = hv[c];
            h_out[base + c] = v;
            x_out[base + c] = from_float<T>(v * scale);
        }
    }
}

template <typename T>
__global__ void pack_kernel(int d, int F, int S, const T* __restrict__ Wgate, const T* __restrict__ Wup,
                            const T* __restrict__ Wdown, T* __restrict__ Wp) {
    // one thread per packed element of planes 0/1; plane 2 is a transpose and gets its own index space
    const size_t n = static_cast<size_t>(F) * d;
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= n) return;
    const int neuron = static_cast<int>(idx / d), c = static_cast<int>(idx % d);
    const int g = neuron / S, j = neuron % S;
    const size_t group_base = static_cast<size_t>(g) * 3 * S * d;
    Wp[group_base + (static_cast<size_t>(0) * S + j) * d + c] = Wgate[idx];
    Wp[group_base + (static_cast<size_t>(1) * S + j) * d + c] = Wup[idx];
    Wp[group_base + (static_cast<size_t>(2) * S + j) * d + c] = Wdown[static_cast<size_t>(c) * F + neuron];
}

halo_status launch_merge(const float* partials, const uint8_t* arrived, int n_dev, int n_tok, int d, float* y,
                         cudaStream_t st) {
    const size_t n = static_cast<size_t>(n_tok) * d;
    merge_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(partials, arrived, n_dev, n, y);
    HALO_CHECK_LAUNCH();
    return HALO_OK;
}

namespace {
// the four-column path needs d % 4 == 0 and every buffer 16-byte aligned
bool all_aligned16(std::initializer_list<const void*> ptrs) {
    for (const void* p : ptrs)
        if (p && (reinterpret_cast<uintptr_t>(p) & 15u)) return false;
    return true;
}
}  // namespace

halo_status launch_glue(int d, int n_tok, halo_dtype xdtype, const float* h, const float* y, float* h_out,
                        void* x_out, cudaStream_t st) {
    const size_t smem = sizeof(float) * static_cast<size_t>(d);
    const int vec = (d % 4 == 0) && all_aligned16({h, y, h_out, x_out});
    if (xdtype == HALO_BF16)
        glue_kernel<__nv_bfloat16, false><<<n_tok, 1024, smem, st>>>(d, h, y, nullptr, nullptr, 0, 0, h_out,
                                                                      static_cast<__nv_bfloat16*>(x_out), nullptr, vec, nullptr);
    else
        glue_kernel<float, false><<<n_tok, 1024, smem, st>>>(d, h, y, nullptr, nullptr, 0, 0, h_out,
                                                             static_cast<float*>(x_out), nullptr, vec, nullptr);
    HALO_CHECK_LAUNCH();
    return HALO_OK;
}

halo_status launch_merge_glue(const float* partials, const uint8_t* arrived, int n_dev, int n_tok, int d,
                              halo_dtype xdtype, const float* h, float* h_out, void* x_out, float* y_tap,
                              cudaStream_t st, bool zero_after) {
    float* zero_slots = zero_after ? const_cast<float*>(partials) : nullptr;
    const size_t smem = sizeof(float) * static_cast<size_t>(d);
    const size_t stride = static_cast<size_t>(n_tok) * d;
    const int vec = (d % 4 == 0) && all_aligned16({partials, h, h_out, x_out, y_tap});
    if (xdtype == HALO_BF16)
        glue_kernel<__nv_bfloat16, true><<<n_tok, 1024, smem, st>>>(d, h, nullptr, partials, arrived, n_dev, stride,
                                                                     h_out, static_cast<__nv_bfloat16*>(x_out), y_tap, vec,
                                                                     zero_slots);
    else
        glue_kernel<float, true><<<n_tok, 1024, smem, st>>>(d, h, nullptr, partials, arrived, n_dev, stride, h_out,
                                                            static_cast<float*>(x_out), y_tap, vec, zero_slots);
    HALO_CHECK_LAUNCH();
    return HALO_OK;
}

halo_status launch_pack(const halo_ffn_shape& sh, const void* Wgate, const void* Wup, const void* Wdown,
                        void* Wpacked, cudaStream_t st) {
    const size_t n = static_cast<size_t>(sh.d_ffn) * sh.d_model;
    const unsigned blocks = static_cast<unsigned>((n + 255) / 256);
    if (sh.wdtype == HALO_BF16)
        pack_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(
            sh.d_model, sh.d_ffn, sh.group_size, static_cast<const __nv_bfloat16*>(Wgate),
            static_cast<const __nv_bfloat16*>(Wup), static_cast<const __nv_bfloat16*>(Wdown),
            static_cast<__nv_bfloat16*>(Wpacked));
    else
        pack_kernel<float><<<blocks, 256, 0, st>>>(sh.d_model, sh.d_ffn, sh.group_size,
                                                   static_cast<const float*>(Wgate), static_cast<const float*>(Wup),
                                                   static_cast<const float*>(Wdown), static_cast<float*>(Wpacked));
    HALO_CHECK_LAUNCH();
    return HALO_OK;
}

}  // namespace halo
