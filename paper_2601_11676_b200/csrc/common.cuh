// Shared declarations of the CUDA side of libhalo (internal; the public ABI is include/halo.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "halo.h"

namespace halo {

constexpr int kSmCount = 148;  // B200: 2 dies x 74 SMs

// Assignment-phase tables in the form the selection kernel takes by value.
struct PlanDev {
    int n_dev;
    int mode;           // halo_sel_mode
    int k_critical;
    float threshold;
    uint32_t seed_lo, seed_hi;
    int dev_order[HALO_MAX_DEVICES];                 // ascending loss rate
    unsigned long long loss_thresh[HALO_MAX_DEVICES];  // T_i = round(rho_i * 2^32), by device index
    unsigned long long cum_weight[HALO_MAX_DEVICES];   // cumulative share weight in dev_order
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline halo_status cuda_status(cudaError_t e) { return e == cudaSuccess ? HALO_OK : HALO_ERR_CUDA; }

// Opt a kernel in to `bytes` of dynamic shared memory, once per device (the attribute is per device; the flag
// array belongs to the calling site, one per kernel instantiation).
template <typename Kernel>
inline bool ensure_dynamic_smem(Kernel kernel, size_t bytes, bool (&done)[64]) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (done[dev]) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)) != cudaSuccess)
        return false;
    done[dev] = true;
    return true;
}

#define HALO_CHECK_LAUNCH()                                   \
    do {                                                      \
        cudaError_t e__ = cudaGetLastError();                 \
        if (e__ != cudaSuccess) return HALO_ERR_CUDA;         \
    } while (0)

// ---- device helpers ------------------------------------------------------

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// 16-byte streaming load: weights are read once, keep them out of L1.
__device__ __forceinline__ uint4 ldg_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// Element traits: how many elements one 16-byte chunk holds and how to widen it.
template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kPerChunk = 4;
    __device__ static __forceinline__ void widen(const uint4& w, float (&f)[4]) {
        f[0] = __uint_as_float(w.x); f[1] = __uint_as_float(w.y);
        f[2] = __uint_as_float(w.z); f[3] = __uint_as_float(w.w);
    }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kPerChunk = 8;
    __device__ static __forceinline__ void widen(const uint4& w, float (&f)[8]) {
        f[0] = bf16_lo(w.x); f[1] = bf16_hi(w.x); f[2] = bf16_lo(w.y); f[3] = bf16_hi(w.y);
        f[4] = bf16_lo(w.z); f[5] = bf16_hi(w.z); f[6] = bf16_lo(w.w); f[7] = bf16_hi(w.w);
    }
};

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ void flag_status(uint32_t* status, uint32_t bits) {
    if (status) atomicOr(status, bits);
}

// ---- launchers implemented in the .cu files (host side, all asynchronous) --

halo_status check_pred_shape(const halo_pred_shape* s);   // argument rules of the predictor (capi.cu)

// Process-wide options set through halo_set_option (capi.cu).  A value of -1 means "not set: use the default".
enum OptionId { OPT_CROSS_STAGES = 0, OPT_L2_AHEAD, OPT_MAX_STEPS_PER_LAUNCH, OPT_PREFILL_TWO_LAUNCHES, OPT_PREFILL_KCUTS,
                OPT_PREFILL_KRATIO_PERCENT, OPT_MHA_THREE_LAUNCHES, OPT_I4_NO_RING, OPT_PROMPT_KCUTS, OPT_PROMPT_L2_AHEAD, OPT_TMEM_RING,
                OPT_COUNT };
int option_value(OptionId id);

halo_status launch_predict(const halo_pred_shape& sh, const void* W1, const void* W2, const void* feat, int n_tok,
                           int mean_pool, float* scores, float* workspace, uint32_t* dev_status, cudaStream_t st);
halo_status launch_select(const PlanDev& plan, int G, const float* scores, uint32_t step, uint32_t layer,
                          int force_all, int32_t* order, int32_t* dev_of_group, uint8_t* arrived, uint8_t* keep,
                          int32_t* keep_list, int32_t* n_keep, uint32_t* dev_status, cudaStream_t st);
// Second predictor layer + selection in one block (decode path of the stack).
halo_status launch_score_select(const halo_pred_shape& sh, const void* W2, const float* hidden,
                                const PlanDev& plan, uint32_t step, uint32_t layer, int force_all, float* scores,
                                int32_t* order, int32_t* dev_of_group, uint8_t* arrived, uint8_t* keep,
                                int32_t* keep_list, int32_t* n_keep, uint32_t* dev_status, cudaStream_t st);
halo_status launch_predict_hidden(const halo_pred_shape& sh, const void* W1, const void* feat, int n_tok,
                                  float* hidden, cudaStream_t st);
// already_zero: the caller guarantees that `partials` is zero (otherwise the call zeroes it first).
halo_status launch_group_ffn_decode(const halo_ffn_shape& sh, const void* W, const void* x, int n_tok,
                                    const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group,
                                    int n_dev, float* partials, uint32_t* dev_status, cudaStream_t st,
                                    bool already_zero = false);
halo_status launch_group_ffn_stream(const halo_ffn_shape& sh, const void* W, const void* x, int n_tok,
                                    const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group,
                                    int n_dev, float* partials, uint32_t* dev_status, cudaStream_t st,
                                    bool zero_first = false);
// Prefill form (tensor cores); workspace = bf16 [n_tok][d_ffn]; partials must already be zero.
bool prefill_supported(const halo_ffn_shape& sh, int n_tok);
size_t prefill_workspace_bytes(const halo_ffn_shape& sh, int n_tok);
// true when launch_group_ffn_prefill with collapse != 0 ADDS into slot 0 of `partials` (K-split reductions), so the
// caller may pass a buffer that already holds a value to add to
bool prefill_accumulates(const halo_ffn_shape& sh, int n_tok);
halo_status launch_group_ffn_prefill(const halo_ffn_shape& sh, const void* W, const void* x, int n_tok,
                                     const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group,
                                     int n_dev, int collapse, float* partials, void* workspace, uint32_t* dev_status,
                                     cudaStream_t st, bool ctl_clean = false);
bool pred_gemm_supported(const halo_pred_shape& sh, int n_tok);
halo_status launch_pred_hidden_gemm(const halo_pred_shape& sh, const void* W1, const void* feat, int n_tok,
                                    float* hidden, uint32_t* dev_status, cudaStream_t st);
halo_status launch_merge(const float* partials, const uint8_t* arrived, int n_dev, int n_tok, int d, float* y,
                         cudaStream_t st);
halo_status launch_glue(int d, int n_tok, halo_dtype xdtype, const float* h, const float* y, float* h_out,
                        void* x_out, cudaStream_t st);
// merge + residual + normalise in one launch (stack path); y_tap may be NULL.
// zero_after: every slot of `partials` is left zeroed (for a following kernel that adds into them).
halo_status launch_merge_glue(const float* partials, const uint8_t* arrived, int n_dev, int n_tok, int d,
                              halo_dtype xdtype, const float* h, float* h_out, void* x_out, float* y_tap,
                              cudaStream_t st, bool zero_after = false);
// Zero-fill of partial slots by a kernel that releases a programmatically dependent launch at once (the dependent
// kernel executes griddepcontrol.wait before it first adds to the slots); n_floats a multiple of 4.
halo_status launch_zero_partials(float* partials, size_t n_floats, cudaStream_t st);
// halo_mha_block without argument checks; already_zero: the caller guarantees that `partials` is zero.
halo_status launch_mha_block(const halo_mha_shape& sh, const void* W_packed, const void* Wk, const void* Wv, const void* x,
                             void* K_cache, void* V_cache, int pos, const int32_t* keep_list, const int32_t* n_keep,
                             const int32_t* dev_of_group, int n_dev, float* partials, uint32_t* dev_status, cudaStream_t st,
                             bool already_zero);
// int4 codes + scales of the kept groups (all groups when keep_list is null) -> bf16 rows in the packed layout
halo_status launch_dequantize_i4(const halo_ffn_shape& sh, const void* Q, const void* scales, const int32_t* keep_list,
                                 const int32_t* n_keep, void* W_out, uint32_t* dev_status, cudaStream_t st);
// halo_group_ffn_i4 without argument checks; already_zero: the caller guarantees that `partials` is zero
halo_status launch_group_ffn_i4(const halo_ffn_shape& sh, const void* Q, const void* scales, const void* x, int n_tok,
                                const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group, int n_dev,
                                float* partials, uint32_t* dev_status, cudaStream_t st, bool already_zero);
// the same block on int4 weights: Qp/Sp, Qk/Sk, Qv/Sv = codes and scales of W_packed, Wk, Wv (halo_quantize_rows_i4)
halo_status launch_mha_block_i4(const halo_mha_shape& sh, const void* Qp, const void* Sp, const void* Qk, const void* Sk,
                                const void* Qv, const void* Sv, const void* x, void* K_cache, void* V_cache, int pos,
                                const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group, int n_dev,
                                float* partials, uint32_t* dev_status, cudaStream_t st, bool already_zero);
halo_status launch_pack(const halo_ffn_shape& sh, const void* Wgate, const void* Wup, const void* Wdown,
                        void* Wpacked, cudaStream_t st);

}  // namespace halo

// Host-side plan object behind the opaque halo_plan.
struct halo_plan {
    int n_groups;
    int n_dev;
    double loss_rate[HALO_MAX_DEVICES];
    uint32_t share_weight[HALO_MAX_DEVICES];
    halo::PlanDev dev;
};
