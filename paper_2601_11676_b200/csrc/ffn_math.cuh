// Inner arithmetic of the decode FFN consumers (bf16 weights and activations, fp32 accumulation).
#pragma once
#include <stdint.h>

namespace halo {

// acc0 += w.lo * x.lo, acc1 += w.hi * x.hi for one packed pair of bf16: sm_100 mixed-precision FMA
// (fp32 accumulator, bf16 multiplicands; the product of two bf16 is exact in fp32, one rounding).
__device__ __forceinline__ void fma_bf16x2(uint32_t w, uint32_t x, float& acc0, float& acc1) {
    asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\t"
        "mov.b32 {wl, wh}, %2;\n\t"
        "mov.b32 {xl, xh}, %3;\n\t"
        "fma.rn.f32.bf16 %0, wl, xl, %0;\n\t"
        "fma.rn.f32.bf16 %1, wh, xh, %1;\n\t}"
        : "+f"(acc0), "+f"(acc1)
        : "r"(w), "r"(x));
}

// eight products of a 16-byte chunk into two accumulator chains
__device__ __forceinline__ void dot_bf16x8(const uint4& w, const uint4& x, float& acc0, float& acc1) {
    fma_bf16x2(w.x, x.x, acc0, acc1);
    fma_bf16x2(w.y, x.y, acc0, acc1);
    fma_bf16x2(w.z, x.z, acc0, acc1);
    fma_bf16x2(w.w, x.w, acc0, acc1);
}

// acc[e] += h * w[e] for a 16-byte chunk of bf16 (h stays fp32)
__device__ __forceinline__ void axpy_bf16x8(float h, const uint4& w, float (&acc)[8]) {
    acc[0] = fmaf(h, __uint_as_float(w.x << 16), acc[0]);
    acc[1] = fmaf(h, __uint_as_float(w.x & 0xffff0000u), acc[1]);
    acc[2] = fmaf(h, __uint_as_float(w.y << 16), acc[2]);
    acc[3] = fmaf(h, __uint_as_float(w.y & 0xffff0000u), acc[3]);
    acc[4] = fmaf(h, __uint_as_float(w.z << 16), acc[4]);
    acc[5] = fmaf(h, __uint_as_float(w.z & 0xffff0000u), acc[5]);
    acc[6] = fmaf(h, __uint_as_float(w.w << 16), acc[6]);
    acc[7] = fmaf(h, __uint_as_float(w.w & 0xffff0000u), acc[7]);
}

// SiLU(a) * b with the fast exponential and reciprocal (a few ulp; far inside the output tolerance)
__device__ __forceinline__ float silu_mul(float a, float b) {
    return __fdividef(a, 1.0f + __expf(-a)) * b;
}

// sum of the WPR partial dot products of one row, stored contiguously
template <int WPR>
__device__ __forceinline__ float sum_parts(const float* p) {
    if constexpr (WPR == 4) {
        const float4 v = *reinterpret_cast<const float4*>(p);
        return (v.x + v.y) + (v.z + v.w);
    } else if constexpr (WPR == 2) {
        const float2 v = *reinterpret_cast<const float2*>(p);
        return v.x + v.y;
    } else if constexpr (WPR == 8) {
        const float4 u = *reinterpret_cast<const float4*>(p);
        const float4 v = *reinterpret_cast<const float4*>(p + 4);
        return ((u.x + u.y) + (u.z + u.w)) + ((v.x + v.y) + (v.z + v.w));
    } else {
        float s = 0.0f;
#pragma unroll
        for (int q = 0; q < WPR; ++q) s += p[q];
        return s;
    }
}

}  // namespace halo
