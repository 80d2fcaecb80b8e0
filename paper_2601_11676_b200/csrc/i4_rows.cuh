// Row products on int4 rows (format of halo_quantize_rows_i4: nibble = code + 8, element 2i in the low half of byte i,
// one bf16 scale per 128 consecutive elements of a row) against a bf16 vector x kept in shared memory in the nibble
// pairing: for 16-byte code chunk c (32 weights) and its word w, xp[w * chunks16 + c] holds the four pairs
// (x[32c + 8w + k], x[32c + 8w + k + 4]), k = 0..3, as bf16x2, and xsum[c] the plain sum of the chunk's 32 elements of x.
// Nibbles k and k + 4 of a word become the bf16 pair {128 + n_k, 128 + n_k+4} by mask and OR and feed the
// mixed-precision FMA; 136 * xsum[c] is taken off per chunk, the block's scale multiplies the chunk's sum.
#pragma once

#include "common.cuh"
#include "ffn_math.cuh"
#include "i4_math.cuh"

namespace halo {

// Block-wide: arranges x (d bf16 elements, d % 128 == 0) as described above.  The caller synchronises afterwards.
__device__ __forceinline__ void stage_x_paired(const __nv_bfloat16* __restrict__ x, uint4* xp, float* xsum, int d) {
    const int chunks16 = d / 32;
    const uint16_t* xb = reinterpret_cast<const uint16_t*>(x);
    uint32_t* xp_words = reinterpret_cast<uint32_t*>(xp);
    for (int i = threadIdx.x; i < d / 2; i += blockDim.x) {
        const int c = i / 16, r = i - c * 16, w = r >> 2, k = r & 3;
        const uint32_t lo16 = xb[32 * c + 8 * w + k], hi16 = xb[32 * c + 8 * w + k + 4];
        xp_words[(static_cast<size_t>(w) * chunks16 + c) * 4 + k] = lo16 | (hi16 << 16);
    }
    for (int c = threadIdx.x; c < chunks16; c += blockDim.x) {
        float sx = 0.0f;
        for (int e = 0; e < 32; ++e) sx += __bfloat162float(x[32 * c + e]);
        xsum[c] = sx;
    }
}

// <row_a, x> and <row_b, x> by one warp (row_a may equal row_b); four 16-byte code chunks per row and lane in flight.
__device__ __forceinline__ void warp_two_rows_dot_i4(const uint8_t* __restrict__ Q, const __nv_bfloat16* __restrict__ scales,
                                                     size_t row_a, size_t row_b, int d, const uint4* xp,
                                                     const float* xsum, int lane, float& out_a, float& out_b) {
    const int chunks16 = d / 32, nb = d / 128;
    const uint4* a4 = reinterpret_cast<const uint4*>(Q + row_a * (static_cast<size_t>(d) / 2));
    const uint4* b4 = reinterpret_cast<const uint4*>(Q + row_b * (static_cast<size_t>(d) / 2));
    float acc_a = 0.0f, acc_b = 0.0f;
    for (int c0 = lane; c0 < chunks16; c0 += 128) {
        uint4 wa[4], wb[4];
        float sa[4], sb[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = c0 + 32 * u;
            if (c < chunks16) {
                wa[u] = ldg_stream16(a4 + c);
                wb[u] = ldg_stream16(b4 + c);
                sa[u] = __bfloat162float(scales[row_a * nb + (c >> 2)]);
                sb[u] = __bfloat162float(scales[row_b * nb + (c >> 2)]);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = c0 + 32 * u;
            if (c < chunks16) {
                float ta0 = 0.0f, ta1 = 0.0f, tb0 = 0.0f, tb1 = 0.0f;
                const uint32_t aw[4] = {wa[u].x, wa[u].y, wa[u].z, wa[u].w};
                const uint32_t bw[4] = {wb[u].x, wb[u].y, wb[u].z, wb[u].w};
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const uint4 xq = xp[static_cast<size_t>(w) * chunks16 + c];
                    const uint32_t xk[4] = {xq.x, xq.y, xq.z, xq.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        fma_bf16x2(nibble_pair_bf16(aw[w], k), xk[k], ta0, ta1);
                        fma_bf16x2(nibble_pair_bf16(bw[w], k), xk[k], tb0, tb1);
                    }
                }
                const float off = kNibbleBias * xsum[c];
                acc_a = fmaf(sa[u], (ta0 + ta1) - off, acc_a);
                acc_b = fmaf(sb[u], (tb0 + tb1) - off, acc_b);
            }
        }
    }
    out_a = warp_sum(acc_a);
    out_b = warp_sum(acc_b);
}

}  // namespace halo
