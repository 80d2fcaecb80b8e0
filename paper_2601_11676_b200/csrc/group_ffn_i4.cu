// int4 group-quantised weights for the decode FFN (steps a6..a8 on 4-bit weights).  The paper evaluates models
// quantised to 4-bit integers (Sec. IV-A) without giving a format; the one used here: symmetric, one bf16 scale
// per block of 128 consecutive elements of a packed row, s = bf16(amax / 7) rounded up to 5 significant bits,
// q = clamp(rint(w / s), -8, 7), nibble = q + 8, element 2i in the low half of byte i.  With 5 bits in the scale every
// dequantised value (nibble - 8) * s is exactly a bf16 number: the tensor-core prompt path loses nothing on the weights.
//
// halo_quantize_weights_i4: one warp per (row, block); decisions in fp32 with IEEE division and round-half-even.
// halo_group_ffn_i4, generic form: the structure of the generic decode kernel (a thread block walks a contiguous range of kept
// neurons in batches of 8; phase 1 one warp per neuron against x in shared memory; phase 2 fixed columns per
// thread, sums kept in registers until the holder changes).  Nibbles are never converted one by one: a word's
// nibbles k and k+4 are masked into the two halves of a register and OR-ed with 0x4300, which makes them the bf16
// numbers 128 + nibble; phase 1 feeds those pairs to the mixed-precision FMA against x pre-arranged in the same
// pairing, phase 2 splits the pair into two fp32 values.  The offset (128 + 8) times the plain sum of x (or of
// the row factors) is subtracted once per block.
#include <algorithm>
#include <cstdlib>

#include "common.cuh"
#include "ffn_math.cuh"
#include "i4_math.cuh"
#include "tma.cuh"

namespace halo {

namespace {
constexpr int kQBlock = 128;
constexpr int kI4Threads = 256;
constexpr int kI4Warps = kI4Threads / 32;
constexpr int kI4BlocksPerSm = 2;

// The same pair with the right shift done as the high half of a product (word * 2^(32 - 4k)), which runs on the
// multiply-add pipe; the logic pipe, half as wide, is what bounds the unpacking.  `mul` = 2^(32 - 4k) must reach the
// kernel as a run-time value, else the compiler turns the product back into a shift.
__device__ __forceinline__ uint32_t nibble_pair_mulhi(uint32_t word, uint32_t mul) {
    return (__umulhi(word, mul) & 0x000F000Fu) | 0x43004300u;
}



template <typename T>
__global__ void __launch_bounds__(256)
quantize_i4_kernel(int d, long long n_rows, const T* __restrict__ W, uint8_t* __restrict__ Q,
                   __nv_bfloat16* __restrict__ scales) {
    const int lane = threadIdx.x & 31;
    const long long wid = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int nb = d / kQBlock;
    if (wid >= n_rows * nb) return;
    const long long row = wid / nb;
    const int b = static_cast<int>(wid - row * nb);
    const size_t base = static_cast<size_t>(row) * d + static_cast<size_t>(b) * kQBlock + 4 * lane;
    float w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) w[e] = to_float(W[base + e]);
    float amax = fmaxf(fmaxf(fabsf(w[0]), fabsf(w[1])), fmaxf(fabsf(w[2]), fabsf(w[3])));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    __nv_bfloat16 sb = __float2bfloat16_rn(__fdiv_rn(amax, 7.0f));
    {
        // up to the next bf16 number with at most 5 significant bits (the carry may reach the exponent): code * scale
        // then has at most 8 significant bits, i.e. every dequantised value is itself a bf16 number
        uint16_t bits = __bfloat16_as_ushort(sb);
        if (bits & 7u) bits = static_cast<uint16_t>((bits | 7u) + 1u);
        sb = __ushort_as_bfloat16(bits);
    }
    const float s = __bfloat162float(sb);
    if (lane == 0) scales[static_cast<size_t>(row) * nb + b] = sb;
    uint32_t packed = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        float t = s > 0.0f ? rintf(__fdiv_rn(w[e], s)) : 0.0f;
        t = fminf(fmaxf(t, -8.0f), 7.0f);
        packed |= static_cast<uint32_t>(static_cast<int>(t) + 8) << (4 * e);
    }
    reinterpret_cast<uint16_t*>(Q)[base / 4] = static_cast<uint16_t>(packed);   // 4 elements = 2 bytes
}

// Kept groups (or all of them) back to bf16 in the packed layout, for the tensor-core prompt path: a thread turns one
// word of codes into 8 values = one 16-byte store, neighbouring lanes neighbouring words, so every store instruction
// of a warp covers 512 contiguous bytes.  value = (nibble - 8) * s, EXACT in bf16 for scales of the quantiser above (5
// significant bits; a foreign scale with more bits is rounded once).  No integer-to-float conversion: nibbles k and
// k+4 of the word become the bf16 pair {128 + n_k, 128 + n_k+4} by mask and OR, 136 is subtracted (exact) and the pair
// is multiplied by the scale in bf16x2; a byte permute puts neighbouring elements back side by side.  Groups outside
// the kept set are not touched.
__device__ __forceinline__ uint4 dequant_word(uint32_t word, __nv_bfloat16 scale) {
    const __nv_bfloat162 s2 = __halves2bfloat162(scale, scale);
    const uint32_t bias_bits = 0x43084308u;                       // {136, 136}
    const __nv_bfloat162 bias = *reinterpret_cast<const __nv_bfloat162*>(&bias_bits);
    uint32_t r[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t pr = nibble_pair_bf16(word, k);            // {128 + e_k, 128 + e_k+4}
        const __nv_bfloat162 v = __hmul2(__hsub2(*reinterpret_cast<const __nv_bfloat162*>(&pr), bias), s2);
        r[k] = *reinterpret_cast<const uint32_t*>(&v);
    }
    return make_uint4(__byte_perm(r[0], r[1], 0x5410), __byte_perm(r[2], r[3], 0x5410),
                      __byte_perm(r[0], r[1], 0x7632), __byte_perm(r[2], r[3], 0x7632));
}

__global__ void __launch_bounds__(256)
dequantize_i4_kernel(int d, int S, int G, const uint8_t* __restrict__ Q, const __nv_bfloat16* __restrict__ scales,
                     const int32_t* __restrict__ keep_list, const int32_t* __restrict__ n_keep_ptr,
                     __nv_bfloat16* __restrict__ W, uint32_t* dev_status) {
    int nk = G;
    if (keep_list) {
        nk = *n_keep_ptr;
        if (nk < 0 || nk > G) {
            if (threadIdx.x == 0 && blockIdx.x == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
            nk = nk < 0 ? 0 : G;
        }
    }
    // a group's rows are contiguous in all three arrays: word j of the group's codes holds elements 8j..8j+7 of the
    // group and uses scale j / 16
    const long long per_group = 3ll * S * (d / 8);               // code words per group
    const long long total = static_cast<long long>(nk) * per_group;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    constexpr int kU = 4;                                        // loads in flight per thread
    for (long long i0 = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i0 < total; i0 += kU * stride) {
        uint32_t word[kU];
        __nv_bfloat16 sc[kU];
        uint4* dst[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            dst[u] = nullptr;
            const long long i = i0 + u * stride;
            if (i >= total) continue;
            const int kp = static_cast<int>(i / per_group);
            const long long j = i - kp * per_group;
            const int g = keep_list ? keep_list[kp] : kp;
            if (g < 0 || g >= G) {
                flag_status(dev_status, HALO_DEV_BAD_INDEX);
                continue;
            }
            const size_t gbase = static_cast<size_t>(g) * per_group;
            word[u] = __ldg(reinterpret_cast<const uint32_t*>(Q) + gbase + j);
            sc[u] = scales[(gbase + j) / 16];
            dst[u] = reinterpret_cast<uint4*>(W) + gbase + j;
        }
#pragma unroll
        for (int u = 0; u < kU; ++u)
            if (dst[u]) *dst[u] = dequant_word(word[u], sc[u]);
    }
}

template <int ITERS>
__global__ void __launch_bounds__(kI4Threads, kI4BlocksPerSm)
group_ffn_i4_kernel(int d, int S, int G, const uint8_t* __restrict__ Q, const __nv_bfloat16* __restrict__ scales,
                    const __nv_bfloat16* __restrict__ x_all, const int32_t* __restrict__ keep_list,
                    const int32_t* __restrict__ n_keep_ptr, const int32_t* __restrict__ dev_of_group, int n_dev,
                    int n_tok, float* __restrict__ partials, uint32_t* dev_status) {
    extern __shared__ __align__(16) unsigned char smem_b[];
    const int chunks16 = d / 32;           // 16-byte chunks (32 weights) per row
    const int chunks8 = d / 16;            // 8-byte chunks (16 weights) per row
    const int nb = d / kQBlock;
    uint4* xp = reinterpret_cast<uint4*>(smem_b);                       // [4][chunks16]: x in nibble pairing
    float* xsum = reinterpret_cast<float*>(smem_b + static_cast<size_t>(d) * 2);   // [chunks16]
    float* hs = xsum + chunks16;                                        // [kI4Warps]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tok = blockIdx.y;

    int nk = *n_keep_ptr;
    if (nk < 0 || nk > G) {
        if (tid == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
        nk = nk < 0 ? 0 : G;
    }
    const long long total = static_cast<long long>(nk) * S;
    const int lo = static_cast<int>(total * blockIdx.x / gridDim.x);
    const int hi = static_cast<int>(total * (blockIdx.x + 1) / gridDim.x);
    if (lo >= hi) return;

    // x: for chunk c and word w of a weight chunk, the four pairs (x[8w+k], x[8w+k+4]), k = 0..3, as bf16x2
    const uint16_t* xb = reinterpret_cast<const uint16_t*>(x_all + static_cast<size_t>(tok) * d);
    uint32_t* xp_words = reinterpret_cast<uint32_t*>(xp);
    for (int i = tid; i < d / 2; i += kI4Threads) {
        const int c = i / 16, r = i - c * 16, w = r >> 2, k = r & 3;
        const uint32_t lo16 = xb[32 * c + 8 * w + k], hi16 = xb[32 * c + 8 * w + k + 4];
        xp_words[(static_cast<size_t>(w) * chunks16 + c) * 4 + k] = lo16 | (hi16 << 16);
    }
    for (int c = tid; c < chunks16; c += kI4Threads) {
        float sx = 0.0f;
        for (int e = 0; e < 32; ++e) sx += __bfloat162float(x_all[static_cast<size_t>(tok) * d + 32 * c + e]);
        xsum[c] = sx;
    }
    __syncthreads();

    float acc[ITERS][16];
    float corr[ITERS];
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
        corr[i] = 0.0f;
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[i][e] = 0.0f;
    }
    int cur_slot = -1;
    const size_t slot_stride = static_cast<size_t>(n_tok) * d;

    auto flush = [&](int slot) {
        float* dst = partials + static_cast<size_t>(slot) * slot_stride + static_cast<size_t>(tok) * d;
#pragma unroll
        for (int i = 0; i < ITERS; ++i) {
            const int c = tid + kI4Threads * i;
            if (c < chunks8) {
                const float off = kNibbleBias * corr[i];
#pragma unroll
                for (int e = 0; e < 16; e += 4)
                    red_add_v4f(dst + c * 16 + e, acc[i][e] - off, acc[i][e + 1] - off, acc[i][e + 2] - off,
                                acc[i][e + 3] - off);
            }
            corr[i] = 0.0f;
#pragma unroll
            for (int e = 0; e < 16; ++e) acc[i][e] = 0.0f;
        }
    };

    const size_t row_bytes = static_cast<size_t>(d) / 2;

    // A batch = up to 8 consecutive neurons of one kept group.  (Issuing the gate/up loads of batch t+1 before the
    // down rows of batch t are consumed was measured and is slower: the extra live registers cost more than the
    // overlap gains.)
    struct Batch { int n_next, g, j0, cnt, slot; bool any; };
    auto find_batch = [&](int n) {
        Batch bt{n, 0, 0, 0, 0, false};
        while (n < hi) {
            const int ki = n / S, j0 = n - ki * S;
            const int g = keep_list[ki];
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
            bt.g = g; bt.j0 = j0; bt.slot = slot; bt.any = true;
            bt.cnt = min(kI4Warps, min(hi - n, S - j0));
            bt.n_next = n + bt.cnt;
            return bt;
        }
        bt.n_next = hi;
        return bt;
    };
    // phase-1 operands of this warp's neuron of a batch: 4 chunks of the gate row, 4 of the up row, their scales
    uint4 wg[4], wu[4];
    float fg[4], fu[4];
    auto load_phase1 = [&](const Batch& bt) {
        if (bt.any && warp < bt.cnt && chunks16 <= 128) {
            const size_t rg = static_cast<size_t>(bt.g) * 3 * S + bt.j0 + warp, ru = rg + S;
            const uint4* gate = reinterpret_cast<const uint4*>(Q + rg * row_bytes);
            const uint4* up = reinterpret_cast<const uint4*>(Q + ru * row_bytes);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int c = lane + 32 * u;
                if (c < chunks16) {
                    wg[u] = ldg_stream16(gate + c);
                    wu[u] = ldg_stream16(up + c);
                    fg[u] = __bfloat162float(scales[rg * nb + (c >> 2)]);
                    fu[u] = __bfloat162float(scales[ru * nb + (c >> 2)]);
                }
            }
        }
    };
    auto dot_chunk = [&](const uint4& g4, const uint4& u4, float sgf, float suf, int c, float& a, float& b) {
        float tg0 = 0.0f, tg1 = 0.0f, tu0 = 0.0f, tu1 = 0.0f;
        const uint32_t gw[4] = {g4.x, g4.y, g4.z, g4.w};
        const uint32_t uw[4] = {u4.x, u4.y, u4.z, u4.w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const uint4 xq = xp[static_cast<size_t>(w) * chunks16 + c];
            const uint32_t xk[4] = {xq.x, xq.y, xq.z, xq.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                fma_bf16x2(nibble_pair_bf16(gw[w], k), xk[k], tg0, tg1);
                fma_bf16x2(nibble_pair_bf16(uw[w], k), xk[k], tu0, tu1);
            }
        }
        const float off = kNibbleBias * xsum[c];
        a = fmaf(sgf, (tg0 + tg1) - off, a);
        b = fmaf(suf, (tu0 + tu1) - off, b);
    };

    Batch cur = find_batch(lo);
    while (cur.any) {
        load_phase1(cur);
        if (cur.slot != cur_slot) {
            if (cur_slot >= 0) flush(cur_slot);
            cur_slot = cur.slot;
        }
        const size_t group_row = static_cast<size_t>(cur.g) * 3 * S;     // first packed row of the group

        // ---- phase 1: gate / up products, one neuron per warp --------------------------------------------
        if (warp < cur.cnt) {
            float a = 0.0f, b = 0.0f;
            if (chunks16 <= 128) {              // the whole row was fetched ahead
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int c = lane + 32 * u;
                    if (c < chunks16) dot_chunk(wg[u], wu[u], fg[u], fu[u], c, a, b);
                }
            } else {                            // rows longer than 4096: fetched here, 4 chunks at a time
                const size_t rg = group_row + cur.j0 + warp, ru = rg + S;
                const uint4* gate = reinterpret_cast<const uint4*>(Q + rg * row_bytes);
                const uint4* up = reinterpret_cast<const uint4*>(Q + ru * row_bytes);
                for (int c0 = lane; c0 < chunks16; c0 += 128) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int c = c0 + 32 * u;
                        if (c < chunks16) {
                            wg[u] = ldg_stream16(gate + c);
                            wu[u] = ldg_stream16(up + c);
                            fg[u] = __bfloat162float(scales[rg * nb + (c >> 2)]);
                            fu[u] = __bfloat162float(scales[ru * nb + (c >> 2)]);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int c = c0 + 32 * u;
                        if (c < chunks16) dot_chunk(wg[u], wu[u], fg[u], fu[u], c, a, b);
                    }
                }
            }
            a = warp_sum(a);
            b = warp_sum(b);
            if (lane == 0) hs[warp] = silu_mul(a, b);
        }
        __syncthreads();

        // ---- phase 2: down rows, block-wide, 16 fixed columns per thread and turn ---------------------------
        for (int jb = 0; jb < cur.cnt; jb += 4) {
            uint2 wd[4][ITERS];
            float hsv[4][ITERS];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj)
#pragma unroll
                for (int i = 0; i < ITERS; ++i) {
                    const int c = tid + kI4Threads * i;
                    if (jb + jj < cur.cnt && c < chunks8) {
                        const size_t rd = group_row + 2 * S + cur.j0 + jb + jj;
                        wd[jj][i] = __ldg(reinterpret_cast<const uint2*>(Q + rd * row_bytes) + c);
                        hsv[jj][i] = __bfloat162float(scales[rd * nb + (c >> 3)]);
                    }
                }
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                if (jb + jj < cur.cnt) {
                    const float h = hs[jb + jj];
#pragma unroll
                    for (int i = 0; i < ITERS; ++i) {
                        const int c = tid + kI4Threads * i;
                        if (c < chunks8) {
                            const float f = h * hsv[jj][i];
                            corr[i] += f;
                            const uint32_t words[2] = {wd[jj][i].x, wd[jj][i].y};
#pragma unroll
                            for (int v = 0; v < 2; ++v)
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    const uint32_t p = nibble_pair_bf16(words[v], k);
                                    acc[i][8 * v + k] = fmaf(f, __uint_as_float(p << 16), acc[i][8 * v + k]);
                                    acc[i][8 * v + k + 4] = fmaf(f, __uint_as_float(p & 0xffff0000u), acc[i][8 * v + k + 4]);
                                }
                        }
                    }
                }
            }
        }
        const Batch nxt = find_batch(cur.n_next);
        __syncthreads();  // hs is rewritten by the next batch
        cur = nxt;
    }
    if (cur_slot >= 0) flush(cur_slot);
}

// ------------------------------------------------------------------------------------------------------------
// Ring form of the same computation for d_model 2048 / 4096 (group size a multiple of 8): a producer warp streams
// batches of 8 neurons (their gate, up and down code rows and the three runs of scales: six bulk copies per stage)
// into a shared-memory ring, the consumer warps work from shared memory, so no consumer ever waits on a global load
// and the bytes in flight are set by the ring depth.
//   phase 1  a warp per row (or per gate/up pair of rows); the lane's chunks against x kept in shared memory in the
//            nibble pairing; the two products of a neuron meet in shared memory;
//   phase 2  REP replicas of d/16 threads; a replica takes every REP-th down row, a thread owns 16 columns.
// The unpacking is bound by the logic pipe (half as wide as the multiply-add pipe), so work is moved off it: mask and
// exponent bits sit in registers (one three-input logic instruction per pair of weights), some right shifts are done
// as high halves of products, the lower element of a pair is moved up by a multiplication, and the upper element is
// used without masking the lower one off (its surplus is subtracted once per flush).
// Every mbarrier wait is bounded; on a timeout the block flags HALO_DEV_TIMEOUT, drains its copies and returns.
// ------------------------------------------------------------------------------------------------------------
constexpr int kRingNB = 8;
constexpr int kRingConsumers = 512;            // consumer threads of the tensor-core form further down
constexpr int kRingConsumerWarps = kRingConsumers / 32;
template <int N>
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ring_consumer_barrier() { consumer_barrier<kRingConsumers>(); }

struct RingHeader {
    uint64_t full[8];
    uint64_t empty[8];
    int slot[8];        // holder slot of the batch in each stage, -1 = skip
    int abort_flag;
    int pad[3];
    __align__(16) float red[2][2 * kRingNB];
};
constexpr int kRingHeaderBytes = 1024;
static_assert(sizeof(RingHeader) <= kRingHeaderBytes, "ring header region");

// NCW consumer warps + one producer warp.  NCW = 8 with two stages is sized so that TWO thread blocks share an SM
// (2 x 113 KB of shared memory, 2 x 288 threads): while one block sits at the barrier between its phases or waits for
// a stage, the other one computes, and the blocks of the next launch move in as soon as one of this launch leaves.
// NCW = 16 with four stages is the one-block-per-SM form.  Phase 1: warp w takes rows w, w + NCW, ... of the 16
// (8 gate, then 8 up), so with NCW = 8 a warp has the gate and the up row of one neuron and reads x once for both.
template <int XC, int REP, int STAGES, int NCW>
__global__ void __launch_bounds__(NCW * 32 + 32, NCW == 8 ? 2 : 1)
group_ffn_i4_ring_kernel(int d, int S, int G, const uint8_t* __restrict__ Q, const __nv_bfloat16* __restrict__ scales,
                         const __nv_bfloat16* __restrict__ x_all, const int32_t* __restrict__ keep_list,
                         const int32_t* __restrict__ n_keep_ptr, const int32_t* __restrict__ dev_of_group, int n_dev,
                         int n_tok, float* __restrict__ partials, uint32_t* dev_status) {
    constexpr int NB = kRingNB;
    constexpr int kConsumers = NCW * 32;
    constexpr int RPW = 2 * NB / NCW;            // rows of phase 1 per warp
    static_assert(STAGES <= 8 && NB % REP == 0 && (NCW == 8 || NCW == 16), "ring / replica shape");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    RingHeader& hd = *reinterpret_cast<RingHeader*>(smem_raw);
    const int chunks16 = d / 32, chunks8 = d / 16, nb = d / kQBlock;
    const uint32_t row_bytes = static_cast<uint32_t>(d) / 2u;
    const uint32_t plane_bytes = row_bytes * NB;                 // codes of one of gate / up / down for a batch
    const uint32_t sc_bytes = static_cast<uint32_t>(nb) * 2u * NB;   // scales of one plane of a batch
    const uint32_t stage_bytes = 3u * (plane_bytes + sc_bytes);
    uint4* xp = reinterpret_cast<uint4*>(smem_raw + kRingHeaderBytes);                                  // [4][chunks16]
    float* xsum = reinterpret_cast<float*>(smem_raw + kRingHeaderBytes + static_cast<size_t>(d) * 2);   // [chunks16]
    unsigned char* ring =
        smem_raw + kRingHeaderBytes + static_cast<size_t>(d) * 2 + ((static_cast<size_t>(chunks16) * 4 + 127) & ~size_t(127));

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tok = blockIdx.y;
    // Run-time copies of constants (n_tok > 0, so the added term is zero): the multipliers stand in for shifts (see
    // nibble_pair_mulhi), and mask / exponent bits held in registers make "and, then or" one instruction (PairBits).
    const uint32_t rt_zero = static_cast<uint32_t>(n_tok) >> 31;
    const uint32_t mul1 = 0x10000000u + rt_zero, mul2 = 0x01000000u + rt_zero, mul3 = 0x00100000u + rt_zero;
    const uint32_t mul16 = 0x00010000u + rt_zero;
    const PairBits pb{0x000F000Fu + rt_zero, 0x43004300u + rt_zero};
    int nk = *n_keep_ptr;
    if (nk < 0 || nk > G) {
        if (tid == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
        nk = nk < 0 ? 0 : G;
    }
    // the zero-fill of the partial slots runs ahead of this kernel as a programmatic dependency: released here for the
    // next call's zero-fill, waited for below before the first sum leaves this block
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int per_group = S / NB;
    const long long total = static_cast<long long>(nk) * per_group;  // batches
    const int lo = static_cast<int>(total * blockIdx.x / gridDim.x);
    const int hi = static_cast<int>(total * (blockIdx.x + 1) / gridDim.x);
    if (lo >= hi) return;
    const int n_it = hi - lo;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&hd.full[s], 1); mbar_init(&hd.empty[s], NCW); }
        hd.abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    volatile int* abort_flag = &hd.abort_flag;

    if (warp == NCW) {
        // ---------------- producer ----------------
        if (lane == 0) {
            int issued = 0;
            for (int it = 0; it < n_it; ++it) {
                if (*abort_flag) break;
                const int s = it % STAGES;
                const uint32_t use = static_cast<uint32_t>(it / STAGES);
                if (it >= STAGES && !mbar_wait_bounded(&hd.empty[s], (use - 1u) & 1u, abort_flag)) { *abort_flag = 1; break; }
                const int b = lo + it;
                const int ki = b / per_group, j0 = (b - ki * per_group) * NB;
                const int g = keep_list[ki];
                int slot = 0;
                bool ok = (g >= 0 && g < G);
                if (ok && dev_of_group) { slot = dev_of_group[g] + 1; ok = (slot >= 0 && slot <= n_dev); }
                issued = it + 1;
                if (!ok) {
                    flag_status(dev_status, HALO_DEV_BAD_INDEX);
                    hd.slot[s] = -1;
                    mbar_arrive(&hd.full[s]);
                    continue;
                }
                hd.slot[s] = slot;
                unsigned char* dst = ring + static_cast<size_t>(s) * stage_bytes;
                mbar_arrive_expect_tx(&hd.full[s], stage_bytes);
#pragma unroll
                for (int plane = 0; plane < 3; ++plane) {
                    const size_t row = static_cast<size_t>(g) * 3 * S + static_cast<size_t>(plane) * S + j0;
                    bulk_copy_g2s(dst + plane * plane_bytes, Q + row * row_bytes, plane_bytes, &hd.full[s]);
                    bulk_copy_g2s(dst + 3 * plane_bytes + plane * sc_bytes, scales + row * nb, sc_bytes, &hd.full[s]);
                }
            }
            if (*abort_flag) {
                const int first = issued > STAGES ? issued - STAGES : 0;
                for (int it = first; it < issued; ++it) {
                    int never = 0;
                    mbar_wait_bounded(&hd.full[it % STAGES], static_cast<uint32_t>(it / STAGES) & 1u, &never);
                }
                flag_status(dev_status, HALO_DEV_TIMEOUT);
            }
        }
        return;
    }

    // ---------------- consumers ----------------
    {   // x in the nibble pairing, and its plain sums per 32 elements
        const uint16_t* xb = reinterpret_cast<const uint16_t*>(x_all + static_cast<size_t>(tok) * d);
        uint32_t* xp_words = reinterpret_cast<uint32_t*>(xp);
        for (int i = tid; i < d / 2; i += kConsumers) {
            const int c = i / 16, r = i - c * 16, w = r >> 2, k = r & 3;
            const uint32_t lo16 = xb[32 * c + 8 * w + k], hi16 = xb[32 * c + 8 * w + k + 4];
            xp_words[(static_cast<size_t>(w) * chunks16 + c) * 4 + k] = lo16 | (hi16 << 16);
        }
        for (int c = tid; c < chunks16; c += kConsumers) {
            float sx = 0.0f;
            for (int e = 0; e < 32; ++e) sx += __bfloat162float(x_all[static_cast<size_t>(tok) * d + 32 * c + e]);
            xsum[c] = sx;
        }
    }
    consumer_barrier<kConsumers>();
    const int rep = tid / (kConsumers / REP);              // phase 2 replica and 8-byte column chunk
    const int col = tid % (kConsumers / REP);
    float acc[16], corr = 0.0f;
#pragma unroll
    for (int e = 0; e < 16; ++e) acc[e] = 0.0f;
    int cur_slot = -1;
    const size_t slot_stride = static_cast<size_t>(n_tok) * d;

    bool dep_waited = false;
    auto flush = [&](int slot) {
        if (!dep_waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            dep_waited = true;
        }
        if (col < chunks8) {
            float* dst = partials + static_cast<size_t>(slot) * slot_stride + static_cast<size_t>(tok) * d + col * 16;
            const float off = kNibbleBias * corr;
            // upper elements (e + 4): sum f * (128 + 0x4300 / 65536 + n_hi + n_lo / 65536), n_lo from element e
            const float off_hi = (kNibbleBias + 17152.0f / 65536.0f) * corr;
#pragma unroll
            for (int v = 0; v < 16; v += 8) {
                float lo4[4], hi4[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    lo4[k] = acc[v + k] - off;
                    hi4[k] = (acc[v + k + 4] - off_hi) - (acc[v + k] - 128.0f * corr) * (1.0f / 65536.0f);
                }
                red_add_v4f(dst + v, lo4[0], lo4[1], lo4[2], lo4[3]);
                red_add_v4f(dst + v + 4, hi4[0], hi4[1], hi4[2], hi4[3]);
            }
        }
        corr = 0.0f;
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[e] = 0.0f;
    };

    for (int it = 0; it < n_it; ++it) {
        const int s = it % STAGES;
        const uint32_t parity = static_cast<uint32_t>(it / STAGES) & 1u;
        if (!*abort_flag && !mbar_wait_bounded(&hd.full[s], parity, abort_flag)) *abort_flag = 1;
        const int slot = *abort_flag ? -1 : hd.slot[s];
        const unsigned char* stage = ring + static_cast<size_t>(s) * stage_bytes;
        const __nv_bfloat16* stage_sc = reinterpret_cast<const __nv_bfloat16*>(stage + 3 * plane_bytes);   // [3][NB][nb]
        float* red = hd.red[it & 1];
        if (slot >= 0) {
            if (slot != cur_slot) {
                if (cur_slot >= 0) flush(cur_slot);
                cur_slot = slot;
            }
            // phase 1: code rows 0..15 of the stage are the 8 gate rows then the 8 up rows (planes 0, 1 adjacent)
            float a[RPW];
#pragma unroll
            for (int r = 0; r < RPW; ++r) a[r] = 0.0f;
#pragma unroll
            for (int u = 0; u < XC; ++u) {
                const int c = lane + 32 * u;
                uint32_t ww[RPW][4];
                float t0[RPW], t1[RPW];
#pragma unroll
                for (int r = 0; r < RPW; ++r) {
                    const uint4 w4 = reinterpret_cast<const uint4*>(stage + static_cast<size_t>(warp + r * NCW) * row_bytes)[c];
                    ww[r][0] = w4.x; ww[r][1] = w4.y; ww[r][2] = w4.z; ww[r][3] = w4.w;
                    t0[r] = 0.0f; t1[r] = 0.0f;
                }
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const uint4 xq = xp[static_cast<size_t>(w) * chunks16 + c];
#pragma unroll
                    for (int r = 0; r < RPW; ++r) {
                        fma_bf16x2(nibble_pair_r(ww[r][w], pb), xq.x, t0[r], t1[r]);
                        fma_bf16x2(nibble_pair_r(ww[r][w] >> 4, pb), xq.y, t0[r], t1[r]);
                        fma_bf16x2(nibble_pair_r(ww[r][w] >> 8, pb), xq.z, t0[r], t1[r]);
                        fma_bf16x2(nibble_pair_r(__umulhi(ww[r][w], mul3), pb), xq.w, t0[r], t1[r]);
                    }
                }
                const float off = kNibbleBias * xsum[c];
#pragma unroll
                for (int r = 0; r < RPW; ++r)
                    a[r] = fmaf(__bfloat162float(stage_sc[static_cast<size_t>(warp + r * NCW) * nb + (c >> 2)]),
                                (t0[r] + t1[r]) - off, a[r]);
            }
#pragma unroll
            for (int r = 0; r < RPW; ++r) {
                a[r] = warp_sum(a[r]);
                if (lane == 0) red[warp + r * NCW] = a[r];
            }
        }
        consumer_barrier<kConsumers>();
        if (slot >= 0 && col < chunks8) {
            // phase 2: this replica's down rows, 16 columns of each
            const unsigned char* down = stage + 2 * plane_bytes;
            const __nv_bfloat16* ds = stage_sc + static_cast<size_t>(2 * NB) * nb;
#pragma unroll
            for (int jj = 0; jj < NB / REP; ++jj) {
                const int j = jj * REP + rep;
                const float h = silu_mul(red[j], red[NB + j]);
                const float f = h * __bfloat162float(ds[static_cast<size_t>(j) * nb + (col >> 3)]);
                corr += f;
                const uint2 w2 = reinterpret_cast<const uint2*>(down + static_cast<size_t>(j) * row_bytes)[col];
                const uint32_t words[2] = {w2.x, w2.y};
                // The pair register itself, read as fp32, is 128 + (upper nibble) + (0x4300 + lower nibble) / 65536: it is
                // used as it stands for the upper element (no mask), and the surplus is taken off once, at the flush.
#pragma unroll
                for (int v = 0; v < 2; ++v) {
                    const uint32_t pk[4] = {nibble_pair_r(words[v], pb), nibble_pair_r(__umulhi(words[v], mul1), pb),
                                            nibble_pair_r(__umulhi(words[v], mul2), pb),
                                            nibble_pair_r(__umulhi(words[v], mul3), pb)};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        acc[8 * v + k] = fmaf(f, __uint_as_float(pk[k] * mul16), acc[8 * v + k]);
                        acc[8 * v + k + 4] = fmaf(f, __uint_as_float(pk[k]), acc[8 * v + k + 4]);
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&hd.empty[s]);
    }
    if (cur_slot >= 0) flush(cur_slot);
    if (tid == 0 && *abort_flag) flag_status(dev_status, HALO_DEV_TIMEOUT);
}

__device__ __forceinline__ void mma_16816_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ------------------------------------------------------------------------------------------------------------
// Ring form with the products on the tensor cores (mma.sync m16n8k16, bf16 x bf16 -> fp32); an option, not the default
// (see the dispatch below for the measurement).  The plain ring kernel is bound by instruction issue: every weight
// costs a mask-and-bias plus a multiply-add on the CUDA cores.  Here the CUDA cores only turn nibbles into bf16
// numbers (128 + nibble, one shift and one logic instruction per pair) and the multiply-adds of 256 weights go into
// one warp-wide MMA.  A batch is 8 neurons: its 8 gate rows and 8 up rows are the 16 rows of the A operand.
//   phase 1  warp w owns a slice of d/16 input elements.  Thread (g = lane / 4, t = lane % 4) takes word t of each
//            16-byte chunk of rows g (gate) and 8 + g (up): a word's nibbles k and k + 4 form one register pair, so
//            the K order of an MMA is "pairs (k, k + 4)"; x is laid out in the same pairing and sits in column 0 of
//            the B operand.  After the 8 MMAs of a 128-element block the accumulator of a row is corrected by the
//            offset (136 x the plain sum of x over the block) and scaled by the row's block scale.
//   phase 2  y[c] = sum_j f_j * (nibble_j[c] - 8), f_j = silu(a_j) * b_j * scale_j: the M dimension is 16 columns,
//            the K dimension the 8 neurons (K slots 8..15 are zero).  Thread (g, t) takes word g of a 64-column
//            group from rows 2t and 2t + 1 and pairs the two rows' nibbles column by column (one byte permutation per
//            column); f is split into a bf16 high and low part that sit in columns 0 and 1 of B, so nothing is lost
//            to bf16 rounding.  The column sums stay in the MMA accumulators across batches.
// Rows are staged with a pitch of (d/2 + 16) bytes so that the word loads above are free of bank conflicts.
// ------------------------------------------------------------------------------------------------------------
struct MmaRingHeader {
    uint64_t full[8];
    uint64_t empty[8];
    int slot[8];
    int abort_flag;
    int pad[3];
    __align__(16) float red[3][2 * kRingNB];     // gate / up sums of the batch, by batch number modulo 3
};

// KG = 64-column groups per warp in phase 2 = d / 1024.  512 threads, no producer warp: with 17 warps one of the four
// register files of an SM would hold five warps and cap every thread at 96 registers, too few for the 64 accumulator
// registers of phase 2.  Instead, right after the barrier between the two phases of batch `it` (every warp is then
// done with batch it-1), lane 0 of every warp issues one or two of the copies of batch it + STAGES - 1 into the stage
// batch it-1 occupied.
template <int KG, int STAGES>
__global__ void __launch_bounds__(kRingConsumers, 1)
group_ffn_i4_mma_kernel(int d, int S, int G, const uint8_t* __restrict__ Q, const __nv_bfloat16* __restrict__ scales,
                        const __nv_bfloat16* __restrict__ x_all, const int32_t* __restrict__ keep_list,
                        const int32_t* __restrict__ n_keep_ptr, const int32_t* __restrict__ dev_of_group, int n_dev,
                        int n_tok, float* __restrict__ partials, uint32_t* dev_status) {
    constexpr int NB = kRingNB;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    MmaRingHeader& hd = *reinterpret_cast<MmaRingHeader*>(smem_raw);
    const int chunks16 = d / 32, nb = d / kQBlock;
    const uint32_t row_bytes = static_cast<uint32_t>(d) / 2u;
    const uint32_t pitch = row_bytes + 16u;
    const uint32_t sc_bytes = static_cast<uint32_t>(nb) * 2u * NB;      // scales of one plane of a batch
    const uint32_t codes_bytes = 3u * NB * pitch;
    const uint32_t stage_bytes = codes_bytes + 3u * sc_bytes;
    uint4* xp = reinterpret_cast<uint4*>(smem_raw + 1024);                                  // [4][chunks16]
    float* xsum = reinterpret_cast<float*>(smem_raw + 1024 + static_cast<size_t>(d) * 2);   // [nb]: per 128 elements
    unsigned char* ring = smem_raw + 1024 + static_cast<size_t>(d) * 2 + ((static_cast<size_t>(nb) * 4 + 127) & ~size_t(127));

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tok = blockIdx.y;
    int nk = *n_keep_ptr;
    if (nk < 0 || nk > G) {
        if (tid == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
        nk = nk < 0 ? 0 : G;
    }
    const int per_group = S / NB;
    const long long total = static_cast<long long>(nk) * per_group;
    const int lo = static_cast<int>(total * blockIdx.x / gridDim.x);
    const int hi = static_cast<int>(total * (blockIdx.x + 1) / gridDim.x);
    if (lo >= hi) return;
    const int n_it = hi - lo;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(&hd.full[s], 1);
        hd.abort_flag = 0;
        mbar_fence_init();
    }
    if (tid < 3 * 2 * NB) (&hd.red[0][0])[tid] = 0.0f;
    __syncthreads();
    volatile int* abort_flag = &hd.abort_flag;

    // Copies of batch `bi` into its stage, shared out over the warps: copy number cp = 0..26 (24 code rows with the
    // padded pitch, 3 planes of scales) goes to warp cp % 16.  Warp 0 also posts the expected bytes (or marks the
    // stage as skipped); copies of other warps may complete before that, which the transaction count allows.
    auto issue_batch = [&](int bi) {
        if (lane != 0 || bi >= n_it) return;
        const int s = bi % STAGES;
        const int b = lo + bi;
        const int ki = b / per_group, j0 = (b - ki * per_group) * NB;
        const int gq = keep_list[ki];
        int slot = 0;
        bool ok = (gq >= 0 && gq < G);
        if (ok && dev_of_group) { slot = dev_of_group[gq] + 1; ok = (slot >= 0 && slot <= n_dev); }
        if (warp == 0) {
            if (!ok) {
                flag_status(dev_status, HALO_DEV_BAD_INDEX);
                hd.slot[s] = -1;
                mbar_arrive(&hd.full[s]);
            } else {
                hd.slot[s] = slot;
                mbar_arrive_expect_tx(&hd.full[s], 3u * NB * row_bytes + 3u * sc_bytes);
            }
        }
        if (!ok) return;
        unsigned char* dst = ring + static_cast<size_t>(s) * stage_bytes;
        const size_t row0 = static_cast<size_t>(gq) * 3 * S + j0;      // row of plane 0; plane p adds p * S
        for (int cp = warp; cp < 3 * NB + 3; cp += kRingConsumerWarps) {
            if (cp < 3 * NB) {
                const int plane = cp / NB, j = cp - plane * NB;
                bulk_copy_g2s(dst + cp * pitch, Q + (row0 + static_cast<size_t>(plane) * S + j) * row_bytes, row_bytes, &hd.full[s]);
            } else {
                const int plane = cp - 3 * NB;
                bulk_copy_g2s(dst + codes_bytes + plane * sc_bytes, scales + (row0 + static_cast<size_t>(plane) * S) * nb, sc_bytes,
                              &hd.full[s]);
            }
        }
    };
    for (int bi = 0; bi < STAGES - 1; ++bi) issue_batch(bi);

    // ---------------- consumers ----------------
    {   // x in the nibble pairing, and its plain sums per block of 128 elements
        const uint16_t* xb = reinterpret_cast<const uint16_t*>(x_all + static_cast<size_t>(tok) * d);
        uint32_t* xp_words = reinterpret_cast<uint32_t*>(xp);
        for (int i = tid; i < d / 2; i += kRingConsumers) {
            const int c = i / 16, r = i - c * 16, w = r >> 2, k = r & 3;
            const uint32_t lo16 = xb[32 * c + 8 * w + k], hi16 = xb[32 * c + 8 * w + k + 4];
            xp_words[(static_cast<size_t>(w) * chunks16 + c) * 4 + k] = lo16 | (hi16 << 16);
        }
        for (int b = tid; b < nb; b += kRingConsumers) {
            float sx = 0.0f;
            for (int e = 0; e < kQBlock; ++e) sx += __bfloat162float(x_all[static_cast<size_t>(tok) * d + kQBlock * b + e]);
            xsum[b] = sx;
        }
    }
    ring_consumer_barrier();
    const int g = lane >> 2, t = lane & 3;
    constexpr int CPW_BLOCKS = KG / 2;            // 128-element blocks of the K slice of a warp in phase 1 (d / 16 / 128)
    static_assert(KG == 2 || KG == 4, "d must be 2048 or 4096");
    float acc[KG][4][4];                           // phase-2 accumulators: [64-column group][column pair][MMA fragment]
    float corr[KG];                                // sum of f per 64-column group's scale block (offset correction)
#pragma unroll
    for (int q = 0; q < KG; ++q) {
        corr[q] = 0.0f;
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[q][i][e] = 0.0f;
    }
    int cur_slot = -1;
    const size_t slot_stride = static_cast<size_t>(n_tok) * d;

    auto flush = [&](int slot) {
        float* dst = partials + static_cast<size_t>(slot) * slot_stride + static_cast<size_t>(tok) * d;
#pragma unroll
        for (int q = 0; q < KG; ++q) {
            const float off = kNibbleBias * corr[q];
            if (t == 0) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    // columns 2i and 2i + 1 of word g of this group: high part (B column 0) + low part (B column 1)
                    const int col = (warp * KG + q) * 64 + g * 8 + 2 * i;
                    asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(dst + col),
                                 "f"(acc[q][i][0] + acc[q][i][1] - off), "f"(acc[q][i][2] + acc[q][i][3] - off)
                                 : "memory");
                }
            }
            corr[q] = 0.0f;
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[q][i][e] = 0.0f;
        }
    };

    for (int it = 0; it < n_it; ++it) {
        const int s = it % STAGES;
        const uint32_t parity = static_cast<uint32_t>(it / STAGES) & 1u;
        if (!*abort_flag && !mbar_wait_bounded(&hd.full[s], parity, abort_flag)) *abort_flag = 1;
        const int slot = *abort_flag ? -1 : hd.slot[s];
        const unsigned char* stage = ring + static_cast<size_t>(s) * stage_bytes;
        const __nv_bfloat16* stage_sc = reinterpret_cast<const __nv_bfloat16*>(stage + codes_bytes);   // [3][NB][nb]
        float* red = hd.red[it % 3];
        if (slot >= 0) {
            if (slot != cur_slot) {
                if (cur_slot >= 0) flush(cur_slot);
                cur_slot = slot;
            }
            // ---- phase 1: this warp's slice of the 16 gate / up rows on the tensor cores ----
            const unsigned char* row_g = stage + static_cast<size_t>(g) * pitch + t * 4;
            const unsigned char* row_u = stage + static_cast<size_t>(NB + g) * pitch + t * 4;
            float a_g = 0.0f, a_u = 0.0f;
#pragma unroll
            for (int blk = 0; blk < CPW_BLOCKS; ++blk) {
                const int block = warp * CPW_BLOCKS + blk;       // 128-element block of the rows
                float c4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    const int c = block * 4 + cc;
                    const uint32_t wg = *reinterpret_cast<const uint32_t*>(row_g + c * 16);
                    const uint32_t wu = *reinterpret_cast<const uint32_t*>(row_u + c * 16);
                    uint4 xb = make_uint4(0u, 0u, 0u, 0u);
                    if (g == 0) xb = xp[static_cast<size_t>(t) * chunks16 + c];
                    mma_16816_bf16(c4, nibble_pair_bf16(wg, 0), nibble_pair_bf16(wu, 0), nibble_pair_bf16(wg, 1),
                                   nibble_pair_bf16(wu, 1), xb.x, xb.y);
                    mma_16816_bf16(c4, nibble_pair_bf16(wg, 2), nibble_pair_bf16(wu, 2), nibble_pair_bf16(wg, 3),
                                   nibble_pair_bf16(wu, 3), xb.z, xb.w);
                    asm volatile("" ::: "memory");
                }
                if (t == 0) {   // column 0 of the accumulator: rows g (gate) and 8 + g (up)
                    const float off = kNibbleBias * xsum[block];
                    a_g = fmaf(__bfloat162float(stage_sc[static_cast<size_t>(g) * nb + block]), c4[0] - off, a_g);
                    a_u = fmaf(__bfloat162float(stage_sc[static_cast<size_t>(NB + g) * nb + block]), c4[2] - off, a_u);
                }
            }
            if (t == 0) {
                atomicAdd(&red[g], a_g);
                atomicAdd(&red[NB + g], a_u);
            }
        }
        ring_consumer_barrier();
        if (tid < 2 * NB) hd.red[(it + 2) % 3][tid] = 0.0f;     // the buffer of the batch after next
        if (!*abort_flag) issue_batch(it + STAGES - 1);        // into the stage of batch it-1, which everybody has left
        if (slot >= 0) {
            // ---- phase 2: this warp's d/16 columns of the 8 down rows on the tensor cores ----
            const float h0 = silu_mul(red[2 * t], red[NB + 2 * t]);
            const float h1 = silu_mul(red[2 * t + 1], red[NB + 2 * t + 1]);
            const __nv_bfloat16* ds = stage_sc + static_cast<size_t>(2 * NB) * nb;
            const unsigned char* d0 = stage + static_cast<size_t>(2 * NB + 2 * t) * pitch + g * 4;
            const unsigned char* d1 = d0 + pitch;
#pragma unroll
            for (int q = 0; q < KG; ++q) {
                const int grp = warp * KG + q;                  // 64-column group; its scale block is grp / 2
                const float f0 = h0 * __bfloat162float(ds[static_cast<size_t>(2 * t) * nb + (grp >> 1)]);
                const float f1 = h1 * __bfloat162float(ds[static_cast<size_t>(2 * t + 1) * nb + (grp >> 1)]);
                // sum of f over the 8 neurons (lanes with the same g hold the 4 pairs)
                float fs = f0 + f1;
                fs += __shfl_xor_sync(0xffffffffu, fs, 1);
                fs += __shfl_xor_sync(0xffffffffu, fs, 2);
                corr[q] += fs;
                // f = high + low, both bf16: column 0 of B carries the high parts, column 1 the low parts
                const __nv_bfloat16 f0h = __float2bfloat16_rn(f0), f1h = __float2bfloat16_rn(f1);
                const __nv_bfloat162 hi2 = __halves2bfloat162(f0h, f1h);
                const __nv_bfloat162 lo2 = __floats2bfloat162_rn(f0 - __bfloat162float(f0h), f1 - __bfloat162float(f1h));
                uint32_t bfrag = 0u;
                if (g == 0) bfrag = *reinterpret_cast<const uint32_t*>(&hi2);
                else if (g == 1) bfrag = *reinterpret_cast<const uint32_t*>(&lo2);
                const uint32_t w0 = *reinterpret_cast<const uint32_t*>(d0 + grp * 32);
                const uint32_t w1 = *reinterpret_cast<const uint32_t*>(d1 + grp * 32);
                uint32_t p0[4], p1[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) { p0[k] = nibble_pair_bf16(w0, k); p1[k] = nibble_pair_bf16(w1, k); }
                // column c < 4 is the low half of pair c, column c >= 4 the high half of pair c - 4; an A register holds
                // one column of the two rows
                mma_16816_bf16(acc[q][0], __byte_perm(p0[0], p1[0], 0x5410), __byte_perm(p0[1], p1[1], 0x5410), 0u, 0u, bfrag, 0u);
                mma_16816_bf16(acc[q][1], __byte_perm(p0[2], p1[2], 0x5410), __byte_perm(p0[3], p1[3], 0x5410), 0u, 0u, bfrag, 0u);
                mma_16816_bf16(acc[q][2], __byte_perm(p0[0], p1[0], 0x7632), __byte_perm(p0[1], p1[1], 0x7632), 0u, 0u, bfrag, 0u);
                mma_16816_bf16(acc[q][3], __byte_perm(p0[2], p1[2], 0x7632), __byte_perm(p0[3], p1[3], 0x7632), 0u, 0u, bfrag, 0u);
                asm volatile("" ::: "memory");   // keeps the next group's loads behind this group's MMAs (register pressure)
            }
        }
    }
    if (cur_slot >= 0) flush(cur_slot);
    if (*abort_flag) {
        // a wait ran out: every copy that was issued must have landed before the block goes away
        __syncthreads();
        if (tid == 0) {
            for (int bi = max(0, n_it - STAGES); bi < n_it; ++bi) {
                int never = 0;
                mbar_wait_bounded(&hd.full[bi % STAGES], static_cast<uint32_t>(bi / STAGES) & 1u, &never);
            }
            flag_status(dev_status, HALO_DEV_TIMEOUT);
        }
    }
}

halo_status check_i4_shape(const halo_ffn_shape* s) {
    if (!s) return HALO_ERR_ARG;
    if (s->d_model <= 0 || s->d_model % kQBlock != 0 || s->d_model > 8192 || s->group_size <= 0 || s->d_ffn <= 0 ||
        s->d_ffn % s->group_size != 0 || s->d_ffn / s->group_size > HALO_MAX_GROUPS)
        return HALO_ERR_SHAPE;
    return HALO_OK;
}
}  // namespace

halo_status launch_dequantize_i4(const halo_ffn_shape& sh, const void* Q, const void* scales, const int32_t* keep_list,
                                 const int32_t* n_keep, void* W_out, uint32_t* dev_status, cudaStream_t st) {
    const int d = sh.d_model, S = sh.group_size, G = sh.d_ffn / S;
    int dev = 0, sms = kSmCount;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long threads = static_cast<long long>(G) * 3 * S * (d / 32);
    const unsigned blocks = static_cast<unsigned>(std::min<long long>((threads + 255) / 256, static_cast<long long>(sms) * 16));
    dequantize_i4_kernel<<<blocks, 256, 0, st>>>(d, S, G, static_cast<const uint8_t*>(Q),
                                                  static_cast<const __nv_bfloat16*>(scales), keep_list, n_keep,
                                                  static_cast<__nv_bfloat16*>(W_out), dev_status);
    return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}

}  // namespace halo

using namespace halo;

extern "C" halo_status halo_quantize_rows_i4(int d_model, long long n_rows, halo_dtype wdtype, const void* W, void* Q,
                                             void* scales, void* stream) {
    if (d_model <= 0 || d_model % kQBlock != 0 || d_model > 8192 || n_rows <= 0) return HALO_ERR_SHAPE;
    if (wdtype != HALO_F32 && wdtype != HALO_BF16) return HALO_ERR_DTYPE;
    if (!W || !Q || !scales) return HALO_ERR_ARG;
    if (!aligned16(W) || !aligned16(Q) || !aligned16(scales)) return HALO_ERR_ALIGN;
    const long long warps = n_rows * (d_model / kQBlock);
    if ((warps + 7) / 8 > 0x7fffffffll) return HALO_ERR_SHAPE;
    const unsigned blocks = static_cast<unsigned>((warps + 7) / 8);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (wdtype == HALO_BF16)
        quantize_i4_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(d_model, n_rows, static_cast<const __nv_bfloat16*>(W),
                                                                  static_cast<uint8_t*>(Q),
                                                                  static_cast<__nv_bfloat16*>(scales));
    else
        quantize_i4_kernel<float><<<blocks, 256, 0, st>>>(d_model, n_rows, static_cast<const float*>(W),
                                                          static_cast<uint8_t*>(Q), static_cast<__nv_bfloat16*>(scales));
    return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}

extern "C" halo_status halo_quantize_weights_i4(const halo_ffn_shape* shape, const void* W_packed, void* Q,
                                                void* scales, void* stream) {
    halo_status rc = check_i4_shape(shape);
    if (rc != HALO_OK) return rc;
    return halo_quantize_rows_i4(shape->d_model, 3ll * shape->d_ffn, shape->wdtype, W_packed, Q, scales, stream);
}

extern "C" halo_status halo_dequantize_weights_i4(const halo_ffn_shape* shape, const void* Q, const void* scales,
                                                  const int32_t* keep_list, const int32_t* n_keep, void* W_packed,
                                                  uint32_t* dev_status, void* stream) {
    halo_status rc = check_i4_shape(shape);
    if (rc != HALO_OK) return rc;
    if (!Q || !scales || !W_packed || (keep_list && !n_keep)) return HALO_ERR_ARG;
    if (!aligned16(Q) || !aligned16(scales) || !aligned16(W_packed)) return HALO_ERR_ALIGN;
    return launch_dequantize_i4(*shape, Q, scales, keep_list, n_keep, W_packed, dev_status, static_cast<cudaStream_t>(stream));
}

extern "C" halo_status halo_group_ffn_i4(const halo_ffn_shape* shape, const void* Q, const void* scales, const void* x,
                                         int n_tok, const int32_t* keep_list, const int32_t* n_keep,
                                         const int32_t* dev_of_group, int n_dev, float* partials, uint32_t* dev_status,
                                         void* stream) {
    halo_status rc = check_i4_shape(shape);
    if (rc != HALO_OK) return rc;
    if (!Q || !scales || !x || !keep_list || !n_keep || !partials || n_tok <= 0) return HALO_ERR_ARG;
    if (n_dev < 0 || n_dev > HALO_MAX_DEVICES || (!dev_of_group && n_dev != 0)) return HALO_ERR_ARG;
    if (!aligned16(Q) || !aligned16(scales) || !aligned16(x) || !aligned16(partials)) return HALO_ERR_ALIGN;
    return launch_group_ffn_i4(*shape, Q, scales, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials, dev_status,
                               static_cast<cudaStream_t>(stream), false);
}

// already_zero: the caller guarantees that `partials` is zero (otherwise the call zeroes it first).  Without the
// zero-fill in front of it the ring kernel is an ordinary launch: as a programmatic dependent it would start under
// whatever precedes it in the stream, which may be the kernel that writes x.
halo_status halo::launch_group_ffn_i4(const halo_ffn_shape& sh, const void* Q, const void* scales, const void* x, int n_tok,
                                      const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group,
                                      int n_dev, float* partials, uint32_t* dev_status, cudaStream_t st, bool already_zero) {
    const halo_ffn_shape* shape = &sh;
    const int d = shape->d_model, S = shape->group_size, G = shape->d_ffn / S;
    const size_t bytes = sizeof(float) * static_cast<size_t>(n_dev + 1) * n_tok * d;
    const int form_early = option_value(OPT_I4_NO_RING);
    const bool ring_form = (d == 2048 || d == 4096) && S % kRingNB == 0 && form_early != 1 && form_early != 3;
    if (already_zero) {
    } else if (ring_form) {
        if (launch_zero_partials(partials, bytes / sizeof(float), st) != HALO_OK) return HALO_ERR_CUDA;
    } else if (cudaMemsetAsync(partials, 0, bytes, st) != cudaSuccess) {
        return HALO_ERR_CUDA;
    }
    const uint8_t* q = static_cast<const uint8_t*>(Q);
    const __nv_bfloat16* sc = static_cast<const __nv_bfloat16*>(scales);
    const __nv_bfloat16* xt = static_cast<const __nv_bfloat16*>(x);
    int dev = 0, sms = kSmCount;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    // 3: ring with the products on the tensor cores.  Correct, and measured SLOWER than the CUDA-core ring: with one
    // token only one of the 8 columns of an m16n8k16 MMA carries data, and at the rate of the legacy mma.sync path of this
    // GPU (about 8 cycles per instruction and SM sub-partition) that costs as many cycles per weight as the FMA it replaces.
    const int form = form_early;
    if ((d == 2048 || d == 4096) && S % kRingNB == 0 && form == 3) {
        constexpr int kStages = 4;
        const size_t nbk = static_cast<size_t>(d) / kQBlock;
        const size_t stage = 3 * kRingNB * (static_cast<size_t>(d) / 2 + 16) + 3 * nbk * 2 * kRingNB;
        const size_t smem_m = 1024 + static_cast<size_t>(d) * 2 + ((nbk * 4 + 127) & ~size_t(127)) + kStages * stage;
        const long long batches = static_cast<long long>(G) * (S / kRingNB);
        const dim3 grid_m(static_cast<unsigned>(std::min<long long>(batches, sms)), n_tok);
        if (d == 4096) {
            auto k = group_ffn_i4_mma_kernel<4, kStages>;
            static bool once[64] = {};
            if (!ensure_dynamic_smem(k, smem_m, once)) return HALO_ERR_CUDA;
            k<<<grid_m, kRingConsumers, smem_m, st>>>(d, S, G, q, sc, xt, keep_list, n_keep, dev_of_group, n_dev, n_tok,
                                                     partials, dev_status);
        } else {
            auto k = group_ffn_i4_mma_kernel<2, kStages>;
            static bool once[64] = {};
            if (!ensure_dynamic_smem(k, smem_m, once)) return HALO_ERR_CUDA;
            k<<<grid_m, kRingConsumers, smem_m, st>>>(d, S, G, q, sc, xt, keep_list, n_keep, dev_of_group, n_dev, n_tok,
                                                   partials, dev_status);
        }
        return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
    }
    if (ring_form) {
        // ring form.  Default: two thread blocks per SM (8 consumer warps, 2 stages each); option value 2: one block
        // per SM (16 consumer warps, 4 stages).
        const bool two = form_early != 2;
        const int stages = two ? 2 : 4;
        const size_t stage = 3 * (static_cast<size_t>(d) / 2 * kRingNB + static_cast<size_t>(d) / kQBlock * 2 * kRingNB);
        const size_t smem_r = kRingHeaderBytes + static_cast<size_t>(d) * 2 +
                              ((static_cast<size_t>(d) / 32 * 4 + 127) & ~size_t(127)) + stages * stage;
        const long long batches = static_cast<long long>(G) * (S / kRingNB);
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(static_cast<unsigned>(std::min<long long>(batches, static_cast<long long>(sms) * (two ? 2 : 1))), n_tok);
        cfg.blockDim = dim3(two ? 8 * 32 + 32 : 16 * 32 + 32);
        cfg.dynamicSmemBytes = smem_r;
        cfg.stream = st;
        cudaLaunchAttribute attr{};
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = already_zero ? 0 : 1;
        auto go = [&](auto k, bool (&once)[64]) {
            if (!ensure_dynamic_smem(k, smem_r, once)) return HALO_ERR_CUDA;
            return cudaLaunchKernelEx(&cfg, k, d, S, G, q, sc, xt, keep_list, n_keep, dev_of_group, n_dev, n_tok, partials,
                                      dev_status) == cudaSuccess
                       ? HALO_OK
                       : HALO_ERR_CUDA;
        };
        static bool once_a[64] = {}, once_b[64] = {}, once_c[64] = {}, once_d[64] = {};
        if (d == 4096) return two ? go(group_ffn_i4_ring_kernel<4, 1, 2, 8>, once_a) : go(group_ffn_i4_ring_kernel<4, 2, 4, 16>, once_b);
        return two ? go(group_ffn_i4_ring_kernel<2, 2, 2, 8>, once_c) : go(group_ffn_i4_ring_kernel<2, 4, 4, 16>, once_d);
    }
    const int chunks8 = d / 16;
    const int iters = (chunks8 + kI4Threads - 1) / kI4Threads;
    const long long max_batches = (static_cast<long long>(G) * S + kI4Warps - 1) / kI4Warps;
    const int gx = static_cast<int>(std::min<long long>(max_batches, static_cast<long long>(sms) * kI4BlocksPerSm));
    const dim3 grid(gx, n_tok);
    const size_t smem = static_cast<size_t>(d) * 2 + sizeof(float) * (d / 32 + kI4Warps);
    switch (iters) {
        case 1:
            group_ffn_i4_kernel<1><<<grid, kI4Threads, smem, st>>>(d, S, G, q, sc, xt, keep_list, n_keep, dev_of_group,
                                                                   n_dev, n_tok, partials, dev_status);
            break;
        case 2:
            group_ffn_i4_kernel<2><<<grid, kI4Threads, smem, st>>>(d, S, G, q, sc, xt, keep_list, n_keep, dev_of_group,
                                                                   n_dev, n_tok, partials, dev_status);
            break;
        default: return HALO_ERR_SHAPE;
    }
    return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}
