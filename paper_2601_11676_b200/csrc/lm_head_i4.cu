// LM-head neuron groups on int4 rows (Sec. II-A, Sec. III-B.3 for the block; Sec. IV-A: the evaluated models are 4-bit).
// Format of halo_quantize_rows_i4: symmetric, one bf16 scale per 128 consecutive elements of a row, nibble = code + 8.
// logits[t][v] = sum over the row's blocks of s_b * sum_e (nibble - 8) * x: a warp takes two vocabulary rows at a time
// against x kept in shared memory in the nibble pairing (nibbles k and k+4 of a word become the bf16 pair
// {128 + n_k, 128 + n_k+4} by mask and OR and feed the mixed-precision FMA; 136 times the plain sum of x over the 32
// elements of a 16-byte chunk is taken off per chunk).  Thread blocks walk (group, 16-row item) pairs in a stride; three
// thread blocks per SM cover each other's loads (holding the next item's rows in registers instead, at two thread blocks
// per SM, was measured slower, and moving a shift to the multiplier and the mask constants into registers, which pays
// in the FFN kernel, changed nothing here: no single pipe is the bound, the issue slots are 55 % busy at 24 warps per SM).
#include <algorithm>

#include "common.cuh"
#include "ffn_math.cuh"
#include "i4_math.cuh"

namespace halo {

namespace {
constexpr int kLmI4Threads = 256;
constexpr int kLmI4Warps = kLmI4Threads / 32;
constexpr int kLmI4RowsPerItem = 2 * kLmI4Warps;                     // a warp takes two rows of an item
constexpr int kLmI4BlocksPerSm = 3;

// Operands of one row pair held by a lane: chunks lane + 32u of both rows and their scales (rows up to 4096 wide), or,
// for wider rows, the chunks of one 4096-element slice at a time.
struct PairRegs {
    uint4 wa[4], wb[4];
    float sa[4], sb[4];
    int v0;            // first row, or -1 when this warp has nothing to do in the item
    bool two;
};

__global__ void __launch_bounds__(kLmI4Threads, kLmI4BlocksPerSm)
lm_head_i4_kernel(int d, int vocab, int S, int n_tok, const uint8_t* __restrict__ Q,
                  const __nv_bfloat16* __restrict__ scales, const __nv_bfloat16* __restrict__ x,
                  const int32_t* __restrict__ keep_list, const int32_t* __restrict__ n_keep_ptr,
                  float* __restrict__ logits, uint32_t* dev_status) {
    extern __shared__ __align__(16) unsigned char smem_b[];
    const int chunks16 = d / 32;                                     // 16-byte code chunks (32 weights) per row
    const int nb = d / 128;
    uint4* xp = reinterpret_cast<uint4*>(smem_b);                    // [4][chunks16]: x in nibble pairing
    float* xsum = reinterpret_cast<float*>(smem_b + static_cast<size_t>(d) * 2);   // [chunks16]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_groups = (vocab + S - 1) / S;
    const int items_per_group = (S + kLmI4RowsPerItem - 1) / kLmI4RowsPerItem;
    int nk = n_groups;
    if (keep_list) nk = max(0, min(*n_keep_ptr, n_groups));
    const long long total = static_cast<long long>(nk) * items_per_group;
    const size_t row_bytes = static_cast<size_t>(d) / 2;
    // rows of this warp in an item (and whether the item is valid at all)
    auto rows_of = [&](long long item, int& v0, bool& two, bool report) {
        v0 = -1;
        two = false;
        if (item >= total) return;
        const int ki = static_cast<int>(item / items_per_group), rb = static_cast<int>(item - ki * items_per_group);
        const int g = keep_list ? keep_list[ki] : ki;
        if (g < 0 || g >= n_groups) {
            if (report && tid == 0 && rb == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
            return;
        }
        const int v_end = min(min(vocab, (g + 1) * S), g * S + (rb + 1) * kLmI4RowsPerItem);
        const int v = g * S + rb * kLmI4RowsPerItem + 2 * warp;
        if (v < v_end) {
            v0 = v;
            two = v + 1 < v_end;
        }
    };
    // the chunks c0 + 32u of the pair's rows
    auto fetch = [&](PairRegs& r, int c0) {
        if (r.v0 < 0) return;
        const size_t ra = static_cast<size_t>(r.v0), rb = r.two ? ra + 1 : ra;   // a lone last row: read twice, used once
        const uint4* a4 = reinterpret_cast<const uint4*>(Q + ra * row_bytes);
        const uint4* b4 = reinterpret_cast<const uint4*>(Q + rb * row_bytes);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = c0 + 32 * u;
            if (c < chunks16) {
                r.wa[u] = ldg_stream16(a4 + c);
                r.wb[u] = ldg_stream16(b4 + c);
                r.sa[u] = __bfloat162float(scales[ra * nb + (c >> 2)]);
                r.sb[u] = __bfloat162float(scales[rb * nb + (c >> 2)]);
            }
        }
    };
    auto dot = [&](const PairRegs& r, int c0, float& acc_a, float& acc_b) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = c0 + 32 * u;
            if (c < chunks16) {
                float ta0 = 0.0f, ta1 = 0.0f, tb0 = 0.0f, tb1 = 0.0f;
                const uint32_t aw[4] = {r.wa[u].x, r.wa[u].y, r.wa[u].z, r.wa[u].w};
                const uint32_t bw[4] = {r.wb[u].x, r.wb[u].y, r.wb[u].z, r.wb[u].w};
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
                acc_a = fmaf(r.sa[u], (ta0 + ta1) - off, acc_a);
                acc_b = fmaf(r.sb[u], (tb0 + tb1) - off, acc_b);
            }
        }
    };

    for (int t = 0; t < n_tok; ++t) {
        if (t > 0) __syncthreads();                                  // everybody is done with the previous x
        // for chunk c and word w of a code chunk, the four pairs (x[8w+k], x[8w+k+4]), k = 0..3, as bf16x2
        const uint16_t* xb = reinterpret_cast<const uint16_t*>(x + static_cast<size_t>(t) * d);
        uint32_t* xp_words = reinterpret_cast<uint32_t*>(xp);
        PairRegs cur;
        for (int i = tid; i < d / 2; i += kLmI4Threads) {
            const int c = i / 16, r = i - c * 16, w = r >> 2, k = r & 3;
            const uint32_t lo16 = xb[32 * c + 8 * w + k], hi16 = xb[32 * c + 8 * w + k + 4];
            xp_words[(static_cast<size_t>(w) * chunks16 + c) * 4 + k] = lo16 | (hi16 << 16);
        }
        for (int c = tid; c < chunks16; c += kLmI4Threads) {
            float sx = 0.0f;
            for (int e = 0; e < 32; ++e) sx += __bfloat162float(x[static_cast<size_t>(t) * d + 32 * c + e]);
            xsum[c] = sx;
        }
        __syncthreads();

        for (long long item = blockIdx.x; item < total; item += gridDim.x) {
            float acc_a = 0.0f, acc_b = 0.0f;
            rows_of(item, cur.v0, cur.two, t == 0);
            if (cur.v0 >= 0)
                for (int c0 = lane; c0 < chunks16; c0 += 128) {
                    fetch(cur, c0);
                    dot(cur, c0, acc_a, acc_b);
                }
            if (cur.v0 >= 0) {                                       // warp-uniform
                acc_a = warp_sum(acc_a);
                acc_b = warp_sum(acc_b);
                float* out = logits + static_cast<size_t>(t) * vocab + cur.v0;
                if (lane == 0) out[0] = acc_a;
                if (lane == 1 && cur.two) out[1] = acc_b;
            }
        }
    }
}
}  // namespace

}  // namespace halo

using namespace halo;

extern "C" halo_status halo_group_lm_head_i4(const halo_lm_shape* shape, const void* Q, const void* scales, const void* x,
                                             int n_tok, const int32_t* keep_list, const int32_t* n_keep, float* logits,
                                             uint32_t* dev_status, void* stream) {
    if (!shape || !Q || !scales || !x || !logits || !dev_status) return HALO_ERR_ARG;
    if ((keep_list == nullptr) != (n_keep == nullptr)) return HALO_ERR_ARG;
    if (shape->d_model <= 0 || shape->d_model % 128 != 0 || shape->d_model > 8192 || shape->vocab <= 0 ||
        shape->group_size <= 0 || n_tok <= 0)
        return HALO_ERR_SHAPE;
    if (!aligned16(Q) || !aligned16(scales) || !aligned16(x)) return HALO_ERR_ALIGN;
    const int d = shape->d_model, S = shape->group_size;
    const long long n_groups = (static_cast<long long>(shape->vocab) + S - 1) / S;
    const long long items = n_groups * ((S + kLmI4RowsPerItem - 1) / kLmI4RowsPerItem);
    int dev = 0, sms = kSmCount;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const unsigned grid = static_cast<unsigned>(std::min<long long>(items, static_cast<long long>(sms) * kLmI4BlocksPerSm));
    const size_t smem = static_cast<size_t>(d) * 2 + sizeof(float) * (d / 32);
    lm_head_i4_kernel<<<grid, kLmI4Threads, smem, static_cast<cudaStream_t>(stream)>>>(
        d, shape->vocab, S, n_tok, static_cast<const uint8_t*>(Q), static_cast<const __nv_bfloat16*>(scales),
        static_cast<const __nv_bfloat16*>(x), keep_list, n_keep, logits, dev_status);
    return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}
