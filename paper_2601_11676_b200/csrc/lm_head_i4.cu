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

#include "i4_rows.cuh"
#include "tma.cuh"

namespace halo {

namespace {
constexpr int kLmI4Threads = 256;
constexpr int kLmI4Warps = kLmI4Threads / 32;
constexpr int kLmI4RowsPerItem = 2 * kLmI4Warps;                     // a warp takes two rows of an item
constexpr int kLmI4BlocksPerSm = 3;

__global__ void __launch_bounds__(kLmI4Threads, kLmI4BlocksPerSm)
lm_head_i4_kernel(int d, int vocab, int S, int n_tok, const uint8_t* __restrict__ Q,
                  const __nv_bfloat16* __restrict__ scales, const __nv_bfloat16* __restrict__ x,
                  const int32_t* __restrict__ keep_list, const int32_t* __restrict__ n_keep_ptr,
                  float* __restrict__ logits, uint32_t* dev_status) {
    extern __shared__ __align__(16) unsigned char smem_b[];
    uint4* xp = reinterpret_cast<uint4*>(smem_b);                    // [4][chunks16]: x in nibble pairing
    float* xsum = reinterpret_cast<float*>(smem_b + static_cast<size_t>(d) * 2);   // [chunks16]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_groups = (vocab + S - 1) / S;
    const int items_per_group = (S + kLmI4RowsPerItem - 1) / kLmI4RowsPerItem;
    int nk = n_groups;
    if (keep_list) nk = max(0, min(*n_keep_ptr, n_groups));
    const long long total = static_cast<long long>(nk) * items_per_group;
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
    for (int t = 0; t < n_tok; ++t) {
        if (t > 0) __syncthreads();                                  // everybody is done with the previous x
        stage_x_paired(x + static_cast<size_t>(t) * d, xp, xsum, d);
        __syncthreads();

        for (long long item = blockIdx.x; item < total; item += gridDim.x) {
            int v0;
            bool two;
            rows_of(item, v0, two, t == 0);
            if (v0 >= 0) {                                           // warp-uniform
                float acc_a, acc_b;
                const size_t ra = static_cast<size_t>(v0);           // a lone last row: read twice, used once
                warp_two_rows_dot_i4(Q, scales, ra, two ? ra + 1 : ra, d, xp, xsum, lane, acc_a, acc_b);
                float* out = logits + static_cast<size_t>(t) * vocab + v0;
                if (lane == 0) out[0] = acc_a;
                if (lane == 1 && two) out[1] = acc_b;
            }
        }
    }
}

// One token, d_model 2048 / 4096: the streaming form.  One thread block per SM; a producer thread streams batches of 32
// consecutive rows (their codes and their scales: two bulk copies) into a shared-memory ring, 16 consumer warps take two
// rows each against x kept in REGISTERS in the nibble pairing (a lane always meets the same chunks of x), so a consumer
// neither waits on a global load nor reads x from shared memory.  Every mbarrier wait is bounded.
constexpr int kLmI4RingWarps = 16;
constexpr int kLmI4RingRows = 2 * kLmI4RingWarps;
constexpr int kLmI4RingThreads = kLmI4RingWarps * 32 + 32;

struct LmI4RingHeader {
    uint64_t full[8];
    uint64_t empty[8];
    int row0[8];        // first vocabulary row of the batch in each stage
    int n_rows[8];      // rows of the batch (0 = skip)
    int abort_flag;
};

template <int XC, int STAGES>
__global__ void __launch_bounds__(kLmI4RingThreads, 1)
lm_head_i4_ring_kernel(int d, int vocab, int S, const uint8_t* __restrict__ Q, const __nv_bfloat16* __restrict__ scales,
                       const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ keep_list,
                       const int32_t* __restrict__ n_keep_ptr, float* __restrict__ logits, uint32_t* dev_status) {
    static_assert(STAGES <= 8, "ring depth");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    LmI4RingHeader& hd = *reinterpret_cast<LmI4RingHeader*>(smem_raw);
    unsigned char* ring = smem_raw + 1024;
    const uint32_t crow_bytes = static_cast<uint32_t>(d) / 2u;            // codes of a row
    const uint32_t srow_bytes = static_cast<uint32_t>(d) / 64u;           // scales of a row (bf16 per 128 elements)
    const uint32_t stage_bytes = (crow_bytes + srow_bytes) * kLmI4RingRows;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_groups = (vocab + S - 1) / S;
    int nk = n_groups;
    if (keep_list) nk = max(0, min(*n_keep_ptr, n_groups));
    const int per_group = (S + kLmI4RingRows - 1) / kLmI4RingRows;
    const long long total = static_cast<long long>(nk) * per_group;          // batches
    const int lo = static_cast<int>(total * blockIdx.x / gridDim.x);
    const int hi = static_cast<int>(total * (blockIdx.x + 1) / gridDim.x);
    if (lo >= hi) return;
    const int n_it = hi - lo;
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&hd.full[s], 1); mbar_init(&hd.empty[s], kLmI4RingWarps); }
        hd.abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    volatile int* abort_flag = &hd.abort_flag;

    if (warp == kLmI4RingWarps) {
        // ---------------- producer ----------------
        if (lane == 0) {
            int issued = 0;
            for (int it = 0; it < n_it; ++it) {
                if (*abort_flag) break;
                const int s = it % STAGES;
                const uint32_t use = static_cast<uint32_t>(it / STAGES);
                if (it >= STAGES && !mbar_wait_bounded(&hd.empty[s], (use - 1u) & 1u, abort_flag)) { *abort_flag = 1; break; }
                const int b = lo + it;
                const int ki = b / per_group, jb = b - ki * per_group;
                const int g = keep_list ? keep_list[ki] : ki;
                issued = it + 1;
                int n = 0, row0 = 0;
                if (g < 0 || g >= n_groups) {
                    flag_status(dev_status, HALO_DEV_BAD_INDEX);
                } else {
                    row0 = g * S + jb * kLmI4RingRows;
                    n = max(0, min(kLmI4RingRows, min(vocab, (g + 1) * S) - row0));
                }
                hd.row0[s] = row0;
                hd.n_rows[s] = n;
                if (n == 0) {
                    mbar_arrive(&hd.full[s]);
                    continue;
                }
                unsigned char* dst = ring + static_cast<size_t>(s) * stage_bytes;
                mbar_arrive_expect_tx(&hd.full[s], static_cast<uint32_t>(n) * (crow_bytes + srow_bytes));
                bulk_copy_g2s(dst, Q + static_cast<size_t>(row0) * crow_bytes, static_cast<uint32_t>(n) * crow_bytes, &hd.full[s]);
                bulk_copy_g2s(dst + kLmI4RingRows * crow_bytes,
                              reinterpret_cast<const unsigned char*>(scales) + static_cast<size_t>(row0) * srow_bytes,
                              static_cast<uint32_t>(n) * srow_bytes, &hd.full[s]);
            }
            if (*abort_flag) {
                // the consumers stopped waiting: every copy this block issued lands before it exits
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

    // ---------------- consumers: warp w takes rows 2w and 2w + 1 of every batch ----------------
    // this lane's chunks lane + 32u of x: for word w of a chunk the four pairs (x[8w+k], x[8w+k+4]) as bf16x2, and the
    // chunk's plain sum
    uint4 xq[XC][4];
    float xs[XC];
    {
        const uint16_t* xb = reinterpret_cast<const uint16_t*>(x);
#pragma unroll
        for (int u = 0; u < XC; ++u) {
            const int c = lane + 32 * u;
            const uint4* src = reinterpret_cast<const uint4*>(xb + 32 * c);
            float sx = 0.0f;
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const uint4 v = __ldg(src + w);                      // elements 8w .. 8w+7 of the chunk
                // pairs (e_k, e_k+4): low halves of v.x, v.y with low halves of v.z, v.w, and the same for the high halves
                xq[u][w] = make_uint4(__byte_perm(v.x, v.z, 0x5410), __byte_perm(v.x, v.z, 0x7632),
                                      __byte_perm(v.y, v.w, 0x5410), __byte_perm(v.y, v.w, 0x7632));
                const uint32_t ws[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) sx += bf16_lo(ws[e]) + bf16_hi(ws[e]);
            }
            xs[u] = sx;
        }
    }
    // constants that must reach the arithmetic as run-time values (else the compiler folds them back into immediates
    // and shifts): a zero it cannot see through
    const uint32_t rt_zero = static_cast<uint32_t>(d) >> 31;
    const uint32_t mul3 = 0x00100000u + rt_zero;                   // word * 2^20 >> 32 = word >> 12 (a second shift
                                                                   // moved to the multiplier measured slower: 25.0 against 23.2 us)
    const PairBits pb{0x000F000Fu + rt_zero, 0x43004300u + rt_zero};
    const int ra = 2 * warp;
    for (int it = 0; it < n_it; ++it) {
        const int s = it % STAGES;
        const uint32_t parity = static_cast<uint32_t>(it / STAGES) & 1u;
        if (!*abort_flag && !mbar_wait_bounded(&hd.full[s], parity, abort_flag)) *abort_flag = 1;
        if (*abort_flag) break;
        const int n = hd.n_rows[s], row0 = hd.row0[s];
        if (ra < n) {
            const bool two = ra + 1 < n;
            const unsigned char* base = ring + static_cast<size_t>(s) * stage_bytes;
            const int rb = two ? ra + 1 : ra;
            const uint4* a4 = reinterpret_cast<const uint4*>(base + static_cast<size_t>(ra) * crow_bytes);
            const uint4* b4 = reinterpret_cast<const uint4*>(base + static_cast<size_t>(rb) * crow_bytes);
            const __nv_bfloat16* sca = reinterpret_cast<const __nv_bfloat16*>(base + kLmI4RingRows * crow_bytes + ra * srow_bytes);
            const __nv_bfloat16* scb = reinterpret_cast<const __nv_bfloat16*>(base + kLmI4RingRows * crow_bytes + rb * srow_bytes);
            float acc_a = 0.0f, acc_b = 0.0f;
#pragma unroll
            for (int u = 0; u < XC; ++u) {
                const int c = lane + 32 * u;
                const uint4 wa = a4[c], wb = b4[c];
                const uint32_t aw[4] = {wa.x, wa.y, wa.z, wa.w};
                const uint32_t bw[4] = {wb.x, wb.y, wb.z, wb.w};
                float ta0 = 0.0f, ta1 = 0.0f, tb0 = 0.0f, tb1 = 0.0f;
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const uint32_t xk[4] = {xq[u][w].x, xq[u][w].y, xq[u][w].z, xq[u][w].w};
                    // the logic pipe bounds this loop: mask and exponent bits come from registers (one three-input
                    // instruction per pair) and the widest shift is done as the high half of a product
                    fma_bf16x2(nibble_pair_r(aw[w], pb), xk[0], ta0, ta1);
                    fma_bf16x2(nibble_pair_r(bw[w], pb), xk[0], tb0, tb1);
                    fma_bf16x2(nibble_pair_r(aw[w] >> 4, pb), xk[1], ta0, ta1);
                    fma_bf16x2(nibble_pair_r(bw[w] >> 4, pb), xk[1], tb0, tb1);
                    fma_bf16x2(nibble_pair_r(aw[w] >> 8, pb), xk[2], ta0, ta1);
                    fma_bf16x2(nibble_pair_r(bw[w] >> 8, pb), xk[2], tb0, tb1);
                    fma_bf16x2(nibble_pair_r(__umulhi(aw[w], mul3), pb), xk[3], ta0, ta1);
                    fma_bf16x2(nibble_pair_r(__umulhi(bw[w], mul3), pb), xk[3], tb0, tb1);
                }
                const float off = kNibbleBias * xs[u];
                acc_a = fmaf(__bfloat162float(sca[c >> 2]), (ta0 + ta1) - off, acc_a);
                acc_b = fmaf(__bfloat162float(scb[c >> 2]), (tb0 + tb1) - off, acc_b);
            }
            acc_a = warp_sum(acc_a);
            acc_b = warp_sum(acc_b);
            if (lane == 0) logits[row0 + ra] = acc_a;
            if (lane == 1 && two) logits[row0 + ra + 1] = acc_b;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&hd.empty[s]);
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
    if (n_tok == 1 && (d == 2048 || d == 4096)) {
        constexpr int kStages = 3;
        const long long batches = n_groups * ((S + kLmI4RingRows - 1) / kLmI4RingRows);
        const unsigned grid_r = static_cast<unsigned>(std::min<long long>(batches, sms));
        const size_t smem_r = 1024 + static_cast<size_t>(kStages) * kLmI4RingRows * (d / 2 + d / 64);
        const uint8_t* q8 = static_cast<const uint8_t*>(Q);
        const __nv_bfloat16* sc = static_cast<const __nv_bfloat16*>(scales);
        const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        if (d == 4096) {
            auto k = lm_head_i4_ring_kernel<4, kStages>;
            static bool once[64] = {};
            if (!ensure_dynamic_smem(k, smem_r, once)) return HALO_ERR_CUDA;
            k<<<grid_r, kLmI4RingThreads, smem_r, st>>>(d, shape->vocab, S, q8, sc, xb, keep_list, n_keep, logits, dev_status);
        } else {
            auto k = lm_head_i4_ring_kernel<2, kStages>;
            static bool once[64] = {};
            if (!ensure_dynamic_smem(k, smem_r, once)) return HALO_ERR_CUDA;
            k<<<grid_r, kLmI4RingThreads, smem_r, st>>>(d, shape->vocab, S, q8, sc, xb, keep_list, n_keep, logits, dev_status);
        }
        return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
    }
    const unsigned grid = static_cast<unsigned>(std::min<long long>(items, static_cast<long long>(sms) * kLmI4BlocksPerSm));
    const size_t smem = static_cast<size_t>(d) * 2 + sizeof(float) * (d / 32);
    lm_head_i4_kernel<<<grid, kLmI4Threads, smem, static_cast<cudaStream_t>(stream)>>>(
        d, shape->vocab, S, n_tok, static_cast<const uint8_t*>(Q), static_cast<const __nv_bfloat16*>(scales),
        static_cast<const __nv_bfloat16*>(x), keep_list, n_keep, logits, dev_status);
    return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}
