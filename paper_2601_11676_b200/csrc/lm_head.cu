// LM-head neuron groups (Sec. II-A: an up-projection only, a collection of groups of vocabulary rows;
// Sec. III-B.3: delivered reliably, so nothing is dropped): logits[t][v] = <W[v], x_t> for the rows of the listed
// groups.  Bandwidth-bound: the rows are streamed once, a warp takes two rows at a time with sixteen 16-byte loads
// per lane in flight; further tokens re-read the block's 32 rows while they are still cached.
//
// One token, bf16, d_model 2048 / 4096: lm_head_ring_kernel, the streaming form of the FFN kernels.  One thread block
// per SM; a producer thread streams batches of 8 rows (one bulk copy each) into a shared-memory ring, 8 consumer warps
// take a row each against x kept in registers: no consumer waits on a global load, no barrier between warps, and the
// bytes in flight are set by the ring (192 KB per SM).  Every mbarrier wait is bounded.
#include <algorithm>

#include "common.cuh"
#include "ffn_math.cuh"
#include "tma.cuh"

namespace halo {

namespace {
constexpr int kLmRingRows = 8;                         // rows per stage = consumer warps
constexpr int kLmRingThreads = kLmRingRows * 32 + 32;

struct LmRingHeader {
    uint64_t full[8];
    uint64_t empty[8];
    int row0[8];        // first vocabulary row of the batch in each stage
    int n_rows[8];      // rows of the batch (0 = skip)
    int abort_flag;
};

template <int XC, int STAGES>
__global__ void __launch_bounds__(kLmRingThreads, 1)
lm_head_ring_kernel(int d, int vocab, int S, const __nv_bfloat16* __restrict__ W, const __nv_bfloat16* __restrict__ x,
                    const int32_t* __restrict__ keep_list, const int32_t* __restrict__ n_keep_ptr,
                    float* __restrict__ logits, uint32_t* dev_status) {
    static_assert(STAGES <= 8, "ring depth");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    LmRingHeader& hd = *reinterpret_cast<LmRingHeader*>(smem_raw);
    unsigned char* ring = smem_raw + 1024;
    const uint32_t row_bytes = static_cast<uint32_t>(d) * 2u;
    const uint32_t stage_bytes = row_bytes * kLmRingRows;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_groups = (vocab + S - 1) / S;
    int nk = n_groups;
    if (keep_list) nk = max(0, min(*n_keep_ptr, n_groups));
    const int per_group = (S + kLmRingRows - 1) / kLmRingRows;
    const long long total = static_cast<long long>(nk) * per_group;          // batches
    const int lo = static_cast<int>(total * blockIdx.x / gridDim.x);
    const int hi = static_cast<int>(total * (blockIdx.x + 1) / gridDim.x);
    if (lo >= hi) return;
    const int n_it = hi - lo;
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&hd.full[s], 1); mbar_init(&hd.empty[s], kLmRingRows); }
        hd.abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    volatile int* abort_flag = &hd.abort_flag;

    if (warp == kLmRingRows) {
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
                    row0 = g * S + jb * kLmRingRows;
                    n = max(0, min(kLmRingRows, min(vocab, (g + 1) * S) - row0));
                }
                hd.row0[s] = row0;
                hd.n_rows[s] = n;
                if (n == 0) {
                    mbar_arrive(&hd.full[s]);
                    continue;
                }
                mbar_arrive_expect_tx(&hd.full[s], static_cast<uint32_t>(n) * row_bytes);
                bulk_copy_g2s(ring + static_cast<size_t>(s) * stage_bytes, W + static_cast<size_t>(row0) * d,
                              static_cast<uint32_t>(n) * row_bytes, &hd.full[s]);
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

    // ---------------- consumers: warp w takes row w of every batch ----------------
    uint4 xq[XC];
    {
        const uint4* xg = reinterpret_cast<const uint4*>(x);
#pragma unroll
        for (int i = 0; i < XC; ++i) xq[i] = __ldg(xg + lane + 32 * i);
    }
    for (int it = 0; it < n_it; ++it) {
        const int s = it % STAGES;
        const uint32_t parity = static_cast<uint32_t>(it / STAGES) & 1u;
        if (!*abort_flag && !mbar_wait_bounded(&hd.full[s], parity, abort_flag)) *abort_flag = 1;
        if (*abort_flag) break;
        const int n = hd.n_rows[s], row0 = hd.row0[s];
        if (warp < n) {
            const uint4* rp = reinterpret_cast<const uint4*>(ring + static_cast<size_t>(s) * stage_bytes +
                                                             static_cast<size_t>(warp) * row_bytes);
            float dot0 = 0.0f, dot1 = 0.0f;
#pragma unroll
            for (int i = 0; i < XC; ++i) dot_bf16x8(rp[lane + 32 * i], xq[i], dot0, dot1);
            const float v = warp_sum(dot0 + dot1);
            if (lane == 0) logits[row0 + warp] = v;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&hd.empty[s]);
    }
}

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
    if (shape->wdtype == HALO_BF16 && n_tok == 1 && (d == 2048 || d == 4096)) {
        int dev = 0, sms = kSmCount;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const long long batches = n_groups * ((S + kLmRingRows - 1) / kLmRingRows);
        const unsigned grid = static_cast<unsigned>(std::min<long long>(batches, sms));
        const __nv_bfloat16* Wb = static_cast<const __nv_bfloat16*>(W);
        const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
        if (d == 4096) {
            constexpr int kStages = 3;
            const size_t smem_r = 1024 + static_cast<size_t>(kStages) * kLmRingRows * d * 2;
            auto k = lm_head_ring_kernel<16, kStages>;
            static bool once[64] = {};
            if (!ensure_dynamic_smem(k, smem_r, once)) return HALO_ERR_CUDA;
            k<<<grid, kLmRingThreads, smem_r, st>>>(d, shape->vocab, S, Wb, xb, keep_list, n_keep, logits, dev_status);
        } else {
            constexpr int kStages = 6;
            const size_t smem_r = 1024 + static_cast<size_t>(kStages) * kLmRingRows * d * 2;
            auto k = lm_head_ring_kernel<8, kStages>;
            static bool once[64] = {};
            if (!ensure_dynamic_smem(k, smem_r, once)) return HALO_ERR_CUDA;
            k<<<grid, kLmRingThreads, smem_r, st>>>(d, shape->vocab, S, Wb, xb, keep_list, n_keep, logits, dev_status);
        }
        return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
    }
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
