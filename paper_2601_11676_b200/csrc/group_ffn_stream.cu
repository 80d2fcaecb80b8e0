// halo_group_ffn, decode form, fast path for bf16 (steps a6..a8).
//
// One thread block per SM.  The kept neurons are cut into batches of NB consecutive neurons of one group
// (their gate rows, up rows and down rows are three contiguous byte ranges of the packed layout) and the
// batches are dealt evenly and contiguously to the blocks.  A producer warp streams each batch into a ring
// of shared-memory stages with bulk asynchronous copies (cp.async.bulk, completion counted on an mbarrier),
// so the bytes in flight are set by the ring depth, not by registers.  512 consumer threads work from shared
// memory:
//   phase 1  the 2*NB gate/up rows are split over the 16 warps (16/(2*NB) warps per row); each lane keeps its
//            slice of x in registers for the whole launch; partial dot products meet in shared memory;
//   phase 2  every thread owns fixed 16-byte column chunks of the down rows and keeps their fp32 sums in
//            registers across batches.
// Sums are added to partials[slot] with vector fp32 reductions when the holder changes and at the end.
// Every wait on an mbarrier is bounded: if one runs out the block flags HALO_DEV_TIMEOUT, stops waiting,
// drains its outstanding copies (bounded) and returns.
#include "common.cuh"
#include "ffn_math.cuh"
#include "tma.cuh"

namespace halo {

constexpr int kConsumers = 512;
constexpr int kConsumerWarps = kConsumers / 32;
constexpr int kStreamThreads = kConsumers + 32;
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }

struct StreamSmemHeader {
    uint64_t full[8];
    uint64_t empty[8];
    int slot[8];        // holder slot of the batch in each stage, -1 = skip
    int abort_flag;
    int pad[3];
    __align__(16) float red[2][32];   // [parity][row * warps_per_row + part]
};

// NB   neurons per batch; XC  16-byte chunks of a row per lane in phase 1;
// P2   column passes per thread in phase 2 (chunks > 512); REP  thread replicas per column (chunks < 512).
template <int NB, int XC, int P2, int REP, int STAGES>
__global__ void __launch_bounds__(kStreamThreads, 1)
group_ffn_stream_kernel(int d, int S, int G, const __nv_bfloat16* __restrict__ W,
                        const __nv_bfloat16* __restrict__ x_all, const int32_t* __restrict__ keep_list,
                        const int32_t* __restrict__ n_keep_ptr, const int32_t* __restrict__ dev_of_group, int n_dev,
                        int n_tok, float* __restrict__ partials, uint32_t* dev_status) {
    constexpr int ROWS = 2 * NB;
    constexpr int WPR = kConsumerWarps / ROWS;  // warps per row in phase 1
    static_assert(WPR * ROWS == kConsumerWarps, "rows must divide the consumer warps");
    static_assert(STAGES <= 8 && NB % REP == 0, "ring / replica shape");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    StreamSmemHeader& hd = *reinterpret_cast<StreamSmemHeader*>(smem_raw);
    unsigned char* ring = smem_raw + 1024;
    const int chunks = d >> 3;
    const uint32_t row_bytes = static_cast<uint32_t>(d) * 2u;
    const uint32_t plane_bytes = row_bytes * NB;      // one of gate / up / down for a batch
    const uint32_t stage_bytes = 3u * plane_bytes;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tok = blockIdx.y;
    // A following launch that declares itself a programmatic dependent (the zero-fill of the next call of this entry
    // point does) may be scheduled as this kernel's thread blocks retire; it waits for this kernel's completion itself
    // before it touches anything.  Ordinary launches behind this kernel are not affected.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    int nk = *n_keep_ptr;
    if (nk < 0 || nk > G) {
        if (tid == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
        nk = nk < 0 ? 0 : G;
    }
    const int per_group = S / NB;
    const long long total = static_cast<long long>(nk) * per_group;  // batches
    const int lo = static_cast<int>(total * blockIdx.x / gridDim.x);
    const int hi = static_cast<int>(total * (blockIdx.x + 1) / gridDim.x);
    if (lo >= hi) return;
    const int n_it = hi - lo;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&hd.full[s], 1); mbar_init(&hd.empty[s], kConsumerWarps); }
        hd.abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    volatile int* abort_flag = &hd.abort_flag;

    if (warp == kConsumerWarps) {
        // ---------------- producer ----------------
        if (lane == 0) {
            int issued = 0;
            for (int it = 0; it < n_it; ++it) {
                if (*abort_flag) break;  // a wait ran out somewhere in the block: issue nothing more
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
                const __nv_bfloat16* group = W + static_cast<size_t>(g) * 3 * S * d;
                unsigned char* dst = ring + static_cast<size_t>(s) * stage_bytes;
                mbar_arrive_expect_tx(&hd.full[s], stage_bytes);
                bulk_copy_g2s(dst, group + static_cast<size_t>(j0) * d, plane_bytes, &hd.full[s]);
                bulk_copy_g2s(dst + plane_bytes, group + static_cast<size_t>(S + j0) * d, plane_bytes, &hd.full[s]);
                bulk_copy_g2s(dst + 2 * plane_bytes, group + static_cast<size_t>(2 * S + j0) * d, plane_bytes,
                              &hd.full[s]);
            }
            if (*abort_flag) {
                // consumers stopped waiting: make sure every copy this block issued has landed before it exits
                const int first = issued > STAGES ? issued - STAGES : 0;
                for (int it = first; it < issued; ++it) {
                    const int s = it % STAGES;
                    const uint32_t parity = static_cast<uint32_t>(it / STAGES) & 1u;
                    int never = 0;
                    mbar_wait_bounded(&hd.full[s], parity, &never);
                }
                flag_status(dev_status, HALO_DEV_TIMEOUT);
            }
        }
        return;
    }

    // ---------------- consumers ----------------
    const int row = warp / WPR, part = warp % WPR;   // phase 1: which row, which slice of it
    const int p1_base = part * (XC * 32) + lane;      // chunk index of this lane's first chunk; stride 32
    uint4 xq[XC];  // this lane's slice of x, packed bf16
    {
        const uint4* xg = reinterpret_cast<const uint4*>(x_all + static_cast<size_t>(tok) * d);
#pragma unroll
        for (int i = 0; i < XC; ++i) xq[i] = __ldg(xg + p1_base + 32 * i);
    }
    const int rep = (REP > 1) ? tid / (kConsumers / REP) : 0;   // phase 2 replica
    const int col0 = (REP > 1) ? tid % (kConsumers / REP) : tid;
    float acc[P2][8];
#pragma unroll
    for (int p = 0; p < P2; ++p)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[p][e] = 0.0f;
    int cur_slot = -1;
    const size_t slot_stride = static_cast<size_t>(n_tok) * d;

    bool dep_waited = false;
    auto flush = [&](int slot) {
        // The zero-fill of `partials` may still be running (this kernel is launched as its programmatic dependent, so
        // that the weight stream starts under it): nothing is added before it has completed.  A no-op otherwise.
        if (!dep_waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); dep_waited = true; }
        float* dst = partials + static_cast<size_t>(slot) * slot_stride + static_cast<size_t>(tok) * d;
#pragma unroll
        for (int p = 0; p < P2; ++p) {
            const int c = col0 + kConsumers * p;
            if (c < chunks) {
                red_add_v4f(dst + c * 8, acc[p][0], acc[p][1], acc[p][2], acc[p][3]);
                red_add_v4f(dst + c * 8 + 4, acc[p][4], acc[p][5], acc[p][6], acc[p][7]);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[p][e] = 0.0f;
        }
    };

    for (int it = 0; it < n_it; ++it) {
        const int s = it % STAGES;
        const uint32_t parity = static_cast<uint32_t>(it / STAGES) & 1u;
        if (!*abort_flag && !mbar_wait_bounded(&hd.full[s], parity, abort_flag)) *abort_flag = 1;
        const int slot = hd.slot[s];
        const unsigned char* stage = ring + static_cast<size_t>(s) * stage_bytes;
        float* red = hd.red[it & 1];
        if (slot >= 0) {
            if (slot != cur_slot) {
                if (cur_slot >= 0) flush(cur_slot);
                cur_slot = slot;
            }
            // phase 1: rows 0..NB-1 are gate rows, NB..2NB-1 the up rows (planes 0 and 1 are adjacent)
            const uint4* rp = reinterpret_cast<const uint4*>(stage + static_cast<size_t>(row) * row_bytes);
            float dot0 = 0.0f, dot1 = 0.0f;
#pragma unroll
            for (int i = 0; i < XC; ++i) dot_bf16x8(rp[p1_base + 32 * i], xq[i], dot0, dot1);
            const float dot = warp_sum(dot0 + dot1);
            if (lane == 0) red[row * WPR + part] = dot;
        }
        consumer_barrier();
        if (slot >= 0) {
            // phase 2
            const unsigned char* down = stage + 2 * plane_bytes;
#pragma unroll
            for (int jj = 0; jj < NB / REP; ++jj) {
                const int j = jj * REP + rep;
                const float h = silu_mul(sum_parts<WPR>(red + j * WPR), sum_parts<WPR>(red + (NB + j) * WPR));
                const uint4* dr = reinterpret_cast<const uint4*>(down + static_cast<size_t>(j) * row_bytes);
#pragma unroll
                for (int p = 0; p < P2; ++p) {
                    const int c = col0 + kConsumers * p;
                    if (P2 == 1 || c < chunks) axpy_bf16x8(h, dr[c], acc[p]);
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&hd.empty[s]);
    }
    if (cur_slot >= 0) flush(cur_slot);
    if (tid == 0 && *abort_flag) flag_status(dev_status, HALO_DEV_TIMEOUT);
}

// Zero-fill of the partial slots; lets the dependent streaming kernel start at once.
__global__ void __launch_bounds__(256)
zero_partials_kernel(float4* __restrict__ p, size_t n4) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // itself launched as a programmatic dependent: whatever ran before it on the stream (say the previous call's
    // streaming kernel, which may still be adding to these very slots) must have completed before anything is zeroed
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n4) p[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
}

halo_status launch_zero_partials(float* partials, size_t n_floats, cudaStream_t st) {
    const size_t n4 = n_floats / 4;     // a multiple of 4: d_model % 8 == 0
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>((n4 + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, zero_partials_kernel, reinterpret_cast<float4*>(partials), n4) == cudaSuccess ? HALO_OK
                                                                                                                 : HALO_ERR_CUDA;
}

// ---- host side ---------------------------------------------------------------------------------------------

namespace {

struct StreamConfig { int nb, xc, p2, rep, stages; };

bool pick_stream_config(int d, int S, StreamConfig* cfg) {
    const int chunks = d / 8;
    switch (d) {
        case 2048: *cfg = {4, 4, 1, 2, 4}; break;
        case 4096: *cfg = {2, 4, 1, 1, 4}; break;
        case 5120: *cfg = {2, 5, 2, 1, 3}; break;
        case 8192: *cfg = {1, 4, 2, 1, 4}; break;
        default: return false;
    }
    (void)chunks;
    return S % cfg->nb == 0;
}

template <int NB, int XC, int P2, int REP, int STAGES>
halo_status launch_stream_cfg(const halo_ffn_shape& sh, const void* W, const void* x, int n_tok,
                              const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group, int n_dev,
                              float* partials, uint32_t* dev_status, cudaStream_t st, bool zero_first) {
    auto kernel = group_ffn_stream_kernel<NB, XC, P2, REP, STAGES>;
    const size_t smem = 1024 + static_cast<size_t>(STAGES) * 3 * NB * sh.d_model * 2;
    static bool configured[64] = {};
    if (!ensure_dynamic_smem(kernel, smem, configured)) return HALO_ERR_CUDA;
    int dev = 0, sms = kSmCount;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int G = sh.d_ffn / sh.group_size;
    const long long max_batches = static_cast<long long>(G) * (sh.group_size / NB);
    dim3 grid(static_cast<unsigned>(std::min<long long>(max_batches, sms)), n_tok);
    if (!zero_first) {
        kernel<<<grid, kStreamThreads, smem, st>>>(sh.d_model, sh.group_size, G, static_cast<const __nv_bfloat16*>(W),
                                                   static_cast<const __nv_bfloat16*>(x), keep_list, n_keep, dev_of_group,
                                                   n_dev, n_tok, partials, dev_status);
        HALO_CHECK_LAUNCH();
        return HALO_OK;
    }
    // zero-fill as a kernel that releases its dependent at once, then the streaming kernel as that dependent: its
    // prologue and its weight stream run under the zero-fill; it waits for it only before it first adds to `partials`
    if (launch_zero_partials(partials, static_cast<size_t>(n_dev + 1) * n_tok * sh.d_model, st) != HALO_OK) return HALO_ERR_CUDA;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kStreamThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, sh.d_model, sh.group_size, G, static_cast<const __nv_bfloat16*>(W),
                                               static_cast<const __nv_bfloat16*>(x), keep_list, n_keep, dev_of_group, n_dev,
                                               n_tok, partials, dev_status);
    return err == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}

}  // namespace

// Returns HALO_ERR_UNIMPLEMENTED when the shape has no streaming configuration (the caller falls back to the
// generic kernel, having zeroed nothing).  zero_first: the call zeroes partials itself; otherwise they must be zero.
halo_status launch_group_ffn_stream(const halo_ffn_shape& sh, const void* W, const void* x, int n_tok,
                                    const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group,
                                    int n_dev, float* partials, uint32_t* dev_status, cudaStream_t st, bool zero_first) {
    StreamConfig cfg;
    if (sh.wdtype != HALO_BF16 || !pick_stream_config(sh.d_model, sh.group_size, &cfg)) return HALO_ERR_UNIMPLEMENTED;
    switch (sh.d_model) {
        case 2048: return launch_stream_cfg<4, 4, 1, 2, 4>(sh, W, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials, dev_status, st, zero_first);
        case 4096: return launch_stream_cfg<2, 4, 1, 1, 4>(sh, W, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials, dev_status, st, zero_first);
        case 5120: return launch_stream_cfg<2, 5, 2, 1, 3>(sh, W, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials, dev_status, st, zero_first);
        case 8192: return launch_stream_cfg<1, 4, 2, 1, 4>(sh, W, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials, dev_status, st, zero_first);
    }
    return HALO_ERR_UNIMPLEMENTED;
}

}  // namespace halo
