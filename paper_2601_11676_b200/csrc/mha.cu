// MHA neuron groups (Sec. II-A: one head and its output-projection weight form an independent neuron group),
// decode form, under the same selection / holder-slot / merge machinery as the FFN groups.
//   halo_mha_kv_append   k = Wk x, v = Wv x for ALL heads into the caches (every device keeps a full KV cache,
//                        Sec. III-B.3; keys and values are never dropped)
//   halo_group_mha       for every kept head h:  q = Wq_h x;  w = softmax(q K_h^T / sqrt(dh)) over positions 0..pos;
//                        o = w V_h;  partials[slot(h)] += sum_j o_j * Wo_h[j]
// halo_group_mha is ONE launch: a cluster of eight thread blocks per kept head (query rows shared through
// distributed shared memory, positions split over the blocks with an online softmax, each block then streams its
// part of the head's output-projection slice and adds its column sums to the holder's slot with vector
// reductions).  The earlier three-launch form (query rows; attention per (head, 128-position chunk) with a
// running-max partial (m, l, o); combination + output-projection rows) is kept for comparison
// (HALO_TUNE_MHA_THREE_LAUNCHES=1).  Bandwidth-bound like the FFN decode path.
#include <cstdlib>

#include "common.cuh"
#include "i4_rows.cuh"
#include "tma.cuh"

namespace halo {

constexpr int kAttnChunk = 128;   // positions per attention block
constexpr int kOutRows = 16;      // output-projection rows per block

constexpr int kRowsPerWarp = 2;   // rows a warp of the row-product kernels takes, both at once
constexpr int kRowsPerBlock = 8 * kRowsPerWarp;

// x (d elements, 16-byte aligned) widened into shared memory, 16 bytes per thread and step
template <typename T>
__device__ __forceinline__ void stage_x(const T* __restrict__ x, float* xs, int d) {
    constexpr int E = Elem<T>::kPerChunk;
    const uint4* x4 = reinterpret_cast<const uint4*>(x);
    for (int c = threadIdx.x; c < d / E; c += blockDim.x) {
        float xf[E];
        Elem<T>::widen(__ldg(x4 + c), xf);
#pragma unroll
        for (int e = 0; e < E; ++e) xs[c * E + e] = xf[e];
    }
}

// <row_a, x> and <row_b, x> by one warp; eight 16-byte loads per row and lane in flight (sixteen per lane)
template <typename T>
__device__ __forceinline__ void warp_two_rows_dot(const T* __restrict__ row_a, const T* __restrict__ row_b,
                                                  const float* __restrict__ xs, int chunks, int lane, float& out_a,
                                                  float& out_b) {
    constexpr int E = Elem<T>::kPerChunk;
    const uint4* a4 = reinterpret_cast<const uint4*>(row_a);
    const uint4* b4 = reinterpret_cast<const uint4*>(row_b);
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
    out_a = warp_sum(acc_a);
    out_b = warp_sum(acc_b);
}

// rows of [Wk; Wv]: rows 0..H*dh-1 are keys, the rest values; a warp takes kRowsPerWarp consecutive rows
template <typename T>
__global__ void __launch_bounds__(256)
mha_kv_append_kernel(int d, int H, int dh, int Lmax, const T* __restrict__ Wk, const T* __restrict__ Wv,
                     const T* __restrict__ x, int pos, T* __restrict__ Kc, T* __restrict__ Vc) {
    extern __shared__ __align__(16) float xs[];
    stage_x(x, xs, d);
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n = H * dh;                       // even (dh % 16 == 0): a pair of rows never straddles keys/values
    const int r0 = blockIdx.x * kRowsPerBlock + warp * kRowsPerWarp;
#pragma unroll
    for (int i = 0; i < kRowsPerWarp; i += 2) {
        const int r = r0 + i;
        if (r >= 2 * n) return;
        const bool is_v = r >= n;
        const int rr = is_v ? r - n : r;
        const T* base = (is_v ? Wv : Wk) + static_cast<size_t>(rr) * d;
        float va, vb;
        warp_two_rows_dot(base, base + d, xs, d / Elem<T>::kPerChunk, lane, va, vb);
        if (lane < 2) {
            const int row = rr + lane, h = row / dh, j = row - h * dh;
            (is_v ? Vc : Kc)[(static_cast<size_t>(h) * Lmax + pos) * dh + j] = from_float<T>(lane == 0 ? va : vb);
        }
    }
}

// q[ki][j] = <Wq_h[j], x> / sqrt(dh) for the kept heads; a warp takes kRowsPerWarp consecutive rows of one head
template <typename T>
__global__ void __launch_bounds__(256)
mha_q_kernel(int d, int H, int dh, const T* __restrict__ Wp, const T* __restrict__ x,
             const int32_t* __restrict__ keep_list, const int32_t* __restrict__ n_keep_ptr, float* __restrict__ q_ws,
             uint32_t* dev_status) {
    extern __shared__ __align__(16) float xs[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int nk = *n_keep_ptr;
    nk = max(0, min(nk, H));
    if (blockIdx.x * kRowsPerBlock >= nk * dh) return;     // the whole block lies beyond the kept heads
    stage_x(x, xs, d);
    __syncthreads();
    const int r0 = blockIdx.x * kRowsPerBlock + warp * kRowsPerWarp;   // dh % 16 == 0: the four rows share a head
    const int ki = r0 / dh, j0 = r0 - ki * dh;
    if (ki >= nk) return;
    const int h = keep_list[ki];
    if (h < 0 || h >= H) {
        if (lane == 0 && j0 == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
        return;
    }
    const float scale = rsqrtf(static_cast<float>(dh));
#pragma unroll
    for (int i = 0; i < kRowsPerWarp; i += 2) {
        const T* base = Wp + ((static_cast<size_t>(h) * 2 + 0) * dh + j0 + i) * d;
        float va, vb;
        warp_two_rows_dot(base, base + d, xs, d / Elem<T>::kPerChunk, lane, va, vb);
        if (lane < 2) q_ws[static_cast<size_t>(ki) * dh + j0 + i + lane] = (lane == 0 ? va : vb) * scale;
    }
}

// attention partial of one (kept head, chunk of 128 positions): m = max score, l = sum exp(s - m),
// o[j] = sum_p exp(s_p - m) V[p][j]; record layout [m, l, o[dh]]
template <typename T>
__global__ void __launch_bounds__(kAttnChunk)
mha_attn_kernel(int H, int dh, int Lmax, int pos, const T* __restrict__ Kc, const T* __restrict__ Vc,
                const int32_t* __restrict__ keep_list, const int32_t* __restrict__ n_keep_ptr,
                const float* __restrict__ q_ws, float* __restrict__ attn_ws, int n_chunks) {
    __shared__ float q[256];
    __shared__ float w[kAttnChunk];
    __shared__ float red[8];
    const int ki = blockIdx.x, chunk = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int nk = *n_keep_ptr;
    nk = max(0, min(nk, H));
    if (ki >= nk) return;
    const int h = keep_list[ki];
    if (h < 0 || h >= H) return;
    for (int j = tid; j < dh; j += kAttnChunk) q[j] = q_ws[static_cast<size_t>(ki) * dh + j];
    __syncthreads();
    constexpr int E = Elem<T>::kPerChunk;
    const int p = chunk * kAttnChunk + tid;
    const bool valid = p <= pos;
    float s = -INFINITY;
    if (valid) {
        const uint4* krow = reinterpret_cast<const uint4*>(Kc + (static_cast<size_t>(h) * Lmax + p) * dh);
        float acc = 0.0f;
        for (int c = 0; c < dh / E; ++c) {
            float kf[E];
            Elem<T>::widen(__ldg(krow + c), kf);
#pragma unroll
            for (int e = 0; e < E; ++e) acc = fmaf(kf[e], q[c * E + e], acc);
        }
        s = acc;
    }
    // block max
    float m = s;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) red[warp] = m;
    __syncthreads();
    m = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
    const float e = valid ? __expf(s - m) : 0.0f;
    w[tid] = e;
    float l = warp_sum(e);
    if (lane == 0) red[4 + warp] = l;
    __syncthreads();
    l = red[4] + red[5] + red[6] + red[7];
    float* rec = attn_ws + (static_cast<size_t>(ki) * n_chunks + chunk) * (dh + 2);
    if (tid == 0) { rec[0] = m; rec[1] = l; }
    const int n_valid = min(kAttnChunk, pos + 1 - chunk * kAttnChunk);
    // o[j] = sum_p w_p V[p][j]: a thread takes one 16-byte column group and every (128 / groups)-th position,
    // the position groups meet in shared memory
    const int col_groups = dh / E;                      // 16-byte groups per value row
    const int pos_groups = kAttnChunk / col_groups;     // threads per column group
    const int cg = tid % col_groups, pg = tid / col_groups;
    float part[E];
#pragma unroll
    for (int e = 0; e < E; ++e) part[e] = 0.0f;
    if (pg < pos_groups) {
        const uint4* vbase = reinterpret_cast<const uint4*>(Vc + (static_cast<size_t>(h) * Lmax + static_cast<size_t>(chunk) * kAttnChunk) * dh) + cg;
#pragma unroll 4
        for (int pp = pg; pp < n_valid; pp += pos_groups) {
            float vf[E];
            Elem<T>::widen(__ldg(vbase + static_cast<size_t>(pp) * col_groups), vf);
            const float wp = w[pp];
#pragma unroll
            for (int e = 0; e < E; ++e) part[e] = fmaf(wp, vf[e], part[e]);
        }
    }
    __syncthreads();                                    // q[] is no longer needed: reuse it as the meeting place
    float* o_acc = q;
    for (int j = tid; j < dh; j += kAttnChunk) o_acc[j] = 0.0f;
    __syncthreads();
    if (pg < pos_groups) {
#pragma unroll
        for (int e = 0; e < E; ++e) atomicAdd(&o_acc[cg * E + e], part[e]);
    }
    __syncthreads();
    for (int j = tid; j < dh; j += kAttnChunk) rec[2 + j] = o_acc[j];
}

// combine the chunk partials of the block's values o_j, then stream their output-projection rows
template <typename T, int ITERS>
__global__ void __launch_bounds__(256)
mha_out_kernel(int d, int H, int dh, const T* __restrict__ Wp, const int32_t* __restrict__ keep_list,
               const int32_t* __restrict__ n_keep_ptr, const int32_t* __restrict__ dev_of_group, int n_dev,
               const float* __restrict__ attn_ws, int n_chunks, float* __restrict__ partials, uint32_t* dev_status) {
    constexpr int E = Elem<T>::kPerChunk;
    __shared__ float o_s[kOutRows];
    const int ki = blockIdx.x, j0 = blockIdx.y * kOutRows, tid = threadIdx.x;
    int nk = *n_keep_ptr;
    nk = max(0, min(nk, H));
    if (ki >= nk) return;
    const int h = keep_list[ki];
    if (h < 0 || h >= H) return;   // flagged by the query kernel
    int slot = 0;
    if (dev_of_group) {
        slot = dev_of_group[h] + 1;
        if (slot < 0 || slot > n_dev) {
            if (tid == 0 && j0 == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
            return;
        }
    }
    if (tid < kOutRows) {
        const float* rec0 = attn_ws + static_cast<size_t>(ki) * n_chunks * (dh + 2);
        float M = -INFINITY;
        for (int c = 0; c < n_chunks; ++c) M = fmaxf(M, rec0[static_cast<size_t>(c) * (dh + 2)]);
        float L = 0.0f, o = 0.0f;
        for (int c = 0; c < n_chunks; ++c) {
            const float* rec = rec0 + static_cast<size_t>(c) * (dh + 2);
            const float f = __expf(rec[0] - M);
            L = fmaf(rec[1], f, L);
            o = fmaf(rec[2 + j0 + tid], f, o);
        }
        o_s[tid] = o / L;
    }
    __syncthreads();
    const int chunks = d / E;
    float acc[ITERS][E];
#pragma unroll
    for (int i = 0; i < ITERS; ++i)
#pragma unroll
        for (int e = 0; e < E; ++e) acc[i][e] = 0.0f;
    const T* rows = Wp + ((static_cast<size_t>(h) * 2 + 1) * dh + j0) * d;
    for (int jb = 0; jb < kOutRows; jb += 4) {
        uint4 wv[4][ITERS];
#pragma unroll
        for (int jj = 0; jj < 4; ++jj)
#pragma unroll
            for (int i = 0; i < ITERS; ++i) {
                const int c = tid + 256 * i;
                if (c < chunks) wv[jj][i] = ldg_stream16(reinterpret_cast<const uint4*>(rows + static_cast<size_t>(jb + jj) * d) + c);
            }
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const float o = o_s[jb + jj];
#pragma unroll
            for (int i = 0; i < ITERS; ++i) {
                const int c = tid + 256 * i;
                if (c < chunks) {
                    float w8[E];
                    Elem<T>::widen(wv[jj][i], w8);
#pragma unroll
                    for (int e = 0; e < E; ++e) acc[i][e] = fmaf(o, w8[e], acc[i][e]);
                }
            }
        }
    }
    float* dst = partials + static_cast<size_t>(slot) * d;
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
        const int c = tid + 256 * i;
        if (c < chunks) {
#pragma unroll
            for (int e = 0; e < E; e += 4) red_add_v4f(dst + c * E + e, acc[i][e], acc[i][e + 1], acc[i][e + 2], acc[i][e + 3]);
        }
    }
}

// ------------------------------------------------------------------------------------------------------------
// The three steps above in ONE launch: a cluster of kMhaCluster thread blocks per kept head.  Block r computes
// dh / 8 query rows and hands them to all blocks of its cluster through distributed shared memory; then takes
// every 8th run of positions (online softmax over pieces of up to 256 positions); the blocks exchange their (m, l) and the
// slices of o that each other needs; block r finally streams the dh / 8 output-projection rows of its slice.
// The only waits are the cluster barriers, which the hardware guarantees to be reachable (a cluster is
// co-scheduled); a block never leaves before the last remote write into its shared memory has been synchronised.
// ------------------------------------------------------------------------------------------------------------
constexpr int kMhaCluster = 8;
constexpr int kMhaMaxRows = 32;     // dh <= 256: at most 32 rows of a head per block

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// store a float into the same shared-memory location of another block of the cluster
__device__ __forceinline__ void st_remote_f32(float* local_smem_ptr, uint32_t target_rank, float v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local_smem_ptr)), "r"(target_rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}

// APPEND: the whole MHA block of a token in this one launch.  The grid then has one cluster per head (kept or not):
// block r first computes dh / 8 rows each of the head's keys and values for this token and writes them into the
// caches at `pos` (every head, never dropped); clusters of heads that are not kept end there.  The cluster barrier
// that completes the query also orders those cache writes before the attention reads them.
// Shared memory for a thread block's K and V rows (see kv_smem in the kernel): used when every block of a cluster has
// a single piece of positions and the two pieces fit in 64 KB (so that two thread blocks still share an SM).
constexpr size_t kKvSmemMax = 64 * 1024;
constexpr size_t kMhaSmemLimit = 32 * 1024 + kKvSmemMax;   // x widened (at most 8192 floats) + the K / V rows
static size_t kv_smem_bytes(int pos, int dh, size_t elem) {
    const int n_pos = pos + 1;
    const int piece = std::min(256, std::max(32, ((n_pos + kMhaCluster - 1) / kMhaCluster + 31) & ~31));
    if (n_pos > kMhaCluster * piece) return 0;          // several pieces per block: the loop fetches them itself
    const size_t bytes = 2 * static_cast<size_t>(piece) * dh * elem;
    return (bytes <= kKvSmemMax && (static_cast<size_t>(dh) * elem) % 16 == 0) ? bytes : 0;
}

// I4 (with APPEND, T = bf16): Wp, Wk and Wv hold int4 codes (halo_quantize_rows_i4 of the same row matrices), Sp, Sk
// and Sv their scales; x and the caches stay bf16.  The row products go against x in the nibble pairing, the
// output-projection rows are unpacked into 16 columns per thread; everything between is the same code.
template <typename T, int ITERS, bool APPEND, bool I4 = false>
__global__ void __cluster_dims__(kMhaCluster, 1, 1) __launch_bounds__(256)
mha_fused_kernel(int d, int H, int dh, int Lmax, int pos, const T* __restrict__ Wp, const T* __restrict__ x,
                 const T* Kc, const T* Vc, const int32_t* __restrict__ keep_list,
                 const int32_t* __restrict__ n_keep_ptr, const int32_t* __restrict__ dev_of_group, int n_dev,
                 float* __restrict__ partials, uint32_t* dev_status, const T* __restrict__ Wk, const T* __restrict__ Wv,
                 T* Kw, T* Vw, int kv_smem, const __nv_bfloat16* __restrict__ Sp = nullptr,
                 const __nv_bfloat16* __restrict__ Sk = nullptr, const __nv_bfloat16* __restrict__ Sv = nullptr) {
    static_assert(!I4 || (APPEND && sizeof(T) == 2), "int4 weights: fused block on bf16 activations only");
    constexpr int E = Elem<T>::kPerChunk;
    extern __shared__ __align__(16) float xs[];          // [d]: x widened; behind it (kv_smem): this block's K and V rows
    // int4: the same d floats hold x in the nibble pairing (2d bytes) and its sums per 32 elements (d/8 bytes)
    uint4* xp = reinterpret_cast<uint4*>(xs);
    float* xsum = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(xs) + static_cast<size_t>(d) * 2);
    __shared__ uint64_t kv_bar;
    __shared__ float q_s[256];                           // the head's full query (written by all blocks of the cluster)
    __shared__ float o_acc[256];                         // this block's running o over its positions
    __shared__ float w_s[256];                           // softmax weights of the current piece
    __shared__ float red[16];
    __shared__ float ml_in[kMhaCluster][2];              // (m, l) of every block of the cluster
    __shared__ float o_in[kMhaCluster][kMhaMaxRows];     // their o restricted to this block's rows
    __shared__ float o_s[kMhaMaxRows];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r = static_cast<int>(cluster_rank());
    int nk = *n_keep_ptr;
    nk = max(0, min(nk, H));
    const int rows = dh / kMhaCluster;                   // rows of the head per block (even: dh % 16 == 0)
    const int j0 = r * rows;
    const int chunks = d / E;
    int h, slot = 0;
    if constexpr (APPEND) {
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // see group_ffn_stream_kernel
        h = blockIdx.y;
        // keys and values of this token for head h, rows j0 .. j0 + rows of each, two rows per warp and turn
        if constexpr (I4) stage_x_paired(reinterpret_cast<const __nv_bfloat16*>(x), xp, xsum, d);
        else stage_x(x, xs, d);
        __syncthreads();
        for (int i = 2 * warp; i < 2 * rows; i += 16) {
            const bool is_v = i >= rows;
            const int j = j0 + (is_v ? i - rows : i);
            float va, vb;
            if constexpr (I4) {
                const size_t row = static_cast<size_t>(h) * dh + j;
                warp_two_rows_dot_i4(reinterpret_cast<const uint8_t*>(is_v ? Wv : Wk), is_v ? Sv : Sk, row, row + 1, d, xp,
                                     xsum, lane, va, vb);
            } else {
                const T* base = (is_v ? Wv : Wk) + (static_cast<size_t>(h) * dh + j) * d;
                warp_two_rows_dot(base, base + d, xs, chunks, lane, va, vb);
            }
            if (lane < 2) (is_v ? Vw : Kw)[(static_cast<size_t>(h) * Lmax + pos) * dh + j + lane] = from_float<T>(lane == 0 ? va : vb);
        }
        // is this head kept, and by whom?  (the list is short: one pass of the block over it)
        int found = 0;
        for (int i = tid; i < nk; i += 256) {
            const int e = keep_list[i];
            if (e == h) found = 1;
            if ((e < 0 || e >= H) && h == 0 && r == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
        }
        if (!__syncthreads_or(found)) return;            // the same decision in every block of the cluster
        if (dev_of_group) {
            slot = dev_of_group[h] + 1;
            if (slot < 0 || slot > n_dev) {
                if (tid == 0 && r == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
                return;
            }
        }
    } else {
        const int ki = blockIdx.y;
        if (ki >= nk) return;                            // the same decision in every block of the cluster
        h = keep_list[ki];
        if (h < 0 || h >= H) {
            if (tid == 0 && r == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
            return;
        }
        if (dev_of_group) {
            slot = dev_of_group[h] + 1;
            if (slot < 0 || slot > n_dev) {
                if (tid == 0 && r == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
                return;
            }
        }
    }

    // Distributed shared memory may be written only once every block of the cluster is known to be running:
    // arrive now, wait before the first remote store (the staging of x lies in between, and the blocks of a cluster
    // are scheduled together, so the wait costs next to nothing).  The early returns above are taken by all blocks
    // of a cluster or by none.
    cluster_arrive();
    // ---- query rows j0 .. j0 + rows, two per warp and turn, sent to every block of the cluster ----
    if constexpr (!APPEND) stage_x(x, xs, d);
    for (int j = tid; j < dh; j += 256) o_acc[j] = 0.0f;
    // piece = positions a block takes at a time: an eighth of the context (so that all eight blocks work) in
    // multiples of 32, at most one position per thread
    const int n_pos = pos + 1;
    const int piece = min(256, max(32, ((n_pos + kMhaCluster - 1) / kMhaCluster + 31) & ~31));
    // kv_smem (the host sets it when a block has one piece and it fits): the cached K and V rows of this block's
    // positions are fetched into shared memory by two bulk copies NOW, under the query rows, instead of by dependent
    // loads in the position loop.  The row of the current token is not among them when this launch writes it itself.
    unsigned char* kvs = reinterpret_cast<unsigned char*>(xs + d);
    const size_t row_b = static_cast<size_t>(dh) * sizeof(T);
    const int pf_first = r * piece;
    const int pf_valid = max(0, min(piece, n_pos - pf_first));
    int pf_rows = pf_valid;
    if (APPEND && pf_valid > 0 && pf_first + pf_valid - 1 == pos) pf_rows -= 1;
    const bool pf = kv_smem != 0 && pf_valid > 0;
    if (pf && tid == 0) { mbar_init(&kv_bar, 1); mbar_fence_init(); }
    __syncthreads();
    if (pf && tid == 0 && pf_rows > 0) {
        const uint32_t bytes = static_cast<uint32_t>(pf_rows * row_b);
        mbar_arrive_expect_tx(&kv_bar, 2u * bytes);
        bulk_copy_g2s(kvs, Kc + (static_cast<size_t>(h) * Lmax + pf_first) * dh, bytes, &kv_bar);
        bulk_copy_g2s(kvs + piece * row_b, Vc + (static_cast<size_t>(h) * Lmax + pf_first) * dh, bytes, &kv_bar);
    }
    const float scale = rsqrtf(static_cast<float>(dh));
    cluster_wait();                                      // every block of the cluster has started
    for (int i = 2 * warp; i < rows; i += 16) {
        float va, vb;
        if constexpr (I4) {
            const size_t row = (static_cast<size_t>(h) * 2 + 0) * dh + j0 + i;
            warp_two_rows_dot_i4(reinterpret_cast<const uint8_t*>(Wp), Sp, row, row + 1, d, xp, xsum, lane, va, vb);
        } else {
            const T* base = Wp + ((static_cast<size_t>(h) * 2 + 0) * dh + j0 + i) * d;
            warp_two_rows_dot(base, base + d, xs, chunks, lane, va, vb);
        }
        if (lane < kMhaCluster) {
            st_remote_f32(&q_s[j0 + i], lane, va * scale);
            st_remote_f32(&q_s[j0 + i + 1], lane, vb * scale);
        }
    }
    cluster_barrier();                                   // q_s complete everywhere

    // ---- this block's positions: pieces r, r + 8, r + 16, ... of 256 positions; running (m, l, o) ----
    float m_run = -INFINITY, l_run = 0.0f;
    const int col_groups = dh / E;                       // 16-byte groups per value row
    const int pos_groups = 256 / col_groups;             // threads per column group
    const int cg = tid % col_groups, pg = tid / col_groups;
    if (pf) {
        if (pf_rows > 0) {
            int never = 0;
            if (!mbar_wait_bounded(&kv_bar, 0u, &never) && tid == 0) flag_status(dev_status, HALO_DEV_TIMEOUT);
        }
        if (pf_rows < pf_valid) {
            // the current token's row, written by this cluster before the barrier above: 16 bytes per thread
            const int rl = pf_valid - 1;
            if (tid < 2 * col_groups) {
                const bool is_v = tid >= col_groups;
                const int c = is_v ? tid - col_groups : tid;
                const uint4* src = reinterpret_cast<const uint4*>((is_v ? Vc : Kc) + (static_cast<size_t>(h) * Lmax + pos) * dh) + c;
                reinterpret_cast<uint4*>(kvs + (is_v ? piece * row_b : 0) + rl * row_b)[c] = __ldcg(src);
            }
            __syncthreads();
        }
    }
    for (int p0 = r * piece; p0 < n_pos; p0 += kMhaCluster * piece) {
        const int p = p0 + tid;
        const bool valid = tid < piece && p < n_pos;
        float sc = -INFINITY;
        if (valid) {
            float acc = 0.0f;
            if (pf) {
                // a row per thread out of shared memory; the threads of a quarter warp start at different 16-byte groups
                const uint4* krow = reinterpret_cast<const uint4*>(kvs + tid * row_b);
#pragma unroll 8
                for (int c = 0; c < col_groups; ++c) {
                    int cc = c + tid;
                    cc -= (cc / col_groups) * col_groups;
                    float kf[E];
                    Elem<T>::widen(krow[cc], kf);
#pragma unroll
                    for (int e = 0; e < E; ++e) acc = fmaf(kf[e], q_s[cc * E + e], acc);
                }
            } else {
            const uint4* krow = reinterpret_cast<const uint4*>(Kc + (static_cast<size_t>(h) * Lmax + p) * dh);
#pragma unroll 8
            for (int c = 0; c < col_groups; ++c) {
                float kf[E];
                Elem<T>::widen(APPEND ? __ldcg(krow + c) : __ldg(krow + c), kf);
#pragma unroll
                for (int e = 0; e < E; ++e) acc = fmaf(kf[e], q_s[c * E + e], acc);
            }
            }
            sc = acc;
        }
        float m = sc;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) red[warp] = m;
        __syncthreads();
        m = red[0];
#pragma unroll
        for (int w = 1; w < 8; ++w) m = fmaxf(m, red[w]);
        const float m_new = fmaxf(m_run, m);             // finite: the piece holds at least one position
        const float keep_old = __expf(m_run - m_new);    // 0 on the first piece (m_run = -inf)
        const float e = valid ? __expf(sc - m_new) : 0.0f;
        w_s[tid] = e;
        float l = warp_sum(e);
        if (lane == 0) red[8 + warp] = l;
        for (int j = tid; j < dh; j += 256) o_acc[j] *= keep_old;
        __syncthreads();
        l = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) l += red[8 + w];
        l_run = l_run * keep_old + l;
        m_run = m_new;
        const int n_valid = min(piece, n_pos - p0);
        if (pg < pos_groups) {
            float part[E];
#pragma unroll
            for (int k = 0; k < E; ++k) part[k] = 0.0f;
            const uint4* vbase = pf ? reinterpret_cast<const uint4*>(kvs + piece * row_b) + cg
                                    : reinterpret_cast<const uint4*>(Vc + (static_cast<size_t>(h) * Lmax + p0) * dh) + cg;
#pragma unroll 8
            for (int pp = pg; pp < n_valid; pp += pos_groups) {
                float vf[E];
                const uint4* vp = vbase + static_cast<size_t>(pp) * col_groups;
                Elem<T>::widen(pf ? *vp : (APPEND ? __ldcg(vp) : __ldg(vp)), vf);
                const float wp = w_s[pp];
#pragma unroll
                for (int k = 0; k < E; ++k) part[k] = fmaf(wp, vf[k], part[k]);
            }
#pragma unroll
            for (int k = 0; k < E; ++k) atomicAdd(&o_acc[cg * E + k], part[k]);
        }
        __syncthreads();                                 // o_acc, w_s and red are free for the next piece
    }

    // ---- exchange: block r' gets (m, l) of this block and the o values of ITS rows ----
    if (tid < kMhaCluster) {
        st_remote_f32(&ml_in[r][0], tid, m_run);
        st_remote_f32(&ml_in[r][1], tid, l_run);
    }
    for (int j = tid; j < dh; j += 256) st_remote_f32(&o_in[r][j % rows], j / rows, o_acc[j]);
    cluster_barrier();                                   // the last remote access to anybody's shared memory
    if (tid < rows) {
        float M = -INFINITY;
#pragma unroll
        for (int c = 0; c < kMhaCluster; ++c) M = fmaxf(M, ml_in[c][0]);
        float L = 0.0f, o = 0.0f;
#pragma unroll
        for (int c = 0; c < kMhaCluster; ++c) {
            const float f = ml_in[c][1] > 0.0f ? __expf(ml_in[c][0] - M) : 0.0f;   // blocks without positions: 0
            L = fmaf(ml_in[c][1], f, L);
            o = fmaf(o_in[c][tid], f, o);
        }
        o_s[tid] = o / L;
    }
    __syncthreads();

    // ---- output-projection rows j0 .. j0 + rows of the head's slice: column sums into the holder's slot ----
    if constexpr (I4) {
        // a thread owns 8-byte code chunks (16 columns each); sums of f * (128 + nibble) with f = o_j * scale, and of f
        // alone, whose 136-fold is taken off at the end
        const int chunks8 = d / 16, nb = d / 128;
        const size_t row_bytes = static_cast<size_t>(d) / 2;
        const uint8_t* Qp = reinterpret_cast<const uint8_t*>(Wp);
        const size_t row0 = (static_cast<size_t>(h) * 2 + 1) * dh + j0;
        float acc4[ITERS][16], corr[ITERS];
#pragma unroll
        for (int i = 0; i < ITERS; ++i) {
            corr[i] = 0.0f;
#pragma unroll
            for (int k = 0; k < 16; ++k) acc4[i][k] = 0.0f;
        }
        constexpr int kRowsInFlight = ITERS == 1 ? 8 : 4;
        for (int jb = 0; jb < rows; jb += kRowsInFlight) {
            uint2 wv[kRowsInFlight][ITERS];
            float sv[kRowsInFlight][ITERS];
#pragma unroll
            for (int jj = 0; jj < kRowsInFlight; ++jj)
#pragma unroll
                for (int i = 0; i < ITERS; ++i) {
                    const int c = tid + 256 * i;
                    if (c < chunks8 && jb + jj < rows) {
                        const size_t rw = row0 + jb + jj;
                        wv[jj][i] = __ldg(reinterpret_cast<const uint2*>(Qp + rw * row_bytes) + c);
                        sv[jj][i] = __bfloat162float(Sp[rw * nb + (c >> 3)]);
                    } else {
                        wv[jj][i] = make_uint2(0u, 0u);
                        sv[jj][i] = 0.0f;
                    }
                }
#pragma unroll
            for (int jj = 0; jj < kRowsInFlight; ++jj) {
                const float o = jb + jj < rows ? o_s[jb + jj] : 0.0f;
#pragma unroll
                for (int i = 0; i < ITERS; ++i) {
                    const float f = o * sv[jj][i];               // 0 for the padded rows and columns
                    corr[i] += f;
                    const uint32_t words[2] = {wv[jj][i].x, wv[jj][i].y};
#pragma unroll
                    for (int v = 0; v < 2; ++v)
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const uint32_t p = nibble_pair_bf16(words[v], k);
                            acc4[i][8 * v + k] = fmaf(f, __uint_as_float(p << 16), acc4[i][8 * v + k]);
                            acc4[i][8 * v + k + 4] = fmaf(f, __uint_as_float(p & 0xffff0000u), acc4[i][8 * v + k + 4]);
                        }
                }
            }
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");       // the zero-fill of the slots (see below)
        float* dst4 = partials + static_cast<size_t>(slot) * d;
#pragma unroll
        for (int i = 0; i < ITERS; ++i) {
            const int c = tid + 256 * i;
            if (c < chunks8) {
                const float off = kNibbleBias * corr[i];
#pragma unroll
                for (int k = 0; k < 16; k += 4)
                    red_add_v4f(dst4 + c * 16 + k, acc4[i][k] - off, acc4[i][k + 1] - off, acc4[i][k + 2] - off,
                                acc4[i][k + 3] - off);
            }
        }
    } else {
    float acc[ITERS][E];
#pragma unroll
    for (int i = 0; i < ITERS; ++i)
#pragma unroll
        for (int k = 0; k < E; ++k) acc[i][k] = 0.0f;
    const T* wrows = Wp + ((static_cast<size_t>(h) * 2 + 1) * dh + j0) * d;
    constexpr int kAtOnce = ITERS <= 2 ? 8 : 4;          // rows whose 16-byte pieces a thread has in flight
    for (int jb = 0; jb < rows; jb += kAtOnce) {
        uint4 wv[kAtOnce][ITERS];
#pragma unroll
        for (int jj = 0; jj < kAtOnce; ++jj)
#pragma unroll
            for (int i = 0; i < ITERS; ++i) {
                const int c = tid + 256 * i;
                wv[jj][i] = (c < chunks && jb + jj < rows)
                                ? ldg_stream16(reinterpret_cast<const uint4*>(wrows + static_cast<size_t>(jb + jj) * d) + c)
                                : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
        for (int jj = 0; jj < kAtOnce; ++jj) {
            const float o = jb + jj < rows ? o_s[jb + jj] : 0.0f;
#pragma unroll
            for (int i = 0; i < ITERS; ++i) {
                const int c = tid + 256 * i;
                if (c < chunks) {
                    float w8[E];
                    Elem<T>::widen(wv[jj][i], w8);
#pragma unroll
                    for (int k = 0; k < E; ++k) acc[i][k] = fmaf(o, w8[k], acc[i][k]);
                }
            }
        }
    }
    // the zero-fill of the slots may still be running when this kernel was launched as its programmatic dependent
    if constexpr (APPEND) asm volatile("griddepcontrol.wait;" ::: "memory");
    float* dst = partials + static_cast<size_t>(slot) * d;
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
        const int c = tid + 256 * i;
        if (c < chunks) {
#pragma unroll
            for (int k = 0; k < E; k += 4) red_add_v4f(dst + c * E + k, acc[i][k], acc[i][k + 1], acc[i][k + 2], acc[i][k + 3]);
        }
    }
    }
}

template <typename T>
__global__ void mha_pack_kernel(int d, int H, int dh, const T* __restrict__ Wq, const T* __restrict__ Wo, T* __restrict__ Wp) {
    const size_t n = static_cast<size_t>(H) * dh * d;
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= n) return;
    const int row = static_cast<int>(idx / d), c = static_cast<int>(idx % d);
    const int h = row / dh, j = row % dh;
    Wp[((static_cast<size_t>(h) * 2 + 0) * dh + j) * d + c] = Wq[idx];
    Wp[((static_cast<size_t>(h) * 2 + 1) * dh + j) * d + c] = Wo[static_cast<size_t>(c) * H * dh + row];
}

}  // namespace halo

using namespace halo;

namespace {
halo_status check_mha_shape(const halo_mha_shape* s) {
    if (!s) return HALO_ERR_ARG;
    if (s->wdtype != HALO_F32 && s->wdtype != HALO_BF16) return HALO_ERR_DTYPE;
    if (s->d_model <= 0 || s->d_model % 8 != 0 || s->d_model > 8192 || s->n_heads <= 0 ||
        s->n_heads > HALO_MAX_GROUPS || s->max_len <= 0)
        return HALO_ERR_SHAPE;
    if (s->head_dim < kOutRows || s->head_dim > 256 || s->head_dim % kOutRows != 0) return HALO_ERR_SHAPE;
    const int per_chunk = s->wdtype == HALO_F32 ? 4 : 8;
    if (s->d_model / per_chunk > 1024) return HALO_ERR_SHAPE;
    return HALO_OK;
}
}  // namespace

extern "C" halo_status halo_pack_mha_weights(const halo_mha_shape* shape, const void* Wq, const void* Wo, void* W_packed,
                                             void* stream) {
    halo_status rc = check_mha_shape(shape);
    if (rc != HALO_OK) return rc;
    if (!Wq || !Wo || !W_packed) return HALO_ERR_ARG;
    const size_t n = static_cast<size_t>(shape->n_heads) * shape->head_dim * shape->d_model;
    const unsigned blocks = static_cast<unsigned>((n + 255) / 256);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (shape->wdtype == HALO_BF16)
        mha_pack_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(shape->d_model, shape->n_heads, shape->head_dim,
                                                               static_cast<const __nv_bfloat16*>(Wq),
                                                               static_cast<const __nv_bfloat16*>(Wo),
                                                               static_cast<__nv_bfloat16*>(W_packed));
    else
        mha_pack_kernel<float><<<blocks, 256, 0, st>>>(shape->d_model, shape->n_heads, shape->head_dim,
                                                       static_cast<const float*>(Wq), static_cast<const float*>(Wo),
                                                       static_cast<float*>(W_packed));
    return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}

extern "C" halo_status halo_mha_kv_append(const halo_mha_shape* shape, const void* Wk, const void* Wv, const void* x,
                                          int pos, void* K_cache, void* V_cache, void* stream) {
    halo_status rc = check_mha_shape(shape);
    if (rc != HALO_OK) return rc;
    if (!Wk || !Wv || !x || !K_cache || !V_cache) return HALO_ERR_ARG;
    if (pos < 0 || pos >= shape->max_len) return HALO_ERR_ARG;
    if (!aligned16(Wk) || !aligned16(Wv) || !aligned16(x) || !aligned16(K_cache) || !aligned16(V_cache)) return HALO_ERR_ALIGN;
    const int d = shape->d_model, H = shape->n_heads, dh = shape->head_dim;
    const unsigned blocks = static_cast<unsigned>((2 * H * dh + kRowsPerBlock - 1) / kRowsPerBlock);
    const size_t smem = sizeof(float) * d;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (shape->wdtype == HALO_BF16)
        mha_kv_append_kernel<__nv_bfloat16><<<blocks, 256, smem, st>>>(
            d, H, dh, shape->max_len, static_cast<const __nv_bfloat16*>(Wk), static_cast<const __nv_bfloat16*>(Wv),
            static_cast<const __nv_bfloat16*>(x), pos, static_cast<__nv_bfloat16*>(K_cache),
            static_cast<__nv_bfloat16*>(V_cache));
    else
        mha_kv_append_kernel<float><<<blocks, 256, smem, st>>>(d, H, dh, shape->max_len, static_cast<const float*>(Wk),
                                                               static_cast<const float*>(Wv), static_cast<const float*>(x),
                                                               pos, static_cast<float*>(K_cache),
                                                               static_cast<float*>(V_cache));
    return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}

extern "C" size_t halo_group_mha_workspace_bytes(const halo_mha_shape* shape) {
    if (check_mha_shape(shape) != HALO_OK) return 0;
    const size_t H = shape->n_heads, dh = shape->head_dim;
    const size_t chunks = (static_cast<size_t>(shape->max_len) + kAttnChunk - 1) / kAttnChunk;
    return sizeof(float) * (H * dh + H * chunks * (dh + 2));
}

template <typename T>
static halo_status group_mha_typed(const halo_mha_shape& sh, const void* Wp, const void* x, const void* Kc, const void* Vc,
                                   int pos, const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group,
                                   int n_dev, float* partials, float* ws, uint32_t* dev_status, cudaStream_t st) {
    constexpr int E = Elem<T>::kPerChunk;
    const int d = sh.d_model, H = sh.n_heads, dh = sh.head_dim;
    float* q_ws = ws;
    float* attn_ws = ws + static_cast<size_t>(H) * dh;
    const int n_chunks = pos / kAttnChunk + 1;
    if (cudaMemsetAsync(partials, 0, sizeof(float) * static_cast<size_t>(n_dev + 1) * d, st) != cudaSuccess) return HALO_ERR_CUDA;
    const bool three_launches = option_value(OPT_MHA_THREE_LAUNCHES) == 1;
    if (!three_launches) {
        // one launch: a cluster of eight thread blocks per kept head
        const int iters_f = (d / E + 255) / 256;
        const dim3 grid_f(kMhaCluster, H);
        const size_t kv_b = kv_smem_bytes(pos, dh, sizeof(T));
        const size_t smem_f = sizeof(float) * d + kv_b;
#define HALO_MHA_FUSED(I)                                                                                            \
    case I: {                                                                                                        \
        static bool once[64] = {};                                                                                   \
        if (!ensure_dynamic_smem(mha_fused_kernel<T, I, false>, kMhaSmemLimit, once)) return HALO_ERR_CUDA; \
        mha_fused_kernel<T, I, false><<<grid_f, 256, smem_f, st>>>(                                                   \
            d, H, dh, sh.max_len, pos, static_cast<const T*>(Wp), static_cast<const T*>(x), static_cast<const T*>(Kc), \
            static_cast<const T*>(Vc), keep_list, n_keep, dev_of_group, n_dev, partials, dev_status, nullptr, nullptr,  \
            nullptr, nullptr, kv_b ? 1 : 0);                                                                         \
        break;                                                                                                       \
    }
        switch (iters_f) {
            HALO_MHA_FUSED(1)
            HALO_MHA_FUSED(2)
            HALO_MHA_FUSED(3)
            HALO_MHA_FUSED(4)
            default: return HALO_ERR_SHAPE;
        }
#undef HALO_MHA_FUSED
        HALO_CHECK_LAUNCH();
        return HALO_OK;
    }
    mha_q_kernel<T><<<(H * dh + kRowsPerBlock - 1) / kRowsPerBlock, 256, sizeof(float) * d, st>>>(d, H, dh, static_cast<const T*>(Wp),
                                                                      static_cast<const T*>(x), keep_list, n_keep, q_ws,
                                                                      dev_status);
    HALO_CHECK_LAUNCH();
    mha_attn_kernel<T><<<dim3(H, n_chunks), kAttnChunk, 0, st>>>(H, dh, sh.max_len, pos, static_cast<const T*>(Kc),
                                                                 static_cast<const T*>(Vc), keep_list, n_keep, q_ws,
                                                                 attn_ws, n_chunks);
    HALO_CHECK_LAUNCH();
    const int iters = (d / E + 255) / 256;
    const dim3 grid(H, dh / kOutRows);
#define HALO_MHA_OUT(I)                                                                                              \
    case I:                                                                                                          \
        mha_out_kernel<T, I><<<grid, 256, 0, st>>>(d, H, dh, static_cast<const T*>(Wp), keep_list, n_keep, dev_of_group, \
                                                   n_dev, attn_ws, n_chunks, partials, dev_status);                   \
        break;
    switch (iters) {
        HALO_MHA_OUT(1)
        HALO_MHA_OUT(2)
        HALO_MHA_OUT(3)
        HALO_MHA_OUT(4)
        default: return HALO_ERR_SHAPE;
    }
#undef HALO_MHA_OUT
    HALO_CHECK_LAUNCH();
    return HALO_OK;
}

extern "C" halo_status halo_group_mha(const halo_mha_shape* shape, const void* W_packed, const void* x,
                                      const void* K_cache, const void* V_cache, int pos, const int32_t* keep_list,
                                      const int32_t* n_keep, const int32_t* dev_of_group, int n_dev, float* partials,
                                      void* workspace, size_t workspace_bytes, uint32_t* dev_status, void* stream) {
    halo_status rc = check_mha_shape(shape);
    if (rc != HALO_OK) return rc;
    if (!W_packed || !x || !K_cache || !V_cache || !keep_list || !n_keep || !partials) return HALO_ERR_ARG;
    if (pos < 0 || pos >= shape->max_len) return HALO_ERR_ARG;
    if (n_dev < 0 || n_dev > HALO_MAX_DEVICES || (!dev_of_group && n_dev != 0)) return HALO_ERR_ARG;
    if (!aligned16(W_packed) || !aligned16(x) || !aligned16(K_cache) || !aligned16(V_cache) || !aligned16(partials) ||
        !aligned16(workspace))
        return HALO_ERR_ALIGN;
    if (!workspace || workspace_bytes < halo_group_mha_workspace_bytes(shape)) return HALO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* ws = static_cast<float*>(workspace);
    if (shape->wdtype == HALO_BF16)
        return group_mha_typed<__nv_bfloat16>(*shape, W_packed, x, K_cache, V_cache, pos, keep_list, n_keep, dev_of_group,
                                              n_dev, partials, ws, dev_status, st);
    return group_mha_typed<float>(*shape, W_packed, x, K_cache, V_cache, pos, keep_list, n_keep, dev_of_group, n_dev,
                                  partials, ws, dev_status, st);
}

template <typename T>
static halo_status mha_block_typed(const halo_mha_shape& sh, const void* Wp, const void* Wk, const void* Wv, const void* x,
                                   void* Kc, void* Vc, int pos, const int32_t* keep_list, const int32_t* n_keep,
                                   const int32_t* dev_of_group, int n_dev, float* partials, uint32_t* dev_status,
                                   cudaStream_t st, bool already_zero) {
    constexpr int E = Elem<T>::kPerChunk;
    const int d = sh.d_model, H = sh.n_heads, dh = sh.head_dim;
    // the zero-fill releases this launch at once: the row products and the attention run under it
    if (!already_zero && launch_zero_partials(partials, static_cast<size_t>(n_dev + 1) * d, st) != HALO_OK) return HALO_ERR_CUDA;
    const int iters = (d / E + 255) / 256;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(kMhaCluster, H);
    cfg.blockDim = dim3(256);
    const size_t kv_b = kv_smem_bytes(pos, dh, sizeof(T));
    cfg.dynamicSmemBytes = sizeof(float) * d + kv_b;
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = already_zero ? 0 : 1;
    const T* Wp_t = static_cast<const T*>(Wp); const T* x_t = static_cast<const T*>(x);
    const T* Kc_t = static_cast<const T*>(Kc); const T* Vc_t = static_cast<const T*>(Vc);
    const T* Wk_t = static_cast<const T*>(Wk); const T* Wv_t = static_cast<const T*>(Wv);
    T* Kw_t = static_cast<T*>(Kc); T* Vw_t = static_cast<T*>(Vc);
    const int Lmax = sh.max_len;
    cudaError_t err = cudaSuccess;
    const int kv_flag = kv_b ? 1 : 0;
    const __nv_bfloat16* no_scales = nullptr;
#define HALO_MHA_BLOCK(I)                                                                                            \
    case I: {                                                                                                        \
        static bool once[64] = {};                                                                                   \
        if (!ensure_dynamic_smem(mha_fused_kernel<T, I, true>, kMhaSmemLimit, once)) return HALO_ERR_CUDA; \
        err = cudaLaunchKernelEx(&cfg, mha_fused_kernel<T, I, true>, d, H, dh, Lmax, pos, Wp_t, x_t, Kc_t, Vc_t,      \
                                 keep_list, n_keep, dev_of_group, n_dev, partials, dev_status, Wk_t, Wv_t, Kw_t, Vw_t, \
                                 kv_flag, no_scales, no_scales, no_scales);                                           \
        break;                                                                                                       \
    }
    switch (iters) {
        HALO_MHA_BLOCK(1)
        HALO_MHA_BLOCK(2)
        HALO_MHA_BLOCK(3)
        HALO_MHA_BLOCK(4)
        default: return HALO_ERR_SHAPE;
    }
#undef HALO_MHA_BLOCK
    return err == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}

// The fused block on int4 weights (activations and caches bf16).
halo_status halo::launch_mha_block_i4(const halo_mha_shape& sh, const void* Qp, const void* Sp, const void* Qk, const void* Sk,
                                      const void* Qv, const void* Sv, const void* x, void* Kc, void* Vc, int pos,
                                      const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group, int n_dev,
                                      float* partials, uint32_t* dev_status, cudaStream_t st, bool already_zero) {
    using T = __nv_bfloat16;
    const int d = sh.d_model, H = sh.n_heads, dh = sh.head_dim;
    if (!already_zero && launch_zero_partials(partials, static_cast<size_t>(n_dev + 1) * d, st) != HALO_OK) return HALO_ERR_CUDA;
    const int iters = (d / 16 + 255) / 256;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(kMhaCluster, H);
    cfg.blockDim = dim3(256);
    const size_t kv_b = kv_smem_bytes(pos, dh, sizeof(T));
    cfg.dynamicSmemBytes = sizeof(float) * d + kv_b;
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = already_zero ? 0 : 1;
    const T* Wp_t = static_cast<const T*>(Qp); const T* x_t = static_cast<const T*>(x);
    const T* Kc_t = static_cast<const T*>(Kc); const T* Vc_t = static_cast<const T*>(Vc);
    const T* Wk_t = static_cast<const T*>(Qk); const T* Wv_t = static_cast<const T*>(Qv);
    T* Kw_t = static_cast<T*>(Kc); T* Vw_t = static_cast<T*>(Vc);
    const T* Sp_t = static_cast<const T*>(Sp); const T* Sk_t = static_cast<const T*>(Sk); const T* Sv_t = static_cast<const T*>(Sv);
    const int Lmax = sh.max_len, kv_flag = kv_b ? 1 : 0;
    cudaError_t err = cudaSuccess;
#define HALO_MHA_BLOCK_I4(I)                                                                                         \
    case I: {                                                                                                        \
        static bool once[64] = {};                                                                                   \
        if (!ensure_dynamic_smem(mha_fused_kernel<T, I, true, true>, kMhaSmemLimit, once)) return HALO_ERR_CUDA;      \
        err = cudaLaunchKernelEx(&cfg, mha_fused_kernel<T, I, true, true>, d, H, dh, Lmax, pos, Wp_t, x_t, Kc_t, Vc_t, \
                                 keep_list, n_keep, dev_of_group, n_dev, partials, dev_status, Wk_t, Wv_t, Kw_t, Vw_t, \
                                 kv_flag, Sp_t, Sk_t, Sv_t);                                                          \
        break;                                                                                                       \
    }
    switch (iters) {
        HALO_MHA_BLOCK_I4(1)
        HALO_MHA_BLOCK_I4(2)
        default: return HALO_ERR_SHAPE;
    }
#undef HALO_MHA_BLOCK_I4
    return err == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}

halo_status halo::launch_mha_block(const halo_mha_shape& sh, const void* W_packed, const void* Wk, const void* Wv, const void* x,
                                   void* K_cache, void* V_cache, int pos, const int32_t* keep_list, const int32_t* n_keep,
                                   const int32_t* dev_of_group, int n_dev, float* partials, uint32_t* dev_status,
                                   cudaStream_t st, bool already_zero) {
    if (sh.wdtype == HALO_BF16)
        return mha_block_typed<__nv_bfloat16>(sh, W_packed, Wk, Wv, x, K_cache, V_cache, pos, keep_list, n_keep, dev_of_group,
                                              n_dev, partials, dev_status, st, already_zero);
    return mha_block_typed<float>(sh, W_packed, Wk, Wv, x, K_cache, V_cache, pos, keep_list, n_keep, dev_of_group, n_dev,
                                  partials, dev_status, st, already_zero);
}

extern "C" halo_status halo_mha_block(const halo_mha_shape* shape, const void* W_packed, const void* Wk, const void* Wv,
                                      const void* x, void* K_cache, void* V_cache, int pos, const int32_t* keep_list,
                                      const int32_t* n_keep, const int32_t* dev_of_group, int n_dev, float* partials,
                                      uint32_t* dev_status, void* stream) {
    halo_status rc = check_mha_shape(shape);
    if (rc != HALO_OK) return rc;
    if (!W_packed || !Wk || !Wv || !x || !K_cache || !V_cache || !keep_list || !n_keep || !partials) return HALO_ERR_ARG;
    if (pos < 0 || pos >= shape->max_len) return HALO_ERR_ARG;
    if (n_dev < 0 || n_dev > HALO_MAX_DEVICES || (!dev_of_group && n_dev != 0)) return HALO_ERR_ARG;
    if (shape->head_dim % (2 * kMhaCluster) != 0) return HALO_ERR_SHAPE;
    if (!aligned16(W_packed) || !aligned16(Wk) || !aligned16(Wv) || !aligned16(x) || !aligned16(K_cache) ||
        !aligned16(V_cache) || !aligned16(partials))
        return HALO_ERR_ALIGN;
    return halo::launch_mha_block(*shape, W_packed, Wk, Wv, x, K_cache, V_cache, pos, keep_list, n_keep, dev_of_group, n_dev,
                                  partials, dev_status, static_cast<cudaStream_t>(stream), false);
}

extern "C" halo_status halo_mha_block_i4(const halo_mha_shape* shape, const void* Qp, const void* Sp, const void* Qk,
                                         const void* Sk, const void* Qv, const void* Sv, const void* x, void* K_cache,
                                         void* V_cache, int pos, const int32_t* keep_list, const int32_t* n_keep,
                                         const int32_t* dev_of_group, int n_dev, float* partials, uint32_t* dev_status,
                                         void* stream) {
    halo_status rc = check_mha_shape(shape);
    if (rc != HALO_OK) return rc;
    if (!Qp || !Sp || !Qk || !Sk || !Qv || !Sv || !x || !K_cache || !V_cache || !keep_list || !n_keep || !partials)
        return HALO_ERR_ARG;
    if (pos < 0 || pos >= shape->max_len) return HALO_ERR_ARG;
    if (n_dev < 0 || n_dev > HALO_MAX_DEVICES || (!dev_of_group && n_dev != 0)) return HALO_ERR_ARG;
    if (shape->wdtype != HALO_BF16) return HALO_ERR_DTYPE;                 // activations and caches
    if (shape->head_dim % (2 * kMhaCluster) != 0 || shape->d_model % 128 != 0) return HALO_ERR_SHAPE;
    if (!aligned16(Qp) || !aligned16(Sp) || !aligned16(Qk) || !aligned16(Sk) || !aligned16(Qv) || !aligned16(Sv) ||
        !aligned16(x) || !aligned16(K_cache) || !aligned16(V_cache) || !aligned16(partials))
        return HALO_ERR_ALIGN;
    return halo::launch_mha_block_i4(*shape, Qp, Sp, Qk, Sk, Qv, Sv, x, K_cache, V_cache, pos, keep_list, n_keep, dev_of_group,
                                     n_dev, partials, dev_status, static_cast<cudaStream_t>(stream), false);
}
