// halo_group_ffn, prefill form (many tokens, bf16): the masked FFN as dense contractions on the tensor cores.
//
//   GEMM-1  for every kept group g (one CTA tile per 128 tokens x one group):
//             Dg = X * Wgate_g^T,  Du = X * Wup_g^T      two fp32 accumulators in TMEM (tcgen05.mma, kind::f16)
//             H[:, kept position of g] = bf16( silu(Dg) * Du )          epilogue straight from TMEM
//   GEMM-2  for every 128-token x 128-column output tile, holder slot by holder slot:
//             partials[slot] = H[:, groups of the slot] * down rows of those groups      (fp32 out)
//           The down rows are read as stored in the packed layout (plane 2: one row of d per neuron), i.e. as an
//           MN-major B operand; no second copy of the weights.
// Operands reach shared memory by tensor-map TMA (128-byte swizzle, no multicast); kept groups are gathered by
// choosing the TMA row coordinate from keep_list, so skipped groups are never read.  Warp roles: warp 0 TMA
// producer, warp 1 MMA issuer (+ TMEM allocation), warps 2..5 epilogue.  All mbarrier waits are bounded; on a
// timeout the CTA stops waiting, skips its stores, flags HALO_DEV_TIMEOUT, drains its copies and frees TMEM.
#include <algorithm>
#include <mutex>

#include "common.cuh"
#include "ffn_math.cuh"
#include "prompt_stack.cuh"
#include "umma.cuh"

namespace halo {

constexpr int kBM = 128;          // tokens per tile
constexpr int kBK = 64;           // K elements per stage (128 bytes of bf16)
constexpr int kUmmaK = 16;
constexpr int kPfThreads = 192;   // 6 warps
constexpr int kEpiPitch = 36;     // floats per staged accumulator row: 32 + 4 keeps 16-byte accesses conflict-free
constexpr size_t kEpiStageBytes = 4 * 32 * kEpiPitch * sizeof(float);   // one 32 x 32 chunk per epilogue warp

struct PfBarriers {
    uint64_t full[8];
    uint64_t empty[8];
    uint64_t tmem_full;
    uint64_t tmem_empty;
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ bool pf_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    if (*abort_flag) return false;
    if (mbar_wait_bounded(bar, parity, abort_flag)) return true;
    *abort_flag = 1;
    return false;
}

// ------------------------------------------------------------------------------------------------------------
// GEMM-1: hidden activations of one kept group for one tile of tokens
// ------------------------------------------------------------------------------------------------------------
// MH = 128-token halves per tile (1 or 2).  With MH = 2 the group's gate and up rows staged for a K-step serve 256
// tokens: twice the FLOP per staged byte, four fp32 accumulators = all 512 TMEM columns at NS = 128.
template <int NS, int MH, int STAGES>
__global__ void __launch_bounds__(kPfThreads, 1)
ffn_hidden_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                  const __grid_constant__ CUtensorMap tmap_w_half, int T, int d, int S, int G, int n_sm,
                  const int32_t* __restrict__ keep_list, const int32_t* __restrict__ n_keep_ptr,
                  __nv_bfloat16* __restrict__ H, int h_cols, uint32_t* dev_status) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    constexpr uint32_t kAHalf = kBM * kBK * 2, kABytes = MH * kAHalf, kBBytes = NS * kBK * 2;
    constexpr uint32_t kStageBytes = kABytes + 2 * kBBytes;
    constexpr uint32_t kTmemCols = MH * 2 * NS;
    PfBarriers& bars = *reinterpret_cast<PfBarriers*>(smem_raw + static_cast<size_t>(STAGES) * kStageBytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // A group of S neurons is computed as S / NS tiles of NS neurons: blockIdx.y counts (kept position, tile).
    const int subs = S / NS;
    const int kv = blockIdx.y, ki = kv / subs, m0 = blockIdx.x * (kBM * MH);
    int nk = *n_keep_ptr;
    nk = max(0, min(nk, G));
    if (ki >= nk) return;
    // Tail balancing: the tiles that fill whole waves of SMs are computed in full (blockIdx.z == 0); those left
    // for the last, partial wave are split into two half-width tiles (blockIdx.z = which half), when those halves
    // fit in one wave, so the tail takes about half a tile's time.
    int n_full = nk * subs;
    {
        const int tiles_x = gridDim.x, total = tiles_x * nk * subs;
        if (total > n_sm) {
            const int full_tiles = (total / n_sm) * n_sm / tiles_x, left = nk * subs - full_tiles;
            if (left > 0 && 2 * left * tiles_x <= n_sm) n_full = full_tiles;
        }
    }
    const bool split = kv >= n_full;
    if (!split && blockIdx.z != 0) return;
    const int ns = split ? NS / 2 : NS;                // neurons of the group this CTA computes
    const int n_off = (kv - ki * subs) * NS + (split ? blockIdx.z * (NS / 2) : 0);   // first of them in the group
    const CUtensorMap* const map_w = split ? &tmap_w_half : &tmap_w;
    const int g = keep_list[ki];
    if (g < 0 || g >= G) {
        if (tid == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
        return;
    }
    const int n_kt = d / kBK;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&bars.full[s], 1); mbar_init(&bars.empty[s], 1); }
        mbar_init(&bars.tmem_full, 1);
        mbar_init(&bars.tmem_empty, 1);
        bars.abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_descriptor(&tmap_x);
        tma_prefetch_descriptor(map_w);
    }
    if (warp == 1) { tmem_alloc(&bars.tmem_base, kTmemCols); tmem_relinquish_alloc_permit(); }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    volatile int* abort_flag = &bars.abort_flag;
    const uint32_t tmem = bars.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            for (int kt = 0; kt < n_kt; ++kt) {
                const int s = kt % STAGES;
                if (kt >= STAGES && !pf_wait(&bars.empty[s], ((kt / STAGES) - 1) & 1, abort_flag)) break;
                unsigned char* st = smem_raw + static_cast<size_t>(s) * kStageBytes;
                mbar_arrive_expect_tx(&bars.full[s], kABytes + 2u * static_cast<uint32_t>(ns) * kBK * 2u);
#pragma unroll
                for (int mh = 0; mh < MH; ++mh)   // rows beyond T read as zeros
                    tma_load_2d(st + mh * kAHalf, &tmap_x, kt * kBK, m0 + mh * kBM, &bars.full[s]);
                // gate rows, then the up rows directly behind them: one B operand of 2 * ns rows
                tma_load_2d(st + kABytes, map_w, kt * kBK, (g * 3 + 0) * S + n_off, &bars.full[s]);
                tma_load_2d(st + kABytes + ns * (kBK * 2), map_w, kt * kBK, (g * 3 + 1) * S + n_off, &bars.full[s]);
                issued = kt + 1;
            }
            if (*abort_flag) {  // let outstanding copies land before the CTA goes away
                int never = 0;
                for (int kt = max(0, issued - STAGES); kt < issued; ++kt)
                    mbar_wait_bounded(&bars.full[kt % STAGES], (kt / STAGES) & 1, &never);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // one MMA of N = 2 * ns per token half: accumulator columns [0, ns) = gate, [ns, 2 ns) = up.  The wide
            // N keeps the A tile's shared-memory reads per FLOP low.
            const uint32_t idesc = umma_idesc_bf16(kBM, 2 * ns, false);
            for (int kt = 0; kt < n_kt; ++kt) {
                const int s = kt % STAGES;
                if (!pf_wait(&bars.full[s], (kt / STAGES) & 1, abort_flag)) break;
                tcgen05_fence_after_sync();
                const uint32_t a0 = smem_u32(smem_raw + static_cast<size_t>(s) * kStageBytes);
#pragma unroll
                for (int kk = 0; kk < kBK / kUmmaK; ++kk) {
                    const uint64_t b = umma_smem_desc(a0 + kABytes + kk * 32, 16, 1024);
                    const bool accumulate = (kt > 0) || (kk > 0);
#pragma unroll
                    for (int mh = 0; mh < MH; ++mh) {
                        const uint64_t a = umma_smem_desc(a0 + mh * kAHalf + kk * 32, 16, 1024);
                        umma_bf16(tmem + mh * 2 * NS, a, b, idesc, accumulate);
                    }
                }
                umma_commit(&bars.empty[s]);   // the stage is free once these MMAs have read it
            }
            umma_commit(&bars.tmem_full);
        }
    } else {
        // epilogue: this warp reads TMEM lanes [32*(warp%4), +32) = 32 tokens of each half, one token per thread
        const bool ok = pf_wait(&bars.tmem_full, 0, abort_flag);
        tcgen05_fence_after_sync();
        const int quad = warp & 3;
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(quad * 32) << 16);
#pragma unroll
        for (int mh = 0; mh < MH; ++mh) {
            const int row = m0 + mh * kBM + quad * 32 + lane;
            for (int c0 = 0; c0 < ns; c0 += 32) {
                uint32_t dg[32], du[32];
                tmem_ld_32x32(lane_base + mh * 2 * NS + c0, dg);
                tmem_ld_32x32(lane_base + mh * 2 * NS + ns + c0, du);
                tmem_ld_wait();
                if (ok && row < T) {
                    uint4* dst = reinterpret_cast<uint4*>(H + static_cast<size_t>(row) * h_cols +
                                                          static_cast<size_t>(ki) * S + n_off + c0);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t packed[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int i = q * 8 + e * 2;
                            const float h0 = silu_mul(__uint_as_float(dg[i]), __uint_as_float(du[i]));
                            const float h1 = silu_mul(__uint_as_float(dg[i + 1]), __uint_as_float(du[i + 1]));
                            const __nv_bfloat162 p = __floats2bfloat162_rn(h0, h1);
                            packed[e] = *reinterpret_cast<const uint32_t*>(&p);
                        }
                        dst[q] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                    }
                }
            }
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tcgen05_fence_after_sync(); tmem_dealloc(tmem, kTmemCols); }
    if (tid == 0 && *abort_flag) flag_status(dev_status, HALO_DEV_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------------------
// GEMM-2: down projection of the kept columns, one accumulation per holder slot
// ------------------------------------------------------------------------------------------------------------
struct DownSmemTail {
    PfBarriers bars;
    uint64_t acc_full[2];                 // accumulator b holds a finished slot
    uint64_t acc_empty[2];                // accumulator b has been drained by the epilogue
    int slot_lo, slot_hi;                 // holder slots this CTA accumulates (the K range is split by slot)
    int slot_start[HALO_MAX_DEVICES + 2];
    int32_t group_of[HALO_MAX_GROUPS];    // group id per position of the slot-sorted order (-1 = skip)
    int16_t kept_pos[HALO_MAX_GROUPS];    // kept position (column block of H) per position of the order
};

// Kept positions sorted by holder slot (stable), by one warp with ballot compaction per slot.  Slots above
// `slot_cap` are folded into slot_cap.  Fills slot_start[0 .. n_slots), group_of and kept_pos; returns the number of
// valid kept positions.
__device__ __forceinline__ int build_slot_order(DownSmemTail& tail, int nk, int G, int n_dev, int n_slots, int slot_cap,
                                                const int32_t* __restrict__ keep_list,
                                                const int32_t* __restrict__ dev_of_group, uint32_t* dev_status,
                                                int lane) {
    int pos = 0;
    for (int slot = 0; slot < n_slots; ++slot) {
        if (lane == 0) tail.slot_start[slot] = pos;
        for (int base = 0; base < nk; base += 32) {
            const int ki = base + lane;
            int g = -1, sl = -1;
            if (ki < nk) {
                g = keep_list[ki];
                if (g >= 0 && g < G) sl = dev_of_group ? dev_of_group[g] + 1 : 0;
                if (sl < 0 || sl > n_dev) { sl = -1; if (slot == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX); }
                else if (sl > slot_cap) sl = slot_cap;
            }
            const bool match = (sl == slot);
            const unsigned ballot = __ballot_sync(0xffffffffu, match);
            if (match) {
                const int p = pos + __popc(ballot & ((1u << lane) - 1u));
                tail.group_of[p] = g;
                tail.kept_pos[p] = static_cast<int16_t>(ki);
            }
            pos += __popc(ballot);
        }
    }
    return pos;
}

// BN2 output columns per tile.  gridDim.z CTAs share an output tile position but take disjoint ranges of holder
// slots: the slots are separate outputs, so splitting K at a slot boundary needs no reduction.
template <int BN2, int STAGES>
__global__ void __launch_bounds__(kPfThreads, 1)
ffn_down_kernel(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_wd, int T, int d,
                int S, int G, const int32_t* __restrict__ keep_list, const int32_t* __restrict__ n_keep_ptr,
                const int32_t* __restrict__ dev_of_group, int n_dev, int collapse, float* __restrict__ partials,
                uint32_t* dev_status) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    constexpr uint32_t kABytes = kBM * kBK * 2, kBBytes = kBK * BN2 * 2, kStageBytes = kABytes + kBBytes;
    constexpr uint32_t kBBlock = kBK * 64 * 2;   // one 64-column block of B: 64 K-rows x 128 B
    DownSmemTail& tail = *reinterpret_cast<DownSmemTail*>(smem_raw + static_cast<size_t>(STAGES) * kStageBytes);
    PfBarriers& bars = tail.bars;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * kBM, n0 = blockIdx.y * BN2;
    int nk = *n_keep_ptr;
    nk = max(0, min(nk, G));
    const int k_per_group = S / kBK;   // K stages per kept group
    // collapse: only two output slots, 0 = groups of the master, 1 = groups of any device (the caller wants the
    // merged sum only and every listed group has arrived); still two slots so that K can be split over two CTAs
    const int n_slots = collapse ? 2 : n_dev + 1;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&bars.full[s], 1); mbar_init(&bars.empty[s], 1); }
        mbar_init(&bars.tmem_full, 1);
        mbar_init(&bars.tmem_empty, 4);
        for (int b = 0; b < 2; ++b) { mbar_init(&tail.acc_full[b], 1); mbar_init(&tail.acc_empty[b], 4); }
        bars.abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_descriptor(&tmap_h);
        tma_prefetch_descriptor(&tmap_wd);
    }
    // two accumulators: the MMAs of the next slot run while the epilogue drains the previous one
    if (warp == 1) { tmem_alloc(&bars.tmem_base, 2 * BN2); tmem_relinquish_alloc_permit(); }
    if (warp == 0) {
        const int pos = build_slot_order(tail, nk, G, n_dev, n_slots, collapse ? 1 : n_dev, keep_list, dev_of_group,
                                         dev_status, lane);
        if (lane == 0) {
            tail.slot_start[n_slots] = pos;
            // this CTA's share of the slots: cut at the slot boundary nearest to half of the kept groups
            int lo = 0, hi = n_slots;
            if (gridDim.z == 2) {
                int cut = n_slots, best = pos + 1;
                for (int sl = 1; sl < n_slots; ++sl) {
                    const int dist = abs(2 * tail.slot_start[sl] - pos);
                    if (dist < best) { best = dist; cut = sl; }
                }
                if (blockIdx.z == 0) hi = cut; else lo = cut;
            }
            tail.slot_lo = lo;
            tail.slot_hi = hi;
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    volatile int* abort_flag = &bars.abort_flag;
    const uint32_t tmem = bars.tmem_base;
    const int slot_lo = tail.slot_lo, slot_hi = tail.slot_hi;

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;
            bool alive = true;
            for (int p = tail.slot_start[slot_lo]; p < tail.slot_start[slot_hi] && alive; ++p) {
                const int g = tail.group_of[p], kp = tail.kept_pos[p];
                for (int kk2 = 0; kk2 < k_per_group; ++kk2, ++it) {
                    const int s = it % STAGES;
                    if (it >= STAGES && !pf_wait(&bars.empty[s], ((it / STAGES) - 1) & 1, abort_flag)) { alive = false; break; }
                    unsigned char* st = smem_raw + static_cast<size_t>(s) * kStageBytes;
                    mbar_arrive_expect_tx(&bars.full[s], kStageBytes);
                    tma_load_2d(st, &tmap_h, kp * S + kk2 * kBK, m0, &bars.full[s]);
                    const int krow = (g * 3 + 2) * S + kk2 * kBK;
#pragma unroll
                    for (int nb = 0; nb < BN2 / 64; ++nb)
                        tma_load_2d(st + kABytes + nb * kBBlock, &tmap_wd, n0 + nb * 64, krow, &bars.full[s]);
                }
            }
            if (*abort_flag) {
                int never = 0;
                for (int k = max(0, it - STAGES); k < it; ++k)
                    mbar_wait_bounded(&bars.full[k % STAGES], (k / STAGES) & 1, &never);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(kBM, BN2, true);
            int it = 0, used = 0;
            bool alive = true;
            for (int slot = slot_lo; slot < slot_hi && alive; ++slot) {
                const int p0 = tail.slot_start[slot], p1 = tail.slot_start[slot + 1];
                if (p0 == p1) continue;
                const int buf = used & 1;
                if (used >= 2 && !pf_wait(&tail.acc_empty[buf], ((used >> 1) - 1) & 1, abort_flag)) break;  // drained
                tcgen05_fence_after_sync();
                const uint32_t tmem_acc = tmem + buf * BN2;
                const int n_it = (p1 - p0) * k_per_group;
                for (int k = 0; k < n_it; ++k, ++it) {
                    const int s = it % STAGES;
                    if (!pf_wait(&bars.full[s], (it / STAGES) & 1, abort_flag)) { alive = false; break; }
                    tcgen05_fence_after_sync();
                    const uint32_t a0 = smem_u32(smem_raw + static_cast<size_t>(s) * kStageBytes);
#pragma unroll
                    for (int kk = 0; kk < kBK / kUmmaK; ++kk) {
                        const uint64_t a = umma_smem_desc(a0 + kk * 32, 16, 1024);
                        // MN-major B: 16 K-rows per MMA = 2 KiB further; 64-column blocks are kBBlock apart
                        const uint64_t b = umma_smem_desc(a0 + kABytes + kk * 2048, kBBlock, 1024);
                        umma_bf16(tmem_acc, a, b, idesc, (k > 0) || (kk > 0));
                    }
                    umma_commit(&bars.empty[s]);
                }
                if (!alive) break;
                umma_commit(&tail.acc_full[buf]);
                ++used;
            }
        }
    } else {
        const int quad = warp & 3;
        const int row = m0 + quad * 32 + lane;
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(quad * 32) << 16);
        int used = 0;
        for (int slot = slot_lo; slot < slot_hi; ++slot) {
            if (tail.slot_start[slot] == tail.slot_start[slot + 1]) continue;
            const int buf = used & 1;
            const bool ok = pf_wait(&tail.acc_full[buf], (used >> 1) & 1, abort_flag);
            tcgen05_fence_after_sync();
            float* out = partials + (static_cast<size_t>(slot) * T + row) * d + n0;
            for (int c0 = 0; c0 < BN2; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32x32(lane_base + buf * BN2 + c0, v);
                tmem_ld_wait();
                if (ok && row < T) {
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        reinterpret_cast<float4*>(out + c0)[q] =
                            make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                        __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                }
            }
            tcgen05_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tail.acc_empty[buf]);
            ++used;
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tcgen05_fence_after_sync(); tmem_dealloc(tmem, 2 * BN2); }
    if (tid == 0 && *abort_flag) flag_status(dev_status, HALO_DEV_TIMEOUT);
}

// Down projection for prompts of more than one 128-token tile: 256 tokens x 256 output columns per CTA (two
// accumulators of 256 TMEM columns), so that each staged byte feeds 1.5x the FLOPs of the 128-token tile.  The K
// range (kept groups in slot order) is cut into gridDim.z equal runs of 64-deep K tiles; every CTA adds its
// accumulators into the zeroed output slots with vector reductions, so a cut may fall anywhere.  A run that crosses
// a slot boundary drains the accumulators there and starts the next slot from zero.
template <int STAGES>
__global__ void __launch_bounds__(kPfThreads, 1)
ffn_down_wide_kernel(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_wd, int T,
                     int d, int S, int G, const int32_t* __restrict__ keep_list,
                     const int32_t* __restrict__ n_keep_ptr, const int32_t* __restrict__ dev_of_group, int n_dev,
                     int collapse, float* __restrict__ partials, uint32_t* dev_status) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    constexpr int BN2 = 256, MH = 2;
    constexpr uint32_t kAHalf = kBM * kBK * 2, kABytes = MH * kAHalf, kBBytes = kBK * BN2 * 2;
    constexpr uint32_t kStageBytes = kABytes + kBBytes;
    constexpr uint32_t kBBlock = kBK * 64 * 2;
    DownSmemTail& tail = *reinterpret_cast<DownSmemTail*>(smem_raw + static_cast<size_t>(STAGES) * kStageBytes);
    float* const epi_stage = reinterpret_cast<float*>(smem_raw + static_cast<size_t>(STAGES) * kStageBytes +
                                                      ((sizeof(DownSmemTail) + 15) & ~size_t(15)));
    PfBarriers& bars = tail.bars;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * (kBM * MH), n0 = blockIdx.y * BN2;
    int nk = *n_keep_ptr;
    nk = max(0, min(nk, G));
    const int k_per_group = S / kBK;
    // collapse: the caller wants the sum over holders only and every listed group has arrived: one slot
    const int n_slots = collapse ? 1 : n_dev + 1;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&bars.full[s], 1); mbar_init(&bars.empty[s], 1); }
        mbar_init(&bars.tmem_full, 1);
        mbar_init(&bars.tmem_empty, 4);
        mbar_init(&tail.acc_full[0], 1);
        mbar_init(&tail.acc_empty[0], 4);
        bars.abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_descriptor(&tmap_h);
        tma_prefetch_descriptor(&tmap_wd);
    }
    if (warp == 1) { tmem_alloc(&bars.tmem_base, MH * BN2); tmem_relinquish_alloc_permit(); }
    if (warp == 0) {
        const int pos = build_slot_order(tail, nk, G, n_dev, n_slots, n_slots - 1, keep_list, dev_of_group, dev_status,
                                         lane);
        if (lane == 0) {
            tail.slot_start[n_slots] = pos;
            // this CTA's run of K tiles, [slot_lo, slot_hi) reused as the K-tile bounds
            const long long units = static_cast<long long>(pos) * k_per_group;
            tail.slot_lo = static_cast<int>(units * blockIdx.z / gridDim.z);
            tail.slot_hi = static_cast<int>(units * (blockIdx.z + 1) / gridDim.z);
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    volatile int* abort_flag = &bars.abort_flag;
    const uint32_t tmem = bars.tmem_base;
    const int kt_lo = tail.slot_lo, kt_hi = tail.slot_hi;

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;
            for (int kt = kt_lo; kt < kt_hi; ++kt, ++it) {
                const int p = kt / k_per_group, kk2 = kt - p * k_per_group;
                const int g = tail.group_of[p], kp = tail.kept_pos[p];
                const int s = it % STAGES;
                if (it >= STAGES && !pf_wait(&bars.empty[s], ((it / STAGES) - 1) & 1, abort_flag)) break;
                unsigned char* st = smem_raw + static_cast<size_t>(s) * kStageBytes;
                mbar_arrive_expect_tx(&bars.full[s], kStageBytes);
#pragma unroll
                for (int mh = 0; mh < MH; ++mh)   // rows beyond T read as zeros
                    tma_load_2d(st + mh * kAHalf, &tmap_h, kp * S + kk2 * kBK, m0 + mh * kBM, &bars.full[s]);
                const int krow = (g * 3 + 2) * S + kk2 * kBK;
#pragma unroll
                for (int nb = 0; nb < BN2 / 64; ++nb)
                    tma_load_2d(st + kABytes + nb * kBBlock, &tmap_wd, n0 + nb * 64, krow, &bars.full[s]);
            }
            if (*abort_flag) {
                int never = 0;
                for (int k = max(0, it - STAGES); k < it; ++k)
                    mbar_wait_bounded(&bars.full[k % STAGES], (k / STAGES) & 1, &never);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(kBM, BN2, true);
            int it = 0, seg = 0;
            bool alive = true;
            for (int slot = 0; slot < n_slots && alive; ++slot) {
                const int k0 = max(kt_lo, tail.slot_start[slot] * k_per_group);
                const int k1 = min(kt_hi, tail.slot_start[slot + 1] * k_per_group);
                if (k0 >= k1) continue;
                // one accumulator set: the previous segment must have been drained
                if (seg >= 1 && !pf_wait(&tail.acc_empty[0], (seg - 1) & 1, abort_flag)) break;
                tcgen05_fence_after_sync();
                for (int kt = k0; kt < k1; ++kt, ++it) {
                    const int s = it % STAGES;
                    if (!pf_wait(&bars.full[s], (it / STAGES) & 1, abort_flag)) { alive = false; break; }
                    tcgen05_fence_after_sync();
                    const uint32_t a0 = smem_u32(smem_raw + static_cast<size_t>(s) * kStageBytes);
#pragma unroll
                    for (int kk = 0; kk < kBK / kUmmaK; ++kk) {
                        const uint64_t b = umma_smem_desc(a0 + kABytes + kk * 2048, kBBlock, 1024);
#pragma unroll
                        for (int mh = 0; mh < MH; ++mh) {
                            const uint64_t a = umma_smem_desc(a0 + mh * kAHalf + kk * 32, 16, 1024);
                            umma_bf16(tmem + mh * BN2, a, b, idesc, (kt > k0) || (kk > 0));
                        }
                    }
                    umma_commit(&bars.empty[s]);
                }
                if (!alive) break;
                umma_commit(&tail.acc_full[0]);
                ++seg;
            }
        }
    } else {
        const int quad = warp & 3;
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(quad * 32) << 16);
        int seg = 0;
        for (int slot = 0; slot < n_slots; ++slot) {
            const int k0 = max(kt_lo, tail.slot_start[slot] * k_per_group);
            const int k1 = min(kt_hi, tail.slot_start[slot + 1] * k_per_group);
            if (k0 >= k1) continue;
            const bool ok = pf_wait(&tail.acc_full[0], seg & 1, abort_flag);
            tcgen05_fence_after_sync();
            // Each thread holds one token row of the accumulator; the 32 x 32 chunk is turned through shared memory
            // so that one reduction instruction covers 4 rows x 128 contiguous bytes instead of 32 rows x 16.
            float* stage = epi_stage + (warp - 2) * (32 * kEpiPitch);
#pragma unroll
            for (int mh = 0; mh < MH; ++mh) {
                const int row0 = m0 + mh * kBM + quad * 32;
                float* out = partials + (static_cast<size_t>(slot) * T + row0) * d + n0;
                for (int c0 = 0; c0 < BN2; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld_32x32(lane_base + mh * BN2 + c0, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        *reinterpret_cast<float4*>(stage + lane * kEpiPitch + 4 * q) =
                            make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                        __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int r = 4 * j + (lane >> 3), cq = (lane & 7) * 4;
                        const float4 w = *reinterpret_cast<const float4*>(stage + r * kEpiPitch + cq);
                        if (ok && row0 + r < T)
                            red_add_v4f(out + static_cast<size_t>(r) * d + c0 + cq, w.x, w.y, w.z, w.w);
                    }
                    __syncwarp();
                }
            }
            tcgen05_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tail.acc_empty[0]);
            ++seg;
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tcgen05_fence_after_sync(); tmem_dealloc(tmem, MH * BN2); }
    if (tid == 0 && *abort_flag) flag_status(dev_status, HALO_DEV_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------------------
// Both contractions of a prompt's FFN in ONE launch: a queue of tiles, hidden-layer tiles first, then the
// down-projection tiles, claimed by the CTAs as they get free.  A down-projection tile reads H columns that
// hidden-layer tiles of OTHER CTAs write, so each finished hidden tile bumps a ready counter of its (token tile,
// kept group) and the loader of a down tile waits on the counters of the groups it is about to fetch.  Every
// hidden tile precedes every down tile in the queue and never waits on anything but its own copies, so a waited
// counter is always owed by a CTA that is already running and will get there: no co-residency is needed.  This
// fills the last, partial wave of hidden tiles with down-projection work.
// ------------------------------------------------------------------------------------------------------------
// K cuts of the down projection, as cumulative 16.16 fixed-point fractions of the K range: run z covers
// [units * cum[z] >> 16, units * cum[z + 1] >> 16).  The runs shrink geometrically, so the tiles claimed last are
// short: the end of the queue is fine-grained, and the runs that need the last hidden tiles are the small ones.
struct KCuts {
    int n;
    unsigned cum[17];
};
__device__ __forceinline__ int kcut(const KCuts& c, int units, int z) {
    return static_cast<int>((static_cast<unsigned long long>(units) * c.cum[z]) >> 16);
}

struct FusedTail {
    DownSmemTail dn;
    uint64_t tile_full[2];    // the loader has published a tile index
    uint64_t tile_empty[2];   // the MMA thread and the four epilogue warps have read it
    int tile_ring[2];
};
constexpr int kCtlHeaderWords = 32;          // word 0 = tile queue; ready counters follow
constexpr unsigned kReadyPerTile = 8;        // 4 epilogue warps x (2 for a full tile | 1 + 1 for its two halves)

struct FusedGeom {
    int tiles_x, n_full, n1_full, n1, n_tiles, n_tn, z_cuts, units;
};
struct FusedTile {
    int kind;   // 0 = hidden (full group), 1 = hidden (half group), 2 = down
    int ki, mt, half, nt, z;
};
__device__ __forceinline__ FusedTile fused_decode(const FusedGeom& q, int t) {
    FusedTile r{};
    if (t < q.n1_full) {
        r.kind = 0; r.ki = t / q.tiles_x; r.mt = t - r.ki * q.tiles_x;
    } else if (t < q.n1) {
        const int u = t - q.n1_full, per = 2 * q.tiles_x;
        r.kind = 1; r.ki = q.n_full + u / per;
        const int w = u % per;
        r.mt = w >> 1; r.half = w & 1;
    } else {
        const int u = t - q.n1, per = q.tiles_x * q.n_tn;
        r.kind = 2; r.z = u / per;
        const int w = u - r.z * per;
        r.nt = w / q.tiles_x; r.mt = w - r.nt * q.tiles_x;
    }
    return r;
}

// Bounded wait for a ready counter written by other CTAs.
__device__ __forceinline__ bool fused_wait_ready(const unsigned* counter, unsigned ready_when, volatile int* abort_flag) {
    if (ld_acquire_gpu(counter) >= ready_when) return true;
    const long long t0 = clock64();
    for (;;) {
        if (*abort_flag) return false;
        if (ld_acquire_gpu(counter) >= ready_when) return true;
        __nanosleep(64);
        if (clock64() - t0 > static_cast<long long>(kWaitLimitCycles)) { *abort_flag = 1; return false; }
    }
}

template <int NS, int STAGES>
__global__ void __launch_bounds__(kPfThreads, 1)
ffn_fused_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                 const __grid_constant__ CUtensorMap tmap_w_half, const __grid_constant__ CUtensorMap tmap_h,
                 const __grid_constant__ CUtensorMap tmap_wd, const __grid_constant__ KCuts cuts, int T, int d, int S,
                 int G, int n_sm,
                 const int32_t* __restrict__ keep_list, const int32_t* __restrict__ n_keep_ptr,
                 const int32_t* __restrict__ dev_of_group, int n_dev, int collapse, __nv_bfloat16* __restrict__ H,
                 int h_cols, float* __restrict__ partials, unsigned* __restrict__ ctl, uint32_t* dev_status) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    constexpr int BN2 = 256, MH = 2;
    const int subs = S / NS;            // a group of S neurons is computed as S / NS hidden tiles of NS neurons
    constexpr uint32_t kAHalf = kBM * kBK * 2, kABytes = MH * kAHalf;
    constexpr uint32_t kStageBytes = kABytes + kBK * BN2 * 2;   // 64 KiB: the down tile's stage; a hidden stage fits
    constexpr uint32_t kBBlock = kBK * 64 * 2;
    constexpr uint32_t kTmemCols = 512;
    static_assert(MH * 2 * NS <= 512, "hidden accumulators must fit in TMEM");
    FusedTail& ft = *reinterpret_cast<FusedTail*>(smem_raw + static_cast<size_t>(STAGES) * kStageBytes);
    DownSmemTail& tail = ft.dn;
    float* const epi_stage = reinterpret_cast<float*>(smem_raw + static_cast<size_t>(STAGES) * kStageBytes +
                                                      ((sizeof(FusedTail) + 15) & ~size_t(15)));
    PfBarriers& bars = tail.bars;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int nk = *n_keep_ptr;
    nk = max(0, min(nk, G));
    const int k_per_group = S / kBK, n_kt1 = d / kBK;
    const int n_slots = collapse ? 1 : n_dev + 1;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&bars.full[s], 1); mbar_init(&bars.empty[s], 1); }
        mbar_init(&bars.tmem_full, 1);
        mbar_init(&bars.tmem_empty, 4);
        mbar_init(&tail.acc_full[0], 1);
        mbar_init(&tail.acc_empty[0], 4);
        for (int b = 0; b < 2; ++b) { mbar_init(&ft.tile_full[b], 1); mbar_init(&ft.tile_empty[b], 5); }
        bars.abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_descriptor(&tmap_x);
        tma_prefetch_descriptor(&tmap_w);
        tma_prefetch_descriptor(&tmap_h);
        tma_prefetch_descriptor(&tmap_wd);
    }
    if (warp == 1) { tmem_alloc(&bars.tmem_base, kTmemCols); tmem_relinquish_alloc_permit(); }
    if (warp == 0) {
        const int pos = build_slot_order(tail, nk, G, n_dev, n_slots, n_slots - 1, keep_list, dev_of_group, dev_status,
                                         lane);
        if (lane == 0) { tail.slot_start[n_slots] = pos; tail.slot_lo = pos; }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    volatile int* abort_flag = &bars.abort_flag;
    const uint32_t tmem = bars.tmem_base;

    // the tile list, derived identically by every role
    FusedGeom q;
    q.tiles_x = (T + kBM * MH - 1) / (kBM * MH);
    q.n_tn = d / BN2;
    q.z_cuts = cuts.n;
    q.units = tail.slot_lo * k_per_group;    // K tiles of the down projection (valid kept groups only)
    const int nkv = nk * subs;          // hidden tiles per token tile; FusedTile::ki counts them
    q.n_full = nkv;
    {
        // hidden tiles of the last, partial wave are cut into two half-width tiles (finer work at the end)
        const int total = q.tiles_x * nkv;
        if (n_sm > 0 && total > n_sm) {
            const int full_tiles = (total / n_sm) * n_sm / q.tiles_x, left = nkv - full_tiles;
            if (left > 0 && 2 * left * q.tiles_x <= n_sm) q.n_full = full_tiles;
        }
    }
    q.n1_full = q.tiles_x * q.n_full;
    q.n1 = q.n1_full + 2 * q.tiles_x * (nkv - q.n_full);
    q.n_tiles = q.n1 + (q.units > 0 ? q.tiles_x * q.n_tn * cuts.n : 0);

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;
            for (int ti = 0;; ++ti) {
                if (ti >= 2 && !pf_wait(&ft.tile_empty[ti & 1], ((ti >> 1) - 1) & 1, abort_flag)) break;
                const int t = static_cast<int>(min(atomicAdd(&ctl[0], 1u), 0x7fffffffu));
                ft.tile_ring[ti & 1] = t;
                mbar_arrive(&ft.tile_full[ti & 1]);
                if (t >= q.n_tiles) break;
                const FusedTile tl = fused_decode(q, t);
                const int m0 = tl.mt * (kBM * MH);
                bool alive = true;
                if (tl.kind < 2) {
                    const int ki = tl.ki / subs;
                    const int g = keep_list[ki];
                    const bool valid = g >= 0 && g < G;     // an invalid entry was flagged by build_slot_order
                    const int ns = tl.kind == 1 ? NS / 2 : NS;
                    const int n_off = (tl.ki - ki * subs) * NS + (tl.kind == 1 ? tl.half * (NS / 2) : 0);
                    const CUtensorMap* const map_w = tl.kind == 1 ? &tmap_w_half : &tmap_w;
                    const int gg = valid ? g : 0;
                    for (int kt = 0; kt < n_kt1; ++kt, ++it) {
                        const int s = it % STAGES;
                        if (it >= STAGES && !pf_wait(&bars.empty[s], ((it / STAGES) - 1) & 1, abort_flag)) { alive = false; break; }
                        unsigned char* st = smem_raw + static_cast<size_t>(s) * kStageBytes;
                        mbar_arrive_expect_tx(&bars.full[s], kABytes + 2u * static_cast<uint32_t>(ns) * kBK * 2u);
#pragma unroll
                        for (int mh = 0; mh < MH; ++mh)
                            tma_load_2d(st + mh * kAHalf, &tmap_x, kt * kBK, m0 + mh * kBM, &bars.full[s]);
                        tma_load_2d(st + kABytes, map_w, kt * kBK, (gg * 3 + 0) * S + n_off, &bars.full[s]);
                        tma_load_2d(st + kABytes + ns * (kBK * 2), map_w, kt * kBK, (gg * 3 + 1) * S + n_off, &bars.full[s]);
                    }
                } else {
                    const int n0 = tl.nt * BN2;
                    const int kt_lo = kcut(cuts, q.units, tl.z);
                    const int kt_hi = kcut(cuts, q.units, tl.z + 1);
                    int checked = -1;
                    for (int kt = kt_lo; kt < kt_hi; ++kt, ++it) {
                        const int p = kt / k_per_group, kk2 = kt - p * k_per_group;
                        const int g = tail.group_of[p], kp = tail.kept_pos[p];
                        if (p != checked) {
                            // the hidden tiles of this group and token tile must have been written
                            if (!fused_wait_ready(&ctl[kCtlHeaderWords + tl.mt * G + kp], kReadyPerTile * subs, abort_flag)) {
                                alive = false;
                                break;
                            }
                            fence_proxy_async_all();   // their generic-proxy stores before this thread's TMA reads
                            checked = p;
                        }
                        const int s = it % STAGES;
                        if (it >= STAGES && !pf_wait(&bars.empty[s], ((it / STAGES) - 1) & 1, abort_flag)) { alive = false; break; }
                        unsigned char* st = smem_raw + static_cast<size_t>(s) * kStageBytes;
                        mbar_arrive_expect_tx(&bars.full[s], kStageBytes);
#pragma unroll
                        for (int mh = 0; mh < MH; ++mh)
                            tma_load_2d(st + mh * kAHalf, &tmap_h, kp * S + kk2 * kBK, m0 + mh * kBM, &bars.full[s]);
                        const int krow = (g * 3 + 2) * S + kk2 * kBK;
#pragma unroll
                        for (int nb = 0; nb < BN2 / 64; ++nb)
                            tma_load_2d(st + kABytes + nb * kBBlock, &tmap_wd, n0 + nb * 64, krow, &bars.full[s]);
                    }
                }
                if (!alive) break;
            }
            if (*abort_flag) {  // let outstanding copies land before the CTA goes away
                int never = 0;
                for (int k = max(0, it - STAGES); k < it; ++k)
                    mbar_wait_bounded(&bars.full[k % STAGES], (k / STAGES) & 1, &never);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc2 = umma_idesc_bf16(kBM, BN2, true);
            int it = 0, seg = 0;
            bool alive = true;
            for (int ti = 0; alive; ++ti) {
                if (!pf_wait(&ft.tile_full[ti & 1], (ti >> 1) & 1, abort_flag)) break;
                const int t = ft.tile_ring[ti & 1];
                mbar_arrive(&ft.tile_empty[ti & 1]);
                if (t >= q.n_tiles) break;
                const FusedTile tl = fused_decode(q, t);
                if (tl.kind < 2) {
                    const int ns = tl.kind == 1 ? NS / 2 : NS;
                    const uint32_t idesc1 = umma_idesc_bf16(kBM, 2 * ns, false);
                    if (seg >= 1 && !pf_wait(&tail.acc_empty[0], (seg - 1) & 1, abort_flag)) break;
                    tcgen05_fence_after_sync();
                    for (int kt = 0; kt < n_kt1; ++kt, ++it) {
                        const int s = it % STAGES;
                        if (!pf_wait(&bars.full[s], (it / STAGES) & 1, abort_flag)) { alive = false; break; }
                        tcgen05_fence_after_sync();
                        const uint32_t a0 = smem_u32(smem_raw + static_cast<size_t>(s) * kStageBytes);
#pragma unroll
                        for (int kk = 0; kk < kBK / kUmmaK; ++kk) {
                            const uint64_t b = umma_smem_desc(a0 + kABytes + kk * 32, 16, 1024);
#pragma unroll
                            for (int mh = 0; mh < MH; ++mh) {
                                const uint64_t a = umma_smem_desc(a0 + mh * kAHalf + kk * 32, 16, 1024);
                                umma_bf16(tmem + mh * 2 * NS, a, b, idesc1, (kt > 0) || (kk > 0));
                            }
                        }
                        umma_commit(&bars.empty[s]);
                    }
                    if (!alive) break;
                    umma_commit(&tail.acc_full[0]);
                    ++seg;
                } else {
                    const int kt_lo = kcut(cuts, q.units, tl.z);
                    const int kt_hi = kcut(cuts, q.units, tl.z + 1);
                    for (int slot = 0; slot < n_slots && alive; ++slot) {
                        const int k0 = max(kt_lo, tail.slot_start[slot] * k_per_group);
                        const int k1 = min(kt_hi, tail.slot_start[slot + 1] * k_per_group);
                        if (k0 >= k1) continue;
                        if (seg >= 1 && !pf_wait(&tail.acc_empty[0], (seg - 1) & 1, abort_flag)) { alive = false; break; }
                        tcgen05_fence_after_sync();
                        for (int kt = k0; kt < k1; ++kt, ++it) {
                            const int s = it % STAGES;
                            if (!pf_wait(&bars.full[s], (it / STAGES) & 1, abort_flag)) { alive = false; break; }
                            tcgen05_fence_after_sync();
                            const uint32_t a0 = smem_u32(smem_raw + static_cast<size_t>(s) * kStageBytes);
#pragma unroll
                            for (int kk = 0; kk < kBK / kUmmaK; ++kk) {
                                const uint64_t b = umma_smem_desc(a0 + kABytes + kk * 2048, kBBlock, 1024);
#pragma unroll
                                for (int mh = 0; mh < MH; ++mh) {
                                    const uint64_t a = umma_smem_desc(a0 + mh * kAHalf + kk * 32, 16, 1024);
                                    umma_bf16(tmem + mh * BN2, a, b, idesc2, (kt > k0) || (kk > 0));
                                }
                            }
                            umma_commit(&bars.empty[s]);
                        }
                        if (!alive) break;
                        umma_commit(&tail.acc_full[0]);
                        ++seg;
                    }
                }
            }
        }
    } else {
        const int quad = warp & 3;
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(quad * 32) << 16);
        float* stage = epi_stage + (warp - 2) * (32 * kEpiPitch);
        int seg = 0;
        for (int ti = 0;; ++ti) {
            if (!pf_wait(&ft.tile_full[ti & 1], (ti >> 1) & 1, abort_flag)) break;
            const int t = ft.tile_ring[ti & 1];
            __syncwarp();
            if (lane == 0) mbar_arrive(&ft.tile_empty[ti & 1]);
            if (t >= q.n_tiles) break;
            const FusedTile tl = fused_decode(q, t);
            const int m0 = tl.mt * (kBM * MH);
            if (tl.kind < 2) {
                const int ki = tl.ki / subs;
                const int ns = tl.kind == 1 ? NS / 2 : NS;
                const int n_off = (tl.ki - ki * subs) * NS + (tl.kind == 1 ? tl.half * (NS / 2) : 0);
                const int g = keep_list[ki];
                const bool ok = pf_wait(&tail.acc_full[0], seg & 1, abort_flag) && g >= 0 && g < G;
                tcgen05_fence_after_sync();
#pragma unroll
                for (int mh = 0; mh < MH; ++mh) {
                    const int row = m0 + mh * kBM + quad * 32 + lane;
                    for (int c0 = 0; c0 < ns; c0 += 32) {
                        uint32_t dg[32], du[32];
                        tmem_ld_32x32(lane_base + mh * 2 * NS + c0, dg);
                        tmem_ld_32x32(lane_base + mh * 2 * NS + ns + c0, du);
                        tmem_ld_wait();
                        if (ok && row < T) {
                            uint4* dst = reinterpret_cast<uint4*>(H + static_cast<size_t>(row) * h_cols +
                                                                  static_cast<size_t>(ki) * S + n_off + c0);
#pragma unroll
                            for (int qq = 0; qq < 4; ++qq) {
                                uint32_t packed[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int i = qq * 8 + e * 2;
                                    const float h0 = silu_mul(__uint_as_float(dg[i]), __uint_as_float(du[i]));
                                    const float h1 = silu_mul(__uint_as_float(dg[i + 1]), __uint_as_float(du[i + 1]));
                                    const __nv_bfloat162 pk = __floats2bfloat162_rn(h0, h1);
                                    packed[e] = *reinterpret_cast<const uint32_t*>(&pk);
                                }
                                dst[qq] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                            }
                        }
                    }
                }
                // publish: every lane orders its own stores (towards the TMA reads of other CTAs too), then one
                // lane bumps the counter.  An aborted tile publishes nothing; its readers give up on their own.
                tcgen05_fence_before_sync();
                fence_proxy_async_all();
                __threadfence();
                __syncwarp();
                if (lane == 0) {
                    if (ok) atomicAdd(&ctl[kCtlHeaderWords + tl.mt * G + ki], tl.kind == 1 ? 1u : 2u);
                    mbar_arrive(&tail.acc_empty[0]);
                }
                ++seg;
            } else {
                const int n0 = tl.nt * BN2;
                const int kt_lo = kcut(cuts, q.units, tl.z);
                const int kt_hi = kcut(cuts, q.units, tl.z + 1);
                for (int slot = 0; slot < n_slots; ++slot) {
                    const int k0 = max(kt_lo, tail.slot_start[slot] * k_per_group);
                    const int k1 = min(kt_hi, tail.slot_start[slot + 1] * k_per_group);
                    if (k0 >= k1) continue;
                    const bool ok = pf_wait(&tail.acc_full[0], seg & 1, abort_flag);
                    tcgen05_fence_after_sync();
#pragma unroll
                    for (int mh = 0; mh < MH; ++mh) {
                        const int row0 = m0 + mh * kBM + quad * 32;
                        float* out = partials + (static_cast<size_t>(slot) * T + row0) * d + n0;
                        for (int c0 = 0; c0 < BN2; c0 += 32) {
                            uint32_t v[32];
                            tmem_ld_32x32(lane_base + mh * BN2 + c0, v);
                            tmem_ld_wait();
#pragma unroll
                            for (int qq = 0; qq < 8; ++qq)
                                *reinterpret_cast<float4*>(stage + lane * kEpiPitch + 4 * qq) =
                                    make_float4(__uint_as_float(v[4 * qq]), __uint_as_float(v[4 * qq + 1]),
                                                __uint_as_float(v[4 * qq + 2]), __uint_as_float(v[4 * qq + 3]));
                            __syncwarp();
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const int r = 4 * j + (lane >> 3), cq = (lane & 7) * 4;
                                const float4 w = *reinterpret_cast<const float4*>(stage + r * kEpiPitch + cq);
                                if (ok && row0 + r < T)
                                    red_add_v4f(out + static_cast<size_t>(r) * d + c0 + cq, w.x, w.y, w.z, w.w);
                            }
                            __syncwarp();
                        }
                    }
                    tcgen05_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&tail.acc_empty[0]);
                    ++seg;
                }
            }
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tcgen05_fence_after_sync(); tmem_dealloc(tmem, kTmemCols); }
    if (tid == 0 && *abort_flag) flag_status(dev_status, HALO_DEV_TIMEOUT);
    // The last CTA to get here (none reads the control words any more) zeroes them for the next launch.
    __shared__ int is_last;
    if (tid == 0) {
        __threadfence();
        is_last = atomicAdd(&ctl[1], 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (is_last) {
        const int n_words = kCtlHeaderWords + q.tiles_x * G;
        for (int i = tid; i < n_words; i += blockDim.x) ctl[i] = 0u;
    }
}

// ------------------------------------------------------------------------------------------------------------
// Predictor hidden layer for many tokens: Z[T][r] = act(X[T][d] * W1[r][d]^T), fp32 out (step a1, prefill)
// ------------------------------------------------------------------------------------------------------------
template <int STAGES>
__global__ void __launch_bounds__(kPfThreads, 1)
pred_hidden_gemm_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w1, int T,
                        int d, int r, int act, float* __restrict__ Z, uint32_t* dev_status) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    constexpr int BN = 128;
    constexpr uint32_t kABytes = kBM * kBK * 2, kBBytes = BN * kBK * 2, kStageBytes = kABytes + kBBytes;
    PfBarriers& bars = *reinterpret_cast<PfBarriers*>(smem_raw + static_cast<size_t>(STAGES) * kStageBytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * kBM, n0 = blockIdx.y * BN;
    const int n_kt = d / kBK;
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&bars.full[s], 1); mbar_init(&bars.empty[s], 1); }
        mbar_init(&bars.tmem_full, 1);
        mbar_init(&bars.tmem_empty, 1);
        bars.abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_descriptor(&tmap_x);
        tma_prefetch_descriptor(&tmap_w1);
    }
    if (warp == 1) { tmem_alloc(&bars.tmem_base, BN); tmem_relinquish_alloc_permit(); }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    volatile int* abort_flag = &bars.abort_flag;
    const uint32_t tmem = bars.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            for (int kt = 0; kt < n_kt; ++kt) {
                const int s = kt % STAGES;
                if (kt >= STAGES && !pf_wait(&bars.empty[s], ((kt / STAGES) - 1) & 1, abort_flag)) break;
                unsigned char* st = smem_raw + static_cast<size_t>(s) * kStageBytes;
                mbar_arrive_expect_tx(&bars.full[s], kStageBytes);
                tma_load_2d(st, &tmap_x, kt * kBK, m0, &bars.full[s]);
                tma_load_2d(st + kABytes, &tmap_w1, kt * kBK, n0, &bars.full[s]);   // rows beyond r read as zeros
                issued = kt + 1;
            }
            if (*abort_flag) {
                int never = 0;
                for (int kt = max(0, issued - STAGES); kt < issued; ++kt)
                    mbar_wait_bounded(&bars.full[kt % STAGES], (kt / STAGES) & 1, &never);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(kBM, BN, false);
            for (int kt = 0; kt < n_kt; ++kt) {
                const int s = kt % STAGES;
                if (!pf_wait(&bars.full[s], (kt / STAGES) & 1, abort_flag)) break;
                tcgen05_fence_after_sync();
                const uint32_t a0 = smem_u32(smem_raw + static_cast<size_t>(s) * kStageBytes);
#pragma unroll
                for (int kk = 0; kk < kBK / kUmmaK; ++kk)
                    umma_bf16(tmem, umma_smem_desc(a0 + kk * 32, 16, 1024),
                              umma_smem_desc(a0 + kABytes + kk * 32, 16, 1024), idesc, (kt > 0) || (kk > 0));
                umma_commit(&bars.empty[s]);
            }
            umma_commit(&bars.tmem_full);
        }
    } else {
        const bool ok = pf_wait(&bars.tmem_full, 0, abort_flag);
        tcgen05_fence_after_sync();
        const int quad = warp & 3;
        const int row = m0 + quad * 32 + lane;
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(quad * 32) << 16);
        for (int c0 = 0; c0 < BN; c0 += 32) {
            uint32_t v[32];
            tmem_ld_32x32(lane_base + c0, v);
            tmem_ld_wait();
            if (ok && row < T) {
                float* out = Z + static_cast<size_t>(row) * r + n0 + c0;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (n0 + c0 + 4 * q < r) {   // r is a multiple of 8
                        float4 o = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                               __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                        if (act == HALO_ACT_RELU) {
                            o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f);
                        }
                        reinterpret_cast<float4*>(out)[q] = o;
                    }
                }
            }
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tcgen05_fence_after_sync(); tmem_dealloc(tmem, BN); }
    if (tid == 0 && *abort_flag) flag_status(dev_status, HALO_DEV_TIMEOUT);
}

// ---- host side ------------------------------------------------------------------------------------------------

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// bf16 matrix [rows][cols] (cols contiguous), box = box_cols x box_rows, 128-byte swizzle, zero fill out of range
bool make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t row_stride_elems,
              uint32_t box_cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {row_stride_elems * 2};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t elem_strides[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem_strides,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool make_bf16_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t row_stride_elems,
                   uint32_t box_cols, uint32_t box_rows) {
    return make_map(map, base, rows, cols, row_stride_elems, box_cols, box_rows);
}

bool prefill_supported(const halo_ffn_shape& sh, int n_tok) {
    return sh.wdtype == HALO_BF16 && n_tok >= 16 && (sh.group_size == 64 || sh.group_size == 128 || sh.group_size == 256) &&
           sh.d_model % 128 == 0 && sh.d_ffn / sh.group_size <= HALO_MAX_GROUPS;
}

bool prefill_accumulates(const halo_ffn_shape& sh, int n_tok) {
    return prefill_supported(sh, n_tok) && n_tok > kBM && sh.d_model % 256 == 0;
}

namespace {
// tile queue + one ready counter per (256-token tile, kept position), in front of H
size_t prefill_ctl_bytes(const halo_ffn_shape& sh, int n_tok) {
    const size_t words = kCtlHeaderWords + static_cast<size_t>((n_tok + 2 * kBM - 1) / (2 * kBM)) * (sh.d_ffn / sh.group_size);
    return (words * sizeof(unsigned) + 1023) & ~static_cast<size_t>(1023);
}
}  // namespace

size_t prefill_workspace_bytes(const halo_ffn_shape& sh, int n_tok) {
    // control words, then H: bf16 [n_tok][d_ffn], kept groups packed to the left
    return prefill_ctl_bytes(sh, n_tok) + static_cast<size_t>(n_tok) * sh.d_ffn * 2;
}

// ctl_clean: the workspace's control words are known to be zero (left so by an earlier launch on this workspace).
// partials must already be zero (slots without kept groups are not written).  collapse != 0: the caller wants the
// sum over holders only and partials has two slots whose SUM is the result; when prefill_accumulates() holds,
// everything is added into slot 0 (slot 1 is not touched), which may then hold a value to add to.
halo_status launch_group_ffn_prefill(const halo_ffn_shape& sh, const void* W, const void* x, int n_tok,
                                     const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group,
                                     int n_dev, int collapse, float* partials, void* workspace, uint32_t* dev_status,
                                     cudaStream_t st, bool ctl_clean) {
    const int d = sh.d_model, S = sh.group_size, G = sh.d_ffn / S, T = n_tok;
    const size_t ctl_bytes = prefill_ctl_bytes(sh, T);
    unsigned* ctl = static_cast<unsigned*>(workspace);
    __nv_bfloat16* H = reinterpret_cast<__nv_bfloat16*>(static_cast<unsigned char*>(workspace) + ctl_bytes);
    const uint64_t w_rows = static_cast<uint64_t>(G) * 3 * S;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return HALO_ERR_CUDA;
    const int NS = std::min(S, 128);     // neurons per hidden tile; a 256-neuron group is two tiles
    // The five tensor maps depend only on the pointers and the shape: they are encoded once per combination and
    // kept (a stack calls this with the same few buffers for every prompt), not once per launch.
    struct MapSet { const void* W; const void* x; const void* H; int T, d, S, G; CUtensorMap m[5]; bool used; };
    constexpr int kMapSets = 256;
    static MapSet cache[kMapSets];
    static std::mutex cache_mutex;
    CUtensorMap map_x, map_w, map_w_half, map_h, map_wd;
    {
        std::lock_guard<std::mutex> lock(cache_mutex);
        size_t hsh = (reinterpret_cast<uintptr_t>(W) >> 8) * 1000003u ^ (reinterpret_cast<uintptr_t>(x) >> 8) * 7919u ^
                     static_cast<size_t>(T) * 31u;
        MapSet* e = &cache[hsh % kMapSets];
        if (!(e->used && e->W == W && e->x == x && e->H == H && e->T == T && e->d == d && e->S == S && e->G == G)) {
            MapSet fresh{};
            fresh.W = W; fresh.x = x; fresh.H = H; fresh.T = T; fresh.d = d; fresh.S = S; fresh.G = G;
            if (!make_map(&fresh.m[0], x, T, d, d, kBK, kBM) || !make_map(&fresh.m[1], W, w_rows, d, d, kBK, NS) ||
                !make_map(&fresh.m[2], W, w_rows, d, d, kBK, NS / 2) ||
                !make_map(&fresh.m[3], H, T, sh.d_ffn, sh.d_ffn, kBK, kBM) || !make_map(&fresh.m[4], W, w_rows, d, d, 64, kBK))
                return HALO_ERR_CUDA;
            fresh.used = true;
            *e = fresh;      // a colliding entry is simply replaced
        }
        map_x = e->m[0]; map_w = e->m[1]; map_w_half = e->m[2]; map_h = e->m[3]; map_wd = e->m[4];
    }
    const bool two_launches = option_value(OPT_PREFILL_TWO_LAUNCHES) == 1;
    if (T > kBM && d % 256 == 0 && !two_launches) {
        // both contractions in one launch, one CTA per SM pulling tiles from a queue
        // the kernel leaves its control words zeroed; a workspace of unknown content is zeroed here
        if (!ctl_clean && cudaMemsetAsync(ctl, 0, ctl_bytes, st) != cudaSuccess) return HALO_ERR_CUDA;
        constexpr int kStagesF = 3;
        const size_t smemf = static_cast<size_t>(kStagesF) * (2 * kBM * kBK * 2 + kBK * 256 * 2) + sizeof(FusedTail) + 16 +
                             kEpiStageBytes + 1024;
        const int tiles2 = ((T + 2 * kBM - 1) / (2 * kBM)) * (d / 256);
        // K cuts of the down projection: six runs per output tile on the 7B shape, each 0.75 of the one before
        // (a model of the tile queue, then a sweep on the GPU: 0.3 ms per 32-block prompt better than six equal
        // runs); fewer runs when there are many output tiles anyway.  The options "prefill_kcuts" and
        // "prefill_kratio_percent" override.
        int z = std::max(1, std::min(7, (n_sm * 4 / 3) / tiles2));
        double ratio = 0.75;
        if (option_value(OPT_PREFILL_KCUTS) > 0) z = option_value(OPT_PREFILL_KCUTS);
        if (option_value(OPT_PREFILL_KRATIO_PERCENT) > 0) ratio = option_value(OPT_PREFILL_KRATIO_PERCENT) / 100.0;
        KCuts cuts{};
        cuts.n = z;
        {
            double total = 0.0, run = 1.0, acc = 0.0;
            for (int i = 0; i < z; ++i, run *= ratio) total += run;
            run = 1.0;
            for (int i = 0; i < z; ++i, run *= ratio) {
                cuts.cum[i] = static_cast<unsigned>(acc / total * 65536.0);
                acc += run;
            }
            cuts.cum[z] = 65536u;
        }
#define HALO_LAUNCH_FUSED(NS_)                                                                                       \
    do {                                                                                                             \
        auto kf = ffn_fused_kernel<NS_, kStagesF>;                                                                   \
        static bool oncef[64] = {};                                                                                  \
        if (!ensure_dynamic_smem(kf, smemf, oncef)) return HALO_ERR_CUDA;                                            \
        kf<<<n_sm, kPfThreads, smemf, st>>>(map_x, map_w, map_w_half, map_h, map_wd, cuts, T, d, S, G, n_sm,         \
                                            keep_list,                                                               \
                                            n_keep, dev_of_group, n_dev, collapse, H, sh.d_ffn, partials, ctl,       \
                                            dev_status);                                                             \
    } while (0)
        if (NS == 128) HALO_LAUNCH_FUSED(128); else HALO_LAUNCH_FUSED(64);
#undef HALO_LAUNCH_FUSED
        HALO_CHECK_LAUNCH();
        return HALO_OK;
    }
    // GEMM-1: 256-token tiles when the prompt has them (more FLOP per staged byte), else 128-token tiles
#define HALO_LAUNCH_HIDDEN(NS_, MH_, STAGES_)                                                                        \
    do {                                                                                                             \
        auto k1 = ffn_hidden_kernel<NS_, MH_, STAGES_>;                                                              \
        const size_t smem1 = static_cast<size_t>(STAGES_) * (MH_ * kBM * kBK * 2 + 2 * NS_ * kBK * 2) +              \
                             sizeof(PfBarriers) + 1024;                                                              \
        static bool once1[64] = {};                                                                                  \
        if (!ensure_dynamic_smem(k1, smem1, once1)) return HALO_ERR_CUDA;                                            \
        const dim3 grid1((T + kBM * MH_ - 1) / (kBM * MH_), G * (S / NS_), 2);                                       \
        k1<<<grid1, kPfThreads, smem1, st>>>(map_x, map_w, map_w_half, T, d, S, G, n_sm, keep_list, n_keep, H,       \
                                             sh.d_ffn, dev_status);                                                  \
    } while (0)
    if (NS == 128) {
        if (T > kBM) HALO_LAUNCH_HIDDEN(128, 2, 3); else HALO_LAUNCH_HIDDEN(128, 1, 4);
    } else {
        if (T > kBM) HALO_LAUNCH_HIDDEN(64, 2, 4); else HALO_LAUNCH_HIDDEN(64, 1, 6);
    }
#undef HALO_LAUNCH_HIDDEN
    HALO_CHECK_LAUNCH();
    if (d % 256 == 0 && T > kBM) {
        // 256 x 256 tiles; K cut into as many runs as fill the SMs once
        constexpr int kStages2 = 3;
        auto k2 = ffn_down_wide_kernel<kStages2>;
        const size_t smem2 = static_cast<size_t>(kStages2) * (2 * kBM * kBK * 2 + kBK * 256 * 2) + sizeof(DownSmemTail) +
                             16 + kEpiStageBytes + 1024;
        static bool once2[64] = {};
        if (!ensure_dynamic_smem(k2, smem2, once2)) return HALO_ERR_CUDA;
        const int tiles = ((T + 2 * kBM - 1) / (2 * kBM)) * (d / 256);
        const int z = std::max(1, std::min(8, n_sm / tiles));
        const dim3 grid2((T + 2 * kBM - 1) / (2 * kBM), d / 256, z);
        k2<<<grid2, kPfThreads, smem2, st>>>(map_h, map_wd, T, d, S, G, keep_list, n_keep, dev_of_group, n_dev, collapse,
                                             partials, dev_status);
    } else if (d % 256 == 0) {
        // 256-column tiles (more FLOP per staged byte); with holder slots the K range is split over two CTAs
        constexpr int kStages2 = 4;
        auto k2 = ffn_down_kernel<256, kStages2>;
        const size_t smem2 = static_cast<size_t>(kStages2) * (kBM * kBK * 2 + kBK * 256 * 2) + sizeof(DownSmemTail) + 1024;
        static bool once2[64] = {};
        if (!ensure_dynamic_smem(k2, smem2, once2)) return HALO_ERR_CUDA;
        const dim3 grid2((T + kBM - 1) / kBM, d / 256, n_dev > 0 ? 2 : 1);
        k2<<<grid2, kPfThreads, smem2, st>>>(map_h, map_wd, T, d, S, G, keep_list, n_keep, dev_of_group, n_dev, collapse, partials,
                                             dev_status);
    } else {
        constexpr int kStages2 = 6;
        auto k2 = ffn_down_kernel<128, kStages2>;
        const size_t smem2 = static_cast<size_t>(kStages2) * (kBM * kBK * 2 + kBK * 128 * 2) + sizeof(DownSmemTail) + 1024;
        static bool once2[64] = {};
        if (!ensure_dynamic_smem(k2, smem2, once2)) return HALO_ERR_CUDA;
        const dim3 grid2((T + kBM - 1) / kBM, d / 128, 1);
        k2<<<grid2, kPfThreads, smem2, st>>>(map_h, map_wd, T, d, S, G, keep_list, n_keep, dev_of_group, n_dev, collapse, partials,
                                             dev_status);
    }
    HALO_CHECK_LAUNCH();
    return HALO_OK;
}

bool pred_gemm_supported(const halo_pred_shape& sh, int n_tok) {
    return sh.wdtype == HALO_BF16 && n_tok >= 16 && sh.d_in % kBK == 0;
}

// Z[n_tok][rank] = act(feat * W1^T) on the tensor cores.
halo_status launch_pred_hidden_gemm(const halo_pred_shape& sh, const void* W1, const void* feat, int n_tok,
                                    float* hidden, uint32_t* dev_status, cudaStream_t st) {
    CUtensorMap map_x, map_w1;
    if (!make_map(&map_x, feat, n_tok, sh.d_in, sh.d_in, kBK, kBM) ||
        !make_map(&map_w1, W1, sh.rank, sh.d_in, sh.d_in, kBK, 128))
        return HALO_ERR_CUDA;
    constexpr int kStages = 6;
    auto k = pred_hidden_gemm_kernel<kStages>;
    const size_t smem = static_cast<size_t>(kStages) * (kBM * kBK * 2 + 128 * kBK * 2) + sizeof(PfBarriers) + 1024;
    static bool once[64] = {};
    if (!ensure_dynamic_smem(k, smem, once)) return HALO_ERR_CUDA;
    const dim3 grid((n_tok + kBM - 1) / kBM, (sh.rank + 127) / 128);
    k<<<grid, kPfThreads, smem, st>>>(map_x, map_w1, n_tok, sh.d_in, sh.rank, sh.act, hidden, dev_status);
    HALO_CHECK_LAUNCH();
    return HALO_OK;
}

}  // namespace halo
