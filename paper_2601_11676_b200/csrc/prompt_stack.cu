// Prompt path of the FFN stack as ONE persistent kernel: every block of the stack (predictor one layer ahead,
// selection, masked FFN on the tensor cores, residual + normalisation) for one prompt in a single launch.
//
// One CTA per SM takes tiles from a queue, block of the stack by block.  The tiles of block l, in order:
//   for every 256-token tile mt:   [last mt]   PRED     hidden layer of block l+1's predictor from x_l, column sums
//                                                       over the tokens; the CTA that finishes the last one computes
//                                                       the scores and steps a2..a5 for block l+1 and publishes them
//                                  HIDDEN(mt)  one kept group (or half of a 256-neuron group) x 256 tokens:
//                                              gate|up in one N = 2 NS MMA, SiLU * up, H in bf16
//   for every mt:                  DOWN(mt)    256 tokens x 256 output columns x one run of the K range (kept groups),
//                                              accumulators ADDED into the residual stream h
// (Token-tile-major on purpose: with the token tiles of a group next to each other the weights come from HBM only
// once, but the tiles of a block then all end together and the block boundary costs more than the second read.)
// Between the blocks the rows of the next input, x_l = bf16(rmsnorm(h)), are written row by row by whichever
// epilogue warps are waiting at that moment (for their tile's accumulators or for their next tile): a row of token
// tile mt is open as soon as every DOWN(l-1, mt) tile has been added.  This keeps the normalisation off the queue: a
// queue item taken by a CTA whose epilogue is still busy with a long tile would hold up every tile behind it.
// A tile waits only for work that comes before it in this order (all waits are on counters in global memory):
// HIDDEN and PRED for the x rows of their token tile, DOWN for the HIDDEN tiles of the groups it is about to read,
// and a CTA enters block l when the selection of block l is out.  Tiles are claimed in order by CTAs that are
// already running, and rows are normalised by warps that are otherwise only waiting, so whatever is waited for is
// owed by a running CTA that waits only for still earlier work: no co-residency assumption and no grid barrier, and
// no SM idles at a block boundary while another token tile still has work.  Only kept groups are computed (the merge is the sum of what
// was computed).  The mean over tokens of the per-token scores is computed as W2 * mean_t act(W1 x_t): the second
// layer is linear, so the two are the same number up to rounding.
// Warp roles: warp 0 claims items and issues the TMA loads, warp 1 issues the MMAs (and owns the 512 TMEM columns),
// warps 2..9 are the epilogue (two per TMEM lane quadrant, each takes half of the columns).  Every wait is bounded;
// a wait that runs out raises a global abort word and HALO_DEV_TIMEOUT, every CTA drains its copies, frees its
// TMEM and returns.
#include <algorithm>

#include "common.cuh"
#include "ffn_math.cuh"
#include "prompt_stack.cuh"
#include "select_device.cuh"
#include "umma.cuh"

namespace halo {

constexpr int kPsEpiWarps = 8;
constexpr int kPsEpiThreads = 32 * kPsEpiWarps;
constexpr int kPsThreads = 64 + kPsEpiThreads;
constexpr int kPsStages = 3;
constexpr int kPsBM = 128, kPsBK = 64, kPsUK = 16;
constexpr int kPsTile = 256;                                   // tokens per tile (two halves of 128)
constexpr int kPsBN = 256;                                     // output columns of a down tile / units of a predictor tile
constexpr uint32_t kPsAHalf = kPsBM * kPsBK * 2;
constexpr uint32_t kPsABytes = 2 * kPsAHalf;
constexpr uint32_t kPsStageBytes = kPsABytes + kPsBK * kPsBN * 2;   // 64 KiB
constexpr uint32_t kPsBBlock = kPsBK * 64 * 2;                 // one 64-column block of an MN-major B tile
constexpr int kPsEpiPitch = 20;                                // floats per staged row of a 32 x 16 chunk
constexpr size_t kPsScratchBytes = static_cast<size_t>(kPsEpiWarps) * 32 * kPsEpiPitch * sizeof(float);
constexpr int kPsCtlHeader = 16;                               // word 0: abort
constexpr int kPsBlockHeader = 8;                              // 0 queue, 1 predictor parts done, 2 selection published
// then per token tile: down tiles done, x rows claimed, x rows done; then per (token tile, kept position): hidden ready
constexpr unsigned kPsReadyPerHidden = kPsEpiWarps;            // counter increments per finished tile

enum PsKind { PS_HIDDEN = 1, PS_PRED = 2, PS_DOWN = 3, PS_NONE = 4 };

struct PsSmem {
    uint64_t full[4];
    uint64_t empty[4];
    uint64_t acc_full;
    uint64_t acc_empty;
    uint64_t item_full[2];
    uint64_t item_empty[2];
    int item_ring[2];
    uint32_t tmem_base;
    int abort_flag;
    int sel_flag;
    int norm_open;     // normalisation stages (block * tiles_x + token tile) known to be open, monotone
};

// scratch of the selection, aliased with the epilogue's staging chunks (never in use at the same time)
struct PsSelScratch {
    float zsum[1024];
    float score[HALO_MAX_GROUPS];
    SelectSmem sel;
};
static_assert(sizeof(PsSelScratch) <= kPsScratchBytes, "selection scratch must fit in the staging area");

struct PsGeom { int nk, nkv, n_pred, units, n_down_mt, per_mt, first_down, n_items; };
struct PsItem { int kind, mt, a, b; };

__device__ __forceinline__ PsGeom ps_geom(const PromptParams& P, int l, int nk) {
    PsGeom q;
    q.nk = nk;
    q.nkv = nk * P.subs;
    q.n_pred = (l + 1 < P.L) ? P.tiles_x * P.n_pn : 0;
    q.units = nk * (P.S / kPsBK);
    q.n_down_mt = q.units > 0 ? P.n_tn * P.z_cuts : 0;
    q.per_mt = q.nkv;
    q.first_down = P.tiles_x * q.per_mt + q.n_pred;
    q.n_items = q.first_down + P.tiles_x * q.n_down_mt;
    return q;
}

// HIDDEN: a = hidden tile of the token tile (kept position * subs + part); PRED: a = unit tile; DOWN: a = column
// tile, b = K run.
__device__ __forceinline__ PsItem ps_decode(const PromptParams& P, const PsGeom& q, int t) {
    PsItem it{PS_NONE, 0, 0, 0};
    if (t < q.first_down) {
        const int last = P.tiles_x - 1;
        int mt = q.per_mt > 0 ? t / q.per_mt : last;
        if (mt > last) mt = last;
        int u = t - mt * q.per_mt;
        if (mt == last) {
            if (u < q.n_pred) { it.kind = PS_PRED; it.mt = u / P.n_pn; it.a = u - it.mt * P.n_pn; return it; }
            u -= q.n_pred;
        }
        it.kind = PS_HIDDEN; it.mt = mt; it.a = u;
        return it;
    }
    const int u = t - q.first_down;
    it.kind = PS_DOWN;
    it.mt = u / q.n_down_mt;
    const int w = u - it.mt * q.n_down_mt;
    it.b = w / P.n_tn;
    it.a = w - it.b * P.n_tn;
    return it;
}

__device__ __forceinline__ unsigned* ps_block_ctl(const PromptParams& P, int l) {
    return P.ctl + kPsCtlHeader + static_cast<size_t>(l) * P.ctl_stride;
}
__device__ __forceinline__ unsigned* ps_ddone(const PromptParams& P, int l, int mt) { return ps_block_ctl(P, l) + kPsBlockHeader + mt; }
__device__ __forceinline__ unsigned* ps_nclaim(const PromptParams& P, int l, int mt) {
    return ps_block_ctl(P, l) + kPsBlockHeader + P.tiles_x + mt;
}
__device__ __forceinline__ unsigned* ps_ndone(const PromptParams& P, int l, int mt) {
    return ps_block_ctl(P, l) + kPsBlockHeader + 2 * P.tiles_x + mt;
}
__device__ __forceinline__ unsigned* ps_hready(const PromptParams& P, int l, int mt, int kp) {
    return ps_block_ctl(P, l) + kPsBlockHeader + 3 * P.tiles_x + mt * P.G + kp;
}

__device__ __forceinline__ bool ps_mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    if (*abort_flag) return false;
    if (mbar_wait_bounded(bar, parity, abort_flag)) return true;
    *abort_flag = 1;
    return false;
}

// Bounded wait until *ctr >= target (acquire); also ends when this CTA or any other has given up.
__device__ __forceinline__ bool ps_wait_ge(const unsigned* ctr, unsigned target, volatile int* abort_flag,
                                           const unsigned* abort_word) {
    if (target == 0u || ld_acquire_gpu(ctr) >= target) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    for (;;) {
        if (*abort_flag) return false;
        if (ld_acquire_gpu(ctr) >= target) return true;
        __nanosleep(32);
        if ((++spins & 15u) == 0u &&
            (ld_acquire_gpu(abort_word) != 0u || clock64() - t0 > static_cast<long long>(kWaitLimitCycles))) {
            *abort_flag = 1;
            return false;
        }
    }
}

__device__ __forceinline__ void ps_epi_barrier() { asm volatile("bar.sync 2, %0;" ::"n"(kPsEpiThreads) : "memory"); }
struct PsEpiSync {
    __device__ __forceinline__ void operator()() const { ps_epi_barrier(); }
};

__device__ __forceinline__ unsigned long long ps_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ int ps_down_units_of(const PromptParams& P, int nk) { return nk * (P.S / kPsBK); }

template <int NS>
__global__ void __launch_bounds__(kPsThreads, 1)
prompt_stack_kernel(const __grid_constant__ PromptParams P) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    PsSmem& sm = *reinterpret_cast<PsSmem*>(smem_raw + static_cast<size_t>(kPsStages) * kPsStageBytes);
    unsigned char* const scratch = smem_raw + static_cast<size_t>(kPsStages) * kPsStageBytes + 256;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int T = P.T, d = P.d, S = P.S, G = P.G, L = P.L;
    const int n_kt1 = d / kPsBK, k_per_group = S / kPsBK;
    unsigned* const abort_word = P.ctl;

    if (tid == 0) {
        for (int s = 0; s < kPsStages; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 1); }
        mbar_init(&sm.acc_full, 1);
        mbar_init(&sm.acc_empty, kPsEpiWarps);
        for (int b = 0; b < 2; ++b) { mbar_init(&sm.item_full[b], 1); mbar_init(&sm.item_empty[b], 1 + kPsEpiWarps); }
        sm.abort_flag = 0;
        sm.sel_flag = 0;
        sm.norm_open = 0;
        mbar_fence_init();
    }
    if (warp == 1) { tmem_alloc(&sm.tmem_base, 512); tmem_relinquish_alloc_permit(); }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    volatile int* abort_flag = &sm.abort_flag;
    const uint32_t tmem = sm.tmem_base;
    const CUtensorMap* const maps_x = P.maps + 3 * L;
    const CUtensorMap* const maps_h = P.maps + 3 * L + 2;

    if (warp == 0) {
        // ======================================== loader ========================================
        if (lane == 0) {
            int it = 0, n_ring = 0;
            bool alive = true;
            // x and H tiles are re-read by many CTAs and must stay in L2 while the weights stream through it
            const uint64_t keep = l2_policy_evict_last(), stream = l2_policy_evict_first();
            const int ahead = P.l2_ahead;
            auto post = [&](int entry) -> bool {
                const int slot = n_ring & 1;
                if (n_ring >= 2 && !ps_mbar_wait(&sm.item_empty[slot], ((n_ring >> 1) - 1) & 1, abort_flag)) return false;
                sm.item_ring[slot] = entry;
                mbar_arrive(&sm.item_full[slot]);
                ++n_ring;
                return true;
            };
            const bool tracing = P.trace != nullptr;
            long long wait_empty = 0, wait_dep = 0, wait_hready = 0, wait_sel = 0;
            auto stage_acquire = [&](int& s) -> bool {
                s = it % kPsStages;
                if (it < kPsStages) return true;
                const long long c0 = tracing ? clock64() : 0;
                const bool ok = ps_mbar_wait(&sm.empty[s], ((it / kPsStages) - 1) & 1, abort_flag);
                if (tracing) wait_empty += clock64() - c0;
                return ok;
            };
            for (int l = 0; l < L && alive; ++l) {
                unsigned* const cb = ps_block_ctl(P, l);
                const long long c_sel = tracing ? clock64() : 0;
                if (l > 0 && !ps_wait_ge(&cb[2], 1u, abort_flag, abort_word)) { alive = false; break; }
                if (tracing) wait_sel += clock64() - c_sel;
                const PersistSel* sb = &P.sel[l];
                const int nk = max(0, min(__ldcg(&sb->n_keep), G));
                const PsGeom q = ps_geom(P, l, nk);
                const CUtensorMap* const map_w = P.maps + 3 * l;
                const CUtensorMap* const map_wd = map_w + 1;
                const CUtensorMap* const map_w1 = P.maps + 3 * (l + 1 < L ? l + 1 : l) + 2;   // predictor of block l+1
                const CUtensorMap* const map_x = maps_x + (l & 1);
                const CUtensorMap* const map_h = maps_h + (l & 1);
                for (;;) {
                    const int t = static_cast<int>(min(atomicAdd(&cb[0], 1u), 0x000fffffu));
                    if (t >= q.n_items) break;
                    if (!post((l << 20) | t)) { alive = false; break; }
                    const PsItem im = ps_decode(P, q, t);
                    const int m0 = im.mt * kPsTile;
                    if (im.kind == PS_HIDDEN || im.kind == PS_PRED) {
                        // the rows of x_l this tile reads must have been written (by NORM items of any CTA)
                        const int mt_lo = im.kind == PS_HIDDEN ? im.mt : 0, mt_hi = im.kind == PS_HIDDEN ? im.mt + 1 : P.tiles_x;
                        const long long c0 = tracing ? clock64() : 0;
                        for (int mt = mt_lo; mt < mt_hi && alive; ++mt)
                            alive = ps_wait_ge(ps_ndone(P, l, mt), kPsTile, abort_flag, abort_word);
                        if (tracing) wait_dep += clock64() - c0;
                        if (!alive) break;
                        fence_proxy_async_all();   // their generic-proxy stores before this thread's TMA reads
                        int row_a, row_b, rows_b;
                        const CUtensorMap* map_b;
                        if (im.kind == PS_HIDDEN) {
                            const int ki = im.a / P.subs, n_off = (im.a - ki * P.subs) * NS;
                            int g = __ldcg(&sb->keep_list[ki]);
                            if (g < 0 || g >= G) g = 0;   // cannot happen: the list is this kernel's own
                            row_a = (g * 3 + 0) * S + n_off;
                            row_b = (g * 3 + 1) * S + n_off;
                            rows_b = NS;
                            map_b = map_w;
                        } else {
                            row_a = im.a * kPsBN;
                            row_b = row_a + 128;
                            rows_b = 128;
                            map_b = map_w1;
                        }
                        // optional: the weight rows (from HBM) are started towards L2 `ahead` K steps early
                        for (int kt = 0; kt < min(ahead, n_kt1); ++kt) {
                            tma_prefetch_2d(map_b, kt * kPsBK, row_a);
                            tma_prefetch_2d(map_b, kt * kPsBK, row_b);
                        }
                        for (int kt = 0; kt < n_kt1; ++kt, ++it) {
                            if (ahead > 0 && kt + ahead < n_kt1) {
                                tma_prefetch_2d(map_b, (kt + ahead) * kPsBK, row_a);
                                tma_prefetch_2d(map_b, (kt + ahead) * kPsBK, row_b);
                            }
                            int s;
                            if (!stage_acquire(s)) { alive = false; break; }
                            unsigned char* st = smem_raw + static_cast<size_t>(s) * kPsStageBytes;
                            mbar_arrive_expect_tx(&sm.full[s], kPsABytes + 2u * static_cast<uint32_t>(rows_b) * kPsBK * 2u);
                            tma_load_2d_hint(st, map_x, kt * kPsBK, m0, &sm.full[s], keep);
                            tma_load_2d_hint(st + kPsAHalf, map_x, kt * kPsBK, m0 + kPsBM, &sm.full[s], keep);
                            tma_load_2d_hint(st + kPsABytes, map_b, kt * kPsBK, row_a, &sm.full[s], stream);
                            tma_load_2d_hint(st + kPsABytes + rows_b * (kPsBK * 2), map_b, kt * kPsBK, row_b, &sm.full[s], stream);
                        }
                    } else if (im.kind == PS_DOWN) {
                        const int n0 = im.a * kPsBN;
                        const int kt_lo = static_cast<int>(static_cast<long long>(q.units) * im.b / P.z_cuts);
                        const int kt_hi = static_cast<int>(static_cast<long long>(q.units) * (im.b + 1) / P.z_cuts);
                        int checked = -1, g = 0;
                        auto prefetch_down = [&](int kt) {
                            const int p = kt / k_per_group, kk2 = kt - p * k_per_group;
                            int gp = __ldcg(&sb->keep_list[p]);
                            if (gp < 0 || gp >= G) gp = 0;
                            const int krow = (gp * 3 + 2) * S + kk2 * kPsBK;
#pragma unroll
                            for (int nb = 0; nb < kPsBN / 64; ++nb) tma_prefetch_2d(map_wd, n0 + nb * 64, krow);
                        };
                        for (int kt = kt_lo; kt < min(kt_lo + ahead, kt_hi); ++kt) prefetch_down(kt);
                        for (int kt = kt_lo; kt < kt_hi; ++kt, ++it) {
                            if (ahead > 0 && kt + ahead < kt_hi) prefetch_down(kt + ahead);
                            const int p = kt / k_per_group, kk2 = kt - p * k_per_group;
                            if (p != checked) {
                                // the hidden tiles of this group and token tile must have been written
                                const long long c0 = tracing ? clock64() : 0;
                                if (!ps_wait_ge(ps_hready(P, l, im.mt, p), kPsReadyPerHidden * P.subs, abort_flag, abort_word)) {
                                    alive = false;
                                    break;
                                }
                                if (tracing) wait_hready += clock64() - c0;
                                fence_proxy_async_all();
                                g = __ldcg(&sb->keep_list[p]);
                                if (g < 0 || g >= G) g = 0;
                                checked = p;
                            }
                            int s;
                            if (!stage_acquire(s)) { alive = false; break; }
                            unsigned char* st = smem_raw + static_cast<size_t>(s) * kPsStageBytes;
                            mbar_arrive_expect_tx(&sm.full[s], kPsStageBytes);
                            tma_load_2d_hint(st, map_h, p * S + kk2 * kPsBK, m0, &sm.full[s], keep);
                            tma_load_2d_hint(st + kPsAHalf, map_h, p * S + kk2 * kPsBK, m0 + kPsBM, &sm.full[s], keep);
                            const int krow = (g * 3 + 2) * S + kk2 * kPsBK;
#pragma unroll
                            for (int nb = 0; nb < kPsBN / 64; ++nb)
                                tma_load_2d_hint(st + kPsABytes + nb * kPsBBlock, map_wd, n0 + nb * 64, krow, &sm.full[s], stream);
                        }
                    }
                    if (!alive) break;
                }
            }
            if (alive) post(-1);
            if (tracing) {
                P.trace[static_cast<size_t>(blockIdx.x) * 16 + 8] = static_cast<unsigned long long>(wait_empty);
                P.trace[static_cast<size_t>(blockIdx.x) * 16 + 9] = static_cast<unsigned long long>(wait_dep);
                P.trace[static_cast<size_t>(blockIdx.x) * 16 + 5] = static_cast<unsigned long long>(wait_hready);
                P.trace[static_cast<size_t>(blockIdx.x) * 16 + 6] = static_cast<unsigned long long>(wait_sel);
            }
            if (*abort_flag) {   // let outstanding copies land before the CTA goes away
                int never = 0;
                for (int k = max(0, it - kPsStages); k < it; ++k)
                    mbar_wait_bounded(&sm.full[k % kPsStages], (k / kPsStages) & 1, &never);
            }
        }
    } else if (warp == 1) {
        // ======================================== MMA issuer ========================================
        if (lane == 0) {
            constexpr uint32_t idesc_down = umma_idesc_bf16(kPsBM, kPsBN, true);
            constexpr uint32_t idesc_hidden = umma_idesc_bf16(kPsBM, 2 * NS, false);
            constexpr uint32_t idesc_pred = umma_idesc_bf16(kPsBM, kPsBN, false);
            int it = 0, seg = 0, cur_l = -1;
            PsGeom q{};
            bool alive = true;
            const bool tracing = P.trace != nullptr;
            long long wait_full[2] = {0, 0}, wait_acc = 0, busy[2] = {0, 0};
            for (int n = 0; alive; ++n) {
                if (!ps_mbar_wait(&sm.item_full[n & 1], (n >> 1) & 1, abort_flag)) break;
                const int entry = sm.item_ring[n & 1];
                mbar_arrive(&sm.item_empty[n & 1]);
                if (entry < 0) break;
                const int l = entry >> 20, t = entry & 0xfffff;
                if (l != cur_l) { cur_l = l; q = ps_geom(P, l, max(0, min(__ldcg(&P.sel[l].n_keep), G))); }
                const PsItem im = ps_decode(P, q, t);
                int k_lo = 0, k_hi = n_kt1;
                if (im.kind == PS_DOWN) {
                    k_lo = static_cast<int>(static_cast<long long>(q.units) * im.b / P.z_cuts);
                    k_hi = static_cast<int>(static_cast<long long>(q.units) * (im.b + 1) / P.z_cuts);
                    if (k_lo >= k_hi) continue;
                }
                const long long c_start = tracing ? clock64() : 0;
                if (seg >= 1 && !ps_mbar_wait(&sm.acc_empty, (seg - 1) & 1, abort_flag)) break;
                if (tracing) wait_acc += clock64() - c_start;
                tcgen05_fence_after_sync();
                const int tk = im.kind == PS_DOWN ? 1 : 0;
                const uint32_t idesc = im.kind == PS_DOWN ? idesc_down : (im.kind == PS_HIDDEN ? idesc_hidden : idesc_pred);
                const uint32_t half_cols = im.kind == PS_HIDDEN ? 2 * NS : kPsBN;   // TMEM columns per 128-token half
                for (int kt = k_lo; kt < k_hi; ++kt, ++it) {
                    const int s = it % kPsStages;
                    const long long c0 = tracing ? clock64() : 0;
                    if (!ps_mbar_wait(&sm.full[s], (it / kPsStages) & 1, abort_flag)) { alive = false; break; }
                    if (tracing) wait_full[tk] += clock64() - c0;
                    tcgen05_fence_after_sync();
                    const uint32_t a0 = smem_u32(smem_raw + static_cast<size_t>(s) * kPsStageBytes);
#pragma unroll
                    for (int kk = 0; kk < kPsBK / kPsUK; ++kk) {
                        // K-major B (weight rows): 32 bytes per MMA further; MN-major B (down rows): 16 K-rows = 2 KiB
                        const uint64_t b = im.kind == PS_DOWN ? umma_smem_desc(a0 + kPsABytes + kk * 2048, kPsBBlock, 1024)
                                                              : umma_smem_desc(a0 + kPsABytes + kk * 32, 16, 1024);
#pragma unroll
                        for (int mh = 0; mh < 2; ++mh) {
                            const uint64_t a = umma_smem_desc(a0 + mh * kPsAHalf + kk * 32, 16, 1024);
                            umma_bf16(tmem + mh * half_cols, a, b, idesc, (kt > k_lo) || (kk > 0));
                        }
                    }
                    umma_commit(&sm.empty[s]);
                }
                if (!alive) break;
                umma_commit(&sm.acc_full);
                ++seg;
                if (tracing) busy[tk] += clock64() - c_start;
            }
            if (tracing) {
                unsigned long long* tr = P.trace + static_cast<size_t>(blockIdx.x) * 16;
                tr[10] = static_cast<unsigned long long>(wait_full[0]);
                tr[11] = static_cast<unsigned long long>(wait_full[1]);
                tr[12] = static_cast<unsigned long long>(wait_acc);
                tr[13] = static_cast<unsigned long long>(busy[0]);
                tr[14] = static_cast<unsigned long long>(busy[1]);
            }
        }
    } else {
        // ======================================== epilogue ========================================
        const int e = warp - 2, quad = warp & 3, half = e >> 2, te = tid - 64;
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(quad * 32) << 16);
        float* const stage = reinterpret_cast<float*>(scratch) + e * (32 * kPsEpiPitch);
        int seg = 0, cur_l = -1;
        PsGeom q{};
        // ---- normalisation in the background: stage = block * tiles_x + token tile, in order ----
        const int n_stages = L * P.tiles_x;
        int norm_stage = 0;
        // One row of the open stage, if there is one left to take.  Returns false when there is nothing to do now.
        auto norm_help = [&]() -> bool {
            while (norm_stage < n_stages) {
                const int l = norm_stage / P.tiles_x, mt = norm_stage - l * P.tiles_x;
                if (norm_stage >= *reinterpret_cast<volatile int*>(&sm.norm_open)) {
                    // is it open?  x_l rows of token tile mt need every down tile of block l-1 on that token tile.
                    // Only the first epilogue warp asks global memory (one poller per CTA); the others follow the
                    // word it leaves in shared memory.  (All eight warps take rows: with one helper per CTA the
                    // prompt took 8 % longer - the rows are on the critical path of the block boundary.)
                    if (e != 0) return false;
                    bool open = true;
                    if (lane == 0 && l > 0) {
                        open = l == 1 || ld_acquire_gpu(ps_block_ctl(P, l - 1) + 2) != 0u;   // block l-1's kept count is out
                        if (open) {
                            const int nk_prev = max(0, min(__ldcg(&P.sel[l - 1].n_keep), G));
                            const unsigned target = ps_down_units_of(P, nk_prev) > 0
                                                        ? static_cast<unsigned>(P.n_tn * P.z_cuts) * kPsEpiWarps : 0u;
                            open = ld_acquire_gpu(ps_ddone(P, l - 1, mt)) >= target;
                        }
                    }
                    open = __shfl_sync(0xffffffffu, open ? 1 : 0, 0) != 0;
                    if (!open) return false;
                    if (lane == 0) atomicMax(&sm.norm_open, norm_stage + 1);
                }
                if (l > 0) (void)ld_acquire_gpu(ps_ddone(P, l - 1, mt));   // every lane orders its own reads of h
                unsigned r = 0;
                if (lane == 0) r = atomicAdd(ps_nclaim(P, l, mt), 1u);
                r = __shfl_sync(0xffffffffu, r, 0);
                if (r >= static_cast<unsigned>(kPsTile)) { ++norm_stage; continue; }   // all rows taken: next stage
                const int row = mt * kPsTile + static_cast<int>(r);
                if (row < T) {
                    const float* hr = P.h + static_cast<size_t>(row) * d;
                    float ss = 0.0f;
                    for (int c = lane * 4; c < d; c += 128) {
                        const float4 v = __ldcg(reinterpret_cast<const float4*>(hr + c));
                        ss = fmaf(v.x, v.x, fmaf(v.y, v.y, fmaf(v.z, v.z, fmaf(v.w, v.w, ss))));
                    }
                    ss = warp_sum(ss);
                    const float scale = 1.0f / sqrtf(ss / static_cast<float>(d) + 1e-5f);
                    __nv_bfloat16* xr = P.x[l & 1] + static_cast<size_t>(row) * d;
                    __nv_bfloat16* xt = P.tap_x ? P.tap_x + (static_cast<size_t>(l) * T + row) * d : nullptr;
                    for (int c = lane * 8; c < d; c += 256) {
                        const float4 a = __ldcg(reinterpret_cast<const float4*>(hr + c));
                        const float4 b = __ldcg(reinterpret_cast<const float4*>(hr + c + 4));
                        const __nv_bfloat162 p0 = __floats2bfloat162_rn(a.x * scale, a.y * scale);
                        const __nv_bfloat162 p1 = __floats2bfloat162_rn(a.z * scale, a.w * scale);
                        const __nv_bfloat162 p2 = __floats2bfloat162_rn(b.x * scale, b.y * scale);
                        const __nv_bfloat162 p3 = __floats2bfloat162_rn(b.z * scale, b.w * scale);
                        const uint4 packed = make_uint4(*reinterpret_cast<const uint32_t*>(&p0), *reinterpret_cast<const uint32_t*>(&p1),
                                                        *reinterpret_cast<const uint32_t*>(&p2), *reinterpret_cast<const uint32_t*>(&p3));
                        *reinterpret_cast<uint4*>(xr + c) = packed;
                        if (xt) *reinterpret_cast<uint4*>(xt + c) = packed;
                    }
                }
                fence_proxy_async_all();   // x is read by TMA
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(ps_ndone(P, l, mt), 1u);
                return true;
            }
            return false;
        };
        // Bounded wait for an mbarrier phase during which this warp normalises rows when any are open.
        auto wait_helping = [&](uint64_t* bar, uint32_t parity) -> bool {
            if (*abort_flag) return false;
            if (mbar_try_wait(bar, parity)) return true;
            const long long t0 = clock64();
            uint32_t spins = 0;
            for (;;) {
                if (mbar_try_wait(bar, parity)) return true;
                if (!norm_help()) __nanosleep(300);
                if ((++spins & 7u) == 0u) {
                    if (*abort_flag) return false;
                    if (ld_acquire_gpu(abort_word) != 0u || clock64() - t0 > static_cast<long long>(kWaitLimitCycles)) {
                        *abort_flag = 1;
                        return false;
                    }
                }
            }
        };
        const bool tracing = P.trace != nullptr && e == 0 && lane == 0;
        unsigned long long t_mark = tracing ? ps_timer_ns() : 0ull, t_first = t_mark;
        unsigned long long acc_ns[6] = {0, 0, 0, 0, 0, 0};
        for (int n = 0;; ++n) {
            if (!wait_helping(&sm.item_full[n & 1], (n >> 1) & 1)) break;
            const int entry = sm.item_ring[n & 1];
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.item_empty[n & 1]);
            if (entry < 0) break;
            if (tracing) { const unsigned long long now = ps_timer_ns(); acc_ns[4] += now - t_mark; t_mark = now; ++acc_ns[5]; }
            unsigned long long* item_log = nullptr;
            if (tracing && n < P.trace_items) {
                item_log = P.trace + static_cast<size_t>(gridDim.x) * 16 + (static_cast<size_t>(blockIdx.x) * P.trace_items + n) * 3;
                item_log[0] = static_cast<unsigned long long>(entry) + 1ull;
                item_log[1] = t_mark;
            }
            const int l = entry >> 20, t = entry & 0xfffff;
            if (l != cur_l) { cur_l = l; q = ps_geom(P, l, max(0, min(__ldcg(&P.sel[l].n_keep), G))); }
            const PsItem im = ps_decode(P, q, t);
            const int m0 = im.mt * kPsTile;
            if (im.kind == PS_HIDDEN) {
                const int ki = im.a / P.subs, n_off = (im.a - ki * P.subs) * NS;
                const bool ok = wait_helping(&sm.acc_full, seg & 1);
                tcgen05_fence_after_sync();
                __nv_bfloat16* Hb = P.H[l & 1];
#pragma unroll
                for (int mh = 0; mh < 2; ++mh) {
                    const int row = m0 + mh * kPsBM + quad * 32 + lane;
                    for (int c0 = half * (NS / 2); c0 < (half + 1) * (NS / 2); c0 += 32) {
                        uint32_t dg[32], du[32];
                        tmem_ld_32x32(lane_base + mh * 2 * NS + c0, dg);
                        tmem_ld_32x32(lane_base + mh * 2 * NS + NS + c0, du);
                        tmem_ld_wait();
                        if (ok && row < T) {
                            uint4* dst = reinterpret_cast<uint4*>(Hb + static_cast<size_t>(row) * P.h_cols +
                                                                  static_cast<size_t>(ki) * S + n_off + c0);
#pragma unroll
                            for (int qq = 0; qq < 4; ++qq) {
                                uint32_t packed[4];
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    const int i = qq * 8 + k * 2;
                                    const float h0 = silu_mul(__uint_as_float(dg[i]), __uint_as_float(du[i]));
                                    const float h1 = silu_mul(__uint_as_float(dg[i + 1]), __uint_as_float(du[i + 1]));
                                    const __nv_bfloat162 pk = __floats2bfloat162_rn(h0, h1);
                                    packed[k] = *reinterpret_cast<const uint32_t*>(&pk);
                                }
                                dst[qq] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                            }
                        }
                    }
                }
                // publish: every lane orders its own stores (towards the TMA reads of other CTAs too), then one lane
                // bumps the counter.  An aborted tile publishes nothing; its readers give up on their own.
                tcgen05_fence_before_sync();
                fence_proxy_async_all();
                __threadfence();
                __syncwarp();
                if (lane == 0) {
                    if (ok) atomicAdd(ps_hready(P, l, im.mt, ki), 1u);
                    mbar_arrive(&sm.acc_empty);
                }
                ++seg;
                if (tracing) { const unsigned long long now = ps_timer_ns(); acc_ns[1] += now - t_mark; t_mark = now; if (item_log) item_log[2] = now; }
                continue;
            }
            if (im.kind == PS_PRED) {
                const bool ok = wait_helping(&sm.acc_full, seg & 1);
                tcgen05_fence_after_sync();
                const int n0 = im.a * kPsBN;
                float* zp = P.zpart + (static_cast<size_t>((l + 1) & 1) * (P.tiles_x * 8)) * P.r_pad;
#pragma unroll
                for (int mh = 0; mh < 2; ++mh) {
                    float* zrow = zp + static_cast<size_t>((im.mt * 2 + mh) * 4 + quad) * P.r_pad + n0;
                    for (int c0 = half * 128; c0 < (half + 1) * 128; c0 += 32) {
                        uint32_t raw[32];
                        tmem_ld_32x32(lane_base + mh * kPsBN + c0, raw);
                        tmem_ld_wait();
                        float v[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            v[i] = __uint_as_float(raw[i]);
                            if (P.act == HALO_ACT_RELU) v[i] = fmaxf(v[i], 0.0f);
                        }
                        // column sums over the warp's 32 token rows by recursive halving: lane j ends with column j
                        // (rows beyond the prompt read as zero inputs and add nothing)
#pragma unroll
                        for (int off = 16; off >= 1; off >>= 1) {
                            const bool upper = (lane & off) != 0;
#pragma unroll
                            for (int i = 0; i < off; ++i) {
                                const float send = upper ? v[i] : v[i + off];
                                const float keep = upper ? v[i + off] : v[i];
                                v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
                            }
                        }
                        if (ok) zrow[c0 + lane] = v[0];
                    }
                }
                tcgen05_fence_before_sync();
                __threadfence();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&sm.acc_empty);
                    unsigned* const cb = ps_block_ctl(P, l);
                    const unsigned target = static_cast<unsigned>(q.n_pred) * kPsEpiWarps;
                    if (ok && atomicAdd(&cb[1], 1u) + 1u == target) sm.sel_flag = 1;
                }
                ++seg;
                ps_epi_barrier();
                if (sm.sel_flag) {
                    // this CTA finished the last part: scores and steps a2..a5 of block l+1, by the 256 epilogue threads
                    __threadfence();
                    PsSelScratch& ss = *reinterpret_cast<PsSelScratch*>(scratch);
                    const int r = P.r, parts = P.tiles_x * 8;
                    for (int c = te; c < r; c += kPsEpiThreads) {
                        float acc = 0.0f;
                        for (int p = 0; p < parts; ++p) acc += __ldcg(zp + static_cast<size_t>(p) * P.r_pad + c);   // fixed order
                        ss.zsum[c] = acc;
                    }
                    ps_epi_barrier();
                    const __nv_bfloat16* W2 = P.W2[l + 1];
                    const float inv_t = 1.0f / static_cast<float>(T);
                    for (int g = e; g < G; g += kPsEpiWarps) {
                        const uint4* wrow = reinterpret_cast<const uint4*>(W2 + static_cast<size_t>(g) * r);
                        float acc = 0.0f;
                        for (int c = lane; c < (r >> 3); c += 32) {
                            float w8[8];
                            Elem<__nv_bfloat16>::widen(__ldg(wrow + c), w8);
#pragma unroll
                            for (int k = 0; k < 8; ++k) acc = fmaf(w8[k], ss.zsum[c * 8 + k], acc);
                        }
                        acc = warp_sum(acc);
                        if (lane == 0) ss.score[g] = acc * inv_t;
                    }
                    ps_epi_barrier();
                    PersistSel* sb = &P.sel[l + 1];
                    select_block<kPsEpiThreads>(ss.sel, P.plan, G, ss.score, P.step, static_cast<uint32_t>(l + 1), 0, nullptr,
                                                sb->dev_of_group, sb->arrived, nullptr, sb->keep_list, &sb->n_keep, P.status,
                                                te, PsEpiSync());
                    __threadfence();
                    ps_epi_barrier();
                    if (te == 0) {
                        st_release_gpu(ps_block_ctl(P, l + 1) + 2, 1u);
                        sm.sel_flag = 0;
                    }
                    // records (optional), after publication
                    const size_t rec = static_cast<size_t>(l + 1);
                    const int n_dev = P.plan.n_dev;
                    for (int g = te; g < G; g += kPsEpiThreads) {
                        if (P.tap_scores) P.tap_scores[rec * G + g] = ss.score[g];
                        if (P.tap_keep_list) P.tap_keep_list[rec * G + g] = __ldcg(&sb->keep_list[g]);
                        if (P.tap_dev_of_group) P.tap_dev_of_group[rec * G + g] = __ldcg(&sb->dev_of_group[g]);
                    }
                    if (te < n_dev && P.tap_arrived) P.tap_arrived[rec * n_dev + te] = static_cast<uint8_t>(ss.sel.arrived[te]);
                    if (te == 0 && P.tap_n_keep) P.tap_n_keep[rec] = __ldcg(&sb->n_keep);
                    ps_epi_barrier();   // the scratch goes back to the staging chunks
                }
                if (tracing) { const unsigned long long now = ps_timer_ns(); acc_ns[2] += now - t_mark; t_mark = now; if (item_log) item_log[2] = now; }
                continue;
            }
            // ---- DOWN ----
            {
                const int n0 = im.a * kPsBN;
                const int k_lo = static_cast<int>(static_cast<long long>(q.units) * im.b / P.z_cuts);
                const int k_hi = static_cast<int>(static_cast<long long>(q.units) * (im.b + 1) / P.z_cuts);
                bool ok = true;
                if (k_lo < k_hi) {
                    ok = wait_helping(&sm.acc_full, seg & 1);
                    tcgen05_fence_after_sync();
#pragma unroll
                    for (int mh = 0; mh < 2; ++mh) {
                        const int row0 = m0 + mh * kPsBM + quad * 32;
                        float* out = P.h + static_cast<size_t>(row0) * d + n0;
                        for (int c0 = half * 128; c0 < (half + 1) * 128; c0 += 16) {
                            uint32_t v[16];
                            tmem_ld_32x16(lane_base + mh * kPsBN + c0, v);
                            tmem_ld_wait();
                            // the 32 x 16 chunk is turned through shared memory so that one reduction instruction
                            // covers 8 rows x 64 contiguous bytes instead of 32 rows x 16
#pragma unroll
                            for (int qq = 0; qq < 4; ++qq)
                                *reinterpret_cast<float4*>(stage + lane * kPsEpiPitch + 4 * qq) =
                                    make_float4(__uint_as_float(v[4 * qq]), __uint_as_float(v[4 * qq + 1]),
                                                __uint_as_float(v[4 * qq + 2]), __uint_as_float(v[4 * qq + 3]));
                            __syncwarp();
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const int rr = 8 * j + (lane >> 2), cq = (lane & 3) * 4;
                                const float4 w = *reinterpret_cast<const float4*>(stage + rr * kPsEpiPitch + cq);
                                if (ok && row0 + rr < T)
                                    red_add_v4f(out + static_cast<size_t>(rr) * d + c0 + cq, w.x, w.y, w.z, w.w);
                            }
                            __syncwarp();
                        }
                    }
                    tcgen05_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.acc_empty);
                    ++seg;
                }
                __threadfence();
                __syncwarp();
                if (lane == 0 && ok) atomicAdd(ps_ddone(P, l, im.mt), 1u);
                if (tracing) { const unsigned long long now = ps_timer_ns(); acc_ns[3] += now - t_mark; t_mark = now; if (item_log) item_log[2] = now; }
            }
        }
        if (tracing) {
            unsigned long long* tr = P.trace + static_cast<size_t>(blockIdx.x) * 16;
            for (int k = 0; k < 5; ++k) tr[k] = acc_ns[k];
            tr[7] = ps_timer_ns() - t_first;
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tcgen05_fence_after_sync(); tmem_dealloc(tmem, 512); }
    if (tid == 0 && *abort_flag) {
        atomicExch(abort_word, 1u);
        flag_status(P.status, HALO_DEV_TIMEOUT);
    }
}

// ---- host side ------------------------------------------------------------------------------------------------

bool prompt_stack_supported(const halo_ffn_shape& ffn, const halo_pred_shape& pred, int n_layers, int n_tok) {
    if (ffn.wdtype != HALO_BF16 || pred.wdtype != HALO_BF16) return false;
    if (n_tok <= kPsBM || ffn.d_model % 256 != 0) return false;
    if (ffn.group_size != 64 && ffn.group_size != 128 && ffn.group_size != 256) return false;
    const int G = ffn.d_ffn / ffn.group_size;
    if (G > HALO_MAX_GROUPS || pred.rank > 1024 || pred.rank % 8 != 0 || pred.d_in % kPsBK != 0) return false;
    if (n_layers >= 2048) return false;
    const long long tiles_x = (n_tok + kPsTile - 1) / kPsTile;
    const long long items = tiles_x * (4ll * G + (pred.rank + 255) / 256 + (ffn.d_model / 256) * 16ll);
    return items < (1ll << 20);
}

int prompt_stack_ctl_stride(int tiles_x, int G) { return (kPsBlockHeader + tiles_x * (G + 3) + 7) & ~7; }

size_t prompt_stack_ctl_bytes(int n_layers, int tiles_x, int G) {
    return sizeof(unsigned) * (kPsCtlHeader + static_cast<size_t>(n_layers) * prompt_stack_ctl_stride(tiles_x, G));
}

halo_status launch_prompt_stack(const PromptParams& P, cudaStream_t st) {
    const size_t smem = static_cast<size_t>(kPsStages) * kPsStageBytes + 256 + kPsScratchBytes + 1024;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return HALO_ERR_CUDA;
    if (P.S >= 128) {
        auto k = prompt_stack_kernel<128>;
        static bool once[64] = {};
        if (!ensure_dynamic_smem(k, smem, once)) return HALO_ERR_CUDA;
        k<<<n_sm, kPsThreads, smem, st>>>(P);
    } else {
        auto k = prompt_stack_kernel<64>;
        static bool once[64] = {};
        if (!ensure_dynamic_smem(k, smem, once)) return HALO_ERR_CUDA;
        k<<<n_sm, kPsThreads, smem, st>>>(P);
    }
    HALO_CHECK_LAUNCH();
    return HALO_OK;
}

}  // namespace halo
