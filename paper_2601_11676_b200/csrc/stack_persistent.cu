// Decode stack as ONE persistent cooperative kernel: all steps x blocks of the FFN stack, steps a1..a9 plus
// the glue between blocks, without leaving the device.
//
// One thread block per SM: a producer warp and 512 consumer threads around a ring of shared-memory stages fed
// by bulk asynchronous copies.  The producer's stream for block l of a step is
//     [rows of W1 of block l+1 owned by this thread block]   predictor hidden layer, one layer ahead (a1)
//     [batches of NB kept neurons of block l]                 gate/up dot products, SiLU*up, down rows (a6..a8)
//     [END marker]
// The last thread block streams nothing: it is the selector.  As soon as all hidden values of block l+1 are in
// (a counter), it computes the scores and steps a2..a5 and publishes the kept set (a flag); it takes no part in
// the grid barrier, so a selection never delays a block unless it takes longer than the block itself.  The
// stream is HBM-bound, so the SM given up for this costs nothing.
// and it runs ahead of the consumers by the ring depth, across the end of the block: while the consumers sit in
// the grid barrier and the glue, the next block's weights are already landing in shared memory.
// Batches are handed out dynamically (one atomic counter per block, fetched one batch ahead), so a slow or busy
// thread block simply takes fewer.  Only kept groups are ever computed, so the merge (a9) is the plain sum of
// what was computed: each thread block stages its column sums in shared memory and adds them to one of
// kAccBufs interleaved global buffers with ONE bulk reduction (cp.reduce.async.bulk, fp32 add, done by the copy
// engine in L2), then one grid-wide barrier, then every thread block redundantly sums the buffers,
// adds the residual, normalises, and keeps its own copy of x for the next block.
// Every wait (mbarrier, grid barrier, flags) is bounded to about a second; on a timeout the thread block takes
// a uniform exit, raises a global abort word and HALO_DEV_TIMEOUT, and every other thread block follows.
#include <algorithm>

#include "common.cuh"
#include "ffn_math.cuh"
#include "i4_math.cuh"
#include "select_device.cuh"
#include "stack_persistent.cuh"
#include "tma.cuh"
#include "umma.cuh"

namespace halo {

constexpr int kPC = 512;                 // consumer threads
constexpr int kPCWarps = kPC / 32;
constexpr int kPThreads = kPC + 32;      // + producer warp
constexpr int kPThreadsTM = kPC + 64;    // + producer warp + the warp that moves stages into tensor memory
constexpr int kTSlots = 5;               // stage slots in tensor memory
constexpr int kTSlotCols = 96;           // 32-bit columns per slot: 128 lanes x 96 x 4 B = 48 KB, one stage
constexpr int kTCols = 512;              // columns allocated (all of the SM's tensor memory)
constexpr int kHeaderBytes = 16 * 1024;  // PersistSmem
constexpr int kAccBufs = 2;              // interleaved accumulation buffers per block of the stack
constexpr int kFetchAhead = 3;           // batch-counter claims a producer keeps in flight (every claim made at the start of
                                         // a block is a batch that can no longer go to whoever turns out to be faster:
                                         // 6 / 4 / 3 / 2 / 1 measured 3080 / 3143 / 3170 / 3157 / 3166 tokens/s on the
                                         // TinyLlama shape, nine batches per thread block, and no difference at 7B)

enum StageType { ST_FFN = 0, ST_PRED = 1, ST_END = 3 };

struct PersistSmem {
    uint64_t full[8];
    uint64_t empty[8];
    int type[8];
    int arg0[8];   // FFN: 0 = compute, -1 = skip; PRED: first row
    int arg1[8];   // PRED: number of rows
    int abort_flag;
    int blocks_done;   // blocks of the stack whose grid barrier this thread block's consumers have passed
    int pad[2];
    __align__(16) float red[2][32];
    float reduce[32];
    float score[HALO_MAX_GROUPS];
    int kept_group[HALO_MAX_GROUPS];   // producer's table for the block it is issuing: group id or -1 per kept position
    SelectSmem sel;
    float red_h[2][2][32];   // I4 form: [half][parity][row]
    // second level of the ring, in tensor memory (TM form of the kernel)
    uint64_t tfull[8];
    uint64_t tempty[8];
    uint64_t tdrain;
    int ttype[8];
    int targ0[8];
    int targ1[8];
    uint32_t tmem_base;
};
static_assert(sizeof(PersistSmem) <= kHeaderBytes, "shared-memory header too large");

__device__ __forceinline__ void pc_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kPC) : "memory"); }
// barrier over the consumers that also ORs a flag across them (uniform result)
__device__ __forceinline__ bool pc_barrier_or(bool flag) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"(static_cast<uint32_t>(flag)), "n"(kPC)
        : "memory");
    return out != 0;
}
// I4 form: the consumers work as two halves of 256 threads on alternate stages; barrier (with OR) over one half
__device__ __forceinline__ bool half_barrier_or(int half, bool flag) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, %2, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"(static_cast<uint32_t>(flag)), "r"(3 + half), "n"(kPC / 2)
        : "memory");
    return out != 0;
}
struct ConsumerSync {
    __device__ __forceinline__ void operator()() const { pc_barrier(); }
};

// Bounded spin until *word >= target (acquire); gives up early when the global abort word is set.
// counter += v with release semantics and no return value: the stores this thread made before it are visible to whoever
// acquires the counter (spin_until_ge), and the thread does not wait for the round trip
__device__ __forceinline__ void red_release_add(unsigned* word, unsigned v) {
    asm volatile("red.release.gpu.add.u32 [%0], %1;" ::"l"(word), "r"(v) : "memory");
}

__device__ __forceinline__ bool spin_until_ge(const unsigned* word, unsigned target, const unsigned* abort_word) {
    if (ld_acquire_gpu(word) >= target) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (true) {
        if (ld_acquire_gpu(word) >= target) return true;
        if ((++spins & 63u) == 0u) {
            if (ld_acquire_gpu(abort_word) != 0u) return false;
            if (clock64() - t0 > kWaitLimitCycles) return false;
        }
    }
}

__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// trace slots per (block of the stack, thread block)
enum TraceSlot { TR_BLOCK_START = 0, TR_FIRST_STAGE = 1, TR_STAGES_DONE = 2, TR_FLUSHED = 3, TR_BARRIER_DONE = 4,
                 TR_MERGED = 5, TR_X_READY = 6, TR_SELECT_NS = 7 };

// consumers + the mover warp, at the end of the TM form: nobody reads tensor memory after it
__device__ __forceinline__ void tm_join_barrier() { asm volatile("bar.sync 2, %0;" ::"n"(kPC + 32) : "memory"); }

// Shared-memory matrix descriptor without swizzle: 8 x 16-byte core matrices, `sbo` bytes from one group of 8 rows
// to the next, `lbo` bytes from one 16-byte column of core matrices to the next.
__device__ __forceinline__ uint64_t smem_desc_plain(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t dsc = 0;
    dsc |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    dsc |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
    dsc |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
    dsc |= 1ull << 46;
    return dsc;
}
// 4 KB of shared memory -> 128 lanes x 8 columns of tensor memory: with sbo = 128 and lbo = 2048, lane i receives the
// 16-byte chunk i of the first 2 KB in columns 0..3 and chunk i of the second 2 KB in columns 4..7.
__device__ __forceinline__ void tmem_cp_4k(uint32_t taddr, uint32_t smem_addr) {
    asm volatile("tcgen05.cp.cta_group::1.128x256b [%0], %1;" ::"r"(taddr), "l"(smem_desc_plain(smem_addr, 2048u, 128u))
                 : "memory");
}
template <int N>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&v)[N]) {
    static_assert(N == 4 || N == 8 || N == 16, "columns per load");
    if constexpr (N == 4) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3])
                     : "r"(taddr)
                     : "memory");
    } else if constexpr (N == 8) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                     : "r"(taddr)
                     : "memory");
    } else {
        tmem_ld_32x16(taddr, v);
    }
}

// TM = true: the ring has a second level in tensor memory.  A stage that has landed in shared memory is moved on at
// once (tcgen05.cp, issued by one thread of a fourth role, the mover warp) into one of kTSlots slots of the SM's
// 256 KB of tensor memory, which frees the shared-memory stage for the next bulk copy; the consumers read their
// operands from tensor memory (tcgen05.ld).  Shared memory plus tensor memory hold 9 stages (432 KB) instead of 4,
// enough for the producer to keep streaming the next block's weights through the whole of the flush / grid barrier /
// merge at the end of a block, so HBM does not fall idle there and does not have to ramp up again afterwards.
//   layout   row rho of a stage (gate rows, up rows, down rows), 2 KB piece pi of it: columns (rho * PPR + pi) * 4 .. + 3
//            of the slot; lane i holds the 16-byte chunk 128 * pi + i of the row.
//   phase 1  warp w reads lanes 32 * (w % 4) ..; the four warps w / 4 = 0..3 take rows w / 4, w / 4 + 4, ...; a thread
//            keeps the PPR chunks of x that meet its lane.
//   phase 2  thread tid owns the same columns as in the plain form (chunk tid % (512 / REP)), piece = chunk / 128.
// I4 = true: the FFN weights are int4 codes with one bf16 scale per 128 elements (the layout of halo_group_ffn_i4).
// A stage is a batch of NB = 8 neurons: three planes of code rows (d / 2 bytes each) and three runs of scales, six bulk
// copies.  Phase 1: warp w takes code row w of the 16 (8 gate, 8 up) against x kept in shared memory in the nibble
// pairing (XC = 16-byte chunks per lane); phase 2: 512 / (d / 16) replicas of d / 16 threads, a thread owns 16 columns;
// the replicas' sums meet in the one vector buffer in turn.  Predictor rows (bf16) ride the same ring, at most
// stage_bytes / (2 d) of them per stage, two warps per row against x (bf16) in shared memory.  Skeleton (selector,
// producer, grid barrier, merge, glue) as for bf16; the modes PRED_SERIAL and DETERMINISTIC are not built for it.
template <int NB, int XC, int P2, int REP, int STAGES, bool TM, bool I4>
__global__ void __launch_bounds__(TM ? kPThreadsTM : kPThreads, 1)
stack_decode_kernel(const __grid_constant__ PersistParams P) {
    static_assert(!I4 || (!TM && NB == 8 && P2 == 1 && REP == 1), "int4 shape");
    constexpr int ROWS = 2 * NB;
    constexpr int WPR = TM ? 4 : kPCWarps / ROWS;
    constexpr int PPR = XC;                       // TM: 2 KB pieces per row = chunks of x per thread
    static_assert((TM || WPR * ROWS == kPCWarps) && STAGES <= 8 && NB % REP == 0, "shape");
    static_assert(!TM || (P2 == 1 && ROWS % 4 == 0 && 3 * NB * PPR * 4 == kTSlotCols && (PPR == 2 || PPR == 4)), "TM shape");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    PersistSmem& sm = *reinterpret_cast<PersistSmem*>(smem_raw);
    // one vector buffer, used in turn for the fp32 column sums on their way out and for x (bf16) on its way in
    constexpr int kVecBytesPerCol = 4 * REP;
    unsigned char* vec_buf = smem_raw + kHeaderBytes;
    __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(vec_buf);
    // I4: behind the vector buffer, x in the nibble pairing [4][d/32] uint4 and its plain sums per 32 elements
    uint4* xp = reinterpret_cast<uint4*>(smem_raw + kHeaderBytes + static_cast<size_t>(P.d) * kVecBytesPerCol);
    float* xsum = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(xp) + static_cast<size_t>(P.d) * 2);
    unsigned char* ring = smem_raw + kHeaderBytes + static_cast<size_t>(P.d) * kVecBytesPerCol +
                          (I4 ? static_cast<size_t>(P.d) * 2 + ((static_cast<size_t>(P.d) / 32 * 4 + 127) & ~size_t(127)) : 0);

    const int d = P.d, S = P.S, G = P.G, L = P.L, r = P.r, n_dev = P.plan.n_dev;
    const int chunks = d >> 3;
    const uint32_t row_bytes = static_cast<uint32_t>(d) * 2u;                 // a bf16 row (predictor rows; FFN rows of the bf16 form)
    const uint32_t crow_bytes = static_cast<uint32_t>(d) / 2u;                // I4: a row of codes
    const uint32_t sc_bytes = static_cast<uint32_t>(d / 128) * 2u * NB;       // I4: scales of one plane of a batch
    const uint32_t plane_bytes = (I4 ? crow_bytes : row_bytes) * NB;
    const uint32_t stage_bytes = I4 ? 3u * (plane_bytes + sc_bytes) : 3u * plane_bytes;
    const int pred_rows = I4 ? min(8, static_cast<int>(stage_bytes / row_bytes)) : ROWS;   // predictor rows per stage
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int grid = gridDim.x, cta = blockIdx.x;
    const int workers = grid - 1;                 // thread blocks that stream weights; the last one selects
    const bool is_selector = (cta == workers);
    const int per_group = S / NB;
    unsigned* const sync_barrier = P.sync + 0;
    unsigned* const sync_abort = P.sync + 1;
    unsigned* const sync_zcount = P.sync + 2;
    unsigned* const sync_selready = P.sync + 3;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], TM ? 1 : (I4 ? kPCWarps / 2 : kPCWarps)); }
        if constexpr (TM) {
            // tfull: one arrival from the copies' completion, one from the mover after it wrote the slot's metadata
            for (int t = 0; t < kTSlots; ++t) { mbar_init(&sm.tfull[t], 2); mbar_init(&sm.tempty[t], kPCWarps); }
            mbar_init(&sm.tdrain, 1);
        }
        sm.abort_flag = 0;
        sm.blocks_done = 0;
        mbar_fence_init();
    }
    if constexpr (TM) {
        if (!is_selector && warp == kPCWarps + 1) {
            tmem_alloc(&sm.tmem_base, kTCols);
            tmem_relinquish_alloc_permit();
        }
        tcgen05_fence_before_sync();
    }
    __syncthreads();
    if constexpr (TM) tcgen05_fence_after_sync();
    volatile int* abort_flag = &sm.abort_flag;

    // =========================================== selector ===========================================
    if (is_selector) {
        if (warp >= kPCWarps) return;   // only the 512 "consumer" threads are used here
        bool bad = false;
        for (int step_i = 0; step_i < P.steps && !bad; ++step_i) {
            for (int lp = 1; lp < L && !bad; ++lp) {
                // prediction number n_pred (1-based over the run) = the selection of block lp of this step; its
                // hidden values are produced by the workers during block lp-1
                const unsigned n_pred = static_cast<unsigned>(step_i) * (L - 1) + lp;
                // W2 of this block is read once per token: start it towards L2 while the hidden values come in
                if (tid == 0) bulk_prefetch_l2(P.W2[lp], (static_cast<uint32_t>(G) * r * 2u) & ~15u);
                bool okz = true;
                if (tid == 0) okz = spin_until_ge(sync_zcount, n_pred * static_cast<unsigned>(r), sync_abort);
                bad = pc_barrier_or(!okz);
                if (bad) break;
                const unsigned long long t_sel = (P.trace && tid == 0) ? global_timer_ns() : 0ull;
                // a1 (second layer): s[g] = <W2[g], z>
                const float* zsrc = P.z + static_cast<size_t>(n_pred & 1u) * r;
                const __nv_bfloat16* W2 = P.W2[lp];
                const int zc = r >> 3;  // 16-byte chunks per W2 row
                for (int c0 = 0; c0 < zc; c0 += 32) {
                    const int c = c0 + lane;
                    float zv[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                    if (c < zc) {
                        const float4 z0 = __ldcg(reinterpret_cast<const float4*>(zsrc) + 2 * c);
                        const float4 z1 = __ldcg(reinterpret_cast<const float4*>(zsrc) + 2 * c + 1);
                        zv[0] = z0.x; zv[1] = z0.y; zv[2] = z0.z; zv[3] = z0.w;
                        zv[4] = z1.x; zv[5] = z1.y; zv[6] = z1.z; zv[7] = z1.w;
                    }
                    // groups warp, warp+16, ...: all row loads of a pass are issued before any is used
                    for (int g0 = warp; g0 < G; g0 += kPCWarps * 8) {
                        uint4 wv[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int g = g0 + u * kPCWarps;
                            wv[u] = (g < G && c < zc) ? __ldg(reinterpret_cast<const uint4*>(W2 + static_cast<size_t>(g) * r) + c)
                                                      : make_uint4(0, 0, 0, 0);
                        }
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int g = g0 + u * kPCWarps;
                            float w8[8];
                            Elem<__nv_bfloat16>::widen(wv[u], w8);
                            float dot = 0.0f;
#pragma unroll
                            for (int e = 0; e < 8; ++e) dot = fmaf(w8[e], zv[e], dot);
                            dot = warp_sum(dot);
                            if (lane == 0 && g < G) sm.score[g] = (c0 == 0 ? 0.0f : sm.score[g]) + dot;
                        }
                    }
                }
                pc_barrier();
                // a2..a5, written where the producers of block lp will read it
                PersistSel* sb = &P.sel[lp & 1];
                select_block<kPC>(sm.sel, P.plan, G, sm.score, P.step0 + static_cast<uint32_t>(step_i),
                                  static_cast<uint32_t>(lp), 0, nullptr, sb->dev_of_group, sb->arrived, nullptr,
                                  sb->keep_list, &sb->n_keep, P.status, tid, ConsumerSync());
                __threadfence();
                pc_barrier();
                if (tid == 0) st_release_gpu(sync_selready, n_pred);
                // records (optional), after publication: off everybody's critical path
                const size_t rec = static_cast<size_t>(step_i) * L + lp;
                for (int g = tid; g < G; g += kPC) {
                    if (P.tap_scores) P.tap_scores[rec * G + g] = sm.score[g];
                    if (P.tap_keep_list) P.tap_keep_list[rec * G + g] = __ldcg(&sb->keep_list[g]);
                    if (P.tap_dev_of_group) P.tap_dev_of_group[rec * G + g] = __ldcg(&sb->dev_of_group[g]);
                }
                if (tid < n_dev && P.tap_arrived) P.tap_arrived[rec * n_dev + tid] = static_cast<uint8_t>(sm.sel.arrived[tid]);
                if (tid == 0 && P.tap_n_keep) P.tap_n_keep[rec] = __ldcg(&sb->n_keep);
                if (P.trace && tid == 0 && n_pred - 1u < static_cast<unsigned>(P.trace_blocks))
                    P.trace[(static_cast<size_t>(n_pred - 1u) * grid + cta) * 8 + TR_SELECT_NS] = global_timer_ns() - t_sel;
                pc_barrier();   // sm.score / sm.sel are reused by the next selection
            }
        }
        if (bad && tid == 0) {
            atomicExch(sync_abort, 1u);
            flag_status(P.status, HALO_DEV_TIMEOUT);
        }
        return;
    }

    // =========================================== producer ===========================================
    if (warp == kPCWarps) {
        // Lane 0 issues every copy; the other lanes only help to build the per-block table of kept groups.
        int it = 0;
        unsigned qp = 0;  // running block counter of the producer
        int issued_in_block = 0;
        bool alive = true;
        volatile int* blocks_done = &sm.blocks_done;
        auto acquire = [&](int& s) -> bool {
            if (*abort_flag) return false;
            // Loads issued while the consumers synchronise delay that synchronisation (it queues behind them in
            // the memory system), so only the first cross_stages stages of a block may be issued before the
            // consumers are through the previous block's barrier.
            if (issued_in_block >= P.cross_stages && *blocks_done < static_cast<int>(qp)) {
                const long long t0 = clock64();
                while (*blocks_done < static_cast<int>(qp)) {
                    if (*abort_flag) return false;
                    if (clock64() - t0 > kWaitLimitCycles) { *abort_flag = 1; return false; }
                }
            }
            ++issued_in_block;
            s = it % STAGES;
            if (it >= STAGES) {
                const uint32_t use = static_cast<uint32_t>(it / STAGES);
                if (!mbar_wait_bounded(&sm.empty[s], (use - 1u) & 1u, abort_flag)) { *abort_flag = 1; return false; }
            }
            return true;
        };
        auto marker = [&](int type, int a0) -> bool {
            int s;
            if (!acquire(s)) return false;
            sm.type[s] = type; sm.arg0[s] = a0; sm.arg1[s] = 0;
            mbar_arrive(&sm.full[s]);
            ++it;
            return true;
        };
        for (int step_i = 0; step_i < P.steps && alive; ++step_i) {
            for (int l = 0; l < L && alive; ++l) {
                const PersistSel* sb = (l == 0) ? &P.sel[2] : &P.sel[l & 1];
                if (lane == 0) {
                    // (a) rows of a predictor that this thread block owns: the next block's, one layer ahead, beside
                    //     this block's stream; or (pred_serial) this block's own, in front of its stream
                    const int lp = P.pred_serial ? l : l + 1;
                    if (lp >= 1 && lp < L) {
                        const int r0 = static_cast<int>(static_cast<long long>(cta) * r / workers);
                        const int r1 = static_cast<int>(static_cast<long long>(cta + 1) * r / workers);
                        const __nv_bfloat16* W1 = P.W1[lp];
                        for (int row = r0; row < r1 && alive; row += pred_rows) {
                            const int n = min(pred_rows, r1 - row);
                            int s;
                            if (!acquire(s)) { alive = false; break; }
                            sm.type[s] = ST_PRED; sm.arg0[s] = row; sm.arg1[s] = n;
                            mbar_arrive_expect_tx(&sm.full[s], n * row_bytes);
                            bulk_copy_g2s(ring + static_cast<size_t>(s) * stage_bytes, W1 + static_cast<size_t>(row) * d,
                                          n * row_bytes, &sm.full[s]);
                            ++it;
                        }
                    }
                    // (b) the selection of this block must have been published
                    if (alive && l > 0) {
                        const unsigned need = static_cast<unsigned>(step_i) * (L - 1) + l;
                        if (!spin_until_ge(sync_selready, need, sync_abort)) { *abort_flag = 1; alive = false; }
                    }
                }
                alive = __shfl_sync(0xffffffffu, alive ? 1 : 0, 0) != 0;
                if (!alive) break;
                // lane 0's acquire orders only lane 0: every lane that is about to read the published selection
                // makes its own acquire load of the flag (it is already set, so this is one L2 read)
                if (l > 0) (void)ld_acquire_gpu(sync_selready);
                // (c) table of kept groups for this block: two dependent L2 reads, once per block instead of per batch
                int nk = __ldcg(&sb->n_keep);
                nk = max(0, min(nk, G));
                for (int ki = lane; ki < nk; ki += 32) {
                    const int g = __ldcg(&sb->keep_list[ki]);
                    bool ok = (g >= 0 && g < G);
                    if (ok) {
                        const int slot = __ldcg(&sb->dev_of_group[g]) + 1;
                        ok = (slot >= 0 && slot <= n_dev);
                    }
                    if (!ok) flag_status(P.status, HALO_DEV_BAD_INDEX);
                    sm.kept_group[ki] = ok ? g : -1;
                }
                __syncwarp();
                const long long U = static_cast<long long>(nk) * per_group;
                // (c') keep HBM busy while the consumers synchronise: the block's first batches go to L2 now, long
                //      before ring slots free up for them (whoever ends up consuming them)
                if (!I4 && lane < P.l2_ahead) {
                    const long long b = cta + static_cast<long long>(workers) * lane;
                    if (b < U) {
                        const int ki = static_cast<int>(b / per_group), j0 = static_cast<int>(b - static_cast<long long>(ki) * per_group) * NB;
                        const int g = sm.kept_group[ki];
                        if (g >= 0) {
                            const __nv_bfloat16* group = P.W[l] + static_cast<size_t>(g) * 3 * S * d;
                            bulk_prefetch_l2(group + static_cast<size_t>(j0) * d, plane_bytes);
                            bulk_prefetch_l2(group + static_cast<size_t>(S + j0) * d, plane_bytes);
                            bulk_prefetch_l2(group + static_cast<size_t>(2 * S + j0) * d, plane_bytes);
                        }
                    }
                }
                if (lane == 0) {
                    // (d) batches of kept neurons, handed out by the block's counter
                    unsigned* const ctr = P.sync + 32 + (qp & 31u);
                    const __nv_bfloat16* Wl = P.W[l];
                    // The first batch is fixed, the rest come from the counter.  kFetchAhead claims are kept in
                    // flight so that the round trip of the atomic (a microsecond and more while HBM is saturated) is
                    // off the issue path: the claims sit in registers with fixed roles (the loop below is unrolled),
                    // and a claim is read only kFetchAhead batches after it was made.
                    // deterministic: batch cta, cta + workers, ...: every thread block sums the same batches in the
                    // same order in every run
                    long long ahead[kFetchAhead];
                    long long det_next = static_cast<long long>(cta) + workers;
                    auto claim = [&]() -> long long {
                        if (P.deterministic) { const long long v = det_next; det_next += workers; return v; }
                        return static_cast<long long>(workers) + atomicAdd(ctr, 1u);
                    };
                    auto issue = [&](long long b) -> bool {
                        int s;
                        if (!acquire(s)) return false;
                        const int ki = static_cast<int>(b / per_group), j0 = static_cast<int>(b - static_cast<long long>(ki) * per_group) * NB;
                        const int g = sm.kept_group[ki];
                        sm.type[s] = ST_FFN; sm.arg0[s] = g >= 0 ? 0 : -1; sm.arg1[s] = 0;
                        if (g < 0) {
                            mbar_arrive(&sm.full[s]);
                        } else {
                            const __nv_bfloat16* group = Wl + static_cast<size_t>(g) * 3 * S * d;
                            unsigned char* dst = ring + static_cast<size_t>(s) * stage_bytes;
                            mbar_arrive_expect_tx(&sm.full[s], stage_bytes);
                            if constexpr (I4) {
                                const unsigned char* Q = reinterpret_cast<const unsigned char*>(Wl);
                                const __nv_bfloat16* Sc = P.Wsc[l];
                                const int nb = d / 128;
#pragma unroll
                                for (int plane = 0; plane < 3; ++plane) {
                                    const size_t rowi = static_cast<size_t>(g) * 3 * S + static_cast<size_t>(plane) * S + j0;
                                    bulk_copy_g2s(dst + plane * plane_bytes, Q + rowi * crow_bytes, plane_bytes, &sm.full[s]);
                                    bulk_copy_g2s(dst + 3 * plane_bytes + plane * sc_bytes, Sc + rowi * nb, sc_bytes, &sm.full[s]);
                                }
                            } else {
                            bulk_copy_g2s(dst, group + static_cast<size_t>(j0) * d, plane_bytes, &sm.full[s]);
                            bulk_copy_g2s(dst + plane_bytes, group + static_cast<size_t>(S + j0) * d, plane_bytes, &sm.full[s]);
                            bulk_copy_g2s(dst + 2 * plane_bytes, group + static_cast<size_t>(2 * S + j0) * d, plane_bytes,
                                          &sm.full[s]);
                            }
                        }
                        ++it;
                        return true;
                    };
                    if (static_cast<long long>(cta) < U) {
#pragma unroll
                        for (int k = 0; k < kFetchAhead; ++k) ahead[k] = claim();
                        if (!issue(cta)) alive = false;
                        bool more = alive;
                        while (more) {
#pragma unroll
                            for (int k = 0; k < kFetchAhead; ++k) {
                                if (more) {
                                    const long long b = ahead[k];
                                    if (b >= U) {
                                        more = false;     // claims only grow: every later one is past the end too
                                    } else if (!issue(b)) {
                                        alive = false;
                                        more = false;
                                    } else {
                                        ahead[k] = claim();
                                    }
                                }
                            }
                        }
                    }
                    if (alive) alive = marker(ST_END, 0);
                    if (I4 && alive) alive = marker(ST_END, 0);   // one for each half of the consumers
                }
                ++qp;
                issued_in_block = 0;
                __syncwarp();  // the table is rewritten for the next block only after lane 0 is done with it
            }
        }
        if (lane == 0 && *abort_flag) {
            // nobody consumes any more: let every copy this thread block issued land before it exits
            const int first = it > STAGES ? it - STAGES : 0;
            int never = 0;
            for (int k = first; k < it; ++k)
                mbar_wait_bounded(&sm.full[k % STAGES], static_cast<uint32_t>(k / STAGES) & 1u, &never);
        }
        return;
    }

    // =========================================== mover (TM) ===========================================
    if constexpr (TM) {
        if (warp == kPCWarps + 1) {
            const uint32_t tbase = sm.tmem_base;
            if (lane == 0) {
                long long blocks_left = static_cast<long long>(P.steps) * L;
                int it = 0;
                bool cps = false;
                while (blocks_left > 0) {
                    const int s = it % STAGES, t = it % kTSlots;
                    if (!mbar_wait_bounded(&sm.full[s], static_cast<uint32_t>(it / STAGES) & 1u, abort_flag)) { *abort_flag = 1; break; }
                    if (it >= kTSlots &&
                        !mbar_wait_bounded(&sm.tempty[t], (static_cast<uint32_t>(it / kTSlots) - 1u) & 1u, abort_flag)) {
                        *abort_flag = 1;
                        break;
                    }
                    const int type = sm.type[s], a0 = sm.arg0[s], a1 = sm.arg1[s];
                    sm.ttype[t] = type; sm.targ0[t] = a0; sm.targ1[t] = a1;
                    int n4k = 0;    // 4 KB pieces to move
                    if (type == ST_FFN && a0 >= 0) n4k = 3 * NB * PPR / 2;
                    else if (type == ST_PRED) n4k = a1 * PPR / 2;
                    if (n4k > 0) {
                        tcgen05_fence_after_sync();
                        const uint32_t src = smem_u32(ring + static_cast<size_t>(s) * stage_bytes);
                        const uint32_t dst = tbase + static_cast<uint32_t>(t * kTSlotCols);
                        for (int k = 0; k < n4k; ++k) tmem_cp_4k(dst + 8u * k, src + 4096u * k);
                        umma_commit(&sm.tfull[t]);    // the slot is complete when the copies are
                        umma_commit(&sm.empty[s]);    // ... and the shared-memory stage is free again
                        mbar_arrive(&sm.tfull[t]);    // releases the metadata written above
                        cps = true;
                    } else {
                        mbar_arrive(&sm.tfull[t]);
                        mbar_arrive(&sm.tfull[t]);
                        mbar_arrive(&sm.empty[s]);
                    }
                    ++it;
                    if (type == ST_END) --blocks_left;
                }
                if (cps) {   // every copy issued has completed before tensor memory is given back
                    umma_commit(&sm.tdrain);
                    int never = 0;
                    mbar_wait_bounded(&sm.tdrain, 0u, &never);
                }
            }
            __syncwarp();
            tcgen05_fence_before_sync();
            tm_join_barrier();
            tcgen05_fence_after_sync();
            tmem_dealloc(tbase, kTCols);
            return;
        }
    }

    // =========================================== consumers ===========================================
    const int row = warp / WPR, part = warp % WPR;
    const int tq = warp & 3, tg = warp >> 2;      // TM: quarter of the lanes this warp can read, and its row group
    const uint32_t tlane = static_cast<uint32_t>(tq * 32) << 16;
    const uint32_t tbase = TM ? sm.tmem_base : 0u;
    const int p1_base = TM ? tq * 32 + lane : part * (XC * 32) + lane;
    constexpr int p1_step = TM ? 128 : 32;        // distance between this thread's chunks of x
    const int rep = (REP > 1) ? tid / (kPC / REP) : 0;
    const int col0 = (REP > 1) ? tid % (kPC / REP) : tid;
    const bool owner = (REP == 1) || (rep == 0);   // threads that carry the residual stream for their columns
    uint4 xq[XC];      // this lane's slice of x, packed bf16
    float acc[P2][8];
    float hreg[P2][8];
    // I4: phase-2 replica and 16-column chunk of this thread, its sums, and the run-time copies of constants that keep
    // the unpacking off the logic pipe (see group_ffn_i4.cu)
    constexpr int kI4Acc = I4 ? 16 : 1;
    float acc16[kI4Acc], corr = 0.0f;
    const int i4_cols = d >> 4;                                   // 16-column chunks per row
    const int i4_reps = kPC / max(i4_cols, 1);
    const int i4_rep = tid / max(i4_cols, 1), i4_col = tid % max(i4_cols, 1);
    const uint32_t rt_zero = static_cast<uint32_t>(P.steps) >> 31;
    const uint32_t mul1 = 0x10000000u + rt_zero, mul2 = 0x01000000u + rt_zero, mul3 = 0x00100000u + rt_zero;
    const uint32_t mul16 = 0x00010000u + rt_zero;
    const PairBits pb{0x000F000Fu + rt_zero, 0x43004300u + rt_zero};
    int it = 0, red_par = 0;
    int it_half = warp >> 3;       // I4 form: the next stage of this thread's half (stages alternate between the halves)
    unsigned q = 0;  // running block counter over steps: partial buffers rotate with it
    const size_t acc_stride = static_cast<size_t>(d);
    const size_t buf_stride = static_cast<size_t>(kAccBufs) * d;
    bool bad = false;
    auto trace = [&](int slot, unsigned long long value) {
        if (P.trace && tid == 0 && q < static_cast<unsigned>(P.trace_blocks))
            P.trace[(static_cast<size_t>(q) * grid + cta) * 8 + slot] = value;
    };

    // normalise hreg -> xs (bf16) -> xr; thread block 0 records x as the input of block `l_next`
    auto normalise_and_load_x = [&](int step_i, int l_next, bool want_x) {
        float ss = 0.0f;
        if (owner) {
#pragma unroll
            for (int p = 0; p < P2; ++p) {
                const int c = col0 + kPC * p;
                if (c < chunks) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) ss = fmaf(hreg[p][e], hreg[p][e], ss);
                }
            }
        }
        ss = warp_sum(ss);
        if (lane == 0) sm.reduce[warp] = ss;
        pc_barrier();
        float tot = 0.0f;
#pragma unroll
        for (int w = 0; w < kPCWarps; ++w) tot += sm.reduce[w];
        const float scale = 1.0f / sqrtf(tot / static_cast<float>(d) + 1e-5f);
        if (owner && want_x) {
#pragma unroll
            for (int p = 0; p < P2; ++p) {
                const int c = col0 + kPC * p;
                if (c < chunks) {
                    __align__(16) __nv_bfloat16 xb[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) xb[e] = __float2bfloat16_rn(hreg[p][e] * scale);
                    const uint4 packed = *reinterpret_cast<const uint4*>(xb);
                    reinterpret_cast<uint4*>(xs)[c] = packed;
                    if (cta == 0 && P.tap_x)
                        reinterpret_cast<uint4*>(P.tap_x + (static_cast<size_t>(step_i) * L + l_next) * d)[c] = packed;
                    if (cta == 0 && P.pred_serial)
                        reinterpret_cast<uint4*>(P.x_hist + static_cast<size_t>(l_next & 1) * d)[c] = packed;
                }
            }
        }
        pc_barrier();  // xs complete; sm.reduce free again
        if constexpr (I4) {
            if (want_x) {
                // one 16-byte piece of x (8 elements e0..e7) per thread: its nibble pairing is (e0,e4) (e1,e5) (e2,e6) (e3,e7);
                // the four threads of a 32-element chunk add up its plain sum
                const int chunks16 = d / 32;
                for (int i = tid; i < (d >> 3); i += kPC) {
                    const int c = i >> 2, w = i & 3;
                    const uint4 v = reinterpret_cast<const uint4*>(xs)[i];
                    uint4 o;
                    o.x = __byte_perm(v.x, v.z, 0x5410); o.y = __byte_perm(v.x, v.z, 0x7632);
                    o.z = __byte_perm(v.y, v.w, 0x5410); o.w = __byte_perm(v.y, v.w, 0x7632);
                    xp[static_cast<size_t>(w) * chunks16 + c] = o;
                    float sx = (__uint_as_float(v.x << 16) + __uint_as_float(v.x & 0xffff0000u)) +
                               (__uint_as_float(v.y << 16) + __uint_as_float(v.y & 0xffff0000u)) +
                               (__uint_as_float(v.z << 16) + __uint_as_float(v.z & 0xffff0000u)) +
                               (__uint_as_float(v.w << 16) + __uint_as_float(v.w & 0xffff0000u));
                    sx += __shfl_xor_sync(0xffffffffu, sx, 1);
                    sx += __shfl_xor_sync(0xffffffffu, sx, 2);
                    if (w == 0) xsum[c] = sx;
                }
            }
            pc_barrier();
        } else if (want_x) {
#pragma unroll
            for (int i = 0; i < XC; ++i) xq[i] = reinterpret_cast<const uint4*>(xs)[p1_base + p1_step * i];
        }
    };

    // column sums -> shared memory (one region per replica), made visible to the copy engine
    auto stage_sums = [&]() {
        float* dst = reinterpret_cast<float*>(vec_buf) + static_cast<size_t>(rep) * d;
#pragma unroll
        for (int p = 0; p < P2; ++p) {
            const int c = col0 + kPC * p;
            if (c < chunks) {
                reinterpret_cast<float4*>(dst + c * 8)[0] = make_float4(acc[p][0], acc[p][1], acc[p][2], acc[p][3]);
                reinterpret_cast<float4*>(dst + c * 8)[1] = make_float4(acc[p][4], acc[p][5], acc[p][6], acc[p][7]);
            }
        }
        fence_proxy_async_smem();
    };

    for (int step_i = 0; step_i < P.steps && !bad; ++step_i) {
        // residual stream of this step, and the first block's input
        if (owner) {
#pragma unroll
            for (int p = 0; p < P2; ++p) {
                const int c = col0 + kPC * p;
                if (c < chunks) {
                    const float4* src = reinterpret_cast<const float4*>(P.h0 + static_cast<size_t>(step_i) * d + c * 8);
                    const float4 a = __ldg(src), b = __ldg(src + 1);
                    hreg[p][0] = a.x; hreg[p][1] = a.y; hreg[p][2] = a.z; hreg[p][3] = a.w;
                    hreg[p][4] = b.x; hreg[p][5] = b.y; hreg[p][6] = b.z; hreg[p][7] = b.w;
                }
            }
        }
        normalise_and_load_x(step_i, 0, true);

        for (int l = 0; l < L && !bad; ++l) {
#pragma unroll
            for (int p = 0; p < P2; ++p)
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[p][e] = 0.0f;
#pragma unroll
            for (int e = 0; e < kI4Acc; ++e) acc16[e] = 0.0f;
            corr = 0.0f;
            bool any = false;
            bool first_stage = true;
            trace(TR_BLOCK_START, global_timer_ns());

            // ------------------------------ stages of this block ------------------------------
            if constexpr (I4) {
                // Two halves of 8 warps take alternate stages (each with its own barrier), so that one half's phase
                // change and waits are covered by the other half's arithmetic.  Phase 1: warp w of the half takes the gate
                // and the up row of neuron w and reads x once for both; phase 2: a thread owns 16 columns, 256 / (d/16)
                // replicas per half.  The producer ends a block with two END markers, one per half.
                const int half = warp >> 3, hw = warp & 7, ht = tid & 255;
                const int chunks16 = d / 32, nbk = d / 128;
                const int rh = (kPC / 2) / max(i4_cols, 1);           // replicas inside a half
                const int hrep = ht / max(i4_cols, 1);
                int hpar = 0;
                bool hbad = false;
                while (true) {
                    const int itx = it_half;
                    const int s = itx % STAGES;
                    const uint32_t parity = static_cast<uint32_t>(itx / STAGES) & 1u;
                    const bool ok = mbar_wait_bounded(&sm.full[s], parity, abort_flag);
                    if (first_stage && half == 0) { trace(TR_FIRST_STAGE, global_timer_ns()); first_stage = false; }
                    const int type = sm.type[s], a0 = sm.arg0[s], a1 = sm.arg1[s];
                    const unsigned char* stage = ring + static_cast<size_t>(s) * stage_bytes;
                    float* red = sm.red_h[half][hpar];
                    if (ok && type == ST_FFN && a0 >= 0) {
                        any = true;
                        const uint4* rg = reinterpret_cast<const uint4*>(stage + static_cast<size_t>(hw) * crow_bytes);
                        const uint4* ru = reinterpret_cast<const uint4*>(stage + static_cast<size_t>(NB + hw) * crow_bytes);
                        const __nv_bfloat16* sc0 = reinterpret_cast<const __nv_bfloat16*>(stage + 3 * plane_bytes);
                        const __nv_bfloat16* sg = sc0 + static_cast<size_t>(hw) * nbk;
                        const __nv_bfloat16* su = sc0 + static_cast<size_t>(NB + hw) * nbk;
                        float ag = 0.0f, au = 0.0f;
#pragma unroll
                        for (int u = 0; u < XC; ++u) {
                            const int c = lane + 32 * u;
                            const uint4 g4 = rg[c], u4 = ru[c];
                            const uint32_t gw[4] = {g4.x, g4.y, g4.z, g4.w};
                            const uint32_t uw[4] = {u4.x, u4.y, u4.z, u4.w};
                            float g0 = 0.0f, g1 = 0.0f, u0 = 0.0f, u1 = 0.0f;
#pragma unroll
                            for (int w = 0; w < 4; ++w) {
                                const uint4 xv = xp[static_cast<size_t>(w) * chunks16 + c];
                                fma_bf16x2(nibble_pair_r(gw[w], pb), xv.x, g0, g1);
                                fma_bf16x2(nibble_pair_r(uw[w], pb), xv.x, u0, u1);
                                fma_bf16x2(nibble_pair_r(gw[w] >> 4, pb), xv.y, g0, g1);
                                fma_bf16x2(nibble_pair_r(uw[w] >> 4, pb), xv.y, u0, u1);
                                fma_bf16x2(nibble_pair_r(gw[w] >> 8, pb), xv.z, g0, g1);
                                fma_bf16x2(nibble_pair_r(uw[w] >> 8, pb), xv.z, u0, u1);
                                fma_bf16x2(nibble_pair_r(__umulhi(gw[w], mul3), pb), xv.w, g0, g1);
                                fma_bf16x2(nibble_pair_r(__umulhi(uw[w], mul3), pb), xv.w, u0, u1);
                            }
                            const float offx = kNibbleBias * xsum[c];
                            ag = fmaf(__bfloat162float(sg[c >> 2]), (g0 + g1) - offx, ag);
                            au = fmaf(__bfloat162float(su[c >> 2]), (u0 + u1) - offx, au);
                        }
                        ag = warp_sum(ag);
                        au = warp_sum(au);
                        if (lane == 0) { red[hw] = ag; red[NB + hw] = au; }
                    } else if (ok && type == ST_PRED) {
                        // bf16 predictor rows: a warp per row, x (bf16) from shared memory
                        if (hw < a1) {
                            const uint4* rp = reinterpret_cast<const uint4*>(stage + static_cast<size_t>(hw) * row_bytes);
                            const uint4* xv = reinterpret_cast<const uint4*>(xs);
                            float dot0 = 0.0f, dot1 = 0.0f;
                            for (int c = lane; c < chunks; c += 32) dot_bf16x8(rp[c], xv[c], dot0, dot1);
                            const float dot = warp_sum(dot0 + dot1);
                            if (lane == 0) red[hw] = dot;
                        }
                    }
                    hbad = half_barrier_or(half, !ok);
                    if (hbad) { *abort_flag = 1; break; }     // the other half's waits give up on this flag
                    if (type == ST_FFN) {
                        if (a0 >= 0 && hrep < rh) {
                            const unsigned char* down = stage + 2 * plane_bytes;
                            const __nv_bfloat16* ds = reinterpret_cast<const __nv_bfloat16*>(stage + 3 * plane_bytes) + static_cast<size_t>(2 * NB) * nbk;
                            for (int j = hrep; j < NB; j += rh) {
                                const float h = silu_mul(red[j], red[NB + j]);
                                const float f = h * __bfloat162float(ds[static_cast<size_t>(j) * nbk + (i4_col >> 3)]);
                                corr += f;
                                const uint2 w2 = reinterpret_cast<const uint2*>(down + static_cast<size_t>(j) * crow_bytes)[i4_col];
                                const uint32_t words[2] = {w2.x, w2.y};
#pragma unroll
                                for (int v = 0; v < 2; ++v) {
                                    const uint32_t pk[4] = {nibble_pair_r(words[v], pb), nibble_pair_r(__umulhi(words[v], mul1), pb),
                                                            nibble_pair_r(__umulhi(words[v], mul2), pb),
                                                            nibble_pair_r(__umulhi(words[v], mul3), pb)};
#pragma unroll
                                    for (int k = 0; k < 4; ++k) {
                                        acc16[(8 * v + k) % kI4Acc] = fmaf(f, __uint_as_float(pk[k] * mul16), acc16[(8 * v + k) % kI4Acc]);
                                        acc16[(8 * v + k + 4) % kI4Acc] = fmaf(f, __uint_as_float(pk[k]), acc16[(8 * v + k + 4) % kI4Acc]);
                                    }
                                }
                            }
                        }
                        hpar ^= 1;
                    } else if (type == ST_PRED) {
                        if (ht == 0) {
                            const unsigned n_pred = static_cast<unsigned>(step_i) * (L - 1) + (l + 1);
                            float* zdst = P.z + static_cast<size_t>(n_pred & 1u) * r;
                            for (int i = 0; i < a1; ++i) {
                                float z = red[i];
                                if (P.act == HALO_ACT_RELU) z = fmaxf(z, 0.0f);
                                zdst[a0 + i] = z;
                            }
                            red_release_add(sync_zcount, static_cast<unsigned>(a1));   // publishes the values above
                        }
                        hpar ^= 1;
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.empty[s]);
                    it_half += 2;
                    if (type == ST_END) break;
                }
                // both halves are through their END marker (or gave up): one decision for the whole thread block
                bad = pc_barrier_or(hbad);
                any = pc_barrier_or(any);
            } else
            while (true) {
                const int s = TM ? it % kTSlots : it % STAGES;
                const uint32_t parity = static_cast<uint32_t>(it / (TM ? kTSlots : STAGES)) & 1u;
                const bool ok = mbar_wait_bounded(TM ? &sm.tfull[s] : &sm.full[s], parity, abort_flag);
                if constexpr (TM) tcgen05_fence_after_sync();
                if (first_stage) { trace(TR_FIRST_STAGE, global_timer_ns()); first_stage = false; }
                const int type = TM ? sm.ttype[s] : sm.type[s], a0 = TM ? sm.targ0[s] : sm.arg0[s],
                          a1 = TM ? sm.targ1[s] : sm.arg1[s];
                const unsigned char* stage = ring + static_cast<size_t>(TM ? 0 : s) * stage_bytes;
                const uint32_t tslot = tbase + tlane + static_cast<uint32_t>(s * kTSlotCols);   // TM: this warp's lanes of the slot
                float* red = sm.red[red_par];
                // ---- before the barrier: nothing in here may block on other consumers ----
                if constexpr (TM) {
                    if ((type == ST_FFN && a0 >= 0) || type == ST_PRED) {
                        if (type == ST_FFN) any = true;
                        const int n_rows = type == ST_FFN ? ROWS : a1;
                        const uint4* xg = reinterpret_cast<const uint4*>(P.x_hist + static_cast<size_t>((l - 1) & 1) * d);
                        const bool x_global = type == ST_PRED && P.pred_serial;   // this block's own predictor
#pragma unroll
                        for (int rr = 0; rr < ROWS / 4; ++rr) {
                            const int rw = tg + 4 * rr;
                            if (rw < n_rows) {       // warp-uniform
                                uint32_t w[4 * PPR];
                                tmem_ld_cols<4 * PPR>(tslot + static_cast<uint32_t>(rw * PPR * 4), w);
                                tmem_ld_wait();
                                float dot0 = 0.0f, dot1 = 0.0f;
#pragma unroll
                                for (int i = 0; i < PPR; ++i) {
                                    const uint4 wv = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
                                    dot_bf16x8(wv, x_global ? __ldcg(xg + p1_base + p1_step * i) : xq[i], dot0, dot1);
                                }
                                const float dot = warp_sum(dot0 + dot1);
                                if (lane == 0) red[rw * WPR + tq] = dot;
                            }
                        }
                    }
                } else if (type == ST_FFN) {
                    if (a0 >= 0) {
                        any = true;
                        const uint4* rp = reinterpret_cast<const uint4*>(stage + static_cast<size_t>(row) * row_bytes);
                        float dot0 = 0.0f, dot1 = 0.0f;
#pragma unroll
                        for (int i = 0; i < XC; ++i) dot_bf16x8(rp[p1_base + 32 * i], xq[i], dot0, dot1);
                        const float dot = warp_sum(dot0 + dot1);
                        if (lane == 0) red[row * WPR + part] = dot;
                    }
                } else if (type == ST_PRED) {
                    if (row < a1) {
                        const uint4* rp = reinterpret_cast<const uint4*>(stage + static_cast<size_t>(row) * row_bytes);
                        float dot0 = 0.0f, dot1 = 0.0f;
                        if (P.pred_serial) {
                            // this block's own predictor: its input is the previous block's x, kept in global memory
                            const uint4* xp = reinterpret_cast<const uint4*>(P.x_hist + static_cast<size_t>((l - 1) & 1) * d);
#pragma unroll
                            for (int i = 0; i < XC; ++i) dot_bf16x8(rp[p1_base + 32 * i], __ldcg(xp + p1_base + 32 * i), dot0, dot1);
                        } else {
#pragma unroll
                        for (int i = 0; i < XC; ++i) dot_bf16x8(rp[p1_base + 32 * i], xq[i], dot0, dot1);
                        }
                        const float dot = warp_sum(dot0 + dot1);
                        if (lane == 0) red[row * WPR + part] = dot;
                    }
                }
                bad = pc_barrier_or(!ok);
                if (bad) break;
                // ---- after the barrier ----
                if (type == ST_FFN) {
                    if (a0 >= 0) {
                        const unsigned char* down = stage + 2 * plane_bytes;
#pragma unroll
                        for (int jj = 0; jj < NB / REP; ++jj) {
                            const int j = jj * REP + rep;
                            const float h = silu_mul(sum_parts<WPR>(red + j * WPR), sum_parts<WPR>(red + (NB + j) * WPR));
                            if constexpr (TM) {
                                // the thread's chunk col0 of down row j: piece col0 / 128, lane col0 % 128 (this warp's quarter)
                                uint32_t w[4];
                                tmem_ld_cols<4>(tslot + static_cast<uint32_t>(((ROWS + j) * PPR + (col0 >> 7)) * 4), w);
                                tmem_ld_wait();
                                axpy_bf16x8(h, make_uint4(w[0], w[1], w[2], w[3]), acc[0]);
                            } else {
                            const uint4* dr = reinterpret_cast<const uint4*>(down + static_cast<size_t>(j) * row_bytes);
#pragma unroll
                            for (int p = 0; p < P2; ++p) {
                                const int c = col0 + kPC * p;
                                if (P2 == 1 || c < chunks) axpy_bf16x8(h, dr[c], acc[p]);
                            }
                            }
                        }
                    }
                    red_par ^= 1;
                } else if (type == ST_PRED) {
                    if (tid == 0) {
                        // hidden values of the prediction made during this block, in the buffer of its parity
                        const unsigned n_pred = static_cast<unsigned>(step_i) * (L - 1) + (P.pred_serial ? l : l + 1);
                        float* zdst = P.z + static_cast<size_t>(n_pred & 1u) * r;
                        for (int i = 0; i < a1; ++i) {
                            float z = 0.0f;
                            for (int w = 0; w < WPR; ++w) z += red[i * WPR + w];
                            if (P.act == HALO_ACT_RELU) z = fmaxf(z, 0.0f);
                            zdst[a0 + i] = z;
                        }
                        red_release_add(sync_zcount, static_cast<unsigned>(a1));   // publishes the values above
                    }
                    red_par ^= 1;
                }
                if constexpr (TM) tcgen05_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(TM ? &sm.tempty[s] : &sm.empty[s]);
                ++it;
                if (type == ST_END) break;
            }
            if (bad) break;

            // ------------------------------ end of the block: flush, grid barrier, merge + glue ------------------------------
            trace(TR_STAGES_DONE, global_timer_ns());
            if constexpr (I4) {
                if (any) {
                    // the replicas' sums meet in the one vector buffer in turn; the offsets of the unpacking come off here
                    // (upper elements: sum f * (128 + 0x4300 / 65536 + n_hi + n_lo / 65536), n_lo from the element 4 below)
                    const float off = kNibbleBias * corr;
                    const float off_hi = (kNibbleBias + 17152.0f / 65536.0f) * corr;
                    float* dst = reinterpret_cast<float*>(vec_buf) + static_cast<size_t>(i4_col) * 16;
                    for (int rr = 0; rr < i4_reps; ++rr) {
                        if (i4_rep == rr) {
#pragma unroll
                            for (int v = 0; v < 16; v += 8) {
                                float4 lo4, hi4;
                                float* lo = reinterpret_cast<float*>(&lo4);
                                float* hi = reinterpret_cast<float*>(&hi4);
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    lo[k] = acc16[(v + k) % kI4Acc] - off;
                                    hi[k] = (acc16[(v + k + 4) % kI4Acc] - off_hi) - (acc16[(v + k) % kI4Acc] - 128.0f * corr) * (1.0f / 65536.0f);
                                }
                                if (rr > 0) {
                                    const float4 a = reinterpret_cast<const float4*>(dst + v)[0], b = reinterpret_cast<const float4*>(dst + v)[1];
                                    lo4.x += a.x; lo4.y += a.y; lo4.z += a.z; lo4.w += a.w;
                                    hi4.x += b.x; hi4.y += b.y; hi4.z += b.z; hi4.w += b.w;
                                }
                                reinterpret_cast<float4*>(dst + v)[0] = lo4;
                                reinterpret_cast<float4*>(dst + v)[1] = hi4;
                            }
                            fence_proxy_async_smem();
                        }
                        if (rr + 1 < i4_reps) pc_barrier();
                    }
                }
            } else {
                if (REP > 1 && !P.deterministic) {
                    // the replicas' sums meet in the first vector buffer in turn, so one bulk reduction leaves the thread block
                    if (any) {
                        float* dst = reinterpret_cast<float*>(vec_buf);
                        for (int rr = 0; rr < REP; ++rr) {
                            if (rep == rr) {
#pragma unroll
                                for (int p = 0; p < P2; ++p) {
                                    const int c = col0 + kPC * p;
                                    if (c < chunks) {
                                        float4 a = make_float4(acc[p][0], acc[p][1], acc[p][2], acc[p][3]);
                                        float4 b = make_float4(acc[p][4], acc[p][5], acc[p][6], acc[p][7]);
                                        if (rr > 0) {
                                            const float4 u = reinterpret_cast<const float4*>(dst + c * 8)[0];
                                            const float4 v = reinterpret_cast<const float4*>(dst + c * 8)[1];
                                            a.x += u.x; a.y += u.y; a.z += u.z; a.w += u.w;
                                            b.x += v.x; b.y += v.y; b.z += v.z; b.w += v.w;
                                        }
                                        reinterpret_cast<float4*>(dst + c * 8)[0] = a;
                                        reinterpret_cast<float4*>(dst + c * 8)[1] = b;
                                    }
                                }
                                fence_proxy_async_smem();
                            }
                            if (rr + 1 < REP) pc_barrier();
                        }
                    }
                } else if (any || P.deterministic) {
                    stage_sums();
                }
            }
            pc_barrier();
            if (P.deterministic) {
                // this thread block's column sums (replicas added in index order) go to its own row
                float* rowp = P.det_rows + (static_cast<size_t>(q & 1u) * grid + cta) * d;
                if (owner) {
#pragma unroll
                    for (int p = 0; p < P2; ++p) {
                        const int c = col0 + kPC * p;
                        if (c < chunks) {
                            float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
#pragma unroll
                            for (int k = 0; k < REP; ++k) {
                                const float* src = reinterpret_cast<const float*>(vec_buf) + static_cast<size_t>(k) * d + c * 8;
                                const float4 u = reinterpret_cast<const float4*>(src)[0], v = reinterpret_cast<const float4*>(src)[1];
                                a.x += u.x; a.y += u.y; a.z += u.z; a.w += u.w;
                                b.x += v.x; b.y += v.y; b.z += v.z; b.w += v.w;
                            }
                            reinterpret_cast<float4*>(rowp + c * 8)[0] = a;
                            reinterpret_cast<float4*>(rowp + c * 8)[1] = b;
                        }
                    }
                }
                __threadfence();
                pc_barrier();
            }
            bool okb = true;
            if (tid == 0) {
                if (any && !P.deterministic) {
                    float* dst = P.partials + (q % 3u) * buf_stride + static_cast<size_t>(cta % kAccBufs) * acc_stride;
                    bulk_reduce_add_f32_s2g(dst, vec_buf, static_cast<uint32_t>(d) * 4u);   // (replicas already added up)
                    bulk_commit_and_wait_all();   // the sums are in global memory (and vec_buf is free again)
                    fence_proxy_async_all();
                }
                trace(TR_FLUSHED, global_timer_ns());
                // Batch counters rotate over 32 words.  A producer leads its consumers by at most the ring depth
                // (<= 13 stages with the tensor-memory level, every block has at least its END stage), so the counter
                // of the block 16 ahead is idle now: its last user finished 16 blocks ago and its next user cannot
                // have started.
                if (cta == 0) P.sync[32 + ((q + 16u) & 31u)] = 0u;
                // Arrival: ONE acquire-release atomic instead of fence + relaxed atomic + fence (0.3 us per block: 3182 ->
                // 3253 tokens/s on the TinyLlama shape, 784 -> 794 at 7B).  Release: this thread's stores and, through the
                // thread-block barrier in front of it, the other threads' (whose reductions are complete and proxy-fenced
                // above).  Acquire: the last arriver reads the head of the others' release sequence on this word; everybody
                // else acquires in spin_until_ge, and the thread-block barrier behind this passes that on.
                const unsigned target = (q + 1u) * static_cast<unsigned>(workers);
                unsigned before;
                asm volatile("atom.add.acq_rel.gpu.u32 %0, [%1], 1;" : "=r"(before) : "l"(sync_barrier) : "memory");
                okb = (before + 1u == target) || spin_until_ge(sync_barrier, target, sync_abort);
            }
            bad = pc_barrier_or(!okb);
            if (bad) break;
            if (tid == 0) *reinterpret_cast<volatile int*>(&sm.blocks_done) = static_cast<int>(q) + 1;
            trace(TR_BARRIER_DONE, global_timer_ns());

            // a9 + residual: every thread block sums the accumulation buffers for its own copy of the stream
            const float* pbuf = P.partials + (q % 3u) * buf_stride;
            float* zbuf = P.partials + ((q + 2u) % 3u) * buf_stride;   // read two blocks ago by everyone: clear it
            const size_t rec = static_cast<size_t>(step_i) * L + l;
            if (owner) {
#pragma unroll
                for (int p = 0; p < P2; ++p) {
                    const int c = col0 + kPC * p;
                    if (c < chunks) {
                        float y[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                        if (P.deterministic) {
                            // the rows of all streaming thread blocks, added in index order
                            const float* rows = P.det_rows + static_cast<size_t>(q & 1u) * grid * d + c * 8;
                            for (int w = 0; w < workers; ++w) {
                                const float4 u = __ldcg(reinterpret_cast<const float4*>(rows + static_cast<size_t>(w) * d));
                                const float4 v = __ldcg(reinterpret_cast<const float4*>(rows + static_cast<size_t>(w) * d) + 1);
                                y[0] += u.x; y[1] += u.y; y[2] += u.z; y[3] += u.w;
                                y[4] += v.x; y[5] += v.y; y[6] += v.z; y[7] += v.w;
                            }
                        } else {
                        float4 va[kAccBufs], vb[kAccBufs];
#pragma unroll
                        for (int k = 0; k < kAccBufs; ++k) {
                            const float4* src = reinterpret_cast<const float4*>(pbuf + static_cast<size_t>(k) * acc_stride + c * 8);
                            va[k] = __ldcg(src);
                            vb[k] = __ldcg(src + 1);
                        }
#pragma unroll
                        for (int k = 0; k < kAccBufs; ++k) {
                            y[0] += va[k].x; y[1] += va[k].y; y[2] += va[k].z; y[3] += va[k].w;
                            y[4] += vb[k].x; y[5] += vb[k].y; y[6] += vb[k].z; y[7] += vb[k].w;
                        }
                        }
#pragma unroll
                        for (int e = 0; e < 8; ++e) hreg[p][e] += y[e];
                        if (cta == 0) {
                            if (P.tap_y) {
                                float4* dst = reinterpret_cast<float4*>(P.tap_y + rec * d + c * 8);
                                dst[0] = make_float4(y[0], y[1], y[2], y[3]);
                                dst[1] = make_float4(y[4], y[5], y[6], y[7]);
                            }
                            if (l == L - 1) {
                                float4* dst = reinterpret_cast<float4*>(P.h_out + static_cast<size_t>(step_i) * d + c * 8);
                                dst[0] = make_float4(hreg[p][0], hreg[p][1], hreg[p][2], hreg[p][3]);
                                dst[1] = make_float4(hreg[p][4], hreg[p][5], hreg[p][6], hreg[p][7]);
                            }
                        }
                        if (cta < kAccBufs) {
                            float4* dst = reinterpret_cast<float4*>(zbuf + static_cast<size_t>(cta) * acc_stride + c * 8);
                            dst[0] = make_float4(0.f, 0.f, 0.f, 0.f);
                            dst[1] = make_float4(0.f, 0.f, 0.f, 0.f);
                        }
                    }
                }
            }
            trace(TR_MERGED, global_timer_ns());
            if (l + 1 < L) normalise_and_load_x(step_i, l + 1, true);
            trace(TR_X_READY, global_timer_ns());
            ++q;
        }
    }
    if (bad && tid == 0) {
        *abort_flag = 1;                 // the producer stops and drains
        atomicExch(sync_abort, 1u);      // every other thread block follows
        flag_status(P.status, HALO_DEV_TIMEOUT);
    }
    if constexpr (TM) {
        tcgen05_fence_before_sync();
        tm_join_barrier();               // the mover frees the tensor memory behind this
    }
}

// ---- host side -----------------------------------------------------------------------------------------

bool persistent_supported_i4(const halo_ffn_shape& sh, int n_tok, int G) {
    return sh.wdtype == HALO_BF16 && n_tok == 1 && G <= kPC && (sh.d_model == 2048 || sh.d_model == 4096) &&
           sh.group_size % 8 == 0;
}

bool persistent_supported(const halo_ffn_shape& sh, int n_tok, int G) {
    if (sh.wdtype != HALO_BF16 || n_tok != 1 || G > kPC) return false;
    switch (sh.d_model) {
        case 2048: return sh.group_size % 4 == 0;  // batches of NB neurons must tile a group
        case 4096: case 5120: return sh.group_size % 2 == 0;
        case 8192: return true;
    }
    return false;
}

template <int NB, int XC, int P2, int REP, int STAGES, bool TM, bool I4 = false>
static halo_status launch_cfg(PersistParams& P, cudaStream_t st) {
    auto kernel = stack_decode_kernel<NB, XC, P2, REP, STAGES, TM, I4>;
    constexpr int kThreads = TM ? kPThreadsTM : kPThreads;
    const size_t dd = static_cast<size_t>(P.d);
    const size_t smem = I4 ? kHeaderBytes + dd * 4 * REP + dd * 2 + ((dd / 32 * 4 + 127) & ~size_t(127)) +
                                 static_cast<size_t>(STAGES) * 3 * NB * (dd / 2 + dd / 128 * 2)
                           : kHeaderBytes + dd * 4 * REP + static_cast<size_t>(STAGES) * 3 * NB * dd * 2;
    static bool configured[64] = {};
    int dev = 0, sms = kSmCount;
    if (cudaGetDevice(&dev) != cudaSuccess) return HALO_ERR_CUDA;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (!ensure_dynamic_smem(kernel, smem, configured)) return HALO_ERR_CUDA;
    int blocks_per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm, kernel, kThreads, smem) != cudaSuccess)
        return HALO_ERR_CUDA;
    if (blocks_per_sm < 1 || sms < 2) return HALO_ERR_UNIMPLEMENTED;   // cannot be made resident: caller falls back
    void* args[] = {&P};
    const cudaError_t err = cudaLaunchCooperativeKernel(reinterpret_cast<void*>(kernel), dim3(sms), dim3(kThreads), args,
                                                        smem, st);
    if (err == cudaErrorCooperativeLaunchTooLarge) {
        // the SMs are not all ours (another context on the device): not an error of this call, the caller runs the
        // one-launch-per-step path instead
        (void)cudaGetLastError();
        return HALO_ERR_UNIMPLEMENTED;
    }
    return err == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}

halo_status launch_stack_persistent(PersistParams& P, cudaStream_t st) {
    if (P.i4) {
        switch (P.d) {
            case 2048: return launch_cfg<8, 2, 1, 1, 4, false, true>(P, st);
            case 4096: return launch_cfg<8, 4, 1, 1, 3, false, true>(P, st);
        }
        return HALO_ERR_UNIMPLEMENTED;
    }
    switch (P.d) {
        case 2048: return P.tmem_ring ? launch_cfg<4, 2, 1, 2, 4, true>(P, st) : launch_cfg<4, 4, 1, 2, 4, false>(P, st);
        case 4096: return P.tmem_ring ? launch_cfg<2, 4, 1, 1, 4, true>(P, st) : launch_cfg<2, 4, 1, 1, 4, false>(P, st);
        case 5120: return launch_cfg<2, 5, 2, 1, 3, false>(P, st);
        case 8192: return launch_cfg<1, 4, 2, 1, 3, false>(P, st);
    }
    return HALO_ERR_UNIMPLEMENTED;
}

}  // namespace halo
