/*
 * halo.h -- C ABI of libhalo: the group-sparse FFN hot path of HALO
 * (arXiv 2601.11676) for NVIDIA B200 (sm_100a).
 *
 * Path: predictor scores per FFN neuron group -> rank / critical choice /
 * assignment of the less-critical groups to virtual unstable devices /
 * seeded per-device arrival mask -> SwiGLU FFN over the kept groups only,
 * accumulated per holder -> merge of the partials that arrived.
 *
 * Conventions
 *   - Every function returns a halo_status (0 = HALO_OK, negative = error).
 *     Argument errors are found on the host before anything is launched.
 *   - Pointers marked "device" are CUDA device pointers owned by the caller,
 *     16-byte aligned; pointers marked "host" are ordinary host memory.
 *   - GPU entry points enqueue work on `stream` (a cudaStream_t passed as
 *     void*; NULL = the default stream) and return without synchronising.
 *     They allocate nothing and print nothing.  Scratch memory, where a call
 *     needs it, is a caller-owned device `workspace` whose size the matching
 *     *_workspace_bytes function reports.
 *   - Conditions found on the device (non-finite score, out-of-range group
 *     index, a wait that ran out) are OR-ed into the caller-owned device word
 *     `dev_status` (may be NULL); read it after synchronising and decode it
 *     with halo_status_message.
 *   - Element type of weights and activations is `halo_dtype`; scores,
 *     partials and outputs are fp32.
 *
 * Weight layout (Sec. II-A, "neuron group": a group owns its gate rows, its
 * up rows and the matching down-projection columns):
 *     W_packed[G][3][S][d]   G = d_ffn / group_size, S = group_size, d = d_model
 *     plane 0: gate rows, plane 1: up rows,
 *     plane 2: the group's down-projection columns, each stored as a row of d.
 *   One group is one contiguous block of 3*S*d elements, so a skipped group is
 *   a skipped address range.
 */
#ifndef HALO_H
#define HALO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int halo_status;
enum {
    HALO_OK = 0,
    HALO_ERR_ARG = -1,           /* NULL pointer, value out of range */
    HALO_ERR_SHAPE = -2,         /* sizes that do not divide / exceed limits */
    HALO_ERR_ALIGN = -3,         /* a device pointer is not 16-byte aligned */
    HALO_ERR_DTYPE = -4,         /* dtype not supported by this entry point */
    HALO_ERR_CUDA = -5,          /* a CUDA runtime call failed */
    HALO_ERR_NOMEM = -6,         /* host or device allocation failed (create calls only) */
    HALO_ERR_UNIMPLEMENTED = -7,
    HALO_ERR_WORKSPACE = -8      /* workspace missing or too small */
};

/* bits of the device status word */
#define HALO_DEV_NONFINITE_SCORE 1u  /* a score was NaN (ranked lowest) or infinite */
#define HALO_DEV_BAD_INDEX 2u        /* a group id or device id was out of range; the item was skipped */
#define HALO_DEV_TIMEOUT 4u          /* a bounded device-side wait ran out */

#define HALO_MAX_DEVICES 32
#define HALO_MAX_GROUPS 1024

typedef enum { HALO_F32 = 0, HALO_BF16 = 1 } halo_dtype;
typedef enum { HALO_SEL_TOPK = 0, HALO_SEL_THRESHOLD = 1 } halo_sel_mode;
typedef enum { HALO_ACT_RELU = 0, HALO_ACT_NONE = 1 } halo_pred_act;

/* d_ffn % group_size == 0; d_model % 8 == 0; d_ffn / group_size <= HALO_MAX_GROUPS. */
typedef struct {
    int d_model, d_ffn, group_size;
    halo_dtype wdtype;
} halo_ffn_shape;

/* Predictor d_in -> rank -> n_groups; d_in % 8 == 0, rank % 8 == 0. */
typedef struct {
    int d_in, rank, n_groups;
    halo_dtype wdtype;
    halo_pred_act act;
} halo_pred_shape;

typedef struct halo_plan halo_plan;   /* host object: Assignment-phase tables */
typedef struct halo_stack halo_stack; /* host object owning device work buffers of an FFN stack */

const char* halo_status_string(halo_status s);
/* Writes a comma-separated description of the bits of a device status word. */
halo_status halo_status_message(uint32_t dev_status_value, char* msg /*host*/, int msg_len);

/* ------------------------------------------------------------------------
 * Assignment phase (Sec. III-B.4, Algorithm 3: PLR-aware ratio-guided
 * scheduler).  Host only, one-off.
 *   loss_rate[n_dev]    (host) packet-loss rate rho_i in [0,1] of virtual device i
 *   share_weight[n_dev] (host) integer workload ratio r_i (any common scale; sum > 0)
 *   mode / k_critical / threshold: how the critical groups (kept by the
 *     reliable master, never dropped) are chosen from the scores: the k
 *     highest, or those with score >= threshold.
 *   seed: key of the arrival draws.
 * Devices are ordered by ascending loss rate (ties: lower index).  The M
 * less-critical groups, in priority order, are cut into n_dev contiguous
 * chunks; the cut after the j-th device in that order is
 * floor((2*M*C_j + C_n) / (2*C_n)), C_j = cumulative weight.  n_dev may be 0.
 * Errors: HALO_ERR_ARG for a rate outside [0,1], all-zero weights, k out of
 * range, NULL pointers; HALO_ERR_SHAPE for n_groups/n_dev beyond the limits.
 * The plan is owned by the library until halo_plan_destroy.
 * ---------------------------------------------------------------------- */
halo_status halo_plan_create(halo_plan** out, int n_groups, int n_dev, const double* loss_rate,
                             const uint32_t* share_weight, halo_sel_mode mode, int k_critical,
                             float threshold, uint64_t seed);
halo_status halo_plan_destroy(halo_plan* plan);
/* For inspection: device order (ascending loss), the 33-bit loss thresholds
 * T_i = round(rho_i * 2^32) by device index, and the n_dev+1 chunk boundaries
 * for M less-critical groups.  All host arrays; any may be NULL. */
halo_status halo_plan_describe(const halo_plan* plan, int M, int32_t* dev_order, uint64_t* loss_thresh,
                               int32_t* boundaries);

/* ------------------------------------------------------------------------
 * Assignment phase, step 1: workload ratios from the devices' memory budgets
 * m_i and computing power c_i (Sec. III-B.4, PLR-aware load-balancing
 * scheduler).  Host only.  All arrays are host arrays of n_dev entries;
 * model_mem is the model's total memory demand in the unit of mem_budget.
 *   halo_schedule_comp_greedy (Algorithm 1): devices in descending computing
 *     power (ties: lower index) are filled to their budget until the model
 *     fits; the last one needed takes the remainder; unused devices get 0.
 *   halo_schedule_min_max (the problem Algorithm 2 solves): u_i = min(m_i, T*c_i)
 *     with the smallest utilisation threshold T whose allocation holds the
 *     model; minimises the slowest device's time.  The paper bisects on T to a
 *     tolerance (1e-3); here the piecewise-linear equation sum_i min(m_i, T*c_i)
 *     = model_mem is solved exactly at its breakpoints m_i/c_i, so the result
 *     is the limit of that bisection.  eps must be positive and is otherwise
 *     not needed.
 *   Both return ratio[i] = u_i / sum(u) (sum = 1).
 *   halo_ratios_to_share_weights: integer weights round(ratio * 65536) for
 *     halo_plan_create (zero-ratio devices get empty chunks).
 * HALO_ERR_ARG: NULL pointers, n_dev outside [1, HALO_MAX_DEVICES], a
 * negative budget, non-positive computing power or eps, or budgets that
 * cannot hold the model.
 * ---------------------------------------------------------------------- */
halo_status halo_schedule_comp_greedy(int n_dev, const double* mem_budget, const double* compute,
                                      double model_mem, double* ratio);
halo_status halo_schedule_min_max(int n_dev, const double* mem_budget, const double* compute, double model_mem,
                                  double eps, double* ratio);
halo_status halo_ratios_to_share_weights(int n_dev, const double* ratio, uint32_t* share_weight);

/* ------------------------------------------------------------------------
 * Late devices (Sec. III-B.3: the master merges what is available after a
 * timeout, so a partial that comes later than the timeout is as good as lost;
 * Eq. 1: device i needs tau * W_i / c_i for the W_i units it holds, plus the
 * synchronisation time T_c).  Host only.
 *   units[i]   groups device i holds per block (e.g. its chunk from
 *              halo_plan_describe's boundaries); compute[i] = c_i > 0;
 *   tau        cost of one group on a device of computing power 1;
 *   t_comm     T_c; timeout in the same unit of time.
 *   late[i] = 1 iff units[i] > 0 and tau * units[i] / compute[i] + t_comm > timeout.
 * The path has no clock: a caller applies the mask by giving the late devices a
 * loss rate of 1 in halo_plan_create (they then hold the least critical groups
 * and their partials never arrive), or reschedules with Algorithm 2.
 * HALO_ERR_ARG: NULL pointers, n_dev outside [1, HALO_MAX_DEVICES], negative
 * units, tau, t_comm or timeout, non-positive computing power.
 * ---------------------------------------------------------------------- */
halo_status halo_late_devices(int n_dev, const int32_t* units, const double* compute, double tau, double t_comm,
                              double timeout, uint8_t* late);

/* ------------------------------------------------------------------------
 * a1. Predictor (Sec. III-B.2, semantic-aware predictors): importance score
 * of every neuron group of a block from semantic features taken one layer
 * ahead.  Bias-free two-layer network
 *     z = act(W1 * f),  s = W2 * z
 *   W1   device [rank][d_in]      (row u = weights of hidden unit u)
 *   W2   device [n_groups][rank]
 *   feat device [n_tok][d_in], wdtype
 *   scores device fp32: [n_groups] if n_tok == 1 or mean_pool != 0 (mean over
 *     the tokens of the per-token scores, fixed token order), else [n_tok][n_groups]
 *   workspace: halo_predict_workspace_bytes(shape, n_tok) bytes, device.
 * fp32 accumulation.  Sets HALO_DEV_NONFINITE_SCORE if a score is not finite.
 * ---------------------------------------------------------------------- */
size_t halo_predict_workspace_bytes(const halo_pred_shape* shape, int n_tok);
halo_status halo_predict_groups(const halo_pred_shape* shape, const void* W1, const void* W2,
                                const void* feat, int n_tok, int mean_pool, float* scores,
                                void* workspace, size_t workspace_bytes, uint32_t* dev_status, void* stream);

/* ------------------------------------------------------------------------
 * The predictor for callers that cannot provide a workspace.  (The paper has no counterpart of this entry
 * point; it exists for the way this library gets embedded.)
 *
 * halo_predict_groups needs a device workspace, and a workspace has to be allocated by somebody.  Some callers
 * cannot do that at the point of the call: a server that handed all device memory to its own pool at start-up,
 * a plug-in living inside another program's memory budget, a latency-critical loop where entering the CUDA
 * allocator (which may synchronise the device) is not acceptable.  This variant computes exactly what
 * halo_predict_groups computes, with the same arguments minus the workspace, and keeps its two intermediate
 * arrays in a fixed array compiled into the library (HALO_STATIC_SCRATCH_FLOATS floats = 2 MiB, held by every
 * GPU that loads the library, from load until the process exits).  It calls no allocation routine of any kind.
 *   Limit: n_tok * (rank + n_groups) <= HALO_STATIC_SCRATCH_FLOATS, else HALO_ERR_WORKSPACE and nothing runs.
 *   Set-up: the first call on each device looks up the device address of the array (with that device
 *     current); make that first call outside any stream capture.  Later calls only launch.
 *   Sharing: all calls on a device use the same array, and it keeps what the last call left in it.  Nothing in
 *     it needs to be zero at entry.  Two calls that overlap on the GPU (different streams, or host threads
 *     without ordering between their streams) race on it and give wrong scores: keep calls on one stream, or
 *     order them with events.
 * Other errors and the device status word are as for halo_predict_groups.
 * ---------------------------------------------------------------------- */
#define HALO_STATIC_SCRATCH_FLOATS (512 * 1024)
halo_status halo_predict_groups_static(const halo_pred_shape* shape, const void* W1, const void* W2,
                                       const void* feat, int n_tok, int mean_pool, float* scores,
                                       uint32_t* dev_status, void* stream);

/* ------------------------------------------------------------------------
 * a2..a5. Rank, critical choice, runtime assignment and arrival mask
 * (Sec. III-B.3, Pred process: the importance rank indexes the priority
 * lists fixed by the Assignment phase; relaxed synchronisation: the master
 * merges what arrived).
 *   scores device fp32 [G].  Order = higher score first, equal scores by
 *     lower group id; NaN ranks as -inf (status bit), -0 equals +0.
 *   step, layer: counter of the arrival draw.  Device i's partial of this
 *     (step, layer) arrives iff word 0 of Philox4x32-10 with counter
 *     (step, layer, i, 0) and key (seed low, seed high) is >= T_i.
 *   force_all != 0: a reliable block (the first layer): everything arrives.
 * Outputs (device; any of order/dev_of_group/arrived/keep may be NULL):
 *   order[G]        group id at each priority position
 *   dev_of_group[G] holder of each group: -1 = master (critical), else device index
 *   arrived[n_dev]  1 if the device's partial arrives
 *   keep[G]         1 if the group's contribution survives
 *   keep_list[G]    kept group ids, ascending, then -1 padding
 *   n_keep[1]       number of kept groups
 * One thread block; G <= HALO_MAX_GROUPS.
 * ---------------------------------------------------------------------- */
halo_status halo_select_groups(const halo_plan* plan, const float* scores, uint32_t step, uint32_t layer,
                               int force_all, int32_t* order, int32_t* dev_of_group, uint8_t* arrived,
                               uint8_t* keep, int32_t* keep_list, int32_t* n_keep, uint32_t* dev_status,
                               void* stream);

/* ------------------------------------------------------------------------
 * a6..a8. Group-masked SwiGLU FFN (Sec. II-A neuron groups; Sec. II-B: the
 * merged features are the sum of the groups' activations).  For each kept
 * group g and neuron j of it
 *     a = <gate_j, x>, b = <up_j, x>, h = a / (1 + exp(-a)) * b,
 *     partials[slot(g)] += h * down_j,   slot = dev_of_group[g] + 1 (0 = master)
 *   W_packed device, layout above;  x device [n_tok][d], wdtype
 *   keep_list device [>= *n_keep] group ids; n_keep device [1]
 *   dev_of_group device [G] or NULL (everything into slot 0; then n_dev is 0)
 *   partials device fp32 [n_dev+1][n_tok][d]; overwritten (zeroed by the call)
 *   workspace: halo_group_ffn_workspace_bytes(shape, n_tok, n_dev) bytes, device
 * Groups that are not listed cost no memory traffic.  bf16/fp32 inputs, fp32
 * accumulation.  n_tok == 1 runs the bandwidth-bound decode kernel; larger
 * n_tok with bf16 weights runs the tensor-core contraction.  Out-of-range ids
 * are skipped and flagged HALO_DEV_BAD_INDEX.
 * ---------------------------------------------------------------------- */
size_t halo_group_ffn_workspace_bytes(const halo_ffn_shape* shape, int n_tok, int n_dev);
halo_status halo_group_ffn(const halo_ffn_shape* shape, const void* W_packed, const void* x, int n_tok,
                           const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group,
                           int n_dev, float* partials, void* workspace, size_t workspace_bytes,
                           uint32_t* dev_status, void* stream);

/* ------------------------------------------------------------------------
 * True importance of the groups (Sec. II-B: the importance of an activation is
 * its L2 norm; Sec. III-B.2: the predictors are trained on activation norms).
 * norms[g] = || p_g ||_2, p_g = sum_{j in g} silu(<gate_j,x>) * <up_j,x> * down_j,
 * for every group of the block and ONE input vector x.  A calibration and
 * diagnostic call (it reads the whole block), not part of the per-token path.
 *   W_packed device; x device [d], wdtype; norms device fp32 [G]
 *   workspace: halo_group_importance_workspace_bytes(shape) bytes, device.
 * ---------------------------------------------------------------------- */
size_t halo_group_importance_workspace_bytes(const halo_ffn_shape* shape);
halo_status halo_group_importance(const halo_ffn_shape* shape, const void* W_packed, const void* x, float* norms,
                                  void* workspace, size_t workspace_bytes, uint32_t* dev_status, void* stream);

/* ------------------------------------------------------------------------
 * a9. Merge (Sec. III-B.3: after the timeout the master merges the
 * activations that are available): y = partials[0] + sum_i arrived[i] * partials[i+1].
 *   partials device fp32 [n_dev+1][n_tok][d]; arrived device [n_dev] or NULL (all)
 *   y device fp32 [n_tok][d]
 * ---------------------------------------------------------------------- */
halo_status halo_merge_partials(const float* partials, const uint8_t* arrived, int n_dev, int n_tok,
                                int d_model, float* y, void* stream);

/* ------------------------------------------------------------------------
 * Helpers around the path.
 * halo_pack_weights: Wgate[F][d], Wup[F][d], Wdown[d][F] (device) -> W_packed (device).
 * halo_glue: element-wise work between the blocks of an FFN stack (Sec. II-A:
 *   normalisation and residual connection): h_out = h + y (y may be NULL),
 *   x_out = cast(h_out / sqrt(mean(h_out^2) + 1e-5)) per token.
 *   h, y, h_out device fp32 [n_tok][d] (h_out may alias h); x_out device [n_tok][d] in `xdtype`.
 * ---------------------------------------------------------------------- */
halo_status halo_pack_weights(const halo_ffn_shape* shape, const void* Wgate, const void* Wup,
                              const void* Wdown, void* W_packed, void* stream);
halo_status halo_glue(int d_model, int n_tok, halo_dtype xdtype, const float* h, const float* y, float* h_out,
                      void* x_out, void* stream);

/* ------------------------------------------------------------------------
 * MHA neuron groups, decode form (Sec. II-A: "one head and its output projection weight are an independent
 * neuron group").  The same scoring / selection / holder slots / merge apply with G = n_heads: score with
 * halo_predict_groups, choose with halo_select_groups, merge with halo_merge_partials.  Keys and values are not
 * part of a group: every device keeps a full KV cache (Sec. III-B.3), so the K/V projections of ALL heads are
 * computed at every token (halo_mha_kv_append) and never dropped.  No positional rotation is applied.
 *   halo_mha_shape: d_model % 8 == 0, head_dim a multiple of 16 (<= 256); max_len = cache capacity.
 *   W_packed device [H][2][head_dim][d]: plane 0 = the head's query rows, plane 1 = the head's slice of the
 *     output projection stored as rows (row j = column h*head_dim+j of Wo[d][H*head_dim]);
 *     halo_pack_mha_weights builds it from Wq[H*head_dim][d] and Wo.
 *   K_cache, V_cache device [H][max_len][head_dim] in wdtype.
 *   halo_mha_kv_append: k = Wk x, v = Wv x (Wk, Wv device [H*head_dim][d]) written at position pos.
 *   halo_group_mha: for each kept head h: q = Wq_h x; w = softmax(q K_h^T / sqrt(head_dim)) over positions
 *     0..pos; o = w V_h; partials[slot(h)] += sum_j o_j * Wo_h[j].  partials device fp32 [n_dev+1][d], zeroed by
 *     the call; keep_list / n_keep / dev_of_group as for halo_group_ffn (device); x device [d].
 *     workspace: halo_group_mha_workspace_bytes(shape) bytes, device.  fp32 accumulation and softmax.
 * ---------------------------------------------------------------------- */
typedef struct {
    int d_model, n_heads, head_dim, max_len;
    halo_dtype wdtype;
} halo_mha_shape;
halo_status halo_pack_mha_weights(const halo_mha_shape* shape, const void* Wq, const void* Wo, void* W_packed,
                                  void* stream);
halo_status halo_mha_kv_append(const halo_mha_shape* shape, const void* Wk, const void* Wv, const void* x, int pos,
                               void* K_cache, void* V_cache, void* stream);
size_t halo_group_mha_workspace_bytes(const halo_mha_shape* shape);
/* halo_mha_block: halo_mha_kv_append and halo_group_mha of one token in ONE launch (a cluster of eight thread blocks
 * per head: keys and values of every head are written at `pos`, then the kept heads attend over positions 0..pos and
 * add their output-projection slices into partials, zeroed by the call).  Same results as the two calls in turn;
 * K_cache / V_cache are read and written; no workspace. */
halo_status halo_mha_block(const halo_mha_shape* shape, const void* W_packed, const void* Wk, const void* Wv,
                           const void* x, void* K_cache, void* V_cache, int pos, const int32_t* keep_list,
                           const int32_t* n_keep, const int32_t* dev_of_group, int n_dev, float* partials,
                           uint32_t* dev_status, void* stream);
/* halo_mha_block on int4 weights (Sec. IV-A): Qp / Sp, Qk / Sk, Qv / Sv = codes and scales written by
 * halo_quantize_rows_i4 for W_packed (as [H*2*head_dim][d_model]), Wk and Wv; x and the caches bf16
 * (shape->wdtype must be HALO_BF16), d_model % 128 == 0, head_dim % 16 == 0.  Results: halo_mha_block on the
 * dequantised weights. */
halo_status halo_mha_block_i4(const halo_mha_shape* shape, const void* Qp, const void* Sp, const void* Qk, const void* Sk,
                              const void* Qv, const void* Sv, const void* x, void* K_cache, void* V_cache, int pos,
                              const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group, int n_dev,
                              float* partials, uint32_t* dev_status, void* stream);
halo_status halo_group_mha(const halo_mha_shape* shape, const void* W_packed, const void* x, const void* K_cache,
                           const void* V_cache, int pos, const int32_t* keep_list, const int32_t* n_keep,
                           const int32_t* dev_of_group, int n_dev, float* partials, void* workspace,
                           size_t workspace_bytes, uint32_t* dev_status, void* stream);

/* ------------------------------------------------------------------------
 * int4 group-quantised weights for the decode FFN (the paper evaluates models "quantized to 4-bit integer
 * precision", Sec. IV-A, and fixes the neuron-group size "for compatibility with quantization", Sec. II-A; it
 * gives no format).  Format used here: symmetric, one bf16 scale per block of 128 consecutive elements of a
 * packed row: s = bf16(amax / 7) rounded UP to the next bf16 number with at most 5 significant bits,
 * q = clamp(rint(w / s), -8, 7) (fp32 division, round half to even; s == 0 gives q = 0), stored as nibble q + 8
 * with element 2i in the low half of byte i.  value = (nibble - 8) * s, which has at most 8 significant bits: every
 * dequantised value is exactly a bf16 number.
 *   shape: as for halo_group_ffn, with d_model % 128 == 0 and d_model <= 8192; wdtype = type of the SOURCE
 *     weights for halo_quantize_weights_i4, ignored by halo_group_ffn_i4.
 *   Q device uint8 [G][3][S][d/2]; scales device bf16 [G][3][S][d/128]; both 16-byte aligned, caller-owned.
 *   halo_quantize_weights_i4: W_packed (device, layout of halo_pack_weights) -> Q, scales.
 *   halo_group_ffn_i4: halo_group_ffn on the dequantised weights; x device bf16 [n_tok][d]; partials device
 *     fp32 [n_dev+1][n_tok][d], zeroed by the call; keep_list / n_keep / dev_of_group / dev_status as there.
 *     Decode form (one pass over the kept groups' weights per token); no workspace.
 *   halo_dequantize_weights_i4: Q, scales -> W_packed (device bf16, layout of halo_pack_weights, 16-byte aligned,
 *     caller-owned), every element (nibble - 8) * s, exact for scales written by the quantisers of this library
 *     (a scale with more than 5 significant bits is rounded once).  keep_list / n_keep
 *     (device, as for halo_group_ffn) name the groups to write, the others are left as they are; keep_list NULL
 *     writes all groups.  For prompts: the tensor cores take bf16 operands, so a prompt on int4 weights is this
 *     call followed by halo_group_ffn on its output (what an int4 stack created for more than one token does per
 *     block).  shape->wdtype is ignored.  An out-of-range index sets HALO_DEV_BAD_INDEX and that entry is skipped.
 * ---------------------------------------------------------------------- */
halo_status halo_quantize_weights_i4(const halo_ffn_shape* shape, const void* W_packed, void* Q, void* scales,
                                     void* stream);
/* The same quantiser for any row matrix: W device [n_rows][d_model] in wdtype (d_model % 128 == 0, <= 8192) ->
 * Q device uint8 [n_rows][d_model/2], scales device bf16 [n_rows][d_model/128]; all 16-byte aligned. */
halo_status halo_quantize_rows_i4(int d_model, long long n_rows, halo_dtype wdtype, const void* W, void* Q, void* scales,
                                  void* stream);
halo_status halo_dequantize_weights_i4(const halo_ffn_shape* shape, const void* Q, const void* scales,
                                       const int32_t* keep_list, const int32_t* n_keep, void* W_packed,
                                       uint32_t* dev_status, void* stream);
halo_status halo_group_ffn_i4(const halo_ffn_shape* shape, const void* Q, const void* scales, const void* x, int n_tok,
                              const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group,
                              int n_dev, float* partials, uint32_t* dev_status, void* stream);
/* halo_group_ffn_i4 for prompts.  halo_group_ffn_i4_workspace_bytes is non-zero for token counts and shapes the
 * tensor-core FFN takes (16 tokens or more, d_model % 128 == 0, group size 64 / 128 / 256): the call then writes the
 * kept groups' dequantised weights (exact in bf16) into the caller's workspace and runs halo_group_ffn's tensor-core
 * form on them; workspace device, 16-byte aligned, at least that many bytes (one bf16 block of 3 * d_ffn * d_model
 * elements + halo_group_ffn's own workspace), else HALO_ERR_WORKSPACE.  Where the size is 0 the call is
 * halo_group_ffn_i4 and the workspace is not used.  Results and every other argument as halo_group_ffn_i4. */
size_t halo_group_ffn_i4_workspace_bytes(const halo_ffn_shape* shape, int n_tok);
halo_status halo_group_ffn_i4_prompt(const halo_ffn_shape* shape, const void* Q, const void* scales, const void* x,
                                     int n_tok, const int32_t* keep_list, const int32_t* n_keep,
                                     const int32_t* dev_of_group, int n_dev, float* partials, void* workspace,
                                     size_t workspace_bytes, uint32_t* dev_status, void* stream);

/* ------------------------------------------------------------------------
 * LM-head neuron groups (Sec. II-A: the LM head "only contains up-projection" and is "also a collection of
 * neuron groups"; Sec. III-B.3: its results are sent reliably "to ensure the logits are accurate").  A group is
 * group_size consecutive vocabulary rows (the last group may be shorter).  Nothing is dropped and nothing is
 * summed: the groups' outputs are concatenated, so there are no holder slots and no arrival mask here; a caller
 * that distributes the groups over devices uses halo_plan_create / halo_select_groups for the assignment only.
 *   W device [vocab][d_model] in wdtype (16-byte aligned, d_model % 8 == 0, d_model <= 8192);
 *   x device [n_tok][d_model] in wdtype; logits device fp32 [n_tok][vocab];
 *   keep_list / n_keep device: the groups to compute (indices < ceil(vocab / group_size)); both NULL = all.
 *   For every listed group and token: logits[t][v] = <W[v], x_t> (fp32 accumulation); entries of unlisted
 *   groups are left untouched.  An index outside the range sets HALO_DEV_BAD_INDEX in *dev_status and that
 *   group is skipped.  Asynchronous on `stream`; no workspace.
 * ---------------------------------------------------------------------- */
typedef struct {
    int d_model, vocab, group_size;
    halo_dtype wdtype;
} halo_lm_shape;
halo_status halo_group_lm_head(const halo_lm_shape* shape, const void* W, const void* x, int n_tok,
                               const int32_t* keep_list, const int32_t* n_keep, float* logits, uint32_t* dev_status,
                               void* stream);
/* halo_group_lm_head on int4 rows (Sec. IV-A: the evaluated models are 4-bit): Q / scales as written by
 * halo_quantize_rows_i4 for W [vocab][d_model] (d_model % 128 == 0); x device bf16 [n_tok][d_model]; shape->wdtype is
 * ignored.  logits[t][v] = <dequantised row v, x_t> (fp32 accumulation); everything else as halo_group_lm_head. */
halo_status halo_group_lm_head_i4(const halo_lm_shape* shape, const void* Q, const void* scales, const void* x, int n_tok,
                                  const int32_t* keep_list, const int32_t* n_keep, float* logits, uint32_t* dev_status,
                                  void* stream);

/* ------------------------------------------------------------------------
 * One block, steps a1..a9 in one call (the Pred, Comp and merge of one block of the generation phase,
 * Sec. III-B.3): scores from `feat` (the input of the previous block: one layer ahead), selection and arrival
 * draw for (step, layer), FFN of `x` over the kept groups, merge of what arrived.  Same results as calling
 * halo_predict_groups (mean-pooled when n_tok > 1), halo_select_groups, halo_group_ffn and halo_merge_partials
 * in turn.
 *   feat, x device [n_tok][d] wdtype; scores device fp32 [G]; dev_of_group device [G]; arrived device [n_dev];
 *   keep device [G] or NULL; y device fp32 [n_tok][d]
 *   workspace: halo_layer_workspace_bytes(ffn, pred, n_tok, plan's n_dev) bytes, device.
 * ---------------------------------------------------------------------- */
size_t halo_layer_workspace_bytes(const halo_ffn_shape* ffn, const halo_pred_shape* pred, int n_tok, int n_dev);
halo_status halo_layer_fused(const halo_ffn_shape* ffn, const halo_pred_shape* pred, const halo_plan* plan,
                             const void* W_packed, const void* W1, const void* W2, const void* feat, const void* x,
                             int n_tok, uint32_t step, uint32_t layer, int force_all, float* scores,
                             int32_t* dev_of_group, uint8_t* arrived, uint8_t* keep, float* y, void* workspace,
                             size_t workspace_bytes, uint32_t* dev_status, void* stream);
/* halo_status_message for a status word the caller has copied to the host. */
halo_status halo_read_status(const uint32_t* dev_status_host_copy, char* msg /*host*/, int msg_len);

/* ------------------------------------------------------------------------
 * FFN stack: L blocks chained by halo_glue, the predictor of block l reading
 * the input of block l-1 (one layer ahead, Sec. III-B.2) and block 0 reliable
 * (Sec. III-B.3: the first layer has no semantic information yet).
 * halo_stack_create copies the per-layer pointer tables and allocates the
 * device work buffers it owns (freed by halo_stack_destroy); the weights stay
 * caller-owned and must outlive the stack.
 *   W_packed[L], W1[L], W2[L]: host arrays of device pointers (W1[0], W2[0] unused, may be NULL)
 * ---------------------------------------------------------------------- */
typedef struct {
    void* x;              /* device [steps][L][n_tok][d] wdtype: input of every block */
    float* scores;        /* device [steps][L][G] (block 0: zeros) */
    int32_t* dev_of_group;/* device [steps][L][G] */
    uint8_t* arrived;     /* device [steps][L][n_dev] */
    int32_t* keep_list;   /* device [steps][L][G] */
    int32_t* n_keep;      /* device [steps][L] */
    float* y;             /* device [steps][L][n_tok][d]: merged output of every block */
} halo_taps;              /* any member may be NULL */

halo_status halo_stack_create(halo_stack** out, const halo_ffn_shape* ffn, const halo_pred_shape* pred,
                              int n_layers, int n_tok, const halo_plan* plan, const void* const* W_packed,
                              const void* const* W1, const void* const* W2);
/* The same stack on int4 group-quantised FFN weights (Sec. IV-A: the evaluated models are 4-bit): Q[L] and scales[L]
 * as written by halo_quantize_weights_i4 for every block; activations, predictor and everything else as above
 * (ffn->wdtype must be HALO_BF16, d_model % 128 == 0).  One token: the persistent decode kernel for d_model 2048 and
 * 4096, else one launch per step of the path.  Prompts of 16 tokens or more on shapes the tensor-core FFN takes: the
 * stack also owns two bf16 scratch blocks (2 x 3 * d_ffn * d_model * 2 bytes), the kept groups of every block are
 * written there by halo_dequantize_weights_i4's kernel and the tensor-core FFN reads them; other token counts go
 * through halo_group_ffn_i4 token by token. */
halo_status halo_stack_create_i4(halo_stack** out, const halo_ffn_shape* ffn, const halo_pred_shape* pred,
                                 int n_layers, int n_tok, const halo_plan* plan, const void* const* Q,
                                 const void* const* scales, const void* const* W1, const void* const* W2);
halo_status halo_stack_destroy(halo_stack* stack);
/* Runs `steps` tokens (or prompts of n_tok tokens) through the stack.
 *   h0    device fp32 [steps][n_tok][d]: residual-stream input of each step
 *   h_out device fp32 [steps][n_tok][d]: residual stream after the last block
 *   step0: arrival-draw counter of the first step
 *   taps: NULL or per-block records for checking
 * Asynchronous on `stream`; no host synchronisation inside. */
halo_status halo_stack_decode(halo_stack* stack, const float* h0, int steps, uint32_t step0, float* h_out,
                              const halo_taps* taps, void* stream);
/* Same with HOST buffers (pinned memory recommended): copies h0 in, runs,
 * copies h_out back and synchronises the stream before returning. */
halo_status halo_stack_decode_host(halo_stack* stack, const float* h0_host, int steps, uint32_t step0,
                                   float* h_out_host, void* stream);
/* How halo_stack_decode runs.  mode = 0 (default) or a sum of the flags below.
 * Default: decode of bf16 stacks with d_model in {2048, 4096, 5120, 8192} runs as ONE persistent cooperative
 * kernel over all steps and blocks, with the two overlaps of the paper's generation phase (Sec. III-B.3): the
 * predictor and selection of block l+1 run beside the weight stream of block l (Pred beside Comp/Comm), and the
 * first weights of block l+1 are fetched while block l is still being merged (Load beside Comp).  Anything else
 * runs one launch per step of the path; for prompts the predictor and selection of block l+1 then run on a side
 * stream beside the tensor-core FFN of block l.
 *   HALO_STACK_PER_STEP_LAUNCHES  always one launch per step of the path (for comparison and checking);
 *   HALO_STACK_PRED_SERIAL        persistent decode kernel with the predictor and selection of a block at the start
 *                                 of that block, in front of its weight stream (the ablation arm "Pred not overlapped");
 *   HALO_STACK_LOAD_SERIAL        persistent decode kernel that fetches no weights of block l+1 before block l is
 *                                 merged (the ablation arm "Load not overlapped");
 *   HALO_STACK_DETERMINISTIC      persistent decode kernel with a fixed assignment of neuron batches to thread blocks
 *                                 and column sums added in a fixed order, so that two runs give bitwise identical
 *                                 results (slower: every thread block reads every other's sums); the default adds
 *                                 them with atomic reductions in arrival order.
 *   HALO_STACK_PROMPT_ONE_LAUNCH  prompts of more than 128 tokens (bf16, d_model % 256 == 0, group size 64/128/256,
 *                                 predictor rank <= 1024, no y records asked for) run as ONE persistent kernel per
 *                                 prompt: a tile queue over all blocks with the predictor, the selection and the
 *                                 normalisation between blocks inside.  No host work between blocks and one launch
 *                                 instead of ~7 per block; measured 4 % slower than the default on the 512-token 7B
 *                                 shape (the normalisation sits on the critical path of every block boundary), so
 *                                 it is not the default.
 * The three flags before it only act on the persistent decode kernel; results are the same numbers in every mode up
 * to the order of fp32 additions. */
#define HALO_STACK_PER_STEP_LAUNCHES 1
#define HALO_STACK_PRED_SERIAL 2
#define HALO_STACK_LOAD_SERIAL 4
#define HALO_STACK_DETERMINISTIC 8
#define HALO_STACK_PROMPT_ONE_LAUNCH 16
halo_status halo_stack_set_mode(halo_stack* stack, int mode);
/* Measurement options, process-wide.  The defaults are the measured best; the options exist so that a sweep or an
 * ablation can be run through the same library.  value = -1 restores the default.  A stack reads the first three
 * when it is created; the others are read at every call of the entry point they belong to.  No environment
 * variable is read anywhere in the library.
 *   "cross_stages" (0..16)            persistent kernel: stages of the next block fetched across the block barrier
 *   "tmem_ring" (0/1)                 persistent kernel, d_model 2048 / 4096: second level of the weight ring in
 *                                     tensor memory (default 0: measured slower, kept as an option)
 *   "l2_ahead" (0..32)                persistent kernel: batches prefetched to L2 on entering a block
 *   "max_steps_per_launch" (0 = auto) persistent kernel: steps per launch before a run is split
 *   "prefill_two_launches" (0/1)      prompt FFN as two launches (hidden, down) instead of one
 *   "prefill_kcuts" (1..16), "prefill_kratio_percent" (30..100)   prompt FFN: K runs per down-projection tile and
 *                                     the ratio between consecutive runs
 *   "mha_three_launches" (0/1)        halo_group_mha as three launches instead of one
 *   "i4_no_ring" (0..3)               halo_group_ffn_i4: 0 shared-memory ring with two thread blocks per SM
 *                                     (default), 1 plain loads, 2 ring with one thread block per SM, 3 ring with
 *                                     the products on the legacy tensor-core path (mma.sync; slower here)
 * HALO_ERR_ARG for an unknown name or a value outside the stated range. */
halo_status halo_set_option(const char* name, int value);
/* Tracing of the persistent kernel (timing statistics of the generation loop): the caller gives a device
 * buffer trace[n_blocks][halo_stack_trace_width()][8] of 64-bit words; for the first n_blocks blocks of a
 * halo_stack_decode run every thread block records global-timer nanoseconds at: 0 block start, 1 first weight
 * stage landed, 2 last stage consumed, 3 partial sums flushed, 4 grid barrier passed, 5 slots merged,
 * 6 next input ready; 7 = duration of the selection (selecting thread block only).  n_blocks = 0 turns it off. */
halo_status halo_stack_set_trace(halo_stack* stack, unsigned long long* trace /*device*/, int n_blocks);
int halo_stack_trace_width(const halo_stack* stack);
/* ------------------------------------------------------------------------
 * Transformer-block stack: the generation loop over whole layers (Sec. III-B.3, Comp process: "MHA then MLP"; Sec. II-A:
 * MHA blocks, MLP blocks and the LM head are all collections of neuron groups; the first layer and the LM head are sent
 * reliably).  Per token at position pos and layer l:
 *     x_a = cast(rmsnorm(h));  keys / values of ALL heads from x_a appended to layer l's caches at pos (never dropped)
 *     kept heads  = selection from the MHA predictor of layer l applied to layer l-1's x_a   (arrival draw (step, 2l))
 *     h += merge(halo_group_mha over the kept heads)
 *     x_f = cast(rmsnorm(h))
 *     kept groups = selection from the MLP predictor of layer l applied to layer l-1's x_f   (arrival draw (step, 2l+1))
 *     h += merge(halo_group_ffn over the kept groups)
 * Layer 0 keeps every head and group.  After the last layer the LM-head groups (all of them) give the logits of
 * cast(rmsnorm(h)).  The residual input h_0 of each token is given by the caller (it stands for the embedding of the
 * previous token).  One launch per step of the path on `stream`, no host synchronisation inside.
 *   halo_block_weights: host arrays of n_layers device pointers (caller-owned, they must outlive the stack):
 *     W_ffn packed FFN weights; W_mha packed MHA weights (halo_pack_mha_weights); Wk, Wv [H*head_dim][d];
 *     W1_ffn / W2_ffn and W1_mha / W2_mha predictor factors (entry 0 unused, may be NULL); K_cache / V_cache
 *     [H][max_len][head_dim], updated by decode; W_lm [vocab][d] (NULL and lm == NULL: no LM head).
 *   plan_ffn over the FFN groups, plan_mha over the heads (n_groups = n_heads).
 *   halo_block_stack_decode: h0 device fp32 [steps][d]; token s sits at position pos0 + s (pos0 + steps <= max_len)
 *     and draws arrivals with counter step0 + s; logits device fp32 [steps][vocab] or NULL; h_out device fp32
 *     [steps][d] or NULL; taps: NULL or records per (step, layer) of either block type (layout of halo_taps with
 *     n_tok = 1; for the MHA block G = n_heads).
 * ---------------------------------------------------------------------- */
typedef struct halo_block_stack halo_block_stack;
typedef struct {
    const void* const* W_ffn;
    const void* const* W_mha;
    const void* const* Wk;
    const void* const* Wv;
    const void* const* W1_ffn;
    const void* const* W2_ffn;
    const void* const* W1_mha;
    const void* const* W2_mha;
    void* const* K_cache;
    void* const* V_cache;
    const void* W_lm;
} halo_block_weights;
typedef struct {
    halo_taps mha;
    halo_taps ffn;
} halo_block_taps;
halo_status halo_block_stack_create(halo_block_stack** out, const halo_ffn_shape* ffn, const halo_mha_shape* mha,
                                    const halo_lm_shape* lm, const halo_pred_shape* pred_ffn,
                                    const halo_pred_shape* pred_mha, int n_layers, const halo_plan* plan_ffn,
                                    const halo_plan* plan_mha, const halo_block_weights* weights);
/* The same stack on int4 weights (Sec. IV-A: the evaluated models are 4-bit): `codes` has the layout of
 * halo_block_weights with W_ffn = codes of halo_quantize_weights_i4, W_mha / Wk / Wv / W_lm = codes of
 * halo_quantize_rows_i4 of the matrices named there; `scales` holds the matching scale arrays (host arrays of n_layers
 * device pointers, 16-byte aligned; S_lm NULL without an LM head).  Predictor factors, activations and the K/V caches
 * stay bf16 (every shape's wdtype must be HALO_BF16); d_model % 128 == 0, head_dim % 16 == 0.  Per layer:
 * halo_mha_block_i4, halo_group_ffn_i4, and halo_group_lm_head_i4 at the end. */
typedef struct {
    const void* const* S_ffn;
    const void* const* S_mha;
    const void* const* Sk;
    const void* const* Sv;
    const void* S_lm;
} halo_block_scales;
halo_status halo_block_stack_create_i4(halo_block_stack** out, const halo_ffn_shape* ffn, const halo_mha_shape* mha,
                                       const halo_lm_shape* lm, const halo_pred_shape* pred_ffn,
                                       const halo_pred_shape* pred_mha, int n_layers, const halo_plan* plan_ffn,
                                       const halo_plan* plan_mha, const halo_block_weights* codes,
                                       const halo_block_scales* scales);
halo_status halo_block_stack_destroy(halo_block_stack* stack);
halo_status halo_block_stack_decode(halo_block_stack* stack, const float* h0, int steps, int pos0, uint32_t step0,
                                    float* logits, float* h_out, const halo_block_taps* taps, void* stream);
halo_status halo_block_stack_status(halo_block_stack* stack, uint32_t* dev_status_value /*host*/, void* stream);
long long halo_block_stack_last_launches(const halo_block_stack* stack);

/* Failure detection self-test.  Every device-side wait of this library (mbarrier phases of the copy rings, the
 * grid barrier, the published-selection flag) is bounded; when one runs out the kernel raises HALO_DEV_TIMEOUT
 * and returns, so a late or missing partner shows up as a status bit, never as a hung GPU (the paper's master
 * likewise proceeds after its receive timeout, Sec. III-B.3).  This call exercises that mechanism harmlessly:
 * one thread block waits, for at most limit_cycles SM cycles each (1 .. 2e9), on an mbarrier phase nobody
 * completes and on the device word never_set_flag (which the caller leaves at 0).  On return (after
 * synchronising) report[0] = number of threads whose mbarrier wait ran out (128), report[1] = 1 if the flag wait
 * ran out, and HALO_DEV_TIMEOUT is set in *dev_status.  All pointers are device pointers. */
halo_status halo_selftest_bounded_wait(const uint32_t* never_set_flag, long long limit_cycles, uint32_t* report,
                                       uint32_t* dev_status, void* stream);
/* Device status word accumulated by the stack's launches (synchronises the stream). */
halo_status halo_stack_status(halo_stack* stack, uint32_t* dev_status_value /*host*/, void* stream);
/* Number of kernel launches the last halo_stack_decode enqueued. */
long long halo_stack_last_launches(const halo_stack* stack);

#ifdef __cplusplus
}
#endif
#endif /* HALO_H */
