/*
 * halo_ref.c -- CPU fp64 oracle for the HALO group-sparse FFN hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what
 * the method computes, used to check the CUDA library and to time a CPU
 * baseline.  Nothing on the product path may call it, and it shares no code,
 * header, table or helper with the CUDA sources.
 *
 * Every function takes HOST pointers.  Weights / activations arrive as the raw
 * bytes the GPU sees (fp32, or bf16 as uint16) and are widened exactly to
 * double; all arithmetic is fp64 unless a step is an integer decision.
 *
 * Passages followed (HALO, arXiv 2601.11676):
 *   Sec. II-A "Neuron group"            -- a group = gate rows + up rows + the
 *                                          matching down-projection columns.
 *   Sec. II-B insight                   -- merged features = sum of all groups'
 *                                          activations (linearity).
 *   Sec. III-B.2 (SAPs)                 -- small predictor, importance score
 *                                          per group, one layer ahead.
 *   Sec. III-B.3 (Pred process)         -- importance rank indexes the
 *                                          priority lists of the Assignment phase.
 *   Sec. III-B.4 + Algorithm 3          -- PLR-aware ratio-guided partition of
 *                                          the priority list over devices.
 *   Sec. III-B.3 (relaxed sync)         -- the master merges whatever arrived;
 *                                          first layer is reliable.
 *
 * Pins (tests/test_oracle_*.py): Philox4x32-10 known answers; the worked
 * example printed with Algorithm 3; 6144/256 = 24 groups; NGLR = 1 - 1/n;
 * brute-force ranking; dense SwiGLU via an fp64 library matmul; linearity;
 * permutation invariance; closed forms; merge flip identity.
 * Parity unpinned: the *meaning* of predictor scores (needs trained weights)
 * and the particular arrival sequence (the paper's loss is physical; the
 * sequence is fixed here by the Philox counter convention only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define REF_OK 0
#define REF_ERR_ARG (-1)
#define REF_ERR_SHAPE (-2)
#define REF_ERR_NOMEM (-6)

#define REF_F32 0
#define REF_BF16 1

#define REF_SEL_TOPK 0
#define REF_SEL_THRESHOLD 1

#define REF_ACT_RELU 0
#define REF_ACT_NONE 1

#define REF_STATUS_NONFINITE 1u

/* ---- exact widening of the stored element types ------------------------- */

static double ref_widen(const void* base, size_t i, int dtype) {
    if (dtype == REF_F32) return (double)((const float*)base)[i];
    uint32_t bits = (uint32_t)((const uint16_t*)base)[i] << 16; /* bf16 = top half of fp32 */
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static size_t ref_elem_size(int dtype) { return dtype == REF_F32 ? 4 : 2; }

/* double -> bf16 with round-to-nearest-even, via the exact fp32 neighbours.
 * Used only by the inter-layer glue (the activation vector is stored bf16). */
static uint16_t ref_double_to_bf16(double v) {
    if (isnan(v)) return 0x7fc0;
    float f = (float)v;             /* RNE to fp32 first (as the GPU does) */
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;             /* RNE on the dropped 16 bits */
    return (uint16_t)(u >> 16);
}

/* ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) ------------------- */
/* Counter-based generator; 10 rounds of two 32x32->64 multiplies with the
 * published multipliers, and Weyl key bumps between rounds. */

static void philox_round(uint32_t c[4], const uint32_t k[2]) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
    uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    uint32_t n0 = hi1 ^ c[1] ^ k[0];
    uint32_t n2 = hi0 ^ c[3] ^ k[1];
    c[0] = n0; c[1] = lo1; c[2] = n2; c[3] = lo0;
}

void halo_ref_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
    uint32_t k[2] = {key[0], key[1]};
    for (int r = 0; r < 10; ++r) {
        if (r > 0) { k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u; }
        philox_round(c, k);
    }
    memcpy(out, c, sizeof c);
}

/* One Bernoulli draw per (seed, step, layer, device): the device's whole
 * partial activation arrives or is lost (relaxed synchronisation, Sec.
 * III-B.3).  counter = (step, layer, device, 0), key = seed halves; word 0 of
 * the output is compared with T = round(rho * 2^32) in 64-bit, so rho = 0
 * always arrives and rho = 1 never does. */
uint64_t halo_ref_loss_threshold(double rho) {
    if (!(rho > 0.0)) return 0;
    if (rho >= 1.0) return (uint64_t)1 << 32;
    double t = floor(rho * 4294967296.0 + 0.5);
    if (t > 4294967296.0) t = 4294967296.0;
    return (uint64_t)t;
}

int halo_ref_arrival(uint64_t seed, uint32_t step, uint32_t layer, uint32_t device, double rho) {
    uint32_t ctr[4] = {step, layer, device, 0u};
    uint32_t key[2] = {(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)};
    uint32_t out[4];
    halo_ref_philox4x32_10(ctr, key, out);
    return ((uint64_t)out[0] >= halo_ref_loss_threshold(rho)) ? 1 : 0;
}

/* ---- weight layout ------------------------------------------------------- */
/* Packed layer buffer W[G][3][S][d]: plane 0 = gate rows of the group, plane 1
 * = up rows, plane 2 = the group's down-projection columns stored as rows
 * (Sec. II-A: one group owns all three slices).  Conventional matrices are
 * Wgate[F][d], Wup[F][d], Wdown[d][F]. */

static size_t packed_index(int g, int plane, int j, int c, int S, int d) {
    return (((size_t)g * 3 + (size_t)plane) * (size_t)S + (size_t)j) * (size_t)d + (size_t)c;
}

int halo_ref_pack_weights(int d, int F, int S, int dtype, const void* Wgate, const void* Wup,
                          const void* Wdown, void* Wpacked) {
    if (d <= 0 || F <= 0 || S <= 0 || F % S != 0) return REF_ERR_SHAPE;
    size_t es = ref_elem_size(dtype);
    const char* wg = (const char*)Wgate;
    const char* wu = (const char*)Wup;
    const char* wd = (const char*)Wdown;
    char* out = (char*)Wpacked;
    int G = F / S;
    for (int g = 0; g < G; ++g)
        for (int j = 0; j < S; ++j) {
            size_t n = (size_t)g * S + j; /* neuron index in [0,F) */
            for (int c = 0; c < d; ++c) {
                memcpy(out + es * packed_index(g, 0, j, c, S, d), wg + es * (n * d + c), es);
                memcpy(out + es * packed_index(g, 1, j, c, S, d), wu + es * (n * d + c), es);
                memcpy(out + es * packed_index(g, 2, j, c, S, d), wd + es * ((size_t)c * F + n), es);
            }
        }
    return REF_OK;
}

int halo_ref_unpack_weights(int d, int F, int S, int dtype, const void* Wpacked, void* Wgate,
                            void* Wup, void* Wdown) {
    if (d <= 0 || F <= 0 || S <= 0 || F % S != 0) return REF_ERR_SHAPE;
    size_t es = ref_elem_size(dtype);
    const char* in = (const char*)Wpacked;
    int G = F / S;
    for (int g = 0; g < G; ++g)
        for (int j = 0; j < S; ++j) {
            size_t n = (size_t)g * S + j;
            for (int c = 0; c < d; ++c) {
                memcpy((char*)Wgate + es * (n * d + c), in + es * packed_index(g, 0, j, c, S, d), es);
                memcpy((char*)Wup + es * (n * d + c), in + es * packed_index(g, 1, j, c, S, d), es);
                memcpy((char*)Wdown + es * ((size_t)c * F + n), in + es * packed_index(g, 2, j, c, S, d), es);
            }
        }
    return REF_OK;
}

/* ---- step a1: predictor -------------------------------------------------- */
/* Bias-free two-layer net, Sec. III-B.2: z = act(W1 f), s = W2 z, with
 * W1[r][d_in] and W2[G][r] (one row per output unit).  Scores leave as fp32:
 * that array is the boundary the selection reads.  With mean_pool the scores
 * of the n_tok tokens are averaged in fp64 (token order fixed) before the
 * cast, giving one score vector for the whole prompt. */
int halo_ref_predict(int d_in, int rank, int G, int dtype, int act, const void* W1, const void* W2,
                     const void* feat, int n_tok, int mean_pool, float* scores) {
    if (d_in <= 0 || rank <= 0 || G <= 0 || n_tok <= 0) return REF_ERR_SHAPE;
    double* z = (double*)malloc(sizeof(double) * (size_t)rank);
    double* pooled = (double*)calloc((size_t)G, sizeof(double));
    if (!z || !pooled) { free(z); free(pooled); return REF_ERR_NOMEM; }
    for (int t = 0; t < n_tok; ++t) {
        for (int u = 0; u < rank; ++u) {
            double acc = 0.0;
            for (int c = 0; c < d_in; ++c)
                acc += ref_widen(W1, (size_t)u * d_in + c, dtype) * ref_widen(feat, (size_t)t * d_in + c, dtype);
            if (act == REF_ACT_RELU && acc < 0.0) acc = 0.0;
            z[u] = acc;
        }
        for (int g = 0; g < G; ++g) {
            double acc = 0.0;
            for (int u = 0; u < rank; ++u) acc += ref_widen(W2, (size_t)g * rank + u, dtype) * z[u];
            if (mean_pool) pooled[g] += acc;
            else scores[(size_t)t * G + g] = (float)acc;
        }
    }
    if (mean_pool)
        for (int g = 0; g < G; ++g) scores[g] = (float)(pooled[g] / (double)n_tok);
    free(z);
    free(pooled);
    return REF_OK;
}

/* ---- Assignment phase: Algorithm 3 -------------------------------------- */
/* q = argsort(rho ascending; ties -> lower device index).  The priority list
 * of M less-critical groups is cut into n contiguous chunks proportional to
 * the ratios taken in q's order; chunk j goes to device q[j].  Ratios are
 * integer weights; the cut after chunk j is round-half-up(M * C_j / C_n) in
 * 64-bit integers, C_j the cumulative weight. */
int halo_ref_plan(int n_dev, const double* loss_rate, const uint32_t* share_weight, int M,
                  int32_t* dev_order /*[n]*/, uint64_t* loss_thresh /*[n], by device index*/,
                  int32_t* boundaries /*[n+1]*/) {
    if (n_dev < 0 || M < 0) return REF_ERR_ARG;
    for (int i = 0; i < n_dev; ++i) {
        if (!(loss_rate[i] >= 0.0 && loss_rate[i] <= 1.0)) return REF_ERR_ARG;
        loss_thresh[i] = halo_ref_loss_threshold(loss_rate[i]);
        dev_order[i] = i;
    }
    /* insertion sort: stable, ascending rho */
    for (int a = 1; a < n_dev; ++a) {
        int32_t v = dev_order[a];
        int b = a - 1;
        while (b >= 0 && loss_rate[dev_order[b]] > loss_rate[v]) { dev_order[b + 1] = dev_order[b]; --b; }
        dev_order[b + 1] = v;
    }
    uint64_t total = 0;
    for (int i = 0; i < n_dev; ++i) total += share_weight[i];
    boundaries[0] = 0;
    if (n_dev == 0) return REF_OK;
    if (total == 0) return REF_ERR_ARG;
    uint64_t cum = 0;
    for (int j = 0; j < n_dev; ++j) {
        cum += share_weight[dev_order[j]];
        boundaries[j + 1] = (int32_t)((2ull * (uint64_t)M * cum + total) / (2ull * total));
    }
    boundaries[n_dev] = M;
    return REF_OK;
}

/* ---- steps a2..a5: rank, critical choice, assignment, arrival mask ------- */
/* Order: higher score first, equal scores -> lower group index (NaN counts as
 * -inf and raises a status bit; -0 == +0).  TOPK: the first k of the order are
 * critical.  THRESHOLD: critical = {s >= theta} (a prefix of the order).
 * Critical groups stay on the master (never lost); the rest, in priority
 * order, are cut by Algorithm 3.  keep = critical OR the holder arrived;
 * force_all (first layer / reliable block) keeps everything. */
int halo_ref_select(int G, int n_dev, const double* loss_rate, const uint32_t* share_weight,
                    int mode, int k_critical, float threshold, uint64_t seed,
                    const float* scores, uint32_t step, uint32_t layer, int force_all,
                    int32_t* order, int32_t* rank, int32_t* dev_of_group, uint8_t* arrived,
                    uint8_t* keep, int32_t* keep_list, int32_t* n_keep, uint32_t* status) {
    if (G <= 0 || n_dev < 0) return REF_ERR_SHAPE;
    if (mode == REF_SEL_TOPK && (k_critical < 0 || k_critical > G)) return REF_ERR_ARG;
    uint32_t st = 0;
    float* s = (float*)malloc(sizeof(float) * (size_t)G);
    int32_t* dev_order = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n_dev + 1));
    uint64_t* thr = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)(n_dev + 1));
    int32_t* bnd = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n_dev + 2));
    if (!s || !dev_order || !thr || !bnd) { free(s); free(dev_order); free(thr); free(bnd); return REF_ERR_NOMEM; }
    for (int g = 0; g < G; ++g) {
        float v = scores[g];
        if (isnan(v)) { v = -INFINITY; st |= REF_STATUS_NONFINITE; }
        else if (isinf(v)) st |= REF_STATUS_NONFINITE;
        if (v == 0.0f) v = 0.0f; /* folds -0 onto +0 */
        s[g] = v;
    }
    /* rank by counting: how many groups come strictly before g */
    for (int g = 0; g < G; ++g) {
        int before = 0;
        for (int o = 0; o < G; ++o)
            if (s[o] > s[g] || (s[o] == s[g] && o < g)) ++before;
        rank[g] = before;
        order[before] = g;
    }
    int k = k_critical;
    if (mode == REF_SEL_THRESHOLD) {
        k = 0;
        for (int g = 0; g < G; ++g) if (s[g] >= threshold) ++k;
    }
    if (n_dev == 0) k = G; /* nobody else to hold them */
    int M = G - k;
    int rc = halo_ref_plan(n_dev, loss_rate, share_weight, M, dev_order, thr, bnd);
    if (rc != REF_OK) { free(s); free(dev_order); free(thr); free(bnd); return rc; }
    for (int i = 0; i < n_dev; ++i)
        arrived[i] = (uint8_t)(force_all ? 1 : halo_ref_arrival(seed, step, layer, (uint32_t)i, loss_rate[i]));
    int nk = 0;
    for (int g = 0; g < G; ++g) {
        int dev = -1;
        if (rank[g] >= k) {
            int p = rank[g] - k;
            for (int j = 0; j < n_dev; ++j)
                if (bnd[j] <= p && p < bnd[j + 1]) { dev = dev_order[j]; break; }
        }
        dev_of_group[g] = dev;
        keep[g] = (uint8_t)((dev < 0) ? 1 : arrived[dev]);
        if (keep[g]) keep_list[nk++] = g;
    }
    for (int i = nk; i < G; ++i) keep_list[i] = -1;
    *n_keep = nk;
    if (status) *status = st;
    free(s); free(dev_order); free(thr); free(bnd);
    return REF_OK;
}

/* ---- steps a6..a8: group-masked SwiGLU FFN ------------------------------- */
/* For every listed group g and neuron j of it:
 *     a = <gate_j, x>, b = <up_j, x>, h = a / (1 + exp(-a)) * b,
 *     p_g += h * down_j          (down_j = column j of the down projection)
 * and the group's partial p_g is added to the slot of its holder
 * (slot 0 = master, slot i+1 = device i).  group_partials, if given, receives
 * every listed group's p_g on its own ([n_list][n_tok][d]) -- the linearity
 * check and the "importance = L2 norm of the group's activation" diagnostic
 * (Sec. II-B) read it. */
int halo_ref_group_ffn(int d, int F, int S, int dtype, const void* Wpacked, const void* x, int n_tok,
                       const int32_t* list, int n_list, const int32_t* dev_of_group, int n_dev,
                       double* partials /*[n_dev+1][n_tok][d]*/, double* group_partials /*or NULL*/) {
    if (d <= 0 || F <= 0 || S <= 0 || F % S != 0 || n_tok <= 0 || n_list < 0) return REF_ERR_SHAPE;
    int G = F / S;
    for (int i = 0; i < n_list; ++i) if (list[i] < 0 || list[i] >= G) return REF_ERR_ARG;
    size_t slot_elems = (size_t)n_tok * d;
    memset(partials, 0, sizeof(double) * slot_elems * (size_t)(n_dev + 1));
    double* pg = group_partials;
    int own = 0;
    if (!pg) {
        pg = (double*)malloc(sizeof(double) * slot_elems * (size_t)(n_list > 0 ? n_list : 1));
        if (!pg) return REF_ERR_NOMEM;
        own = 1;
    }
#pragma omp parallel for schedule(dynamic)
    for (int i = 0; i < n_list; ++i) {
        int g = list[i];
        double* out = pg + (size_t)i * slot_elems;
        for (size_t e = 0; e < slot_elems; ++e) out[e] = 0.0;
        for (int t = 0; t < n_tok; ++t)
            for (int j = 0; j < S; ++j) {
                double a = 0.0, b = 0.0;
                for (int c = 0; c < d; ++c) {
                    double xc = ref_widen(x, (size_t)t * d + c, dtype);
                    a += ref_widen(Wpacked, packed_index(g, 0, j, c, S, d), dtype) * xc;
                    b += ref_widen(Wpacked, packed_index(g, 1, j, c, S, d), dtype) * xc;
                }
                double h = a / (1.0 + exp(-a)) * b;
                for (int c = 0; c < d; ++c)
                    out[(size_t)t * d + c] += h * ref_widen(Wpacked, packed_index(g, 2, j, c, S, d), dtype);
            }
    }
    for (int i = 0; i < n_list; ++i) { /* fixed order: ascending list position */
        int g = list[i];
        int slot = dev_of_group ? dev_of_group[g] + 1 : 0;
        if (slot < 0 || slot > n_dev) { if (own) free(pg); return REF_ERR_ARG; }
        double* dst = partials + (size_t)slot * slot_elems;
        const double* src = pg + (size_t)i * slot_elems;
        for (size_t e = 0; e < slot_elems; ++e) dst[e] += src[e];
    }
    if (own) free(pg);
    return REF_OK;
}

/* ---- step a9: merge ------------------------------------------------------ */
/* y = P[master] + sum over devices that arrived of P[device]; a lost or late
 * device contributes nothing (Sec. III-B.3). */
int halo_ref_merge(const double* partials, const uint8_t* arrived /*NULL => all*/, int n_dev, int n_tok,
                   int d, double* y) {
    if (n_dev < 0 || n_tok <= 0 || d <= 0) return REF_ERR_SHAPE;
    size_t slot_elems = (size_t)n_tok * d;
    for (size_t e = 0; e < slot_elems; ++e) y[e] = partials[e];
    for (int i = 0; i < n_dev; ++i)
        if (!arrived || arrived[i])
            for (size_t e = 0; e < slot_elems; ++e) y[e] += partials[(size_t)(i + 1) * slot_elems + e];
    return REF_OK;
}

/* ---- glue between the layers of an FFN stack ----------------------------- */
/* Residual stream h (fp32 on the GPU, double here): h' = h + y, and the next
 * block's input is the gain-free RMS-normalised stream stored in the
 * activation dtype: x = cast(h' / sqrt(mean(h'^2) + 1e-5)).  y may be NULL
 * (normalise only: the stack's very first input). */
int halo_ref_glue(int d, int n_tok, int dtype, const double* h, const double* y, double* h_out, void* x_out) {
    if (d <= 0 || n_tok <= 0) return REF_ERR_SHAPE;
    for (int t = 0; t < n_tok; ++t) {
        double ss = 0.0;
        for (int c = 0; c < d; ++c) {
            double v = h[(size_t)t * d + c] + (y ? y[(size_t)t * d + c] : 0.0);
            h_out[(size_t)t * d + c] = v;
            ss += v * v;
        }
        double scale = 1.0 / sqrt(ss / (double)d + 1e-5);
        for (int c = 0; c < d; ++c) {
            double v = h_out[(size_t)t * d + c] * scale;
            if (dtype == REF_F32) ((float*)x_out)[(size_t)t * d + c] = (float)v;
            else ((uint16_t*)x_out)[(size_t)t * d + c] = ref_double_to_bf16(v);
        }
    }
    return REF_OK;
}

/* ---- one whole layer, steps a1..a9 in order ------------------------------ */
/* feat is the predictor input (the previous layer's x: one layer ahead); x is
 * this layer's FFN input.  Only kept groups are computed, so the merge adds
 * every slot that exists.  Outputs y (double) and the selection arrays. */
int halo_ref_layer(int d, int F, int S, int dtype, const void* Wpacked, int rank, int act, const void* W1,
                   const void* W2, int n_dev, const double* loss_rate, const uint32_t* share_weight,
                   int mode, int k_critical, float threshold, uint64_t seed, uint32_t step, uint32_t layer,
                   int force_all, const void* feat, const void* x, int n_tok, float* scores,
                   int32_t* order, int32_t* rank_out, int32_t* dev_of_group, uint8_t* arrived,
                   uint8_t* keep, int32_t* keep_list, int32_t* n_keep, uint32_t* status, double* y) {
    if (F % S != 0) return REF_ERR_SHAPE;
    int G = F / S;
    int rc = halo_ref_predict(d, rank, G, dtype, act, W1, W2, feat, n_tok, n_tok > 1, scores);
    if (rc) return rc;
    rc = halo_ref_select(G, n_dev, loss_rate, share_weight, mode, k_critical, threshold, seed, scores, step,
                         layer, force_all, order, rank_out, dev_of_group, arrived, keep, keep_list, n_keep,
                         status);
    if (rc) return rc;
    double* P = (double*)malloc(sizeof(double) * (size_t)(n_dev + 1) * n_tok * d);
    if (!P) return REF_ERR_NOMEM;
    rc = halo_ref_group_ffn(d, F, S, dtype, Wpacked, x, n_tok, keep_list, *n_keep, dev_of_group, n_dev, P, NULL);
    if (!rc) rc = halo_ref_merge(P, NULL, n_dev, n_tok, d, y);
    free(P);
    return rc;
}

/* ---- Assignment phase, step 1: workload ratios (Algorithms 1 and 2) ------ */
/* Algorithm 1, Computation-Greedy: devices in descending computing power are
 * filled to their memory budget until the model fits; the last device needed
 * takes the remainder, the others get nothing.  r = u / sum(u).  Ties in c
 * keep the lower device index first. */
int halo_ref_comp_greedy(int n, const double* m, const double* c, double Mt, double* r) {
    if (n <= 0 || !(Mt > 0.0)) return REF_ERR_ARG;
    double total = 0.0;
    for (int i = 0; i < n; ++i) { if (!(m[i] >= 0.0) || !(c[i] > 0.0)) return REF_ERR_ARG; total += m[i]; }
    if (total < Mt) return REF_ERR_ARG;   /* the model does not fit at all */
    int* sigma = (int*)malloc(sizeof(int) * (size_t)n);
    if (!sigma) return REF_ERR_NOMEM;
    for (int i = 0; i < n; ++i) sigma[i] = i;
    for (int a = 1; a < n; ++a) {          /* stable insertion sort, descending c */
        int v = sigma[a], b = a - 1;
        while (b >= 0 && c[sigma[b]] < c[v]) { sigma[b + 1] = sigma[b]; --b; }
        sigma[b + 1] = v;
    }
    for (int i = 0; i < n; ++i) r[i] = 0.0;
    double placed = 0.0, sum_u = 0.0;
    for (int j = 0; j < n; ++j) {
        int i = sigma[j];
        double u = m[i];
        if (placed + u >= Mt) { u = Mt - placed; r[i] = u; sum_u += u; break; }
        r[i] = u; sum_u += u; placed += u;
    }
    for (int i = 0; i < n; ++i) r[i] /= sum_u;
    free(sigma);
    return REF_OK;
}

/* Algorithm 2, Min-Max: bisection on the utilisation threshold T (memory per
 * unit of computing power): u_i = min(m_i, T c_i); the smallest T (to eps)
 * whose allocation holds the model; r = u / sum(u). */
int halo_ref_min_max(int n, const double* m, const double* c, double Mt, double eps, double* r) {
    if (n <= 0 || !(Mt > 0.0) || !(eps > 0.0)) return REF_ERR_ARG;
    double total = 0.0, mmax = 0.0, cmin = 0.0;
    for (int i = 0; i < n; ++i) {
        if (!(m[i] >= 0.0) || !(c[i] > 0.0)) return REF_ERR_ARG;
        total += m[i];
        if (i == 0 || m[i] > mmax) mmax = m[i];
        if (i == 0 || c[i] < cmin) cmin = c[i];
    }
    if (total < Mt) return REF_ERR_ARG;
    double left = 0.0, right = mmax / cmin, t_opt = right;
    while (right - left > eps) {
        double mid = (left + right) / 2.0, used = 0.0;
        for (int i = 0; i < n; ++i) used += (m[i] < mid * c[i]) ? m[i] : mid * c[i];
        if (used >= Mt) { t_opt = mid; right = mid; } else left = mid;
    }
    double sum_u = 0.0;
    for (int i = 0; i < n; ++i) { r[i] = (m[i] < t_opt * c[i]) ? m[i] : t_opt * c[i]; sum_u += r[i]; }
    for (int i = 0; i < n; ++i) r[i] /= sum_u;
    return REF_OK;
}

/* ---- MHA neuron groups (Sec. II-A: one head and its output-projection slice) ---- */
/* Packed layout Wattn[H][2][dh][d]: plane 0 = the head's query rows, plane 1 =
 * the head's slice of the output projection stored as rows (row j = column
 * h*dh+j of Wo[d][H*dh]).  Keys and values are NOT part of a group: every
 * device keeps a full KV cache (Sec. III-B.3), so K/V projections are computed
 * for all heads at every token and never dropped.  No positional rotation. */
static size_t mha_index(int h, int plane, int j, int c, int dh, int d) {
    return (((size_t)h * 2 + (size_t)plane) * (size_t)dh + (size_t)j) * (size_t)d + (size_t)c;
}

int halo_ref_pack_mha(int d, int H, int dh, int dtype, const void* Wq /*[H*dh][d]*/, const void* Wo /*[d][H*dh]*/,
                      void* Wpacked) {
    if (d <= 0 || H <= 0 || dh <= 0) return REF_ERR_SHAPE;
    size_t es = ref_elem_size(dtype);
    for (int h = 0; h < H; ++h)
        for (int j = 0; j < dh; ++j)
            for (int c = 0; c < d; ++c) {
                size_t n = (size_t)h * dh + j;
                memcpy((char*)Wpacked + es * mha_index(h, 0, j, c, dh, d), (const char*)Wq + es * (n * d + c), es);
                memcpy((char*)Wpacked + es * mha_index(h, 1, j, c, dh, d),
                       (const char*)Wo + es * ((size_t)c * H * dh + n), es);
            }
    return REF_OK;
}

/* k = Wk x, v = Wv x for every head, stored in the cache dtype at position pos.
 * Caches are [H][Lmax][dh]. */
int halo_ref_mha_kv_append(int d, int H, int dh, int Lmax, int dtype, const void* Wk /*[H*dh][d]*/,
                           const void* Wv, const void* x, int pos, void* K_cache, void* V_cache) {
    if (d <= 0 || H <= 0 || dh <= 0 || pos < 0 || pos >= Lmax) return REF_ERR_SHAPE;
    for (int h = 0; h < H; ++h)
        for (int j = 0; j < dh; ++j) {
            double k = 0.0, v = 0.0;
            size_t row = (size_t)h * dh + j;
            for (int c = 0; c < d; ++c) {
                double xc = ref_widen(x, (size_t)c, dtype);
                k += ref_widen(Wk, row * d + c, dtype) * xc;
                v += ref_widen(Wv, row * d + c, dtype) * xc;
            }
            size_t at = ((size_t)h * Lmax + (size_t)pos) * dh + j;
            if (dtype == REF_F32) { ((float*)K_cache)[at] = (float)k; ((float*)V_cache)[at] = (float)v; }
            else { ((uint16_t*)K_cache)[at] = ref_double_to_bf16(k); ((uint16_t*)V_cache)[at] = ref_double_to_bf16(v); }
        }
    return REF_OK;
}

/* For each listed head h: q = Wq_h x; s_p = <q, K_h[p]> / sqrt(dh) for p = 0..pos;
 * w = softmax(s); o = sum_p w_p V_h[p]; p_h = sum_j o_j * Wo_h[j] (width d), added to
 * the slot of the head's holder.  head_partials, if given, gets every p_h. */
int halo_ref_group_mha(int d, int H, int dh, int Lmax, int dtype, const void* Wpacked, const void* x,
                       const void* K_cache, const void* V_cache, int pos, const int32_t* list, int n_list,
                       const int32_t* dev_of_group, int n_dev, double* partials /*[n_dev+1][d]*/,
                       double* head_partials /*[n_list][d] or NULL*/) {
    if (d <= 0 || H <= 0 || dh <= 0 || pos < 0 || pos >= Lmax || n_list < 0) return REF_ERR_SHAPE;
    for (int i = 0; i < n_list; ++i) if (list[i] < 0 || list[i] >= H) return REF_ERR_ARG;
    memset(partials, 0, sizeof(double) * (size_t)(n_dev + 1) * d);
    double* q = (double*)malloc(sizeof(double) * (size_t)dh);
    double* o = (double*)malloc(sizeof(double) * (size_t)dh);
    double* w = (double*)malloc(sizeof(double) * (size_t)(pos + 1));
    double* ph = (double*)malloc(sizeof(double) * (size_t)d);
    if (!q || !o || !w || !ph) { free(q); free(o); free(w); free(ph); return REF_ERR_NOMEM; }
    int rc = REF_OK;
    for (int i = 0; i < n_list && rc == REF_OK; ++i) {
        int h = list[i];
        for (int j = 0; j < dh; ++j) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += ref_widen(Wpacked, mha_index(h, 0, j, c, dh, d), dtype) * ref_widen(x, (size_t)c, dtype);
            q[j] = acc;
        }
        double smax = -INFINITY;
        for (int p = 0; p <= pos; ++p) {
            double acc = 0.0;
            for (int j = 0; j < dh; ++j) acc += q[j] * ref_widen(K_cache, ((size_t)h * Lmax + p) * dh + j, dtype);
            w[p] = acc / sqrt((double)dh);
            if (w[p] > smax) smax = w[p];
        }
        double denom = 0.0;
        for (int p = 0; p <= pos; ++p) { w[p] = exp(w[p] - smax); denom += w[p]; }
        for (int j = 0; j < dh; ++j) {
            double acc = 0.0;
            for (int p = 0; p <= pos; ++p) acc += w[p] * ref_widen(V_cache, ((size_t)h * Lmax + p) * dh + j, dtype);
            o[j] = acc / denom;
        }
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int j = 0; j < dh; ++j) acc += o[j] * ref_widen(Wpacked, mha_index(h, 1, j, c, dh, d), dtype);
            ph[c] = acc;
        }
        int slot = dev_of_group ? dev_of_group[h] + 1 : 0;
        if (slot < 0 || slot > n_dev) { rc = REF_ERR_ARG; break; }
        for (int c = 0; c < d; ++c) partials[(size_t)slot * d + c] += ph[c];
        if (head_partials) memcpy(head_partials + (size_t)i * d, ph, sizeof(double) * (size_t)d);
    }
    free(q); free(o); free(w); free(ph);
    return rc;
}

/* ---------------------------------------------------------------------------------------------
 * LM-head neuron groups (Sec. II-A: the LM head only has an up-projection and is a collection of
 * neuron groups; Sec. III-B.3: its results travel reliably, so nothing is ever lost).
 * A group is `group_size` consecutive vocabulary rows (the last one may be shorter).  For every
 * listed group and every token: logits[t][v] = <W[v], x_t>.  Entries of unlisted groups are left
 * as the caller set them: the groups' outputs are concatenated, never summed.
 * ------------------------------------------------------------------------------------------- */
int halo_ref_group_lm_head(int d, int vocab, int group_size, int dtype, const void* W /*[vocab][d]*/,
                           const void* x /*[n_tok][d]*/, int n_tok, const int32_t* list, int n_list,
                           double* logits /*[n_tok][vocab]*/) {
    if (d <= 0 || vocab <= 0 || group_size <= 0 || n_tok <= 0 || n_list < 0) return REF_ERR_SHAPE;
    int n_groups = (vocab + group_size - 1) / group_size;
    for (int i = 0; i < n_list; ++i) if (list[i] < 0 || list[i] >= n_groups) return REF_ERR_ARG;
    for (int i = 0; i < n_list; ++i) {
        int g = list[i];
        int v0 = g * group_size, v1 = v0 + group_size < vocab ? v0 + group_size : vocab;
        for (int t = 0; t < n_tok; ++t)
            for (int v = v0; v < v1; ++v) {
                double acc = 0.0;
                for (int c = 0; c < d; ++c)
                    acc += ref_widen(W, (size_t)v * d + c, dtype) * ref_widen(x, (size_t)t * d + c, dtype);
                logits[(size_t)t * vocab + v] = acc;
            }
    }
    return REF_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Late devices (Sec. III-B.3: the master merges what is available after a timeout, so a partial
 * that comes later than the timeout counts as lost; Eq. 1: device i needs tau * W_i / c_i for the
 * W_i units it holds, plus the synchronisation time T_c).
 *   late[i] = 1  iff  tau * units[i] / compute[i] + t_comm > timeout
 * A device that holds nothing sends nothing and is never late.
 * ------------------------------------------------------------------------------------------- */
int halo_ref_late_devices(int n_dev, const int32_t* units, const double* compute, double tau,
                          double t_comm, double timeout, uint8_t* late) {
    if (n_dev <= 0 || !units || !compute || !late || tau < 0.0 || t_comm < 0.0 || timeout < 0.0) return REF_ERR_ARG;
    for (int i = 0; i < n_dev; ++i) {
        if (units[i] < 0 || !(compute[i] > 0.0)) return REF_ERR_ARG;
        double t = tau * (double)units[i] / compute[i] + t_comm;
        late[i] = (units[i] > 0 && t > timeout) ? 1 : 0;
    }
    return REF_OK;
}

/* ---------------------------------------------------------------------------------------------
 * int4 group-quantised weights.  The paper evaluates models "quantized to 4-bit integer
 * precision" (Sec. IV-A) and picks the neuron-group size "for compatibility with quantization"
 * (Sec. II-A) but gives no format; the reading taken here: symmetric, one scale per block of 128
 * consecutive elements of a stored (packed) row,
 *   s = up5(bf16(amax / 7))   (fp32 division, round-to-nearest-even to bf16, then UP to the next bf16 number
 *                              with at most 5 significant bits; amax = max |w| of the block)
 *   q = clamp(rint(w / s), -8, 7)   (fp32 division, round-half-even; s == 0 -> q = 0)
 * stored as nibble q + 8; element 2i in the low half of byte i, element 2i+1 in the high half.
 * The decisions are taken in fp32 on both sides (here and on the GPU), so codes and scales
 * compare bit for bit.  Dequantised value: (nibble - 8) * s.  With 5 significant bits in s and at most 3 (or a
 * single one, for -8) in the code, the product has at most 8: every dequantised value is a bf16 number, so a
 * bf16 operand path (tensor cores) carries the weights without any rounding.
 * ------------------------------------------------------------------------------------------- */
#define REF_QBLOCK 128

static float ref_bf16_bits_to_float(uint16_t b) {
    uint32_t bits = (uint32_t)b << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

int halo_ref_quantize_i4(int d, long long n_rows, int dtype, const void* W, uint8_t* Q /*[n_rows][d/2]*/,
                         uint16_t* scales /*[n_rows][d/128]*/) {
    if (d <= 0 || d % REF_QBLOCK != 0 || n_rows < 0 || !W || !Q || !scales) return REF_ERR_SHAPE;
    int nb = d / REF_QBLOCK;
    for (long long r = 0; r < n_rows; ++r)
        for (int b = 0; b < nb; ++b) {
            size_t base = (size_t)r * d + (size_t)b * REF_QBLOCK;
            float amax = 0.0f;
            for (int e = 0; e < REF_QBLOCK; ++e) {
                float w = (float)ref_widen(W, base + e, dtype);     /* exact: the stored types fit fp32 */
                float a = fabsf(w);
                if (a > amax) amax = a;
            }
            float s32 = amax / 7.0f;
            uint16_t sb = ref_double_to_bf16((double)s32);
            if (sb & 7u) sb = (uint16_t)((sb | 7u) + 1u);        /* up to 5 significant bits (may carry into the exponent) */
            float s = ref_bf16_bits_to_float(sb);
            scales[(size_t)r * nb + b] = sb;
            for (int e = 0; e < REF_QBLOCK; e += 2) {
                int q[2];
                for (int k = 0; k < 2; ++k) {
                    float w = (float)ref_widen(W, base + e + k, dtype);
                    float t = s > 0.0f ? rintf(w / s) : 0.0f;
                    if (t < -8.0f) t = -8.0f;
                    if (t > 7.0f) t = 7.0f;
                    q[k] = (int)t;
                }
                Q[(base + e) / 2] = (uint8_t)((q[0] + 8) | ((q[1] + 8) << 4));
            }
        }
    return REF_OK;
}

int halo_ref_dequantize_i4(int d, long long n_rows, const uint8_t* Q, const uint16_t* scales, float* W32) {
    if (d <= 0 || d % REF_QBLOCK != 0 || n_rows < 0 || !Q || !scales || !W32) return REF_ERR_SHAPE;
    int nb = d / REF_QBLOCK;
    for (long long r = 0; r < n_rows; ++r)
        for (int c = 0; c < d; ++c) {
            size_t i = (size_t)r * d + c;
            int nib = (Q[i / 2] >> ((c & 1) * 4)) & 15;
            float s = ref_bf16_bits_to_float(scales[(size_t)r * nb + c / REF_QBLOCK]);
            W32[i] = (float)(nib - 8) * s;     /* at most 8 significant bits: exact, and a bf16 number */
        }
    return REF_OK;
}
