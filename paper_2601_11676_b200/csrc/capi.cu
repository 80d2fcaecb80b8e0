// extern "C" surface of libhalo: argument checks, the host-side Assignment phase, and the stack runner.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"
#include "prompt_stack.cuh"
#include "stack_persistent.cuh"

using namespace halo;

namespace {

bool valid_dtype(int t) { return t == HALO_F32 || t == HALO_BF16; }
size_t elem_size(halo_dtype t) { return t == HALO_F32 ? 4 : 2; }

halo_status check_ffn_shape(const halo_ffn_shape* s) {
    if (!s) return HALO_ERR_ARG;
    if (!valid_dtype(s->wdtype)) return HALO_ERR_DTYPE;
    if (s->d_model <= 0 || s->d_ffn <= 0 || s->group_size <= 0) return HALO_ERR_SHAPE;
    if (s->d_model % 8 != 0 || s->d_ffn % s->group_size != 0) return HALO_ERR_SHAPE;
    if (s->d_ffn / s->group_size > HALO_MAX_GROUPS) return HALO_ERR_SHAPE;
    const int per_chunk = s->wdtype == HALO_F32 ? 4 : 8;
    if (s->d_model / per_chunk > 1024) return HALO_ERR_SHAPE;  // decode kernel: at most 4 chunks per thread
    return HALO_OK;
}

unsigned long long loss_threshold(double rho) {
    if (!(rho > 0.0)) return 0ull;
    if (rho >= 1.0) return 1ull << 32;
    double t = std::floor(rho * 4294967296.0 + 0.5);
    if (t > 4294967296.0) t = 4294967296.0;
    return static_cast<unsigned long long>(t);
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

namespace halo {
// argument rules of the predictor, shared by every entry point that takes a halo_pred_shape
halo_status check_pred_shape(const halo_pred_shape* s) {
    if (!s) return HALO_ERR_ARG;
    if (!valid_dtype(s->wdtype)) return HALO_ERR_DTYPE;
    if (s->act != HALO_ACT_RELU && s->act != HALO_ACT_NONE) return HALO_ERR_ARG;
    if (s->d_in <= 0 || s->rank <= 0 || s->n_groups <= 0) return HALO_ERR_SHAPE;
    if (s->d_in % 8 != 0 || s->rank % 8 != 0) return HALO_ERR_SHAPE;
    if (s->d_in > 12288 || s->rank > 8192 || s->n_groups > HALO_MAX_GROUPS) return HALO_ERR_SHAPE;
    return HALO_OK;
}

namespace {
struct OptionName { const char* name; OptionId id; int lo, hi; };
const OptionName kOptionNames[] = {
    {"cross_stages", OPT_CROSS_STAGES, 0, 16},
    {"l2_ahead", OPT_L2_AHEAD, 0, 32},
    {"max_steps_per_launch", OPT_MAX_STEPS_PER_LAUNCH, 0, 1 << 30},
    {"prefill_two_launches", OPT_PREFILL_TWO_LAUNCHES, 0, 1},
    {"prefill_kcuts", OPT_PREFILL_KCUTS, 1, 16},
    {"prefill_kratio_percent", OPT_PREFILL_KRATIO_PERCENT, 30, 100},
    {"mha_three_launches", OPT_MHA_THREE_LAUNCHES, 0, 1},
    {"i4_no_ring", OPT_I4_NO_RING, 0, 3},
    {"prompt_kcuts", OPT_PROMPT_KCUTS, 1, 16},
    {"prompt_l2_ahead", OPT_PROMPT_L2_AHEAD, 0, 32},
    {"tmem_ring", OPT_TMEM_RING, 0, 1},
};
std::atomic<int> g_options[OPT_COUNT] = {{-1}, {-1}, {-1}, {-1}, {-1}, {-1}, {-1}, {-1}, {-1}, {-1}, {-1}};
}  // namespace

int option_value(OptionId id) { return g_options[id].load(std::memory_order_relaxed); }
}  // namespace halo

extern "C" halo_status halo_set_option(const char* name, int value) {
    if (!name) return HALO_ERR_ARG;
    for (const auto& o : kOptionNames) {
        if (std::strcmp(name, o.name) != 0) continue;
        if (value != -1 && (value < o.lo || value > o.hi)) return HALO_ERR_ARG;
        g_options[o.id].store(value, std::memory_order_relaxed);
        return HALO_OK;
    }
    return HALO_ERR_ARG;
}

// ---------------------------------------------------------------------------------------------------

extern "C" const char* halo_status_string(halo_status s) {
    switch (s) {
        case HALO_OK: return "ok";
        case HALO_ERR_ARG: return "bad argument";
        case HALO_ERR_SHAPE: return "unsupported shape";
        case HALO_ERR_ALIGN: return "pointer not 16-byte aligned";
        case HALO_ERR_DTYPE: return "unsupported dtype";
        case HALO_ERR_CUDA: return "CUDA call failed";
        case HALO_ERR_NOMEM: return "out of memory";
        case HALO_ERR_UNIMPLEMENTED: return "not implemented";
        case HALO_ERR_WORKSPACE: return "workspace missing or too small";
        default: return "unknown status";
    }
}

extern "C" halo_status halo_status_message(uint32_t v, char* msg, int msg_len) {
    if (!msg || msg_len <= 0) return HALO_ERR_ARG;
    std::snprintf(msg, static_cast<size_t>(msg_len), "%s%s%s%s",
                  v == 0 ? "clean" : "",
                  (v & HALO_DEV_NONFINITE_SCORE) ? "non-finite score;" : "",
                  (v & HALO_DEV_BAD_INDEX) ? "index out of range;" : "",
                  (v & HALO_DEV_TIMEOUT) ? "device wait timed out;" : "");
    return HALO_OK;
}

// ---- Assignment phase (Algorithm 3) ------------------------------------------------------------------

extern "C" halo_status halo_plan_create(halo_plan** out, int n_groups, int n_dev, const double* loss_rate,
                                        const uint32_t* share_weight, halo_sel_mode mode, int k_critical,
                                        float threshold, uint64_t seed) {
    if (!out) return HALO_ERR_ARG;
    *out = nullptr;
    if (n_groups <= 0 || n_groups > HALO_MAX_GROUPS || n_dev < 0 || n_dev > HALO_MAX_DEVICES) return HALO_ERR_SHAPE;
    if (n_dev > 0 && (!loss_rate || !share_weight)) return HALO_ERR_ARG;
    if (mode != HALO_SEL_TOPK && mode != HALO_SEL_THRESHOLD) return HALO_ERR_ARG;
    if (mode == HALO_SEL_TOPK && (k_critical < 0 || k_critical > n_groups)) return HALO_ERR_ARG;
    if (mode == HALO_SEL_THRESHOLD && std::isnan(threshold)) return HALO_ERR_ARG;
    unsigned long long total = 0;
    for (int i = 0; i < n_dev; ++i) {
        if (!(loss_rate[i] >= 0.0 && loss_rate[i] <= 1.0)) return HALO_ERR_ARG;
        total += share_weight[i];
    }
    if (n_dev > 0 && total == 0) return HALO_ERR_ARG;
    halo_plan* p = new (std::nothrow) halo_plan();
    if (!p) return HALO_ERR_NOMEM;
    std::memset(p, 0, sizeof(*p));
    p->n_groups = n_groups;
    p->n_dev = n_dev;
    PlanDev& dv = p->dev;
    dv.n_dev = n_dev;
    dv.mode = mode;
    dv.k_critical = mode == HALO_SEL_TOPK ? k_critical : 0;
    dv.threshold = threshold;
    dv.seed_lo = static_cast<uint32_t>(seed & 0xffffffffull);
    dv.seed_hi = static_cast<uint32_t>(seed >> 32);
    for (int i = 0; i < n_dev; ++i) {
        p->loss_rate[i] = loss_rate[i];
        p->share_weight[i] = share_weight[i];
        dv.loss_thresh[i] = loss_threshold(loss_rate[i]);
        dv.dev_order[i] = i;
    }
    // q = argsort(rho ascending), ties keep the lower device index first
    std::stable_sort(dv.dev_order, dv.dev_order + n_dev,
                     [&](int a, int b) { return p->loss_rate[a] < p->loss_rate[b]; });
    unsigned long long cum = 0;
    for (int j = 0; j < n_dev; ++j) {
        cum += p->share_weight[dv.dev_order[j]];
        dv.cum_weight[j] = cum;
    }
    *out = p;
    return HALO_OK;
}

extern "C" halo_status halo_plan_destroy(halo_plan* plan) {
    delete plan;
    return HALO_OK;
}

extern "C" halo_status halo_plan_describe(const halo_plan* plan, int M, int32_t* dev_order, uint64_t* loss_thresh,
                                          int32_t* boundaries) {
    if (!plan || M < 0) return HALO_ERR_ARG;
    const PlanDev& dv = plan->dev;
    for (int i = 0; i < plan->n_dev; ++i) {
        if (dev_order) dev_order[i] = dv.dev_order[i];
        if (loss_thresh) loss_thresh[i] = dv.loss_thresh[i];
    }
    if (boundaries) {
        boundaries[0] = 0;
        if (plan->n_dev > 0) {
            const unsigned long long total = dv.cum_weight[plan->n_dev - 1];
            for (int j = 1; j < plan->n_dev; ++j)
                boundaries[j] = static_cast<int32_t>(
                    (2ull * static_cast<unsigned long long>(M) * dv.cum_weight[j - 1] + total) / (2ull * total));
            boundaries[plan->n_dev] = M;
        }
    }
    return HALO_OK;
}

// ---- Assignment phase, workload ratios (Algorithms 1 and 2) -----------------------------------------------

namespace {
bool valid_devices(int n, const double* m, const double* c, double Mt, double* total) {
    if (n <= 0 || n > HALO_MAX_DEVICES || !m || !c || !(Mt > 0.0)) return false;
    double t = 0.0;
    for (int i = 0; i < n; ++i) {
        if (!(m[i] >= 0.0) || !(c[i] > 0.0)) return false;
        t += m[i];
    }
    *total = t;
    return t >= Mt;   // the budgets must hold the model
}
}  // namespace

extern "C" halo_status halo_schedule_comp_greedy(int n_dev, const double* mem_budget, const double* compute,
                                                 double model_mem, double* ratio) {
    double total;
    if (!ratio || !valid_devices(n_dev, mem_budget, compute, model_mem, &total)) return HALO_ERR_ARG;
    int order[HALO_MAX_DEVICES];
    for (int i = 0; i < n_dev; ++i) order[i] = i;
    std::stable_sort(order, order + n_dev, [&](int a, int b) { return compute[a] > compute[b]; });
    double used[HALO_MAX_DEVICES] = {};
    double remaining = model_mem, sum = 0.0;
    for (int j = 0; j < n_dev && remaining > 0.0; ++j) {
        const int i = order[j];
        const double take = std::min(mem_budget[i], remaining);   // the last device needed takes the remainder
        used[i] = take;
        sum += take;
        remaining -= take;
    }
    for (int i = 0; i < n_dev; ++i) ratio[i] = used[i] / sum;
    return HALO_OK;
}

extern "C" halo_status halo_schedule_min_max(int n_dev, const double* mem_budget, const double* compute,
                                             double model_mem, double eps, double* ratio) {
    double total;
    if (!ratio || !(eps > 0.0) || !valid_devices(n_dev, mem_budget, compute, model_mem, &total)) return HALO_ERR_ARG;
    // The problem behind Algorithm 2: the smallest common finishing time T such that the devices, each loaded up
    // to min(m_i, T * c_i), hold the model.  held(T) = sum_i min(m_i, T * c_i) is continuous, piecewise linear and
    // non-decreasing with one breakpoint per device at T = m_i / c_i (the device is full from there on), so it is
    // solved exactly piece by piece instead of by bisection: with the devices sorted by breakpoint, and the first k
    // of them full, held(T) = (memory of the full ones) + T * (computing power of the rest).
    int by_break[HALO_MAX_DEVICES];
    for (int i = 0; i < n_dev; ++i) by_break[i] = i;
    std::stable_sort(by_break, by_break + n_dev, [&](int a, int b) {
        return mem_budget[a] * compute[b] < mem_budget[b] * compute[a];   // m_a / c_a < m_b / c_b, c > 0
    });
    double open_power = 0.0;
    for (int i = 0; i < n_dev; ++i) open_power += compute[i];
    double full_mem = 0.0, T = 0.0;
    for (int k = 0; k < n_dev; ++k) {
        const int i = by_break[k];
        const double t_break = mem_budget[i] / compute[i];
        T = (model_mem - full_mem) / open_power;       // where this piece reaches the model's demand
        if (T <= t_break) break;                       // inside the piece: found
        T = t_break;                                   // all budgets together hold the model exactly at the last one
        full_mem += mem_budget[i];
        open_power -= compute[i];
    }
    double sum = 0.0;
    for (int i = 0; i < n_dev; ++i) sum += std::min(mem_budget[i], T * compute[i]);
    if (!(sum > 0.0)) return HALO_ERR_ARG;
    for (int i = 0; i < n_dev; ++i) ratio[i] = std::min(mem_budget[i], T * compute[i]) / sum;
    return HALO_OK;
}

extern "C" halo_status halo_ratios_to_share_weights(int n_dev, const double* ratio, uint32_t* share_weight) {
    if (n_dev <= 0 || n_dev > HALO_MAX_DEVICES || !ratio || !share_weight) return HALO_ERR_ARG;
    for (int i = 0; i < n_dev; ++i) {
        if (!(ratio[i] >= 0.0) || ratio[i] > 65535.0) return HALO_ERR_ARG;
        share_weight[i] = static_cast<uint32_t>(std::floor(ratio[i] * 65536.0 + 0.5));
    }
    return HALO_OK;
}

extern "C" halo_status halo_late_devices(int n_dev, const int32_t* units, const double* compute, double tau,
                                         double t_comm, double timeout, uint8_t* late) {
    if (n_dev <= 0 || n_dev > HALO_MAX_DEVICES || !units || !compute || !late) return HALO_ERR_ARG;
    if (!(tau >= 0.0) || !(t_comm >= 0.0) || !(timeout >= 0.0)) return HALO_ERR_ARG;
    for (int i = 0; i < n_dev; ++i)
        if (units[i] < 0 || !(compute[i] > 0.0)) return HALO_ERR_ARG;
    for (int i = 0; i < n_dev; ++i) {
        const double busy = tau * static_cast<double>(units[i]) / compute[i] + t_comm;   // Eq. 1, one block
        late[i] = (units[i] > 0 && busy > timeout) ? 1 : 0;
    }
    return HALO_OK;
}

// ---- a1 ---------------------------------------------------------------------------------------------

extern "C" size_t halo_predict_workspace_bytes(const halo_pred_shape* shape, int n_tok) {
    if (check_pred_shape(shape) != HALO_OK || n_tok <= 0) return 0;
    return sizeof(float) * static_cast<size_t>(n_tok) * (static_cast<size_t>(shape->rank) + shape->n_groups);
}

extern "C" halo_status halo_predict_groups(const halo_pred_shape* shape, const void* W1, const void* W2,
                                           const void* feat, int n_tok, int mean_pool, float* scores,
                                           void* workspace, size_t workspace_bytes, uint32_t* dev_status,
                                           void* stream) {
    halo_status rc = check_pred_shape(shape);
    if (rc != HALO_OK) return rc;
    if (!W1 || !W2 || !feat || !scores) return HALO_ERR_ARG;
    if (n_tok <= 0) return HALO_ERR_SHAPE;
    if (!aligned16(W1) || !aligned16(W2) || !aligned16(feat) || !aligned16(workspace)) return HALO_ERR_ALIGN;
    if (!workspace || workspace_bytes < halo_predict_workspace_bytes(shape, n_tok)) return HALO_ERR_WORKSPACE;
    return launch_predict(*shape, W1, W2, feat, n_tok, mean_pool, scores, static_cast<float*>(workspace), dev_status,
                          static_cast<cudaStream_t>(stream));
}

// ---- a2..a5 -----------------------------------------------------------------------------------------

extern "C" halo_status halo_select_groups(const halo_plan* plan, const float* scores, uint32_t step, uint32_t layer,
                                          int force_all, int32_t* order, int32_t* dev_of_group, uint8_t* arrived,
                                          uint8_t* keep, int32_t* keep_list, int32_t* n_keep, uint32_t* dev_status,
                                          void* stream) {
    if (!plan || !scores || !keep_list || !n_keep) return HALO_ERR_ARG;
    return launch_select(plan->dev, plan->n_groups, scores, step, layer, force_all, order, dev_of_group, arrived,
                         keep, keep_list, n_keep, dev_status, static_cast<cudaStream_t>(stream));
}

// ---- a6..a8 -----------------------------------------------------------------------------------------

extern "C" size_t halo_group_ffn_workspace_bytes(const halo_ffn_shape* shape, int n_tok, int n_dev) {
    (void)n_dev;
    if (check_ffn_shape(shape) != HALO_OK || n_tok <= 0) return 0;
    return prefill_supported(*shape, n_tok) ? prefill_workspace_bytes(*shape, n_tok) : 0;
}

namespace {
// many tokens + bf16 + supported shape -> tensor-core contraction; otherwise the bandwidth-bound kernels
halo_status dispatch_group_ffn(const halo_ffn_shape& sh, const void* W, const void* x, int n_tok,
                               const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group, int n_dev,
                               float* partials, void* workspace, uint32_t* dev_status, cudaStream_t st,
                               bool* collapsed = nullptr) {
    if (prefill_supported(sh, n_tok) && workspace) {
        // a caller that passes `collapsed` only wants the merged sum: two slots (master / devices) are enough
        const bool collapse = collapsed != nullptr && n_dev > 1;
        if (collapsed) *collapsed = collapse;
        const size_t bytes = sizeof(float) * static_cast<size_t>(collapse ? 2 : n_dev + 1) * n_tok * sh.d_model;
        if (cudaMemsetAsync(partials, 0, bytes, st) != cudaSuccess) return HALO_ERR_CUDA;
        return launch_group_ffn_prefill(sh, W, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, collapse ? 1 : 0, partials,
                                        workspace, dev_status, st);
    }
    if (collapsed) *collapsed = false;
    return launch_group_ffn_decode(sh, W, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials, dev_status, st);
}
}  // namespace

extern "C" halo_status halo_group_ffn(const halo_ffn_shape* shape, const void* W_packed, const void* x, int n_tok,
                                      const int32_t* keep_list, const int32_t* n_keep, const int32_t* dev_of_group,
                                      int n_dev, float* partials, void* workspace, size_t workspace_bytes,
                                      uint32_t* dev_status, void* stream) {
    halo_status rc = check_ffn_shape(shape);
    if (rc != HALO_OK) return rc;
    if (!W_packed || !x || !keep_list || !n_keep || !partials) return HALO_ERR_ARG;
    if (n_tok <= 0) return HALO_ERR_SHAPE;
    if (n_dev < 0 || n_dev > HALO_MAX_DEVICES || (!dev_of_group && n_dev != 0)) return HALO_ERR_ARG;
    if (!aligned16(W_packed) || !aligned16(x) || !aligned16(partials)) return HALO_ERR_ALIGN;
    const size_t need = halo_group_ffn_workspace_bytes(shape, n_tok, n_dev);
    if (need > 0 && (!workspace || workspace_bytes < need)) return HALO_ERR_WORKSPACE;
    if (need > 0 && !aligned16(workspace)) return HALO_ERR_ALIGN;
    return dispatch_group_ffn(*shape, W_packed, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials,
                              need > 0 ? workspace : nullptr, dev_status, static_cast<cudaStream_t>(stream));
}

// ---- int4 weights, many tokens: kept groups back to bf16 in the caller's workspace, then the tensor-core FFN ----

extern "C" size_t halo_group_ffn_i4_workspace_bytes(const halo_ffn_shape* shape, int n_tok) {
    if (!shape || n_tok <= 0) return 0;
    halo_ffn_shape sh = *shape;
    sh.wdtype = HALO_BF16;                                   // activations; the tensor cores' operand type
    if (check_ffn_shape(&sh) != HALO_OK || sh.d_model % 128 != 0 || !prefill_supported(sh, n_tok)) return 0;
    return align_up(static_cast<size_t>(sh.d_ffn) * 3 * sh.d_model * 2, 1024) + prefill_workspace_bytes(sh, n_tok);
}

extern "C" halo_status halo_group_ffn_i4_prompt(const halo_ffn_shape* shape, const void* Q, const void* scales, const void* x,
                                                int n_tok, const int32_t* keep_list, const int32_t* n_keep,
                                                const int32_t* dev_of_group, int n_dev, float* partials, void* workspace,
                                                size_t workspace_bytes, uint32_t* dev_status, void* stream) {
    if (!shape) return HALO_ERR_ARG;
    const size_t need = halo_group_ffn_i4_workspace_bytes(shape, n_tok);
    if (need == 0)    // few tokens or a shape the tensor-core FFN does not take: the decode form, token by token
        return halo_group_ffn_i4(shape, Q, scales, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials, dev_status,
                                 stream);
    if (!Q || !scales || !x || !keep_list || !n_keep || !partials) return HALO_ERR_ARG;
    if (n_dev < 0 || n_dev > HALO_MAX_DEVICES || (!dev_of_group && n_dev != 0)) return HALO_ERR_ARG;
    if (!workspace || workspace_bytes < need) return HALO_ERR_WORKSPACE;
    if (!aligned16(Q) || !aligned16(scales) || !aligned16(x) || !aligned16(partials) || !aligned16(workspace))
        return HALO_ERR_ALIGN;
    halo_ffn_shape sh = *shape;
    sh.wdtype = HALO_BF16;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    const size_t block_bytes = align_up(static_cast<size_t>(sh.d_ffn) * 3 * sh.d_model * 2, 1024);
    halo_status rc = launch_dequantize_i4(sh, Q, scales, keep_list, n_keep, ws, dev_status, st);
    if (rc != HALO_OK) return rc;
    return dispatch_group_ffn(sh, ws, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials, ws + block_bytes,
                              dev_status, st);
}

// ---- a9 and helpers -----------------------------------------------------------------------------------

extern "C" halo_status halo_merge_partials(const float* partials, const uint8_t* arrived, int n_dev, int n_tok,
                                           int d_model, float* y, void* stream) {
    if (!partials || !y) return HALO_ERR_ARG;
    if (n_dev < 0 || n_dev > HALO_MAX_DEVICES || n_tok <= 0 || d_model <= 0) return HALO_ERR_SHAPE;
    return launch_merge(partials, arrived, n_dev, n_tok, d_model, y, static_cast<cudaStream_t>(stream));
}

extern "C" halo_status halo_pack_weights(const halo_ffn_shape* shape, const void* Wgate, const void* Wup,
                                         const void* Wdown, void* W_packed, void* stream) {
    halo_status rc = check_ffn_shape(shape);
    if (rc != HALO_OK) return rc;
    if (!Wgate || !Wup || !Wdown || !W_packed) return HALO_ERR_ARG;
    return launch_pack(*shape, Wgate, Wup, Wdown, W_packed, static_cast<cudaStream_t>(stream));
}

extern "C" halo_status halo_glue(int d_model, int n_tok, halo_dtype xdtype, const float* h, const float* y,
                                 float* h_out, void* x_out, void* stream) {
    if (!h || !h_out || !x_out) return HALO_ERR_ARG;
    if (!valid_dtype(xdtype)) return HALO_ERR_DTYPE;
    if (d_model <= 0 || d_model > 12288 || n_tok <= 0) return HALO_ERR_SHAPE;
    return launch_glue(d_model, n_tok, xdtype, h, y, h_out, x_out, static_cast<cudaStream_t>(stream));
}

// ---- one block, a1..a9 ------------------------------------------------------------------------------------

extern "C" size_t halo_layer_workspace_bytes(const halo_ffn_shape* ffn, const halo_pred_shape* pred, int n_tok, int n_dev) {
    if (check_ffn_shape(ffn) != HALO_OK || check_pred_shape(pred) != HALO_OK || n_tok <= 0 || n_dev < 0) return 0;
    const size_t G = static_cast<size_t>(ffn->d_ffn / ffn->group_size);
    size_t b = align_up(halo_predict_workspace_bytes(pred, n_tok), 256);
    b += align_up(halo_group_ffn_workspace_bytes(ffn, n_tok, n_dev), 256);
    b += align_up(sizeof(float) * static_cast<size_t>(n_dev + 1) * n_tok * ffn->d_model, 256);   // partials
    b += align_up(sizeof(int32_t) * G, 256) + 256;                                                // keep_list, n_keep
    return b;
}

extern "C" halo_status halo_layer_fused(const halo_ffn_shape* ffn, const halo_pred_shape* pred, const halo_plan* plan,
                                        const void* W_packed, const void* W1, const void* W2, const void* feat,
                                        const void* x, int n_tok, uint32_t step, uint32_t layer, int force_all,
                                        float* scores, int32_t* dev_of_group, uint8_t* arrived, uint8_t* keep,
                                        float* y, void* workspace, size_t workspace_bytes, uint32_t* dev_status,
                                        void* stream) {
    halo_status rc = check_ffn_shape(ffn);
    if (rc != HALO_OK) return rc;
    rc = check_pred_shape(pred);
    if (rc != HALO_OK) return rc;
    if (!plan || !W_packed || !W1 || !W2 || !feat || !x || !scores || !dev_of_group || !arrived || !y) return HALO_ERR_ARG;
    if (n_tok <= 0) return HALO_ERR_SHAPE;
    const int G = ffn->d_ffn / ffn->group_size, n_dev = plan->n_dev;
    if (pred->n_groups != G || plan->n_groups != G || pred->d_in != ffn->d_model || pred->wdtype != ffn->wdtype)
        return HALO_ERR_SHAPE;
    if (!aligned16(W_packed) || !aligned16(W1) || !aligned16(W2) || !aligned16(feat) || !aligned16(x) || !aligned16(y) ||
        !aligned16(workspace))
        return HALO_ERR_ALIGN;
    if (!workspace || workspace_bytes < halo_layer_workspace_bytes(ffn, pred, n_tok, n_dev)) return HALO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    float* pred_ws = reinterpret_cast<float*>(ws);
    ws += align_up(halo_predict_workspace_bytes(pred, n_tok), 256);
    void* ffn_ws = ws;
    const size_t ffn_ws_bytes = halo_group_ffn_workspace_bytes(ffn, n_tok, n_dev);
    ws += align_up(ffn_ws_bytes, 256);
    float* partials = reinterpret_cast<float*>(ws);
    ws += align_up(sizeof(float) * static_cast<size_t>(n_dev + 1) * n_tok * ffn->d_model, 256);
    int32_t* keep_list = reinterpret_cast<int32_t*>(ws);
    ws += align_up(sizeof(int32_t) * static_cast<size_t>(G), 256);
    int32_t* n_keep = reinterpret_cast<int32_t*>(ws);
    // a1 (mean over tokens for a prompt), a2..a5, a6..a8 over the kept groups, a9
    rc = launch_predict(*pred, W1, W2, feat, n_tok, 1, scores, pred_ws, dev_status, st);
    if (rc != HALO_OK) return rc;
    rc = launch_select(plan->dev, G, scores, step, layer, force_all, nullptr, dev_of_group, arrived, keep, keep_list,
                       n_keep, dev_status, st);
    if (rc != HALO_OK) return rc;
    rc = dispatch_group_ffn(*ffn, W_packed, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials,
                            ffn_ws_bytes ? ffn_ws : nullptr, dev_status, st);
    if (rc != HALO_OK) return rc;
    return launch_merge(partials, arrived, n_dev, n_tok, ffn->d_model, y, st);
}

extern "C" halo_status halo_read_status(const uint32_t* dev_status_host_copy, char* msg, int msg_len) {
    if (!dev_status_host_copy) return HALO_ERR_ARG;
    return halo_status_message(*dev_status_host_copy, msg, msg_len);
}

// ---- FFN stack ----------------------------------------------------------------------------------------

struct halo_stack {
    halo_ffn_shape ffn;
    halo_pred_shape pred;
    int n_layers, n_tok, G, n_dev;
    halo_plan plan;
    std::vector<const void*> W, W1, W2;
    std::vector<const void*> i4_scales;   // non-empty: W holds int4 codes (halo_quantize_weights_i4)
    // int4 stacks made for prompts: the kept groups of a block are turned back into bf16 (the tensor cores' operand
    // type) in one of two scratch blocks, alternating by block, and the tensor-core FFN reads those
    void* i4_deq[2] = {nullptr, nullptr};
    bool i4_prompt = false;
    void* slab;
    // carved from the slab
    float* h;
    void* x[2];
    float* pred_ws;
    float* scores;
    float* zero_scores;
    int32_t* dev_of_group;
    uint8_t* arrived;
    int32_t* keep_list;
    int32_t* n_keep;
    float* partials;
    uint32_t* status;
    float* stage_in;
    float* stage_out;
    int stage_steps;
    long long last_launches;
    // persistent single-kernel path
    int mode;                      // 0 = automatic, 1 = one launch per step of the path
    bool persistent_ok;
    const void** d_W;              // device pointer tables
    const void** d_Wsc;            // ... of the int4 scales (int4 stacks)
    const void** d_W1;
    const void** d_W2;
    float* p_partials;             // [3][2][d]
    float* p_z;
    halo::PersistSel* p_sel;       // [3]
    unsigned* p_sync;              // [64]
    __nv_bfloat16* p_xhist;        // [2][d]
    float* p_det_rows;             // [2][kMaxGrid][d]
    void* ffn_ws;                  // H buffer of the tensor-core path (multi-token stacks), or null
    bool ffn_ws_clean = false;     // its control words are known to be zero
    // multi-token stacks: predictor + selection of block l+1 run on a side stream while block l's FFN runs
    cudaStream_t side;
    cudaEvent_t ev_x, ev_sel;
    float* set_scores[2];          // two selection sets, by parity of the block
    int32_t* set_dev[2];
    uint8_t* set_arr[2];
    int32_t* set_kl[2];
    int32_t* set_nk[2];
    unsigned long long* trace;     // caller-owned, optional
    int trace_blocks;
    int cross_stages, l2_ahead;    // tuning of the persistent kernel
    int tmem_ring;                 // second ring level in tensor memory (d_model 2048 / 4096)
    int max_steps_per_launch;      // 0 = derived from the counters' range
    // multi-token stacks, persistent prompt kernel (one launch per prompt)
    bool prompt_ok = false;
    void* pp_slab = nullptr;
    CUtensorMap* pp_maps = nullptr;        // device
    __nv_bfloat16* pp_H[2] = {nullptr, nullptr};
    float* pp_zpart = nullptr;
    halo::PersistSel* pp_sel = nullptr;    // [L]
    unsigned* pp_ctl = nullptr;
    size_t pp_ctl_bytes = 0;
    int pp_tiles_x = 0, pp_n_pn = 0, pp_z_cuts = 0;
    unsigned long long* pp_trace = nullptr;   // caller-owned, optional
};

namespace {
halo_status stack_create_impl(halo_stack** out, const halo_ffn_shape* ffn, const halo_pred_shape* pred, int n_layers,
                              int n_tok, const halo_plan* plan, const void* const* W_packed, const void* const* i4_scales,
                              const void* const* W1, const void* const* W2);
}  // namespace

extern "C" halo_status halo_stack_create(halo_stack** out, const halo_ffn_shape* ffn, const halo_pred_shape* pred,
                                         int n_layers, int n_tok, const halo_plan* plan, const void* const* W_packed,
                                         const void* const* W1, const void* const* W2) {
    return stack_create_impl(out, ffn, pred, n_layers, n_tok, plan, W_packed, nullptr, W1, W2);
}

extern "C" halo_status halo_stack_create_i4(halo_stack** out, const halo_ffn_shape* ffn, const halo_pred_shape* pred,
                                            int n_layers, int n_tok, const halo_plan* plan, const void* const* Q,
                                            const void* const* scales, const void* const* W1, const void* const* W2) {
    if (!scales || !ffn) return HALO_ERR_ARG;
    if (ffn->wdtype != HALO_BF16) return HALO_ERR_DTYPE;          // activations and predictor stay bf16
    if (ffn->d_model % 128 != 0) return HALO_ERR_SHAPE;
    for (int l = 0; l < n_layers; ++l)
        if (!scales[l] || !aligned16(scales[l])) return scales[l] ? HALO_ERR_ALIGN : HALO_ERR_ARG;
    return stack_create_impl(out, ffn, pred, n_layers, n_tok, plan, Q, scales, W1, W2);
}

namespace {
halo_status stack_create_impl(halo_stack** out, const halo_ffn_shape* ffn, const halo_pred_shape* pred, int n_layers,
                              int n_tok, const halo_plan* plan, const void* const* W_packed, const void* const* i4_scales,
                              const void* const* W1, const void* const* W2) {
    if (!out) return HALO_ERR_ARG;
    *out = nullptr;
    halo_status rc = check_ffn_shape(ffn);
    if (rc != HALO_OK) return rc;
    rc = check_pred_shape(pred);
    if (rc != HALO_OK) return rc;
    if (!plan || !W_packed || !W1 || !W2) return HALO_ERR_ARG;
    if (n_layers <= 0 || n_tok <= 0) return HALO_ERR_SHAPE;
    const int G = ffn->d_ffn / ffn->group_size;
    if (pred->d_in != ffn->d_model || pred->n_groups != G || plan->n_groups != G || pred->wdtype != ffn->wdtype)
        return HALO_ERR_SHAPE;
    for (int l = 0; l < n_layers; ++l) {
        if (!W_packed[l] || !aligned16(W_packed[l])) return W_packed[l] ? HALO_ERR_ALIGN : HALO_ERR_ARG;
        if (l > 0 && (!W1[l] || !W2[l])) return HALO_ERR_ARG;
        if (l > 0 && (!aligned16(W1[l]) || !aligned16(W2[l]))) return HALO_ERR_ALIGN;
    }
    halo_stack* s = new (std::nothrow) halo_stack();
    if (!s) return HALO_ERR_NOMEM;
    s->ffn = *ffn;
    s->pred = *pred;
    s->n_layers = n_layers;
    s->n_tok = n_tok;
    s->G = G;
    s->n_dev = plan->n_dev;
    s->plan = *plan;
    s->W.assign(W_packed, W_packed + n_layers);
    s->W1.assign(W1, W1 + n_layers);
    s->W2.assign(W2, W2 + n_layers);
    if (i4_scales) s->i4_scales.assign(i4_scales, i4_scales + n_layers);
    s->last_launches = 0;

    const size_t d = ffn->d_model, es = elem_size(ffn->wdtype), T = n_tok;
    const size_t step_elems = T * d;
    s->stage_steps = static_cast<int>(std::max<size_t>(1, std::min<size_t>(64, (16u << 20) / (step_elems * 4))));
    size_t off = 0;
    auto carve = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t o_h = carve(step_elems * 4);
    const size_t o_x0 = carve(step_elems * es), o_x1 = carve(step_elems * es);
    const size_t o_pws = carve(sizeof(float) * T * (static_cast<size_t>(pred->rank) + G));
    const size_t o_sc = carve(sizeof(float) * G), o_zs = carve(sizeof(float) * G);
    const size_t o_dg = carve(sizeof(int32_t) * G), o_ar = carve(HALO_MAX_DEVICES);
    const size_t o_kl = carve(sizeof(int32_t) * G), o_nk = carve(sizeof(int32_t));
    const size_t o_pa = carve(sizeof(float) * (s->n_dev + 1) * step_elems);
    const size_t o_st = carve(sizeof(uint32_t));
    const size_t o_si = carve(sizeof(float) * s->stage_steps * step_elems);
    const size_t o_so = carve(sizeof(float) * s->stage_steps * step_elems);
    const size_t o_tw = carve(sizeof(void*) * n_layers), o_tw1 = carve(sizeof(void*) * n_layers);
    const size_t o_tw2 = carve(sizeof(void*) * n_layers);
    const size_t o_tws = carve(sizeof(void*) * n_layers);
    const size_t o_pp = carve(sizeof(float) * 3 * 2 * d);
    const size_t o_pz = carve(sizeof(float) * 2 * pred->rank);
    const size_t o_ps = carve(sizeof(PersistSel) * 3);
    const size_t o_py = carve(sizeof(unsigned) * 64);
    constexpr size_t kMaxGrid = 192;   // thread blocks of the persistent kernel (one per SM)
    const size_t o_xh = carve(2 * d * 2);
    const size_t o_dr = carve(!i4_scales && persistent_supported(*ffn, n_tok, G) ? sizeof(float) * 2 * kMaxGrid * d : 16);
    const size_t ws_bytes = prefill_supported(*ffn, n_tok) ? prefill_workspace_bytes(*ffn, n_tok) : 0;
    const size_t o_ws = carve(ws_bytes ? ws_bytes : 16);
    const size_t o_sc2 = carve(sizeof(float) * G), o_dg2 = carve(sizeof(int32_t) * G);
    const size_t o_ar2 = carve(HALO_MAX_DEVICES), o_kl2 = carve(sizeof(int32_t) * G), o_nk2 = carve(sizeof(int32_t));
    if (cudaMalloc(&s->slab, off) != cudaSuccess) { delete s; return HALO_ERR_NOMEM; }
    if (cudaMemset(s->slab, 0, off) != cudaSuccess) { cudaFree(s->slab); delete s; return HALO_ERR_CUDA; }
    char* base = static_cast<char*>(s->slab);
    s->h = reinterpret_cast<float*>(base + o_h);
    s->x[0] = base + o_x0;
    s->x[1] = base + o_x1;
    s->pred_ws = reinterpret_cast<float*>(base + o_pws);
    s->scores = reinterpret_cast<float*>(base + o_sc);
    s->zero_scores = reinterpret_cast<float*>(base + o_zs);
    s->dev_of_group = reinterpret_cast<int32_t*>(base + o_dg);
    s->arrived = reinterpret_cast<uint8_t*>(base + o_ar);
    s->keep_list = reinterpret_cast<int32_t*>(base + o_kl);
    s->n_keep = reinterpret_cast<int32_t*>(base + o_nk);
    s->partials = reinterpret_cast<float*>(base + o_pa);
    s->status = reinterpret_cast<uint32_t*>(base + o_st);
    s->stage_in = reinterpret_cast<float*>(base + o_si);
    s->stage_out = reinterpret_cast<float*>(base + o_so);
    s->d_W = reinterpret_cast<const void**>(base + o_tw);
    s->d_W1 = reinterpret_cast<const void**>(base + o_tw1);
    s->d_W2 = reinterpret_cast<const void**>(base + o_tw2);
    s->d_Wsc = reinterpret_cast<const void**>(base + o_tws);
    s->p_partials = reinterpret_cast<float*>(base + o_pp);
    s->p_z = reinterpret_cast<float*>(base + o_pz);
    s->p_sel = reinterpret_cast<PersistSel*>(base + o_ps);
    s->p_sync = reinterpret_cast<unsigned*>(base + o_py);
    s->p_xhist = reinterpret_cast<__nv_bfloat16*>(base + o_xh);
    s->p_det_rows = reinterpret_cast<float*>(base + o_dr);
    s->ffn_ws = ws_bytes ? static_cast<void*>(base + o_ws) : nullptr;
    s->set_scores[0] = s->scores; s->set_scores[1] = reinterpret_cast<float*>(base + o_sc2);
    s->set_dev[0] = s->dev_of_group; s->set_dev[1] = reinterpret_cast<int32_t*>(base + o_dg2);
    s->set_arr[0] = s->arrived; s->set_arr[1] = reinterpret_cast<uint8_t*>(base + o_ar2);
    s->set_kl[0] = s->keep_list; s->set_kl[1] = reinterpret_cast<int32_t*>(base + o_kl2);
    s->set_nk[0] = s->n_keep; s->set_nk[1] = reinterpret_cast<int32_t*>(base + o_nk2);
    s->side = nullptr; s->ev_x = nullptr; s->ev_sel = nullptr;
    if (n_tok > 1 || i4_scales || !persistent_supported(*ffn, n_tok, G)) {   // every path that is not the persistent kernel
        // best effort: without them the blocks simply run one after the other on the caller's stream
        // highest priority: the short predictor/selection kernels of the next block must get SMs as they free up,
        // ahead of the waiting CTAs of the long FFN launch (which pulls its tiles from a queue and loses nothing)
        int prio_lo = 0, prio_hi = 0;
        if (cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi) != cudaSuccess) prio_hi = 0;
        if (cudaStreamCreateWithPriority(&s->side, cudaStreamNonBlocking, prio_hi) != cudaSuccess) s->side = nullptr;
        if (s->side && (cudaEventCreateWithFlags(&s->ev_x, cudaEventDisableTiming) != cudaSuccess ||
                        cudaEventCreateWithFlags(&s->ev_sel, cudaEventDisableTiming) != cudaSuccess)) {
            cudaStreamDestroy(s->side);
            s->side = nullptr;
        }
    }
    s->mode = 0;
    s->trace = nullptr;
    s->trace_blocks = 0;
    // Off unless asked for.  Measured: the form is correct and keeps 9 stages (432 KB) in flight per SM, but a stage
    // costs the consumers about as long as HBM takes to deliver it (8.2 us against 9.4 us per 470 KB on the 1.1B
    // shape), so a deeper backlog cannot be worked off inside a block, while batches claimed 9 stages ahead make the
    // thread blocks finish a block further apart (the grid barrier waits 6 us instead of 2).  Net: 20 % slower there.
    s->tmem_ring = option_value(OPT_TMEM_RING) == 1;
    // with the tensor-memory level the producer may run as far ahead as the ring lets it
    s->cross_stages = s->tmem_ring ? 16 : 2;
    s->l2_ahead = 0;
    if (option_value(OPT_CROSS_STAGES) >= 0) s->cross_stages = option_value(OPT_CROSS_STAGES);
    s->max_steps_per_launch = std::max(0, option_value(OPT_MAX_STEPS_PER_LAUNCH));
    if (option_value(OPT_L2_AHEAD) >= 0) s->l2_ahead = option_value(OPT_L2_AHEAD);
    s->persistent_ok = i4_scales ? persistent_supported_i4(*ffn, n_tok, G) : persistent_supported(*ffn, n_tok, G);
    if (i4_scales && ws_bytes) {
        // best effort: without the scratch blocks a prompt runs through the decode form, token by token
        const size_t block_bytes = static_cast<size_t>(ffn->d_ffn) * 3 * d * 2;
        if (cudaMalloc(&s->i4_deq[0], block_bytes) == cudaSuccess && cudaMalloc(&s->i4_deq[1], block_bytes) == cudaSuccess) {
            s->i4_prompt = true;
        } else {
            (void)cudaGetLastError();
            if (s->i4_deq[0]) cudaFree(s->i4_deq[0]);
            s->i4_deq[0] = s->i4_deq[1] = nullptr;
        }
    }
    {
        // pointer tables, and the first block's selection: reliable block, all scores equal -> the priority
        // order is the group order, everything is kept (Sec. III-B.3, first layer)
        std::vector<PersistSel> sel0(1);
        std::memset(&sel0[0], 0, sizeof(PersistSel));
        const PlanDev& dv = plan->dev;
        int k = dv.mode == HALO_SEL_THRESHOLD ? ((0.0f >= dv.threshold) ? G : 0) : dv.k_critical;
        if (dv.n_dev == 0) k = G;
        const int M = G - k;
        std::vector<int32_t> bnd(dv.n_dev + 1, 0);
        halo_plan_describe(plan, M, nullptr, nullptr, bnd.data());
        sel0[0].n_keep = G;
        for (int g = 0; g < HALO_MAX_GROUPS; ++g) { sel0[0].keep_list[g] = g < G ? g : -1; sel0[0].dev_of_group[g] = -1; }
        for (int g = k; g < G; ++g)
            for (int j = 0; j < dv.n_dev; ++j)
                if (bnd[j] <= g - k && g - k < bnd[j + 1]) { sel0[0].dev_of_group[g] = dv.dev_order[j]; break; }
        for (int i = 0; i < dv.n_dev; ++i) sel0[0].arrived[i] = 1;
        bool ok = cudaMemcpy(s->p_sel + 2, sel0.data(), sizeof(PersistSel), cudaMemcpyHostToDevice) == cudaSuccess;
        ok = ok && cudaMemcpy(s->d_W, s->W.data(), sizeof(void*) * n_layers, cudaMemcpyHostToDevice) == cudaSuccess;
        ok = ok && cudaMemcpy(s->d_W1, s->W1.data(), sizeof(void*) * n_layers, cudaMemcpyHostToDevice) == cudaSuccess;
        ok = ok && cudaMemcpy(s->d_W2, s->W2.data(), sizeof(void*) * n_layers, cudaMemcpyHostToDevice) == cudaSuccess;
        if (i4_scales)
            ok = ok && cudaMemcpy(s->d_Wsc, s->i4_scales.data(), sizeof(void*) * n_layers, cudaMemcpyHostToDevice) == cudaSuccess;
        if (!ok) { cudaFree(s->slab); delete s; return HALO_ERR_CUDA; }
        if (n_tok > 1 && !i4_scales && prompt_stack_supported(*ffn, *pred, n_layers, n_tok)) {
            // persistent prompt kernel: tensor maps (encoded once, here), two H buffers, control words, one selection
            // record per block.  Any failure in here only means that prompts run one launch per step of the path.
            const int S = ffn->group_size, NS = std::min(S, 128), dm = ffn->d_model;
            const int tiles_x = (n_tok + 255) / 256, n_pn = (pred->rank + 255) / 256;
            const size_t n_maps = 3 * static_cast<size_t>(n_layers) + 4;
            const size_t h_bytes = align_up(static_cast<size_t>(n_tok) * ffn->d_ffn * 2, 1024);
            const size_t z_bytes = align_up(sizeof(float) * 2 * tiles_x * 8 * static_cast<size_t>(n_pn) * 256, 256);
            const size_t sel_bytes = align_up(sizeof(PersistSel) * n_layers, 256);
            s->pp_ctl_bytes = align_up(prompt_stack_ctl_bytes(n_layers, tiles_x, G), 256);
            const size_t map_bytes = align_up(sizeof(CUtensorMap) * n_maps, 256);
            const size_t total = map_bytes + 2 * h_bytes + z_bytes + sel_bytes + s->pp_ctl_bytes;
            if (cudaMalloc(&s->pp_slab, total) == cudaSuccess) {
                char* pb = static_cast<char*>(s->pp_slab);
                s->pp_maps = reinterpret_cast<CUtensorMap*>(pb); pb += map_bytes;
                s->pp_H[0] = reinterpret_cast<__nv_bfloat16*>(pb); pb += h_bytes;
                s->pp_H[1] = reinterpret_cast<__nv_bfloat16*>(pb); pb += h_bytes;
                s->pp_zpart = reinterpret_cast<float*>(pb); pb += z_bytes;
                s->pp_sel = reinterpret_cast<PersistSel*>(pb); pb += sel_bytes;
                s->pp_ctl = reinterpret_cast<unsigned*>(pb);
                std::vector<CUtensorMap> maps(n_maps);
                const uint64_t w_rows = static_cast<uint64_t>(G) * 3 * S;
                bool good = cudaMemset(s->pp_slab, 0, total) == cudaSuccess;
                for (int l = 0; l < n_layers && good; ++l) {
                    good = make_bf16_map(&maps[3 * l + 0], s->W[l], w_rows, dm, dm, 64, NS) &&
                           make_bf16_map(&maps[3 * l + 1], s->W[l], w_rows, dm, dm, 64, 64);
                    // block 0 has no predictor: its slot repeats the weight map and is never used
                    good = good && (l == 0 ? make_bf16_map(&maps[3 * l + 2], s->W[l], w_rows, dm, dm, 64, 128)
                                           : make_bf16_map(&maps[3 * l + 2], s->W1[l], pred->rank, dm, dm, 64, 128));
                }
                for (int b = 0; b < 2 && good; ++b)
                    good = make_bf16_map(&maps[3 * n_layers + b], s->x[b], n_tok, dm, dm, 64, 128) &&
                           make_bf16_map(&maps[3 * n_layers + 2 + b], s->pp_H[b], n_tok, ffn->d_ffn, ffn->d_ffn, 64, 128);
                good = good && cudaMemcpy(s->pp_maps, maps.data(), sizeof(CUtensorMap) * n_maps, cudaMemcpyHostToDevice) == cudaSuccess;
                good = good && cudaMemcpy(s->pp_sel, sel0.data(), sizeof(PersistSel), cudaMemcpyHostToDevice) == cudaSuccess;
                if (good) {
                    int dev = 0, n_sm = kSmCount;
                    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
                    s->pp_tiles_x = tiles_x;
                    s->pp_n_pn = n_pn;
                    // K runs per output tile of the down projection: short enough that the tiles a block ends with
                    // do not hold up the next block's first items for long
                    s->pp_z_cuts = std::max(1, std::min(8, (n_sm * 4 / 3) / std::max(1, tiles_x * (dm / 256))));
                    if (option_value(OPT_PROMPT_KCUTS) > 0) s->pp_z_cuts = option_value(OPT_PROMPT_KCUTS);
                    s->prompt_ok = true;
                } else {
                    cudaFree(s->pp_slab);
                    s->pp_slab = nullptr;
                    (void)cudaGetLastError();
                }
            } else {
                (void)cudaGetLastError();
            }
        }
    }
    *out = s;
    return HALO_OK;
}
}  // namespace

extern "C" halo_status halo_stack_destroy(halo_stack* s) {
    if (!s) return HALO_OK;
    if (s->side) {
        cudaStreamSynchronize(s->side);
        cudaEventDestroy(s->ev_x);
        cudaEventDestroy(s->ev_sel);
        cudaStreamDestroy(s->side);
    }
    cudaFree(s->slab);
    if (s->pp_slab) cudaFree(s->pp_slab);
    if (s->i4_deq[0]) cudaFree(s->i4_deq[0]);
    if (s->i4_deq[1]) cudaFree(s->i4_deq[1]);
    delete s;
    return HALO_OK;
}

extern "C" halo_status halo_stack_decode(halo_stack* s, const float* h0, int steps, uint32_t step0, float* h_out,
                                         const halo_taps* taps, void* stream) {
    if (!s || !h0 || !h_out) return HALO_ERR_ARG;
    if (steps <= 0) return HALO_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t d = s->ffn.d_model, T = s->n_tok, es = elem_size(s->ffn.wdtype);
    const size_t step_elems = T * d;
    const int L = s->n_layers, G = s->G, n_dev = s->n_dev;
    long long launches = 0;
    halo_status rc;
    // (the int4 form of the kernel has neither the serialised-predictor arm nor the fixed-order sums)
    const bool i4_stack = !s->i4_scales.empty();
    if (s->persistent_ok && !(s->mode & HALO_STACK_PER_STEP_LAUNCHES) &&
        !(i4_stack && (s->mode & (HALO_STACK_PRED_SERIAL | HALO_STACK_DETERMINISTIC)))) {
        // whole run in one cooperative launch
        if (cudaMemsetAsync(s->p_partials, 0, sizeof(float) * 3 * 2 * d, st) != cudaSuccess ||
            cudaMemsetAsync(s->p_sync, 0, sizeof(unsigned) * 64, st) != cudaSuccess)
            return HALO_ERR_CUDA;
        PersistParams P;
        std::memset(&P, 0, sizeof(P));
        P.L = L; P.steps = steps; P.d = static_cast<int>(d); P.S = s->ffn.group_size; P.G = G; P.r = s->pred.rank;
        P.act = s->pred.act; P.step0 = step0;
        P.W = reinterpret_cast<const __nv_bfloat16* const*>(s->d_W);
        P.W1 = reinterpret_cast<const __nv_bfloat16* const*>(s->d_W1);
        P.W2 = reinterpret_cast<const __nv_bfloat16* const*>(s->d_W2);
        P.i4 = i4_stack ? 1 : 0;
        P.Wsc = reinterpret_cast<const __nv_bfloat16* const*>(s->d_Wsc);
        P.h0 = h0; P.h_out = h_out; P.partials = s->p_partials; P.z = s->p_z; P.sel = s->p_sel; P.sync = s->p_sync;
        P.status = s->status;
        P.plan = s->plan.dev;
        P.trace = s->trace; P.trace_blocks = s->trace_blocks;
        P.cross_stages = s->cross_stages; P.l2_ahead = s->l2_ahead; P.tmem_ring = s->tmem_ring;
        if (s->mode & HALO_STACK_LOAD_SERIAL) { P.cross_stages = 0; P.l2_ahead = 0; }
        P.pred_serial = (s->mode & HALO_STACK_PRED_SERIAL) ? 1 : 0;
        P.deterministic = (s->mode & HALO_STACK_DETERMINISTIC) ? 1 : 0;
        P.x_hist = s->p_xhist; P.det_rows = s->p_det_rows;
        if (taps) {
            P.tap_x = static_cast<__nv_bfloat16*>(taps->x); P.tap_scores = taps->scores;
            P.tap_dev_of_group = taps->dev_of_group; P.tap_arrived = taps->arrived; P.tap_keep_list = taps->keep_list;
            P.tap_n_keep = taps->n_keep; P.tap_y = taps->y;
            // records of the first block of every step: its selection is fixed (everything kept, scores zero)
            for (int sidx = 0; sidx < steps; ++sidx) {
                const size_t rec = static_cast<size_t>(sidx) * L;
                const PersistSel* s0 = s->p_sel + 2;
                auto copy = [&](void* dst, const void* src, size_t bytes) {
                    return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
                };
                bool ok = true;
                if (taps->scores) ok = ok && cudaMemsetAsync(taps->scores + rec * G, 0, sizeof(float) * G, st) == cudaSuccess;
                if (taps->dev_of_group) ok = ok && copy(taps->dev_of_group + rec * G, s0->dev_of_group, sizeof(int32_t) * G);
                if (taps->arrived && n_dev > 0) ok = ok && copy(taps->arrived + rec * n_dev, s0->arrived, n_dev);
                if (taps->keep_list) ok = ok && copy(taps->keep_list + rec * G, s0->keep_list, sizeof(int32_t) * G);
                if (taps->n_keep) ok = ok && copy(taps->n_keep + rec, &s0->n_keep, sizeof(int32_t));
                if (!ok) return HALO_ERR_CUDA;
            }
        }
        // The kernel's 32-bit counters (barrier arrivals, hidden rows) grow with steps x blocks: very long runs are
        // cut into several launches.
        const long long per_step = static_cast<long long>(L) * std::max(s->pred.rank, 256);
        int max_steps = static_cast<int>(std::max<long long>(1, (1ll << 30) / per_step));
        if (s->max_steps_per_launch > 0) max_steps = std::min(max_steps, s->max_steps_per_launch);
        long long n_launches = 0;
        bool fell_back = false;
        for (int done = 0; done < steps; done += max_steps) {
            const int n = std::min(max_steps, steps - done);
            if (done > 0 && (cudaMemsetAsync(s->p_partials, 0, sizeof(float) * 3 * 2 * d, st) != cudaSuccess ||
                             cudaMemsetAsync(s->p_sync, 0, sizeof(unsigned) * 64, st) != cudaSuccess))
                return HALO_ERR_CUDA;
            P.steps = n;
            P.step0 = step0 + static_cast<uint32_t>(done);
            P.h0 = h0 + static_cast<size_t>(done) * step_elems;
            P.h_out = h_out + static_cast<size_t>(done) * step_elems;
            if (taps) {
                const size_t rec = static_cast<size_t>(done) * L;
                P.tap_x = taps->x ? static_cast<__nv_bfloat16*>(taps->x) + rec * step_elems : nullptr;
                P.tap_scores = taps->scores ? taps->scores + rec * G : nullptr;
                P.tap_dev_of_group = taps->dev_of_group ? taps->dev_of_group + rec * G : nullptr;
                P.tap_arrived = taps->arrived ? taps->arrived + rec * n_dev : nullptr;
                P.tap_keep_list = taps->keep_list ? taps->keep_list + rec * G : nullptr;
                P.tap_n_keep = taps->n_keep ? taps->n_keep + rec : nullptr;
                P.tap_y = taps->y ? taps->y + rec * step_elems : nullptr;
            }
            rc = launch_stack_persistent(P, st);
            if (rc == HALO_ERR_UNIMPLEMENTED && done == 0) { fell_back = true; break; }   // not resident: loop path below
            if (rc == HALO_ERR_UNIMPLEMENTED) {
                // a later piece of a split run was refused (the SMs are no longer all ours): the remaining steps
                // run on the one-launch-per-step path, so the call still completes
                halo_taps rest{};
                if (taps) {
                    const size_t rec = static_cast<size_t>(done) * L;
                    rest.x = taps->x ? static_cast<char*>(taps->x) + rec * step_elems * es : nullptr;
                    rest.scores = taps->scores ? taps->scores + rec * G : nullptr;
                    rest.dev_of_group = taps->dev_of_group ? taps->dev_of_group + rec * G : nullptr;
                    rest.arrived = taps->arrived ? taps->arrived + rec * n_dev : nullptr;
                    rest.keep_list = taps->keep_list ? taps->keep_list + rec * G : nullptr;
                    rest.n_keep = taps->n_keep ? taps->n_keep + rec : nullptr;
                    rest.y = taps->y ? taps->y + rec * step_elems : nullptr;
                }
                const int saved_mode = s->mode;
                s->mode = 1;
                rc = halo_stack_decode(s, h0 + static_cast<size_t>(done) * step_elems, steps - done,
                                       step0 + static_cast<uint32_t>(done), h_out + static_cast<size_t>(done) * step_elems,
                                       taps ? &rest : nullptr, stream);
                s->mode = saved_mode;
                if (rc != HALO_OK) return rc;
                s->last_launches += n_launches;
                return HALO_OK;
            }
            if (rc != HALO_OK) return rc;
            ++n_launches;
        }
        if (!fell_back) {
            s->last_launches = n_launches;
            return HALO_OK;
        }
    }
#define HALO_TRY(call) do { rc = (call); if (rc != HALO_OK) return rc; } while (0)
#define HALO_COPY(dst, src, bytes)                                                                    \
    do { if (cudaMemcpyAsync((dst), (src), (bytes), cudaMemcpyDeviceToDevice, st) != cudaSuccess)     \
             return HALO_ERR_CUDA; } while (0)
    if (T > 1 && s->prompt_ok && (s->mode & HALO_STACK_PROMPT_ONE_LAUNCH) && !(s->mode & HALO_STACK_PER_STEP_LAUNCHES) &&
        (!taps || !taps->y)) {
        // Prompt path, one launch per prompt: every block of the stack inside one persistent kernel.  The residual
        // stream is updated in place in the caller's h_out.
        PromptParams P;
        std::memset(&P, 0, sizeof(P));
        P.L = L; P.T = static_cast<int>(T); P.d = static_cast<int>(d); P.S = s->ffn.group_size; P.G = G; P.r = s->pred.rank;
        P.act = s->pred.act;
        P.tiles_x = s->pp_tiles_x; P.n_tn = static_cast<int>(d) / 256; P.n_pn = s->pp_n_pn; P.z_cuts = s->pp_z_cuts;
        P.subs = s->ffn.group_size / std::min(s->ffn.group_size, 128);
        P.ctl_stride = prompt_stack_ctl_stride(P.tiles_x, G);
        P.r_pad = P.n_pn * 256;
        P.l2_ahead = std::max(0, option_value(OPT_PROMPT_L2_AHEAD));
        P.maps = s->pp_maps;
        P.W2 = reinterpret_cast<const __nv_bfloat16* const*>(s->d_W2);
        P.x[0] = static_cast<__nv_bfloat16*>(s->x[0]); P.x[1] = static_cast<__nv_bfloat16*>(s->x[1]);
        P.H[0] = s->pp_H[0]; P.H[1] = s->pp_H[1];
        P.h_cols = s->ffn.d_ffn;
        P.zpart = s->pp_zpart; P.sel = s->pp_sel; P.ctl = s->pp_ctl; P.status = s->status;
        P.plan = s->plan.dev;
        P.trace = s->pp_trace;
        {   // what is left of the caller's buffer behind the per-block words holds the tile records
            int width = halo_stack_trace_width(s);
            const long long words = static_cast<long long>(s->trace_blocks) * width * 8 - static_cast<long long>(width) * 16;
            P.trace_items = (s->pp_trace && words > 0) ? static_cast<int>(words / (3ll * width)) : 0;
        }
        for (int sidx = 0; sidx < steps; ++sidx) {
            float* h_run = h_out + sidx * step_elems;
            if (h_run != h0 + sidx * step_elems &&
                cudaMemcpyAsync(h_run, h0 + sidx * step_elems, sizeof(float) * step_elems, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
                return HALO_ERR_CUDA;
            if (cudaMemsetAsync(s->pp_ctl, 0, s->pp_ctl_bytes, st) != cudaSuccess) return HALO_ERR_CUDA;
            P.h = h_run;
            P.step = step0 + static_cast<uint32_t>(sidx);
            if (taps) {
                const size_t rec = static_cast<size_t>(sidx) * L;
                P.tap_x = taps->x ? static_cast<__nv_bfloat16*>(taps->x) + rec * step_elems : nullptr;
                P.tap_scores = taps->scores ? taps->scores + rec * G : nullptr;
                P.tap_dev_of_group = taps->dev_of_group ? taps->dev_of_group + rec * G : nullptr;
                P.tap_arrived = taps->arrived ? taps->arrived + rec * n_dev : nullptr;
                P.tap_keep_list = taps->keep_list ? taps->keep_list + rec * G : nullptr;
                P.tap_n_keep = taps->n_keep ? taps->n_keep + rec : nullptr;
                // records of the first block: its selection is fixed (everything kept, scores zero)
                const PersistSel* s0 = s->pp_sel;
                auto copy = [&](void* dst, const void* src, size_t bytes) {
                    return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
                };
                bool ok = true;
                if (taps->scores) ok = ok && cudaMemsetAsync(P.tap_scores, 0, sizeof(float) * G, st) == cudaSuccess;
                if (taps->dev_of_group) ok = ok && copy(P.tap_dev_of_group, s0->dev_of_group, sizeof(int32_t) * G);
                if (taps->arrived && n_dev > 0) ok = ok && copy(P.tap_arrived, s0->arrived, n_dev);
                if (taps->keep_list) ok = ok && copy(P.tap_keep_list, s0->keep_list, sizeof(int32_t) * G);
                if (taps->n_keep) ok = ok && copy(P.tap_n_keep, &s0->n_keep, sizeof(int32_t));
                if (!ok) return HALO_ERR_CUDA;
            }
            rc = launch_prompt_stack(P, st);
            if (rc != HALO_OK) return rc;
            ++launches;
        }
        s->last_launches = launches;
        return HALO_OK;
    }
    // Decode stacks that cannot take the persistent kernel (int4 weights, other widths) get the same overlap from the side
    // stream, unless the one-launch-per-step arm was asked for.
    const bool overlapped_decode = T == 1 && !(s->mode & HALO_STACK_PER_STEP_LAUNCHES);
    if ((T > 1 || overlapped_decode) && s->side) {
        // Prompt path, one launch per step of the path.  The scores of block l+1 need only x_l (one layer ahead, Sec. III-B.2), which exists before
        // block l's FFN starts: predictor + selection of block l+1 go to the side stream and overlap with the
        // tensor-core GEMMs of block l (the paper's Pred || Comp overlap).  Two selection sets alternate by block.
        cudaStream_t side = s->side;
#define HALO_CU(call) do { if ((call) != cudaSuccess) return HALO_ERR_CUDA; } while (0)
        for (int sidx = 0; sidx < steps; ++sidx) {
            const uint32_t step = step0 + static_cast<uint32_t>(sidx);
            HALO_TRY(launch_glue(static_cast<int>(d), static_cast<int>(T), s->ffn.wdtype, h0 + sidx * step_elems,
                                 nullptr, s->h, s->x[0], st));
            HALO_TRY(launch_select(s->plan.dev, G, s->zero_scores, step, 0u, 1, nullptr, s->set_dev[0], s->set_arr[0],
                                   nullptr, s->set_kl[0], s->set_nk[0], s->status, st));
            launches += 2;
            if (s->i4_prompt) {
                HALO_TRY(launch_dequantize_i4(s->ffn, s->W[0], s->i4_scales[0], s->set_kl[0], s->set_nk[0], s->i4_deq[0],
                                              s->status, st));
                ++launches;
            }
            HALO_CU(cudaEventRecord(s->ev_x, st));   // x_0 is ready (and set[1] is no longer in use)
            for (int l = 0; l < L; ++l) {
                const int cur = l & 1, nxt = (l + 1) & 1;
                void* x_cur = s->x[cur];
                void* x_next = s->x[nxt];
                if (l + 1 < L) {
                    HALO_CU(cudaStreamWaitEvent(side, s->ev_x, 0));
                    if (T == 1) {
                        HALO_TRY(launch_predict_hidden(s->pred, s->W1[l + 1], x_cur, 1, s->pred_ws, side));
                        HALO_TRY(launch_score_select(s->pred, s->W2[l + 1], s->pred_ws, s->plan.dev, step,
                                                     static_cast<uint32_t>(l + 1), 0, s->set_scores[nxt], nullptr,
                                                     s->set_dev[nxt], s->set_arr[nxt], nullptr, s->set_kl[nxt],
                                                     s->set_nk[nxt], s->status, side));
                        launches += 2;
                    } else {
                        HALO_TRY(launch_predict(s->pred, s->W1[l + 1], s->W2[l + 1], x_cur, static_cast<int>(T), 1,
                                                s->set_scores[nxt], s->pred_ws, s->status, side));
                        HALO_TRY(launch_select(s->plan.dev, G, s->set_scores[nxt], step, static_cast<uint32_t>(l + 1), 0,
                                               nullptr, s->set_dev[nxt], s->set_arr[nxt], nullptr, s->set_kl[nxt],
                                               s->set_nk[nxt], s->status, side));
                        launches += 4;
                    }
                    if (s->i4_prompt) {
                        // the scratch block of parity nxt was last read by block l-1, which ev_x is behind
                        HALO_TRY(launch_dequantize_i4(s->ffn, s->W[l + 1], s->i4_scales[l + 1], s->set_kl[nxt], s->set_nk[nxt],
                                                      s->i4_deq[nxt], s->status, side));
                        ++launches;
                    }
                    HALO_CU(cudaEventRecord(s->ev_sel, side));
                }
                float* y_tap = nullptr;
                if (taps) {
                    const size_t rec = static_cast<size_t>(sidx) * L + l;
                    if (taps->x) HALO_COPY(static_cast<char*>(taps->x) + rec * step_elems * es, x_cur, step_elems * es);
                    if (taps->scores) HALO_COPY(taps->scores + rec * G, l == 0 ? s->zero_scores : s->set_scores[cur], sizeof(float) * G);
                    if (taps->dev_of_group) HALO_COPY(taps->dev_of_group + rec * G, s->set_dev[cur], sizeof(int32_t) * G);
                    if (taps->arrived && n_dev > 0) HALO_COPY(taps->arrived + rec * n_dev, s->set_arr[cur], n_dev);
                    if (taps->keep_list) HALO_COPY(taps->keep_list + rec * G, s->set_kl[cur], sizeof(int32_t) * G);
                    if (taps->n_keep) HALO_COPY(taps->n_keep + rec, s->set_nk[cur], sizeof(int32_t));
                    if (taps->y) y_tap = taps->y + rec * step_elems;
                }
                float* h_dst = (l == L - 1) ? h_out + sidx * step_elems : s->h;
                const void* W_l = s->i4_prompt ? s->i4_deq[cur] : s->W[l];
                if (!s->i4_scales.empty() && !s->i4_prompt) {
                    HALO_TRY(halo_group_ffn_i4(&s->ffn, s->W[l], s->i4_scales[l], x_cur, static_cast<int>(T), s->set_kl[cur],
                                               s->set_nk[cur], s->set_dev[cur], n_dev, s->partials, s->status, stream));
                    HALO_TRY(launch_merge_glue(s->partials, s->set_arr[cur], n_dev, static_cast<int>(T), static_cast<int>(d),
                                               s->ffn.wdtype, s->h, h_dst, x_next, y_tap, st));
                    launches += 3;
                } else if (!y_tap && s->ffn_ws && prefill_accumulates(s->ffn, static_cast<int>(T))) {
                    // only kept (= arrived) groups are computed and nobody asked for y itself: the down projection
                    // adds its tiles straight into the residual stream, and the glue only normalises
                    HALO_TRY(launch_group_ffn_prefill(s->ffn, W_l, x_cur, static_cast<int>(T), s->set_kl[cur],
                                                      s->set_nk[cur], s->set_dev[cur], n_dev, 1, s->h, s->ffn_ws,
                                                      s->status, st, s->ffn_ws_clean));
                    s->ffn_ws_clean = true;   // every launch on this workspace leaves the control words zeroed
                    HALO_TRY(launch_glue(static_cast<int>(d), static_cast<int>(T), s->ffn.wdtype, s->h, nullptr, h_dst,
                                         x_next, st));
                    launches += 3;
                } else {
                    bool collapsed = false;   // the sum over holders is all the glue needs
                    HALO_TRY(dispatch_group_ffn(s->ffn, W_l, x_cur, static_cast<int>(T), s->set_kl[cur],
                                                s->set_nk[cur], s->set_dev[cur], n_dev, s->partials, s->ffn_ws,
                                                s->status, st, &collapsed));
                    HALO_TRY(launch_merge_glue(s->partials, collapsed ? nullptr : s->set_arr[cur],
                                               collapsed ? 1 : n_dev, static_cast<int>(T), static_cast<int>(d),
                                               s->ffn.wdtype, s->h, h_dst, x_next, y_tap, st));
                    launches += 2;
                }
                if (l + 1 < L) {
                    HALO_CU(cudaEventRecord(s->ev_x, st));             // x_{l+1} ready; set[cur] free again
                    // join: block l+1 needs its selection, and the glue of block l+1 will overwrite the x that the
                    // side stream has just been reading
                    HALO_CU(cudaStreamWaitEvent(st, s->ev_sel, 0));
                }
            }
        }
#undef HALO_CU
        s->last_launches = launches;
        return HALO_OK;
    }
    for (int sidx = 0; sidx < steps; ++sidx) {
        const uint32_t step = step0 + static_cast<uint32_t>(sidx);
        HALO_TRY(launch_glue(static_cast<int>(d), static_cast<int>(T), s->ffn.wdtype, h0 + sidx * step_elems, nullptr,
                             s->h, s->x[0], st));
        ++launches;
        for (int l = 0; l < L; ++l) {
            void* x_cur = s->x[l & 1];
            void* x_prev = s->x[(l + 1) & 1];
            const float* scores_used = s->scores;
            if (l == 0) {
                // first block: reliable, no semantic information yet -> everything is kept
                scores_used = s->zero_scores;
                HALO_TRY(launch_select(s->plan.dev, G, s->zero_scores, step, 0u, 1, nullptr, s->dev_of_group,
                                       s->arrived, nullptr, s->keep_list, s->n_keep, s->status, st));
                ++launches;
            } else if (T == 1) {
                HALO_TRY(launch_predict_hidden(s->pred, s->W1[l], x_prev, 1, s->pred_ws, st));
                HALO_TRY(launch_score_select(s->pred, s->W2[l], s->pred_ws, s->plan.dev, step,
                                             static_cast<uint32_t>(l), 0, s->scores, nullptr, s->dev_of_group,
                                             s->arrived, nullptr, s->keep_list, s->n_keep, s->status, st));
                launches += 2;
            } else {
                HALO_TRY(launch_predict(s->pred, s->W1[l], s->W2[l], x_prev, static_cast<int>(T), 1, s->scores,
                                        s->pred_ws, s->status, st));
                HALO_TRY(launch_select(s->plan.dev, G, s->scores, step, static_cast<uint32_t>(l), 0, nullptr,
                                       s->dev_of_group, s->arrived, nullptr, s->keep_list, s->n_keep, s->status, st));
                launches += 4;
            }
            float* y_tap = nullptr;
            if (taps) {
                const size_t rec = static_cast<size_t>(sidx) * L + l;
                if (taps->x) HALO_COPY(static_cast<char*>(taps->x) + rec * step_elems * es, x_cur, step_elems * es);
                if (taps->scores) HALO_COPY(taps->scores + rec * G, scores_used, sizeof(float) * G);
                if (taps->dev_of_group) HALO_COPY(taps->dev_of_group + rec * G, s->dev_of_group, sizeof(int32_t) * G);
                if (taps->arrived && n_dev > 0) HALO_COPY(taps->arrived + rec * n_dev, s->arrived, n_dev);
                if (taps->keep_list) HALO_COPY(taps->keep_list + rec * G, s->keep_list, sizeof(int32_t) * G);
                if (taps->n_keep) HALO_COPY(taps->n_keep + rec, s->n_keep, sizeof(int32_t));
                if (taps->y) y_tap = taps->y + rec * step_elems;
            }
            if (s->i4_prompt) {
                HALO_TRY(launch_dequantize_i4(s->ffn, s->W[l], s->i4_scales[l], s->keep_list, s->n_keep, s->i4_deq[0],
                                              s->status, st));
                ++launches;
                HALO_TRY(dispatch_group_ffn(s->ffn, s->i4_deq[0], x_cur, static_cast<int>(T), s->keep_list, s->n_keep,
                                            s->dev_of_group, n_dev, s->partials, s->ffn_ws, s->status, st));
            } else if (!s->i4_scales.empty()) {
                HALO_TRY(halo_group_ffn_i4(&s->ffn, s->W[l], s->i4_scales[l], x_cur, static_cast<int>(T), s->keep_list,
                                           s->n_keep, s->dev_of_group, n_dev, s->partials, s->status, stream));
                ++launches;
            } else {
                HALO_TRY(dispatch_group_ffn(s->ffn, s->W[l], x_cur, static_cast<int>(T), s->keep_list, s->n_keep,
                                            s->dev_of_group, n_dev, s->partials, s->ffn_ws, s->status, st));
            }
            ++launches;
            float* h_dst = (l == L - 1) ? h_out + sidx * step_elems : s->h;
            HALO_TRY(launch_merge_glue(s->partials, s->arrived, n_dev, static_cast<int>(T), static_cast<int>(d),
                                       s->ffn.wdtype, s->h, h_dst, x_prev, y_tap, st));
            ++launches;
        }
    }
#undef HALO_TRY
#undef HALO_COPY
    s->last_launches = launches;
    return HALO_OK;
}

extern "C" halo_status halo_stack_decode_host(halo_stack* s, const float* h0_host, int steps, uint32_t step0,
                                              float* h_out_host, void* stream) {
    if (!s || !h0_host || !h_out_host) return HALO_ERR_ARG;
    if (steps <= 0) return HALO_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t step_elems = static_cast<size_t>(s->n_tok) * s->ffn.d_model;
    long long launches = 0;
    for (int done = 0; done < steps; done += s->stage_steps) {
        const int n = std::min(s->stage_steps, steps - done);
        const size_t bytes = sizeof(float) * n * step_elems;
        if (cudaMemcpyAsync(s->stage_in, h0_host + done * step_elems, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return HALO_ERR_CUDA;
        halo_status rc = halo_stack_decode(s, s->stage_in, n, step0 + static_cast<uint32_t>(done), s->stage_out,
                                           nullptr, stream);
        if (rc != HALO_OK) return rc;
        launches += s->last_launches;
        if (cudaMemcpyAsync(h_out_host + done * step_elems, s->stage_out, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return HALO_ERR_CUDA;
    }
    s->last_launches = launches;
    return cuda_status(cudaStreamSynchronize(st));
}

extern "C" halo_status halo_stack_status(halo_stack* s, uint32_t* value, void* stream) {
    if (!s || !value) return HALO_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(value, s->status, sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return HALO_ERR_CUDA;
    return cuda_status(cudaStreamSynchronize(st));
}

extern "C" halo_status halo_stack_set_mode(halo_stack* s, int mode) {
    if (!s || mode < 0 || mode > 31) return HALO_ERR_ARG;
    s->mode = mode;
    return HALO_OK;
}

extern "C" halo_status halo_stack_set_trace(halo_stack* s, unsigned long long* trace, int n_blocks) {
    if (!s || n_blocks < 0 || (n_blocks > 0 && !trace)) return HALO_ERR_ARG;
    s->trace = n_blocks > 0 ? trace : nullptr;
    s->trace_blocks = n_blocks;
    s->pp_trace = (n_blocks > 0 && s->n_tok > 1) ? trace : nullptr;
    return HALO_OK;
}

extern "C" int halo_stack_trace_width(const halo_stack* s) {
    int dev = 0, sms = kSmCount;
    (void)s;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms;
}

extern "C" long long halo_stack_last_launches(const halo_stack* s) { return s ? s->last_launches : 0; }
