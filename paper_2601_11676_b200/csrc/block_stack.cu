// halo_block_stack_*: the generation loop over whole transformer blocks (Sec. III-B.3: in every layer the MHA block
// and then the MLP block, one predictor each fed one layer ahead, the first layer and the LM head reliable), built
// from the group entry points of this library: one launch per step of the path (the MHA block is one launch, the
// predictors of the next layer run on a side stream), no host synchronisation inside.
#include <algorithm>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"

using namespace halo;

namespace {
size_t bs_align(size_t v) { return (v + 255) / 256 * 256; }
size_t bs_elem(halo_dtype t) { return t == HALO_F32 ? 4 : 2; }
}  // namespace

struct halo_block_stack {
    halo_ffn_shape ffn;
    halo_mha_shape mha;
    halo_lm_shape lm;
    halo_pred_shape pred_ffn, pred_mha;
    int L, G, H, n_dev_f, n_dev_a;
    bool has_lm;
    halo_plan plan_ffn, plan_mha;
    std::vector<const void*> W_ffn, W_mha, Wk, Wv, W1_ffn, W2_ffn, W1_mha, W2_mha;
    std::vector<void*> K, V;
    const void* W_lm;
    // int4 stacks: W_ffn, W_mha, Wk, Wv and W_lm hold codes, these their scales (activations, caches, predictors bf16)
    bool i4 = false;
    std::vector<const void*> S_ffn, S_mha, Sk, Sv;
    const void* S_lm = nullptr;
    void* slab;
    float* h;
    void* x_a[2];
    void* x_f[2];
    // selections of a layer are made one layer ahead on a side stream: two sets each, by parity of the layer
    float* hidden_a; float* hidden_f;
    float* scores_a[2]; float* scores_f[2]; float* zero_scores;
    int32_t* dev_a[2]; int32_t* dev_f[2];
    uint8_t* arr_a[2]; uint8_t* arr_f[2];
    int32_t* kl_a[2]; int32_t* kl_f[2];
    int32_t* nk_a[2]; int32_t* nk_f[2];
    float* part_a; float* part_f;
    cudaStream_t side;
    cudaEvent_t ev_xa, ev_xf, ev_sa, ev_sf;
    void* mha_ws; size_t mha_ws_bytes;
    uint32_t* status;
    long long last_launches;
};

namespace {
halo_status block_stack_create_impl(halo_block_stack** out, const halo_ffn_shape* ffn, const halo_mha_shape* mha,
                                    const halo_lm_shape* lm, const halo_pred_shape* pred_ffn,
                                    const halo_pred_shape* pred_mha, int n_layers, const halo_plan* plan_ffn,
                                    const halo_plan* plan_mha, const halo_block_weights* w, const halo_block_scales* sc);
}  // namespace

extern "C" halo_status halo_block_stack_create(halo_block_stack** out, const halo_ffn_shape* ffn, const halo_mha_shape* mha,
                                               const halo_lm_shape* lm, const halo_pred_shape* pred_ffn,
                                               const halo_pred_shape* pred_mha, int n_layers, const halo_plan* plan_ffn,
                                               const halo_plan* plan_mha, const halo_block_weights* w) {
    return block_stack_create_impl(out, ffn, mha, lm, pred_ffn, pred_mha, n_layers, plan_ffn, plan_mha, w, nullptr);
}

extern "C" halo_status halo_block_stack_create_i4(halo_block_stack** out, const halo_ffn_shape* ffn, const halo_mha_shape* mha,
                                                  const halo_lm_shape* lm, const halo_pred_shape* pred_ffn,
                                                  const halo_pred_shape* pred_mha, int n_layers, const halo_plan* plan_ffn,
                                                  const halo_plan* plan_mha, const halo_block_weights* codes,
                                                  const halo_block_scales* scales) {
    if (!out) return HALO_ERR_ARG;
    *out = nullptr;
    if (!ffn || !mha || !scales) return HALO_ERR_ARG;
    if (ffn->wdtype != HALO_BF16) return HALO_ERR_DTYPE;                   // activations, caches and predictors
    if (ffn->d_model % 128 != 0 || mha->head_dim % 16 != 0) return HALO_ERR_SHAPE;
    if (!scales->S_ffn || !scales->S_mha || !scales->Sk || !scales->Sv || (lm && !scales->S_lm)) return HALO_ERR_ARG;
    for (int l = 0; l < n_layers; ++l) {
        const void* p[4] = {scales->S_ffn[l], scales->S_mha[l], scales->Sk[l], scales->Sv[l]};
        for (const void* q : p) {
            if (!q) return HALO_ERR_ARG;
            if (!aligned16(q)) return HALO_ERR_ALIGN;
        }
    }
    return block_stack_create_impl(out, ffn, mha, lm, pred_ffn, pred_mha, n_layers, plan_ffn, plan_mha, codes, scales);
}

namespace {
halo_status block_stack_create_impl(halo_block_stack** out, const halo_ffn_shape* ffn, const halo_mha_shape* mha,
                                    const halo_lm_shape* lm, const halo_pred_shape* pred_ffn,
                                    const halo_pred_shape* pred_mha, int n_layers, const halo_plan* plan_ffn,
                                    const halo_plan* plan_mha, const halo_block_weights* w, const halo_block_scales* sc) {
    if (!out) return HALO_ERR_ARG;
    *out = nullptr;
    if (!ffn || !mha || !pred_ffn || !pred_mha || !plan_ffn || !plan_mha || !w) return HALO_ERR_ARG;
    if (n_layers <= 0) return HALO_ERR_SHAPE;
    halo_status rc = check_pred_shape(pred_ffn);
    if (rc != HALO_OK) return rc;
    rc = check_pred_shape(pred_mha);
    if (rc != HALO_OK) return rc;
    if (ffn->d_model <= 0 || ffn->group_size <= 0 || ffn->d_ffn % ffn->group_size != 0) return HALO_ERR_SHAPE;
    const int G = ffn->d_ffn / ffn->group_size, H = mha->n_heads, d = ffn->d_model;
    if (mha->d_model != d || pred_ffn->d_in != d || pred_mha->d_in != d || pred_ffn->n_groups != G ||
        pred_mha->n_groups != H || plan_ffn->n_groups != G || plan_mha->n_groups != H)
        return HALO_ERR_SHAPE;
    if (mha->wdtype != ffn->wdtype || pred_ffn->wdtype != ffn->wdtype || pred_mha->wdtype != ffn->wdtype) return HALO_ERR_DTYPE;
    if (lm && (lm->d_model != d || lm->wdtype != ffn->wdtype || !w->W_lm)) return HALO_ERR_SHAPE;
    if (halo_group_mha_workspace_bytes(mha) == 0) return HALO_ERR_SHAPE;
    if (!w->W_ffn || !w->W_mha || !w->Wk || !w->Wv || !w->K_cache || !w->V_cache) return HALO_ERR_ARG;
    if (n_layers > 1 && (!w->W1_ffn || !w->W2_ffn || !w->W1_mha || !w->W2_mha)) return HALO_ERR_ARG;
    for (int l = 0; l < n_layers; ++l) {
        if (!w->W_ffn[l] || !w->W_mha[l] || !w->Wk[l] || !w->Wv[l] || !w->K_cache[l] || !w->V_cache[l]) return HALO_ERR_ARG;
        if (l > 0 && (!w->W1_ffn[l] || !w->W2_ffn[l] || !w->W1_mha[l] || !w->W2_mha[l])) return HALO_ERR_ARG;
    }
    halo_block_stack* s = new (std::nothrow) halo_block_stack();
    if (!s) return HALO_ERR_NOMEM;
    s->ffn = *ffn; s->mha = *mha; s->pred_ffn = *pred_ffn; s->pred_mha = *pred_mha;
    s->has_lm = lm != nullptr;
    if (lm) s->lm = *lm;
    s->L = n_layers; s->G = G; s->H = H;
    s->plan_ffn = *plan_ffn; s->plan_mha = *plan_mha;
    s->n_dev_f = plan_ffn->n_dev; s->n_dev_a = plan_mha->n_dev;
    auto take = [&](std::vector<const void*>& v, const void* const* src) { if (src) v.assign(src, src + n_layers); else v.assign(n_layers, nullptr); };
    take(s->W_ffn, w->W_ffn); take(s->W_mha, w->W_mha); take(s->Wk, w->Wk); take(s->Wv, w->Wv);
    take(s->W1_ffn, w->W1_ffn); take(s->W2_ffn, w->W2_ffn); take(s->W1_mha, w->W1_mha); take(s->W2_mha, w->W2_mha);
    s->K.assign(w->K_cache, w->K_cache + n_layers);
    s->V.assign(w->V_cache, w->V_cache + n_layers);
    s->W_lm = w->W_lm;
    if (sc) {
        s->i4 = true;
        take(s->S_ffn, sc->S_ffn); take(s->S_mha, sc->S_mha); take(s->Sk, sc->Sk); take(s->Sv, sc->Sv);
        s->S_lm = sc->S_lm;
    }
    s->last_launches = 0;

    const size_t es = bs_elem(ffn->wdtype);
    size_t off = 0;
    auto carve = [&](size_t bytes) { size_t o = off; off = bs_align(off + bytes); return o; };
    const size_t o_h = carve(sizeof(float) * d);
    const size_t o_xa0 = carve(es * d), o_xa1 = carve(es * d), o_xf0 = carve(es * d), o_xf1 = carve(es * d);
    const size_t o_hida = carve(sizeof(float) * pred_mha->rank), o_hidf = carve(sizeof(float) * pred_ffn->rank);
    const size_t o_zs = carve(sizeof(float) * std::max(G, H));
    size_t o_sa[2], o_sf[2], o_da[2], o_df[2], o_aa[2], o_af[2], o_ka[2], o_kf[2], o_na[2], o_nf[2];
    for (int k = 0; k < 2; ++k) {
        o_sa[k] = carve(sizeof(float) * H); o_sf[k] = carve(sizeof(float) * G);
        o_da[k] = carve(sizeof(int32_t) * H); o_df[k] = carve(sizeof(int32_t) * G);
        o_aa[k] = carve(HALO_MAX_DEVICES); o_af[k] = carve(HALO_MAX_DEVICES);
        o_ka[k] = carve(sizeof(int32_t) * H); o_kf[k] = carve(sizeof(int32_t) * G);
        o_na[k] = carve(sizeof(int32_t)); o_nf[k] = carve(sizeof(int32_t));
    }
    const size_t o_pa = carve(sizeof(float) * (s->n_dev_a + 1) * d), o_pf = carve(sizeof(float) * (s->n_dev_f + 1) * d);
    s->mha_ws_bytes = halo_group_mha_workspace_bytes(mha);
    const size_t o_mw = carve(s->mha_ws_bytes);
    const size_t o_st = carve(sizeof(uint32_t));
    if (cudaMalloc(&s->slab, off) != cudaSuccess) { delete s; return HALO_ERR_NOMEM; }
    if (cudaMemset(s->slab, 0, off) != cudaSuccess) { cudaFree(s->slab); delete s; return HALO_ERR_CUDA; }
    char* b = static_cast<char*>(s->slab);
    s->h = reinterpret_cast<float*>(b + o_h);
    s->x_a[0] = b + o_xa0; s->x_a[1] = b + o_xa1; s->x_f[0] = b + o_xf0; s->x_f[1] = b + o_xf1;
    s->hidden_a = reinterpret_cast<float*>(b + o_hida); s->hidden_f = reinterpret_cast<float*>(b + o_hidf);
    s->zero_scores = reinterpret_cast<float*>(b + o_zs);
    for (int k = 0; k < 2; ++k) {
        s->scores_a[k] = reinterpret_cast<float*>(b + o_sa[k]); s->scores_f[k] = reinterpret_cast<float*>(b + o_sf[k]);
        s->dev_a[k] = reinterpret_cast<int32_t*>(b + o_da[k]); s->dev_f[k] = reinterpret_cast<int32_t*>(b + o_df[k]);
        s->arr_a[k] = reinterpret_cast<uint8_t*>(b + o_aa[k]); s->arr_f[k] = reinterpret_cast<uint8_t*>(b + o_af[k]);
        s->kl_a[k] = reinterpret_cast<int32_t*>(b + o_ka[k]); s->kl_f[k] = reinterpret_cast<int32_t*>(b + o_kf[k]);
        s->nk_a[k] = reinterpret_cast<int32_t*>(b + o_na[k]); s->nk_f[k] = reinterpret_cast<int32_t*>(b + o_nf[k]);
    }
    s->part_a = reinterpret_cast<float*>(b + o_pa); s->part_f = reinterpret_cast<float*>(b + o_pf);
    s->mha_ws = b + o_mw;
    s->status = reinterpret_cast<uint32_t*>(b + o_st);
    // side stream for the predictors (best effort: without it they run in line on the caller's stream)
    s->side = nullptr;
    s->ev_xa = s->ev_xf = s->ev_sa = s->ev_sf = nullptr;
    int prio_lo = 0, prio_hi = 0;
    if (cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi) != cudaSuccess) prio_hi = 0;
    if (cudaStreamCreateWithPriority(&s->side, cudaStreamNonBlocking, prio_hi) == cudaSuccess) {
        bool ok = true;
        for (cudaEvent_t* e : {&s->ev_xa, &s->ev_xf, &s->ev_sa, &s->ev_sf})
            ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            for (cudaEvent_t e : {s->ev_xa, s->ev_xf, s->ev_sa, s->ev_sf}) if (e) cudaEventDestroy(e);
            cudaStreamDestroy(s->side);
            s->side = nullptr;
        }
    } else {
        s->side = nullptr;
        (void)cudaGetLastError();
    }
    *out = s;
    return HALO_OK;
}
}  // namespace

extern "C" halo_status halo_block_stack_destroy(halo_block_stack* s) {
    if (!s) return HALO_OK;
    if (s->side) {
        cudaStreamSynchronize(s->side);
        for (cudaEvent_t e : {s->ev_xa, s->ev_xf, s->ev_sa, s->ev_sf}) cudaEventDestroy(e);
        cudaStreamDestroy(s->side);
    }
    cudaFree(s->slab);
    delete s;
    return HALO_OK;
}

extern "C" halo_status halo_block_stack_decode(halo_block_stack* s, const float* h0, int steps, int pos0, uint32_t step0,
                                               float* logits, float* h_out, const halo_block_taps* taps, void* stream) {
    if (!s || !h0) return HALO_ERR_ARG;
    if (steps <= 0 || pos0 < 0 || pos0 + steps > s->mha.max_len) return HALO_ERR_SHAPE;
    if (logits && !s->has_lm) return HALO_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int L = s->L, G = s->G, H = s->H, d = s->ffn.d_model;
    const halo_dtype dt = s->ffn.wdtype;
    const size_t es = bs_elem(dt);
    long long launches = 0;
    halo_status rc;
#define BS_TRY(call) do { rc = (call); if (rc != HALO_OK) return rc; } while (0)
#define BS_COPY(dst, src, bytes)                                                                      \
    do { if (cudaMemcpyAsync((dst), (src), (bytes), cudaMemcpyDeviceToDevice, st) != cudaSuccess)     \
             return HALO_ERR_CUDA; } while (0)
#define BS_CU(call) do { if ((call) != cudaSuccess) return HALO_ERR_CUDA; } while (0)
    // The scores of layer l need only layer l-1's inputs (one layer ahead, Sec. III-B.2): predictor and selection of
    // both blocks of layer l run on the side stream while layer l-1's blocks run here.  The partial slots are zeroed
    // once and left zeroed by every merge, so the streaming kernels need no zero-fill in front of them.
    cudaStream_t side = s->side ? s->side : st;
    const bool fork = s->side != nullptr;
    if (cudaMemsetAsync(s->part_a, 0, sizeof(float) * (s->n_dev_a + 1) * d, st) != cudaSuccess ||
        cudaMemsetAsync(s->part_f, 0, sizeof(float) * (s->n_dev_f + 1) * d, st) != cudaSuccess)
        return HALO_ERR_CUDA;
    for (int sidx = 0; sidx < steps; ++sidx) {
        const uint32_t step = step0 + static_cast<uint32_t>(sidx);
        const int pos = pos0 + sidx;
        BS_TRY(launch_glue(d, 1, dt, h0 + static_cast<size_t>(sidx) * d, nullptr, s->h, s->x_a[0], st));
        // layer 0: reliable, nothing to go by yet -> every head and every group is kept
        BS_TRY(launch_select(s->plan_mha.dev, H, s->zero_scores, step, 0u, 1, nullptr, s->dev_a[0], s->arr_a[0], nullptr,
                             s->kl_a[0], s->nk_a[0], s->status, st));
        BS_TRY(launch_select(s->plan_ffn.dev, G, s->zero_scores, step, 1u, 1, nullptr, s->dev_f[0], s->arr_f[0], nullptr,
                             s->kl_f[0], s->nk_f[0], s->status, st));
        launches += 3;
        for (int l = 0; l < L; ++l) {
            const size_t rec = static_cast<size_t>(sidx) * L + l;
            const int cur = l & 1, nxt = (l + 1) & 1;
            void* xa = s->x_a[cur];
            void* xf = s->x_f[cur];
            // ---- MHA block ----
            if (l + 1 < L) {
                // heads of layer l+1 from this layer's attention input
                if (fork) { BS_CU(cudaEventRecord(s->ev_xa, st)); BS_CU(cudaStreamWaitEvent(side, s->ev_xa, 0)); }
                BS_TRY(launch_predict_hidden(s->pred_mha, s->W1_mha[l + 1], xa, 1, s->hidden_a, side));
                BS_TRY(launch_score_select(s->pred_mha, s->W2_mha[l + 1], s->hidden_a, s->plan_mha.dev, step,
                                           static_cast<uint32_t>(2 * (l + 1)), 0, s->scores_a[nxt], nullptr, s->dev_a[nxt],
                                           s->arr_a[nxt], nullptr, s->kl_a[nxt], s->nk_a[nxt], s->status, side));
                if (fork) BS_CU(cudaEventRecord(s->ev_sa, side));
                launches += 2;
            }
            if (s->i4) {
                BS_TRY(launch_mha_block_i4(s->mha, s->W_mha[l], s->S_mha[l], s->Wk[l], s->Sk[l], s->Wv[l], s->Sv[l], xa, s->K[l],
                                           s->V[l], pos, s->kl_a[cur], s->nk_a[cur], s->dev_a[cur], s->n_dev_a, s->part_a,
                                           s->status, st, true));
                ++launches;
            } else if (s->mha.head_dim % 16 == 0) {
                BS_TRY(launch_mha_block(s->mha, s->W_mha[l], s->Wk[l], s->Wv[l], xa, s->K[l], s->V[l], pos, s->kl_a[cur],
                                        s->nk_a[cur], s->dev_a[cur], s->n_dev_a, s->part_a, s->status, st, true));
                ++launches;
            } else {
                BS_TRY(halo_mha_kv_append(&s->mha, s->Wk[l], s->Wv[l], xa, pos, s->K[l], s->V[l], stream));
                BS_TRY(halo_group_mha(&s->mha, s->W_mha[l], xa, s->K[l], s->V[l], pos, s->kl_a[cur], s->nk_a[cur], s->dev_a[cur],
                                      s->n_dev_a, s->part_a, s->mha_ws, s->mha_ws_bytes, s->status, stream));
                launches += 3;
            }
            float* y_tap = nullptr;
            if (taps) {
                const halo_taps& t = taps->mha;
                if (t.x) BS_COPY(static_cast<char*>(t.x) + rec * d * es, xa, d * es);
                if (t.scores) BS_COPY(t.scores + rec * H, l == 0 ? s->zero_scores : s->scores_a[cur], sizeof(float) * H);
                if (t.dev_of_group) BS_COPY(t.dev_of_group + rec * H, s->dev_a[cur], sizeof(int32_t) * H);
                if (t.arrived && s->n_dev_a > 0) BS_COPY(t.arrived + rec * s->n_dev_a, s->arr_a[cur], s->n_dev_a);
                if (t.keep_list) BS_COPY(t.keep_list + rec * H, s->kl_a[cur], sizeof(int32_t) * H);
                if (t.n_keep) BS_COPY(t.n_keep + rec, s->nk_a[cur], sizeof(int32_t));
                if (t.y) y_tap = t.y + rec * d;
            }
            // merge of the heads that arrived + residual; the normalised stream is the MLP block's input
            BS_TRY(launch_merge_glue(s->part_a, s->arr_a[cur], s->n_dev_a, 1, d, dt, s->h, s->h, xf, y_tap, st, true));
            ++launches;
            // ---- MLP block ----
            // this layer's groups were selected on the side stream under the previous layer
            if (fork && l >= 1) BS_CU(cudaStreamWaitEvent(st, s->ev_sf, 0));
            if (l + 1 < L) {
                // groups of layer l+1 from this layer's MLP input
                if (fork) { BS_CU(cudaEventRecord(s->ev_xf, st)); BS_CU(cudaStreamWaitEvent(side, s->ev_xf, 0)); }
                BS_TRY(launch_predict_hidden(s->pred_ffn, s->W1_ffn[l + 1], xf, 1, s->hidden_f, side));
                BS_TRY(launch_score_select(s->pred_ffn, s->W2_ffn[l + 1], s->hidden_f, s->plan_ffn.dev, step,
                                           static_cast<uint32_t>(2 * (l + 1) + 1), 0, s->scores_f[nxt], nullptr, s->dev_f[nxt],
                                           s->arr_f[nxt], nullptr, s->kl_f[nxt], s->nk_f[nxt], s->status, side));
                if (fork) BS_CU(cudaEventRecord(s->ev_sf, side));
                launches += 2;
            }
            if (s->i4) {
                BS_TRY(launch_group_ffn_i4(s->ffn, s->W_ffn[l], s->S_ffn[l], xf, 1, s->kl_f[cur], s->nk_f[cur], s->dev_f[cur],
                                           s->n_dev_f, s->part_f, s->status, st, true));
                ++launches;
            } else {
                BS_TRY(launch_group_ffn_decode(s->ffn, s->W_ffn[l], xf, 1, s->kl_f[cur], s->nk_f[cur], s->dev_f[cur], s->n_dev_f,
                                               s->part_f, s->status, st, true));
                ++launches;
            }
            y_tap = nullptr;
            if (taps) {
                const halo_taps& t = taps->ffn;
                if (t.x) BS_COPY(static_cast<char*>(t.x) + rec * d * es, xf, d * es);
                if (t.scores) BS_COPY(t.scores + rec * G, l == 0 ? s->zero_scores : s->scores_f[cur], sizeof(float) * G);
                if (t.dev_of_group) BS_COPY(t.dev_of_group + rec * G, s->dev_f[cur], sizeof(int32_t) * G);
                if (t.arrived && s->n_dev_f > 0) BS_COPY(t.arrived + rec * s->n_dev_f, s->arr_f[cur], s->n_dev_f);
                if (t.keep_list) BS_COPY(t.keep_list + rec * G, s->kl_f[cur], sizeof(int32_t) * G);
                if (t.n_keep) BS_COPY(t.n_keep + rec, s->nk_f[cur], sizeof(int32_t));
                if (t.y) y_tap = t.y + rec * d;
            }
            // merge + residual; the normalised stream is the next layer's attention input (or the LM head's input).
            // (The joins with the side stream sit where their results are first needed, not here: a join in front of this
            // merge made every layer wait for the side stream's last kernel, 261 against 307 tokens/s at the 7B shape.
            // Chaining the four kernels of a layer as programmatic dependents on top of that measured 1 % slower.)
            BS_TRY(launch_merge_glue(s->part_f, s->arr_f[cur], s->n_dev_f, 1, d, dt, s->h, s->h, s->x_a[nxt], y_tap, st, true));
            ++launches;
            // The next layer's heads were selected on the side stream under this layer.  Every buffer the side stream
            // reads or writes is indexed by layer parity and is next written on this stream two layers on, behind the
            // joins of the layer in between.
            if (fork && l + 1 < L) BS_CU(cudaStreamWaitEvent(st, s->ev_sa, 0));
        }
        if (logits) {
            // LM head: every vocabulary group, sent reliably (Sec. III-B.3)
            if (s->i4)
                BS_TRY(halo_group_lm_head_i4(&s->lm, s->W_lm, s->S_lm, s->x_a[L & 1], 1, nullptr, nullptr,
                                             logits + static_cast<size_t>(sidx) * s->lm.vocab, s->status, stream));
            else
                BS_TRY(halo_group_lm_head(&s->lm, s->W_lm, s->x_a[L & 1], 1, nullptr, nullptr,
                                          logits + static_cast<size_t>(sidx) * s->lm.vocab, s->status, stream));
            ++launches;
        }
        if (h_out) BS_COPY(h_out + static_cast<size_t>(sidx) * d, s->h, sizeof(float) * d);
    }
#undef BS_CU
#undef BS_TRY
#undef BS_COPY
    s->last_launches = launches;
    return HALO_OK;
}

extern "C" halo_status halo_block_stack_status(halo_block_stack* s, uint32_t* value, void* stream) {
    if (!s || !value) return HALO_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(value, s->status, sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return HALO_ERR_CUDA;
    return cuda_status(cudaStreamSynchronize(st));
}

extern "C" long long halo_block_stack_last_launches(const halo_block_stack* s) { return s ? s->last_launches : 0; }
