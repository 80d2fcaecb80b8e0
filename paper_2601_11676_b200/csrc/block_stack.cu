// halo_block_stack_*: the generation loop over whole transformer blocks (Sec. III-B.3: in every layer the MHA block
// and then the MLP block, one predictor each fed one layer ahead, the first layer and the LM head reliable), built
// from the group entry points of this library: one launch per step of the path, no host synchronisation inside.
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
    void* slab;
    float* h;
    void* x_a[2];
    void* x_f[2];
    float* hidden;            // predictor hidden values
    float* scores_a; float* scores_f; float* zero_scores;
    int32_t* dev_a; int32_t* dev_f;
    uint8_t* arr_a; uint8_t* arr_f;
    int32_t* kl_a; int32_t* kl_f;
    int32_t* nk_a; int32_t* nk_f;
    float* part_a; float* part_f;
    void* mha_ws; size_t mha_ws_bytes;
    uint32_t* status;
    long long last_launches;
};

extern "C" halo_status halo_block_stack_create(halo_block_stack** out, const halo_ffn_shape* ffn, const halo_mha_shape* mha,
                                               const halo_lm_shape* lm, const halo_pred_shape* pred_ffn,
                                               const halo_pred_shape* pred_mha, int n_layers, const halo_plan* plan_ffn,
                                               const halo_plan* plan_mha, const halo_block_weights* w) {
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
    s->last_launches = 0;

    const size_t es = bs_elem(ffn->wdtype);
    size_t off = 0;
    auto carve = [&](size_t bytes) { size_t o = off; off = bs_align(off + bytes); return o; };
    const size_t o_h = carve(sizeof(float) * d);
    const size_t o_xa0 = carve(es * d), o_xa1 = carve(es * d), o_xf0 = carve(es * d), o_xf1 = carve(es * d);
    const size_t o_hid = carve(sizeof(float) * std::max(pred_ffn->rank, pred_mha->rank));
    const size_t o_sa = carve(sizeof(float) * H), o_sf = carve(sizeof(float) * G), o_zs = carve(sizeof(float) * std::max(G, H));
    const size_t o_da = carve(sizeof(int32_t) * H), o_df = carve(sizeof(int32_t) * G);
    const size_t o_aa = carve(HALO_MAX_DEVICES), o_af = carve(HALO_MAX_DEVICES);
    const size_t o_ka = carve(sizeof(int32_t) * H), o_kf = carve(sizeof(int32_t) * G);
    const size_t o_na = carve(sizeof(int32_t)), o_nf = carve(sizeof(int32_t));
    const size_t o_pa = carve(sizeof(float) * (s->n_dev_a + 1) * d), o_pf = carve(sizeof(float) * (s->n_dev_f + 1) * d);
    s->mha_ws_bytes = halo_group_mha_workspace_bytes(mha);
    const size_t o_mw = carve(s->mha_ws_bytes);
    const size_t o_st = carve(sizeof(uint32_t));
    if (cudaMalloc(&s->slab, off) != cudaSuccess) { delete s; return HALO_ERR_NOMEM; }
    if (cudaMemset(s->slab, 0, off) != cudaSuccess) { cudaFree(s->slab); delete s; return HALO_ERR_CUDA; }
    char* b = static_cast<char*>(s->slab);
    s->h = reinterpret_cast<float*>(b + o_h);
    s->x_a[0] = b + o_xa0; s->x_a[1] = b + o_xa1; s->x_f[0] = b + o_xf0; s->x_f[1] = b + o_xf1;
    s->hidden = reinterpret_cast<float*>(b + o_hid);
    s->scores_a = reinterpret_cast<float*>(b + o_sa); s->scores_f = reinterpret_cast<float*>(b + o_sf);
    s->zero_scores = reinterpret_cast<float*>(b + o_zs);
    s->dev_a = reinterpret_cast<int32_t*>(b + o_da); s->dev_f = reinterpret_cast<int32_t*>(b + o_df);
    s->arr_a = reinterpret_cast<uint8_t*>(b + o_aa); s->arr_f = reinterpret_cast<uint8_t*>(b + o_af);
    s->kl_a = reinterpret_cast<int32_t*>(b + o_ka); s->kl_f = reinterpret_cast<int32_t*>(b + o_kf);
    s->nk_a = reinterpret_cast<int32_t*>(b + o_na); s->nk_f = reinterpret_cast<int32_t*>(b + o_nf);
    s->part_a = reinterpret_cast<float*>(b + o_pa); s->part_f = reinterpret_cast<float*>(b + o_pf);
    s->mha_ws = b + o_mw;
    s->status = reinterpret_cast<uint32_t*>(b + o_st);
    *out = s;
    return HALO_OK;
}

extern "C" halo_status halo_block_stack_destroy(halo_block_stack* s) {
    if (!s) return HALO_OK;
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
    for (int sidx = 0; sidx < steps; ++sidx) {
        const uint32_t step = step0 + static_cast<uint32_t>(sidx);
        const int pos = pos0 + sidx;
        BS_TRY(launch_glue(d, 1, dt, h0 + static_cast<size_t>(sidx) * d, nullptr, s->h, s->x_a[0], st));
        ++launches;
        for (int l = 0; l < L; ++l) {
            const size_t rec = static_cast<size_t>(sidx) * L + l;
            void* xa = s->x_a[l & 1];
            void* xf = s->x_f[l & 1];
            // ---- MHA block: keys / values of every head, then the kept heads ----
            BS_TRY(halo_mha_kv_append(&s->mha, s->Wk[l], s->Wv[l], xa, pos, s->K[l], s->V[l], stream));
            ++launches;
            const float* sc_a = s->scores_a;
            if (l == 0) {
                sc_a = s->zero_scores;   // first layer: reliable, nothing to go by yet -> every head is kept
                BS_TRY(launch_select(s->plan_mha.dev, H, s->zero_scores, step, 0u, 1, nullptr, s->dev_a, s->arr_a, nullptr,
                                     s->kl_a, s->nk_a, s->status, st));
                ++launches;
            } else {
                BS_TRY(launch_predict_hidden(s->pred_mha, s->W1_mha[l], s->x_a[(l - 1) & 1], 1, s->hidden, st));
                BS_TRY(launch_score_select(s->pred_mha, s->W2_mha[l], s->hidden, s->plan_mha.dev, step,
                                           static_cast<uint32_t>(2 * l), 0, s->scores_a, nullptr, s->dev_a, s->arr_a, nullptr,
                                           s->kl_a, s->nk_a, s->status, st));
                launches += 2;
            }
            BS_TRY(halo_group_mha(&s->mha, s->W_mha[l], xa, s->K[l], s->V[l], pos, s->kl_a, s->nk_a, s->dev_a, s->n_dev_a,
                                  s->part_a, s->mha_ws, s->mha_ws_bytes, s->status, stream));
            launches += 2;
            float* y_tap = nullptr;
            if (taps) {
                const halo_taps& t = taps->mha;
                if (t.x) BS_COPY(static_cast<char*>(t.x) + rec * d * es, xa, d * es);
                if (t.scores) BS_COPY(t.scores + rec * H, sc_a, sizeof(float) * H);
                if (t.dev_of_group) BS_COPY(t.dev_of_group + rec * H, s->dev_a, sizeof(int32_t) * H);
                if (t.arrived && s->n_dev_a > 0) BS_COPY(t.arrived + rec * s->n_dev_a, s->arr_a, s->n_dev_a);
                if (t.keep_list) BS_COPY(t.keep_list + rec * H, s->kl_a, sizeof(int32_t) * H);
                if (t.n_keep) BS_COPY(t.n_keep + rec, s->nk_a, sizeof(int32_t));
                if (t.y) y_tap = t.y + rec * d;
            }
            // merge of the heads that arrived + residual; the normalised stream is the MLP block's input
            BS_TRY(launch_merge_glue(s->part_a, s->arr_a, s->n_dev_a, 1, d, dt, s->h, s->h, xf, y_tap, st));
            ++launches;
            // ---- MLP block ----
            const float* sc_f = s->scores_f;
            if (l == 0) {
                sc_f = s->zero_scores;
                BS_TRY(launch_select(s->plan_ffn.dev, G, s->zero_scores, step, 1u, 1, nullptr, s->dev_f, s->arr_f, nullptr,
                                     s->kl_f, s->nk_f, s->status, st));
                ++launches;
            } else {
                BS_TRY(launch_predict_hidden(s->pred_ffn, s->W1_ffn[l], s->x_f[(l - 1) & 1], 1, s->hidden, st));
                BS_TRY(launch_score_select(s->pred_ffn, s->W2_ffn[l], s->hidden, s->plan_ffn.dev, step,
                                           static_cast<uint32_t>(2 * l + 1), 0, s->scores_f, nullptr, s->dev_f, s->arr_f,
                                           nullptr, s->kl_f, s->nk_f, s->status, st));
                launches += 2;
            }
            BS_TRY(halo_group_ffn(&s->ffn, s->W_ffn[l], xf, 1, s->kl_f, s->nk_f, s->dev_f, s->n_dev_f, s->part_f, nullptr, 0,
                                  s->status, stream));
            launches += 2;
            y_tap = nullptr;
            if (taps) {
                const halo_taps& t = taps->ffn;
                if (t.x) BS_COPY(static_cast<char*>(t.x) + rec * d * es, xf, d * es);
                if (t.scores) BS_COPY(t.scores + rec * G, sc_f, sizeof(float) * G);
                if (t.dev_of_group) BS_COPY(t.dev_of_group + rec * G, s->dev_f, sizeof(int32_t) * G);
                if (t.arrived && s->n_dev_f > 0) BS_COPY(t.arrived + rec * s->n_dev_f, s->arr_f, s->n_dev_f);
                if (t.keep_list) BS_COPY(t.keep_list + rec * G, s->kl_f, sizeof(int32_t) * G);
                if (t.n_keep) BS_COPY(t.n_keep + rec, s->nk_f, sizeof(int32_t));
                if (t.y) y_tap = t.y + rec * d;
            }
            // merge + residual; the normalised stream is the next layer's attention input (or the LM head's input)
            BS_TRY(launch_merge_glue(s->part_f, s->arr_f, s->n_dev_f, 1, d, dt, s->h, s->h, s->x_a[(l + 1) & 1], y_tap, st));
            ++launches;
        }
        if (logits) {
            // LM head: every vocabulary group, sent reliably (Sec. III-B.3)
            BS_TRY(halo_group_lm_head(&s->lm, s->W_lm, s->x_a[L & 1], 1, nullptr, nullptr,
                                      logits + static_cast<size_t>(sidx) * s->lm.vocab, s->status, stream));
            ++launches;
        }
        if (h_out) BS_COPY(h_out + static_cast<size_t>(sidx) * d, s->h, sizeof(float) * d);
    }
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
