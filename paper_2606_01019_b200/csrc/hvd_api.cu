// C ABI of the library: context management, argument checks, kernel launches.
#include <stdlib.h>

#include <new>

#include "hvd_score.cuh"

using namespace hvd;

namespace {

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

void release(hvd_ctx* c) {
    if (!c) return;
    cudaFree(c->d_W1); cudaFree(c->d_b1); cudaFree(c->d_W2); cudaFree(c->d_WhT); cudaFree(c->d_bh);
    cudaFree(c->lk_partial); cudaFree(c->lk_cnt);
    cudaFree(c->fq_occ); cudaFree(c->fq_cnt);
    cudaFree(c->cp_key); cudaFree(c->cp_cnt); cudaFree(c->cp_arrived);
    cudaFree(c->cp_start); cudaFree(c->cp_pos);
    cudaFree(c->rp_key); cudaFree(c->rp_cnt);
    cudaFree(c->vf_next_unit); cudaFree(c->dev_error); cudaFree(c->vf_row_key); cudaFree(c->vf_alive);
    cudaFree(c->host_ws);
    delete c;
}

template <typename P>
cudaError_t alloc_zero(P** p, size_t bytes) {
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), bytes);
    if (e != cudaSuccess) return e;
    return cudaMemset(*p, 0, bytes);
}

}  // namespace

extern "C" {

const char* hvd_status_string(hvd_status s) {
    switch (s) {
        case HVD_OK: return "HVD_OK";
        case HVD_ERR_INVALID_ARG: return "HVD_ERR_INVALID_ARG";
        case HVD_ERR_CUDA: return "HVD_ERR_CUDA";
        case HVD_ERR_UNSUPPORTED: return "HVD_ERR_UNSUPPORTED";
        case HVD_ERR_ALLOC: return "HVD_ERR_ALLOC";
    }
    return "HVD_ERR_UNKNOWN";
}

const char* hvd_last_error(const hvd_ctx* ctx) { return ctx ? ctx->last_error : ""; }

hvd_status hvd_create(hvd_ctx** out, const hvd_config* cfg) {
    if (!out) return HVD_ERR_INVALID_ARG;
    *out = nullptr;
    if (!cfg) return HVD_ERR_INVALID_ARG;
    if (cfg->max_batch < 1 || cfg->max_batch > 8192) return HVD_ERR_INVALID_ARG;
    if (cfg->k_cap < 1 || cfg->k_cap > HVD_MAX_K) return HVD_ERR_INVALID_ARG;
    if (cfg->l_max < 1 || cfg->l_max > HVD_MAX_L) return HVD_ERR_INVALID_ARG;
    if (cfg->min_match < 1) return HVD_ERR_INVALID_ARG;
    if (cfg->hidden < 1 || cfg->hidden > HVD_MAX_HIDDEN) return HVD_ERR_INVALID_ARG;
    if (cfg->max_hist_len < 1 || cfg->max_hist_len > HVD_MAX_HIST_LEN) return HVD_ERR_INVALID_ARG;
    if (cfg->max_rows < 1 || cfg->max_vocab < 1 || cfg->max_vocab > 0x7fffffffLL) return HVD_ERR_INVALID_ARG;
    if (!(cfg->spec_factor == cfg->spec_factor) || !(cfg->spec_offset == cfg->spec_offset)) return HVD_ERR_INVALID_ARG;

    hvd_ctx* c = new (std::nothrow) hvd_ctx();
    if (!c) return HVD_ERR_ALLOC;
    c->cfg = *cfg;
    c->last_error[0] = 0;
    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, c->device);
    if (e != cudaSuccess) { delete c; return HVD_ERR_CUDA; }

    c->lk_max_chunks = (int)(((int64_t)cfg->max_hist_len + 3 + kLookupMinChunk - 1) / kLookupMinChunk);
    if (cfg->max_rows >= 0x7fffffffLL) { delete c; return HVD_ERR_INVALID_ARG; }

    const size_t H = (size_t)cfg->hidden;
    bool ok = true;
    ok = ok && alloc_zero(&c->d_W1, H * 16 * sizeof(float)) == cudaSuccess;  // row stride 8, or 16 for the extended vector
    ok = ok && alloc_zero(&c->d_b1, H * sizeof(float)) == cudaSuccess;
    ok = ok && alloc_zero(&c->d_W2, H * sizeof(float)) == cudaSuccess;
    ok = ok && alloc_zero(&c->d_WhT, (size_t)HVD_MAX_HIDDEN * HVD_MAX_HIDDEN * sizeof(float)) == cudaSuccess;  // row stride 256
    ok = ok && alloc_zero(&c->d_bh, H * sizeof(float)) == cudaSuccess;
    ok = ok && alloc_zero(&c->lk_partial, (size_t)cfg->max_batch * c->lk_max_chunks * sizeof(LookupPartial)) == cudaSuccess;
    ok = ok && alloc_zero(&c->lk_cnt, (size_t)cfg->max_batch * sizeof(uint32_t)) == cudaSuccess;
    ok = ok && alloc_zero(&c->fq_occ, (size_t)cfg->max_batch * HVD_FREQ_MAX_OCC * sizeof(int32_t)) == cudaSuccess;
    ok = ok && alloc_zero(&c->fq_cnt, (size_t)cfg->max_batch * sizeof(uint32_t)) == cudaSuccess;
    ok = ok && alloc_zero(&c->cp_key, (size_t)cfg->max_batch * sizeof(unsigned long long)) == cudaSuccess;
    ok = ok && alloc_zero(&c->cp_cnt, (size_t)cfg->max_batch * (HVD_MAX_L + 1) * sizeof(uint32_t)) == cudaSuccess;
    ok = ok && alloc_zero(&c->cp_arrived, (size_t)cfg->max_batch * sizeof(uint32_t)) == cudaSuccess;
    ok = ok && alloc_zero(&c->vf_row_key, (size_t)cfg->max_rows * sizeof(unsigned long long)) == cudaSuccess;
    ok = ok && alloc_zero(&c->vf_next_unit, (size_t)kVerifyQueues * 32 * sizeof(uint32_t)) == cudaSuccess;
    ok = ok && alloc_zero(&c->vf_alive, (size_t)cfg->max_batch * sizeof(int32_t)) == cudaSuccess;
    ok = ok && alloc_zero(&c->dev_error, sizeof(int)) == cudaSuccess;
    if (ok) ok = cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) { (void)cudaGetLastError(); release(c); return HVD_ERR_ALLOC; }

    const size_t smem = verify_dyn_smem(cfg->max_batch);
    c->vf_blocks_per_sm[0] = verify_occupancy(HVD_F32, smem);
    c->vf_blocks_per_sm[1] = verify_occupancy(HVD_BF16, smem);
    if (c->vf_blocks_per_sm[0] < 1 || c->vf_blocks_per_sm[1] < 1) { release(c); return HVD_ERR_UNSUPPORTED; }
    c->lk_cluster_mode = getenv("HVD_LOOKUP_CLUSTER") ? atoi(getenv("HVD_LOOKUP_CLUSTER")) : 1;
    lookup_cluster_setup(c);
    c->has_predictor = false;
    c->has_predictor_ext = false;
    c->two_layer = false;
    c->score2_ready = false;
    // programmatic dependent launch of the kernels of a step (bit 0 commit, 1 lookup, 2 stream, 3 one-layer
    // scoring): the next kernel's CTAs are resident and past their prologue when the previous one ends;
    // HVD_PDL_MASK=0 turns it off
    c->pdl_mask = getenv("HVD_PDL_MASK") ? atoi(getenv("HVD_PDL_MASK")) : 15;
    c->pdl_commit = (c->pdl_mask & 1) != 0;
    c->vf_small_bytes = getenv("HVD_VERIFY_SMALL_BYTES") ? atoll(getenv("HVD_VERIFY_SMALL_BYTES")) : kVerifySmallBytes;
    c->vf_boundary_bytes = getenv("HVD_PREFIX_BOUNDARY_BYTES") ? atoll(getenv("HVD_PREFIX_BOUNDARY_BYTES")) : kPrefixBoundaryBytes;
    if (c->vf_boundary_bytes < 1) c->vf_boundary_bytes = 1;
    c->host_ws = nullptr;
    c->host_ws_bytes = 0;
    *out = c;
    return HVD_OK;
}

hvd_status hvd_destroy(hvd_ctx* ctx) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    release(ctx);
    return HVD_OK;
}

hvd_status hvd_device_status(hvd_ctx* ctx, int32_t* code) {
    if (!ctx || !code) return HVD_ERR_INVALID_ARG;
    int v = 0;
    HVD_CUDA_TRY(ctx, cudaMemcpy(&v, ctx->dev_error, sizeof(int), cudaMemcpyDeviceToHost));
    *code = v;
    return HVD_OK;
}

hvd_status hvd_set_predictor(hvd_ctx* ctx, const float* W1, const float* b1, const float* W2,
                             float b2, float tau, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (!W1 || !b1 || !W2) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_set_predictor: NULL weights");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t H = (size_t)ctx->cfg.hidden;
    HVD_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_W1, W1, H * HVD_N_FEATURES * sizeof(float), cudaMemcpyHostToDevice, st));
    HVD_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_b1, b1, H * sizeof(float), cudaMemcpyHostToDevice, st));
    HVD_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_W2, W2, H * sizeof(float), cudaMemcpyHostToDevice, st));
    HVD_CUDA_TRY(ctx, cudaStreamSynchronize(st));  // the host arrays may be reused as soon as we return
    ctx->b2 = b2;
    ctx->tau = tau;
    ctx->has_predictor = true;
    ctx->has_predictor_ext = false;
    ctx->two_layer = false;
    return HVD_OK;
}

// second hidden layer: transposed copy with a fixed row stride (coalesced, 16-byte aligned rows on the device)
static hvd_status store_second_layer(hvd_ctx* ctx, const float* Wh, const float* bh, cudaStream_t st, const char* who) {
    const size_t H = (size_t)ctx->cfg.hidden;
    const size_t S = HVD_MAX_HIDDEN;
    float* t = static_cast<float*>(calloc(S * S, sizeof(float)));
    if (!t) return fail(ctx, HVD_ERR_ALLOC, "out of host memory");
    for (size_t j = 0; j < H; ++j)
        for (size_t i = 0; i < H; ++i) t[i * S + j] = Wh[j * H + i];
    cudaError_t e = cudaMemcpyAsync(ctx->d_WhT, t, S * S * sizeof(float), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->d_bh, bh, H * sizeof(float), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    free(t);
    if (e != cudaSuccess) { ctx->has_predictor = false; ctx->has_predictor_ext = false; return cuda_fail(ctx, e, who); }
    ctx->two_layer = true;
    return HVD_OK;
}

hvd_status hvd_set_predictor2(hvd_ctx* ctx, const float* W1, const float* b1, const float* Wh, const float* bh,
                              const float* W2, float b2, float tau, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (!Wh || !bh) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_set_predictor2: NULL weights");
    const hvd_status r = hvd_set_predictor(ctx, W1, b1, W2, b2, tau, stream);
    if (r != HVD_OK) return r;
    return store_second_layer(ctx, Wh, bh, static_cast<cudaStream_t>(stream), "hvd_set_predictor2");
}

hvd_status hvd_set_token_classes(hvd_ctx* ctx, const uint8_t* cls, int64_t V) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (cls == nullptr || V == 0) { ctx->cls = nullptr; ctx->cls_V = 0; return HVD_OK; }
    if (V < 0 || V > 0x7fffffffLL) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_set_token_classes: V outside [0, 2^31 - 1]");
    ctx->cls = cls; ctx->cls_V = (int32_t)V;
    return HVD_OK;
}

hvd_status hvd_set_predictor_ext(hvd_ctx* ctx, const float* W1, const float* b1, const float* Wh, const float* bh,
                                 const float* W2, float b2, float tau, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (!W1 || !b1 || !W2) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_set_predictor_ext: NULL weights");
    if ((Wh == nullptr) != (bh == nullptr)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_set_predictor_ext: Wh and bh go together");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t H = (size_t)ctx->cfg.hidden;
    float* t = static_cast<float*>(calloc(H * 16, sizeof(float)));  // rows padded to 16 floats
    if (!t) return fail(ctx, HVD_ERR_ALLOC, "hvd_set_predictor_ext: out of host memory");
    for (size_t j = 0; j < H; ++j)
        for (size_t i = 0; i < HVD_N_FEATURES_EXT; ++i) t[j * 16 + i] = W1[j * HVD_N_FEATURES_EXT + i];
    cudaError_t e = cudaMemcpyAsync(ctx->d_W1, t, H * 16 * sizeof(float), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->d_b1, b1, H * sizeof(float), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->d_W2, W2, H * sizeof(float), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    free(t);
    ctx->has_predictor = false;
    ctx->has_predictor_ext = false;
    ctx->two_layer = false;
    if (e != cudaSuccess) return cuda_fail(ctx, e, "hvd_set_predictor_ext");
    ctx->b2 = b2;
    ctx->tau = tau;
    ctx->has_predictor_ext = true;
    if (Wh) return store_second_layer(ctx, Wh, bh, st, "hvd_set_predictor_ext");
    return HVD_OK;
}

hvd_status hvd_lookup(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                      const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K,
                      int32_t n_max, int32_t* draft, int32_t* draft_len, int32_t* match_len,
                      int32_t* match_pos, int32_t* match_cnt, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (B < 1 || B > ctx->cfg.max_batch) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup: B outside [1, max_batch]");
    if (!hist || !hist_off || !hist_cap || !hist_len || !K || !draft || !draft_len || !match_len ||
        !match_pos || !match_cnt)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup: NULL pointer");
    if (!aligned(hist, 16)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup: hist must be 16-byte aligned");
    if (n_max < 0 || n_max > ctx->cfg.max_hist_len)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup: n_max outside [0, max_hist_len]");
    return launch_lookup(ctx, B, hist, hist_off, hist_cap, hist_len, K, n_max, draft, draft_len,
                         match_len, match_pos, match_cnt, nullptr, static_cast<cudaStream_t>(stream));
}

hvd_status hvd_set_corpus(hvd_ctx* ctx, const int32_t* corpus, int64_t m) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (corpus == nullptr || m == 0) { release_corpus_index(ctx); return HVD_OK; }
    if (m < 0 || m > 2147483646LL) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_set_corpus: m outside [0, 2^31 - 2]");
    if (!aligned(corpus, 16)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_set_corpus: corpus must be 16-byte aligned");
    return build_corpus_index(ctx, corpus, m);
}

hvd_status hvd_lookup_corpus(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                             const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K, int32_t n_max,
                             int32_t* draft, int32_t* draft_len, int32_t* match_len, int32_t* match_pos,
                             int32_t* match_src, int32_t* match_cnt, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (B < 1 || B > ctx->cfg.max_batch) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_corpus: B outside [1, max_batch]");
    if (!hist || !hist_off || !hist_cap || !hist_len || !K || !draft || !draft_len || !match_len || !match_pos ||
        !match_src || !match_cnt)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_corpus: NULL pointer");
    if (!aligned(hist, 16)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_corpus: hist must be 16-byte aligned");
    if (n_max < 0 || n_max > ctx->cfg.max_hist_len)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_corpus: n_max outside [0, max_hist_len]");
    return launch_lookup_corpus(ctx, B, hist, hist_off, hist_cap, hist_len, K, n_max, draft, draft_len, match_len,
                                match_pos, match_src, match_cnt, static_cast<cudaStream_t>(stream));
}

hvd_status hvd_lookup_freq(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                           const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K, int32_t n_max,
                           float min_prob, int32_t max_occ, float threshold, const int32_t* model_draft,
                           const int32_t* model_len, int32_t* draft, int32_t* draft_len, float* score,
                           int32_t* match_len, int32_t* match_pos, int32_t* match_cnt, int32_t* select,
                           int32_t* sel_draft, int32_t* sel_len, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (B < 1 || B > ctx->cfg.max_batch) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_freq: B outside [1, max_batch]");
    if (!hist || !hist_off || !hist_cap || !hist_len || !K || !draft || !draft_len || !score || !match_len ||
        !match_pos || !match_cnt)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_freq: NULL pointer");
    const int n_sel = (select != nullptr) + (sel_draft != nullptr) + (sel_len != nullptr);
    if (n_sel != 0 && n_sel != 3)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_freq: select, sel_draft and sel_len go together");
    if ((model_draft == nullptr) != (model_len == nullptr))
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_freq: model_draft and model_len go together");
    if (!aligned(hist, 16)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_freq: hist must be 16-byte aligned");
    if (n_max < 0 || n_max > ctx->cfg.max_hist_len)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_freq: n_max outside [0, max_hist_len]");
    if (max_occ < 1 || max_occ > HVD_FREQ_MAX_OCC)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_freq: max_occ outside [1, HVD_FREQ_MAX_OCC]");
    if (!(min_prob >= 0.0f)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_freq: min_prob must be >= 0");
    return launch_lookup_freq(ctx, B, hist, hist_off, hist_cap, hist_len, K, n_max, min_prob, max_occ, threshold,
                              model_draft, model_len, draft, draft_len, score, match_len, match_pos, match_cnt,
                              select, sel_draft, sel_len, static_cast<cudaStream_t>(stream));
}

hvd_status hvd_replay_labels(hvd_ctx* ctx, const int32_t* trace, int32_t n, int32_t K, int32_t* label,
                             int32_t* draft_len, int32_t* match_len, int32_t* match_pos, int32_t* match_cnt,
                             void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (!trace || !label || !draft_len || !match_len || !match_pos || !match_cnt)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_replay_labels: NULL pointer");
    if (n < 1 || n > ctx->cfg.max_hist_len) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_replay_labels: n outside [1, max_hist_len]");
    if (K < 0 || K > ctx->cfg.k_cap) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_replay_labels: K outside [0, k_cap]");
    if (!aligned(trace, 16)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_replay_labels: trace must be 16-byte aligned");
    return launch_replay(ctx, trace, n, K, label, draft_len, match_len, match_pos, match_cnt,
                         static_cast<cudaStream_t>(stream));
}

hvd_status hvd_lookup_score_select(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                                   const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K,
                                   int32_t n_max, const int32_t* prompt_len, const hvd_req_state* state,
                                   const int32_t* model_draft, const int32_t* model_len, int32_t* draft,
                                   int32_t* draft_len, int32_t* match_len, int32_t* match_pos,
                                   int32_t* match_cnt, float* features, float* score, int32_t* select,
                                   int32_t* sel_draft, int32_t* sel_len, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (B < 1 || B > ctx->cfg.max_batch) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_score_select: B outside [1, max_batch]");
    if (!ctx->has_predictor) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_score_select: call hvd_set_predictor first");
    if (!hist || !hist_off || !hist_cap || !hist_len || !K || !prompt_len || !state || !draft || !draft_len ||
        !match_len || !match_pos || !match_cnt || !score || !select || !sel_draft || !sel_len)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_score_select: NULL pointer");
    if ((model_draft == nullptr) != (model_len == nullptr))
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_score_select: model_draft and model_len go together");
    if (!aligned(hist, 16)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_score_select: hist must be 16-byte aligned");
    if (!aligned(state, 8)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_score_select: state must be 8-byte aligned");
    if (n_max < 0 || n_max > ctx->cfg.max_hist_len)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup_score_select: n_max outside [0, max_hist_len]");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (ctx->two_layer) {
        // the two-layer predictor needs a whole CTA per request: lookup, then its own kernel
        const hvd_status r = launch_lookup(ctx, B, hist, hist_off, hist_cap, hist_len, K, n_max, draft, draft_len,
                                           match_len, match_pos, match_cnt, nullptr, st);
        if (r != HVD_OK) return r;
        return launch_score_select(ctx, B, hist_len, prompt_len, state, K, draft, draft_len, match_len, match_pos,
                                   match_cnt, model_draft, model_len, features, score, select, sel_draft, sel_len, st);
    }
    const ScoreArgs sa = make_score_args(ctx, B, hist_len, prompt_len, state, K, draft, draft_len, match_len,
                                         match_pos, match_cnt, model_draft, model_len, features, score,
                                         select, sel_draft, sel_len);
    return launch_lookup(ctx, B, hist, hist_off, hist_cap, hist_len, K, n_max, draft, draft_len,
                         match_len, match_pos, match_cnt, &sa, st);
}

hvd_status hvd_score_select(hvd_ctx* ctx, int32_t B, const int32_t* hist_len,
                            const int32_t* prompt_len, const hvd_req_state* state, const int32_t* K,
                            const int32_t* draft, const int32_t* draft_len, const int32_t* match_len,
                            const int32_t* match_pos, const int32_t* match_cnt,
                            const int32_t* model_draft, const int32_t* model_len, float* features,
                            float* score, int32_t* select, int32_t* sel_draft, int32_t* sel_len,
                            void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (B < 1 || B > ctx->cfg.max_batch) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_score_select: B outside [1, max_batch]");
    if (!ctx->has_predictor) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_score_select: call hvd_set_predictor first");
    if (!hist_len || !prompt_len || !state || !K || !draft || !draft_len || !match_len || !match_pos ||
        !match_cnt || !score || !select || !sel_draft || !sel_len)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_score_select: NULL pointer");
    if ((model_draft == nullptr) != (model_len == nullptr))
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_score_select: model_draft and model_len go together");
    if (!aligned(state, 8)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_score_select: state must be 8-byte aligned");
    return launch_score_select(ctx, B, hist_len, prompt_len, state, K, draft, draft_len, match_len,
                               match_pos, match_cnt, model_draft, model_len, features, score, select,
                               sel_draft, sel_len, static_cast<cudaStream_t>(stream));
}

hvd_status hvd_score_select_ext(hvd_ctx* ctx, int32_t B, const int32_t* hist_len, const int32_t* prompt_len,
                                const hvd_req_state* state, const int32_t* K, const int32_t* draft,
                                const int32_t* draft_len, const int32_t* match_len, const int32_t* match_pos,
                                const int32_t* match_cnt, const int32_t* match_src, const float* suffix_score,
                                const int32_t* model_draft, const int32_t* model_len, float* features, float* score,
                                int32_t* select, int32_t* sel_draft, int32_t* sel_len, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (B < 1 || B > ctx->cfg.max_batch) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_score_select_ext: B outside [1, max_batch]");
    if (!ctx->has_predictor_ext) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_score_select_ext: call hvd_set_predictor_ext first");
    if (!ctx->cls) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_score_select_ext: call hvd_set_token_classes first");
    if (!hist_len || !prompt_len || !state || !K || !draft || !draft_len || !match_len || !match_pos ||
        !match_cnt || !score || !select || !sel_draft || !sel_len)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_score_select_ext: NULL pointer");
    if ((model_draft == nullptr) != (model_len == nullptr))
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_score_select_ext: model_draft and model_len go together");
    if (!aligned(state, 8)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_score_select_ext: state must be 8-byte aligned");
    return launch_score_select_ext(ctx, B, hist_len, prompt_len, state, K, draft, draft_len, match_len, match_pos,
                                   match_cnt, match_src, suffix_score, model_draft, model_len, features, score, select,
                                   sel_draft, sel_len, static_cast<cudaStream_t>(stream));
}

static hvd_status verify_commit_impl(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V,
                             const int64_t* row_off, int32_t k_uniform, int64_t total_rows,
                             const int32_t* sel_draft, const int32_t* sel_len, const int32_t* parent, const int32_t* select,
                             int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                             int32_t* hist_len, hvd_req_state* state, int32_t* accepted,
                             int32_t* committed, int32_t* n_commit, int32_t* target_tok,
                             int32_t* status, void* stream, const hvd_next_cycle* next = nullptr, bool prefix = false,
                             unsigned long long* rows_read = nullptr, VerifyArgs* args_only = nullptr) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (B < 1 || B > ctx->cfg.max_batch) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit: B outside [1, max_batch]");
    if (dtype != HVD_F32 && dtype != HVD_BF16) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit: unknown dtype");
    if (V < 1 || V > ctx->cfg.max_vocab) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit: V outside [1, max_vocab]");
    if (!logits || !sel_draft || !sel_len || !select || !hist || !hist_off || !hist_cap || !hist_len ||
        !state || !accepted || !committed || !n_commit || !status)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit: NULL pointer");
    const size_t esz = dtype == HVD_F32 ? 4 : 2;
    if (!aligned(logits, esz)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit: logits not aligned to its element type");
    if (!aligned(state, 8)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit: state must be 8-byte aligned");
    if (!row_off) {
        if (k_uniform < 0 || k_uniform > ctx->cfg.k_cap)
            return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit: k_uniform outside [0, k_cap]");
        if (total_rows != (int64_t)B * (k_uniform + 1))
            return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit: total_rows != B*(k_uniform+1)");
    }
    if (total_rows < 1 || total_rows > ctx->cfg.max_rows)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit: total_rows outside [1, max_rows]");

    VerifyArgs a;
    a.B = B; a.logits = logits; a.V = V; a.row_off = row_off; a.k_uniform = k_uniform;
    a.sel_draft = sel_draft; a.sel_len = sel_len; a.parent = parent; a.select = select;
    a.hist = hist; a.hist_off = hist_off; a.hist_cap = hist_cap; a.hist_len = hist_len; a.state = state;
    a.accepted = accepted; a.committed = committed; a.n_commit = n_commit; a.target_tok = target_tok;
    a.status = status; a.k_cap = ctx->cfg.k_cap;
    
    a.next_unit = ctx->vf_next_unit; a.dev_error = ctx->dev_error;
    a.row_key = ctx->vf_row_key; a.total_rows = total_rows; a.ext_keys = nullptr;
    if (args_only) { *args_only = a; return HVD_OK; }
    if (prefix) {
        a.rows_read = rows_read;
        return launch_verify_prefix(ctx, a, dtype, static_cast<cudaStream_t>(stream));
    }
    if (!next) return launch_verify(ctx, a, dtype, static_cast<cudaStream_t>(stream));

    // with the next cycle's lookup and scoring behind the commit
    if (!ctx->has_predictor) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit_next: call hvd_set_predictor first");
    if (!next->K || !next->prompt_len || !next->draft || !next->draft_len || !next->match_len || !next->match_pos ||
        !next->match_cnt || !next->score || !next->select || !next->sel_draft || !next->sel_len)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit_next: NULL pointer in next");
    if ((next->model_draft == nullptr) != (next->model_len == nullptr))
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit_next: model_draft and model_len go together");
    if (!aligned(hist, 16)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit_next: hist must be 16-byte aligned");
    if (next->n_max < 0 || next->n_max > ctx->cfg.max_hist_len)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit_next: n_max outside [0, max_hist_len]");
    if (ctx->two_layer || !cycle_fits_one_cta(next->n_max)) {
        const hvd_status r = launch_verify(ctx, a, dtype, static_cast<cudaStream_t>(stream));
        if (r != HVD_OK) return r;
        return hvd_lookup_score_select(ctx, B, hist, hist_off, hist_cap, hist_len, next->K, next->n_max, next->prompt_len,
                                       state, next->model_draft, next->model_len, next->draft, next->draft_len,
                                       next->match_len, next->match_pos, next->match_cnt, next->features, next->score,
                                       next->select, next->sel_draft, next->sel_len, stream);
    }
    const hvd_status r = launch_verify(ctx, a, dtype, static_cast<cudaStream_t>(stream), false);
    if (r != HVD_OK) return r;
    const ScoreArgs sa = make_score_args(ctx, B, hist_len, next->prompt_len, state, next->K, next->draft, next->draft_len,
                                         next->match_len, next->match_pos, next->match_cnt, next->model_draft,
                                         next->model_len, next->features, next->score, next->select, next->sel_draft,
                                         next->sel_len);
    return launch_commit_lookup(ctx, a, next->K, next->n_max, next->draft, next->draft_len, next->match_len,
                                next->match_pos, next->match_cnt, sa, static_cast<cudaStream_t>(stream));
}

hvd_status hvd_verify_commit(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V,
                             const int64_t* row_off, int32_t k_uniform, int64_t total_rows,
                             const int32_t* sel_draft, const int32_t* sel_len, const int32_t* select,
                             int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                             int32_t* hist_len, hvd_req_state* state, int32_t* accepted,
                             int32_t* committed, int32_t* n_commit, int32_t* target_tok,
                             int32_t* status, void* stream) {
    return verify_commit_impl(ctx, B, logits, dtype, V, row_off, k_uniform, total_rows, sel_draft, sel_len, nullptr,
                              select, hist, hist_off, hist_cap, hist_len, state, accepted, committed, n_commit,
                              target_tok, status, stream);
}

extern "C++" {
namespace hvd {
hvd_status make_verify_args(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V, const int64_t* row_off,
                            int32_t k_uniform, int64_t total_rows, const int32_t* sel_draft, const int32_t* sel_len,
                            const int32_t* select, int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                            int32_t* hist_len, hvd_req_state* state, int32_t* accepted, int32_t* committed,
                            int32_t* n_commit, int32_t* status, VerifyArgs* out) {
    return verify_commit_impl(ctx, B, logits, dtype, V, row_off, k_uniform, total_rows, sel_draft, sel_len, nullptr, select,
                              hist, hist_off, hist_cap, hist_len, state, accepted, committed, n_commit, nullptr, status,
                              nullptr, nullptr, false, nullptr, out);
}
}  // namespace hvd
}  // extern "C++"

hvd_status hvd_verify_commit_prefix(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V,
                                    const int64_t* row_off, int32_t k_uniform, int64_t total_rows,
                                    const int32_t* sel_draft, const int32_t* sel_len, const int32_t* select,
                                    int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                                    int32_t* hist_len, hvd_req_state* state, int32_t* accepted,
                                    int32_t* committed, int32_t* n_commit, uint64_t* rows_read,
                                    int32_t* status, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (rows_read && !aligned(rows_read, 8)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit_prefix: rows_read must be 8-byte aligned");
    return verify_commit_impl(ctx, B, logits, dtype, V, row_off, k_uniform, total_rows, sel_draft, sel_len, nullptr,
                              select, hist, hist_off, hist_cap, hist_len, state, accepted, committed, n_commit,
                              nullptr, status, stream, nullptr, true, reinterpret_cast<unsigned long long*>(rows_read));
}

hvd_status hvd_verify_commit_next(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V,
                                  const int64_t* row_off, int32_t k_uniform, int64_t total_rows,
                                  const int32_t* sel_draft, const int32_t* sel_len, const int32_t* select,
                                  int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                                  int32_t* hist_len, hvd_req_state* state, int32_t* accepted,
                                  int32_t* committed, int32_t* n_commit, int32_t* target_tok,
                                  int32_t* status, const hvd_next_cycle* next, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (!next) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit_next: NULL pointer");
    return verify_commit_impl(ctx, B, logits, dtype, V, row_off, k_uniform, total_rows, sel_draft, sel_len, nullptr,
                              select, hist, hist_off, hist_cap, hist_len, state, accepted, committed, n_commit,
                              target_tok, status, stream, next);
}

hvd_status hvd_verify_commit_tree(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V,
                                  const int64_t* row_off, int32_t k_uniform, int64_t total_rows,
                                  const int32_t* sel_draft, const int32_t* sel_len, const int32_t* parent,
                                  const int32_t* select, int32_t* hist, const int64_t* hist_off,
                                  const int32_t* hist_cap, int32_t* hist_len, hvd_req_state* state,
                                  int32_t* accepted, int32_t* committed, int32_t* n_commit, int32_t* target_tok,
                                  int32_t* status, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (!parent) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit_tree: NULL parent");
    return verify_commit_impl(ctx, B, logits, dtype, V, row_off, k_uniform, total_rows, sel_draft, sel_len, parent,
                              select, hist, hist_off, hist_cap, hist_len, state, accepted, committed, n_commit,
                              target_tok, status, stream);
}

// shared checks of the two calls that split verification across vocabulary shards
static hvd_status check_rows(hvd_ctx* ctx, const char* who, int32_t B, const int64_t* row_off, int32_t k_uniform,
                             int64_t total_rows) {
    if (B < 1 || B > ctx->cfg.max_batch) return fail(ctx, HVD_ERR_INVALID_ARG, "B outside [1, max_batch]");
    if (!row_off) {
        if (k_uniform < 0 || k_uniform > ctx->cfg.k_cap) return fail(ctx, HVD_ERR_INVALID_ARG, "k_uniform outside [0, k_cap]");
        if (total_rows != (int64_t)B * (k_uniform + 1)) return fail(ctx, HVD_ERR_INVALID_ARG, "total_rows != B*(k_uniform+1)");
    }
    if (total_rows < 1 || total_rows > ctx->cfg.max_rows) return fail(ctx, HVD_ERR_INVALID_ARG, "total_rows outside [1, max_rows]");
    (void)who;
    return HVD_OK;
}

hvd_status hvd_verify_keys(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V_shard, int64_t v_offset,
                           const int64_t* row_off, int32_t k_uniform, int64_t total_rows, const int32_t* sel_len,
                           const int32_t* hist_len, const int32_t* hist_cap, int64_t* keys, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    const hvd_status c = check_rows(ctx, "hvd_verify_keys", B, row_off, k_uniform, total_rows);
    if (c != HVD_OK) return c;
    if (dtype != HVD_F32 && dtype != HVD_BF16) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_keys: unknown dtype");
    if (V_shard < 1 || V_shard > ctx->cfg.max_vocab || v_offset < 0 || v_offset + V_shard > 0x7fffffffLL)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_keys: shard outside the vocabulary range");
    if (!logits || !sel_len || !hist_len || !hist_cap || !keys) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_keys: NULL pointer");
    const size_t esz = dtype == HVD_F32 ? 4 : 2;
    if (!aligned(logits, esz)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_keys: logits not aligned to its element type");
    if (!aligned(keys, 8)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_keys: keys must be 8-byte aligned");
    VerifyArgs a = {};
    a.B = B; a.logits = logits; a.V = V_shard; a.row_off = row_off; a.k_uniform = k_uniform;
    a.sel_len = sel_len; a.hist_len = const_cast<int32_t*>(hist_len); a.hist_cap = hist_cap; a.k_cap = ctx->cfg.k_cap;
    a.next_unit = ctx->vf_next_unit; a.dev_error = ctx->dev_error; a.total_rows = total_rows; a.ext_keys = nullptr;
    a.row_key = ctx->vf_row_key;
    return launch_verify_keys(ctx, a, dtype, reinterpret_cast<long long*>(keys), v_offset, static_cast<cudaStream_t>(stream));
}

hvd_status hvd_commit_keys(hvd_ctx* ctx, int32_t B, const int64_t* keys, int64_t V, const int64_t* row_off,
                           int32_t k_uniform, int64_t total_rows, const int32_t* sel_draft, const int32_t* sel_len,
                           const int32_t* select, int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                           int32_t* hist_len, hvd_req_state* state, int32_t* accepted, int32_t* committed,
                           int32_t* n_commit, int32_t* target_tok, int32_t* status, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    const hvd_status c = check_rows(ctx, "hvd_commit_keys", B, row_off, k_uniform, total_rows);
    if (c != HVD_OK) return c;
    if (V < 1 || V > 0x7fffffffLL) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_commit_keys: V outside [1, 2^31 - 1]");
    if (!keys || !sel_draft || !sel_len || !select || !hist || !hist_off || !hist_cap || !hist_len || !state ||
        !accepted || !committed || !n_commit || !status)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_commit_keys: NULL pointer");
    if (!aligned(state, 8) || !aligned(keys, 8)) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_commit_keys: state and keys must be 8-byte aligned");
    VerifyArgs a = {};
    a.B = B; a.V = V; a.row_off = row_off; a.k_uniform = k_uniform;
    a.sel_draft = sel_draft; a.sel_len = sel_len; a.parent = nullptr; a.select = select;
    a.hist = hist; a.hist_off = hist_off; a.hist_cap = hist_cap; a.hist_len = hist_len; a.state = state;
    a.accepted = accepted; a.committed = committed; a.n_commit = n_commit; a.target_tok = target_tok;
    a.status = status; a.k_cap = ctx->cfg.k_cap; a.total_rows = total_rows;
    a.ext_keys = reinterpret_cast<const long long*>(keys);
    return launch_commit_keys(ctx, a, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
