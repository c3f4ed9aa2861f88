// Payoff features, predictor and draft selection (Sec. 3.3, Sec. 3.4, App. B feature groups).
//
// Stand-alone kernel: one warp per request (the per-request arithmetic is in hvd_score.cuh).
#include "hvd_score.cuh"

namespace hvd {
namespace {

constexpr int kWarpsPerBlock = 4;

__global__ void __launch_bounds__(kWarpsPerBlock * 32) score_select_kernel(const ScoreArgs a) {
    __shared__ float s_hid[kWarpsPerBlock][HVD_MAX_HIDDEN];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int b = blockIdx.x * kWarpsPerBlock + warp;
    pdl_trigger();
    pdl_wait();
    if (b >= a.B) return;
    const int kc = a.k_cap;
    const int d = max(0, min(a.draft_len[b], kc));
    const int32_t* src = a.draft + (int64_t)b * kc;
    const int tok0 = lane < d ? src[lane] : -1;
    const int tok1 = lane + 32 < d ? src[lane + 32] : -1;
    score_select_request(a, b, lane, s_hid[warp], a.hist_len[b], d, a.match_len[b], a.match_pos[b],
                         a.match_cnt[b], tok0, tok1);
}

}  // namespace

ScoreArgs make_score_args(hvd_ctx* ctx, int32_t B, const int32_t* hist_len, const int32_t* prompt_len,
                          const hvd_req_state* state, const int32_t* K, const int32_t* draft,
                          const int32_t* draft_len, const int32_t* match_len, const int32_t* match_pos,
                          const int32_t* match_cnt, const int32_t* model_draft, const int32_t* model_len,
                          float* features, float* score, int32_t* select, int32_t* sel_draft, int32_t* sel_len) {
    ScoreArgs a;
    a.B = B; a.hist_len = hist_len; a.prompt_len = prompt_len; a.state = state; a.K = K;
    a.draft = draft; a.draft_len = draft_len; a.match_len = match_len; a.match_pos = match_pos;
    a.match_cnt = match_cnt; a.model_draft = model_draft; a.model_len = model_len;
    a.features = features; a.score = score; a.select = select; a.sel_draft = sel_draft;
    a.sel_len = sel_len;
    a.W1 = ctx->d_W1; a.b1 = ctx->d_b1; a.W2 = ctx->d_W2; a.b2 = ctx->b2; a.tau = ctx->tau;
    a.hidden = ctx->cfg.hidden; a.k_cap = ctx->cfg.k_cap;
    return a;
}

hvd_status launch_score_select(hvd_ctx* ctx, int32_t B, const int32_t* hist_len,
                               const int32_t* prompt_len, const hvd_req_state* state, const int32_t* K,
                               const int32_t* draft, const int32_t* draft_len, const int32_t* match_len,
                               const int32_t* match_pos, const int32_t* match_cnt,
                               const int32_t* model_draft, const int32_t* model_len, float* features,
                               float* score, int32_t* select, int32_t* sel_draft, int32_t* sel_len,
                               cudaStream_t stream) {
    const ScoreArgs a = make_score_args(ctx, B, hist_len, prompt_len, state, K, draft, draft_len, match_len,
                                        match_pos, match_cnt, model_draft, model_len, features, score, select,
                                        sel_draft, sel_len);
    const int blocks = (B + kWarpsPerBlock - 1) / kWarpsPerBlock;
    HVD_CUDA_TRY(ctx, launch_kernel(ctx->use_pdl, score_select_kernel, blocks, kWarpsPerBlock * 32, 0, stream, a));
    return HVD_OK;
}

}  // namespace hvd
