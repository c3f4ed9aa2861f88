// Payoff features, predictor and draft selection (Sec. 3.3, Sec. 3.4, App. B feature groups).
//
// One warp per request.  The work is a few hundred flops per request, far too small and too
// irregular for tensor cores: lane j evaluates hidden unit j (and j+32, ...) with a left-to-right
// chain of fused multiply-adds, lane 0 then accumulates the output layer in unit order, so the fp32
// result does not depend on the launch shape.
#include "hvd_internal.cuh"

namespace hvd {
namespace {

constexpr int kWarpsPerBlock = 4;

struct ScoreArgs {
    int32_t B;
    const int32_t* hist_len;
    const int32_t* prompt_len;
    const hvd_req_state* state;
    const int32_t* K;
    const int32_t* draft;
    const int32_t* draft_len;
    const int32_t* match_len;
    const int32_t* match_pos;
    const int32_t* match_cnt;
    const int32_t* model_draft;
    const int32_t* model_len;
    float* features;
    float* score;
    int32_t* select;
    int32_t* sel_draft;
    int32_t* sel_len;
    const float* W1;
    const float* b1;
    const float* W2;
    float b2, tau;
    int32_t hidden, k_cap;
};

__device__ __forceinline__ int bit_width(uint32_t x) { return 32 - __clz((int)x); }

__global__ void __launch_bounds__(kWarpsPerBlock * 32) score_select_kernel(const ScoreArgs a) {
    __shared__ float s_hid[kWarpsPerBlock][HVD_MAX_HIDDEN];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int b = blockIdx.x * kWarpsPerBlock + warp;
    pdl_trigger();
    pdl_wait();
    if (b >= a.B) return;

    int n = a.hist_len[b];
    n = max(n, 0);
    const int P = max(a.prompt_len[b], 0);
    const hvd_req_state st = a.state[b];
    const int kc = a.k_cap;
    const int K = max(0, min(a.K[b], kc));
    const int d = max(0, min(a.draft_len[b], kc));
    const int L = a.match_len[b];
    const int pos = a.match_pos[b];
    const int cnt = max(a.match_cnt[b], 0);

    float phi[HVD_N_FEATURES];
    phi[0] = (float)L;
    phi[1] = (float)d;
    phi[2] = (float)bit_width((uint32_t)cnt);
    phi[3] = (pos < 0 || n == 0) ? 0.0f : __fdiv_rn((float)(n - pos), (float)n);
    phi[4] = (float)bit_width((uint32_t)P);
    phi[5] = (n == 0) ? 0.0f : __fdiv_rn((float)(n - P), (float)n);
    phi[6] = __fdiv_rn((float)__popc(st.sel_bits & 0xFFu), 8.0f);
    // sum of the eight bytes of the accepted-length ring
    uint64_t r = st.acc_ring;
    r = (r & 0x00FF00FF00FF00FFull) + ((r >> 8) & 0x00FF00FF00FF00FFull);
    r = (r & 0x0000FFFF0000FFFFull) + ((r >> 16) & 0x0000FFFF0000FFFFull);
    const int acc_sum = (int)((r & 0xFFFFFFFFull) + (r >> 32));
    phi[7] = __fdiv_rn((float)acc_sum, 8.0f);

    if (a.features && lane < HVD_N_FEATURES) {
        float v = phi[0];
#pragma unroll
        for (int i = 1; i < HVD_N_FEATURES; ++i) v = (lane == i) ? phi[i] : v;
        a.features[(int64_t)b * HVD_N_FEATURES + lane] = v;
    }

    for (int j = lane; j < a.hidden; j += 32) {
        float acc = a.b1[j];
        const float* w = a.W1 + (int64_t)j * HVD_N_FEATURES;
#pragma unroll
        for (int i = 0; i < HVD_N_FEATURES; ++i) acc = __fmaf_rn(w[i], phi[i], acc);
        s_hid[warp][j] = acc > 0.0f ? acc : 0.0f;
    }
    __syncwarp();
    float y = a.b2;
    if (lane == 0) {
        for (int j = 0; j < a.hidden; ++j) y = __fmaf_rn(a.W2[j], s_hid[warp][j], y);
    }
    y = __shfl_sync(0xffffffffu, y, 0);
    const int sel = (d > 0 && y >= a.tau) ? 1 : 0;

    int m;
    const int32_t* src;
    if (sel) {
        m = d;
        src = a.draft + (int64_t)b * kc;
    } else {
        m = 0;
        src = nullptr;
        if (a.model_draft && a.model_len) {
            m = max(0, min(a.model_len[b], K));
            src = a.model_draft + (int64_t)b * kc;
        }
    }
    for (int j = lane; j < kc; j += 32) a.sel_draft[(int64_t)b * kc + j] = (j < m) ? src[j] : -1;
    if (lane == 0) {
        a.score[b] = y;
        a.select[b] = sel;
        a.sel_len[b] = m;
    }
}

}  // namespace

hvd_status launch_score_select(hvd_ctx* ctx, int32_t B, const int32_t* hist_len,
                               const int32_t* prompt_len, const hvd_req_state* state, const int32_t* K,
                               const int32_t* draft, const int32_t* draft_len, const int32_t* match_len,
                               const int32_t* match_pos, const int32_t* match_cnt,
                               const int32_t* model_draft, const int32_t* model_len, float* features,
                               float* score, int32_t* select, int32_t* sel_draft, int32_t* sel_len,
                               cudaStream_t stream) {
    ScoreArgs a;
    a.B = B; a.hist_len = hist_len; a.prompt_len = prompt_len; a.state = state; a.K = K;
    a.draft = draft; a.draft_len = draft_len; a.match_len = match_len; a.match_pos = match_pos;
    a.match_cnt = match_cnt; a.model_draft = model_draft; a.model_len = model_len;
    a.features = features; a.score = score; a.select = select; a.sel_draft = sel_draft;
    a.sel_len = sel_len;
    a.W1 = ctx->d_W1; a.b1 = ctx->d_b1; a.W2 = ctx->d_W2; a.b2 = ctx->b2; a.tau = ctx->tau;
    a.hidden = ctx->cfg.hidden; a.k_cap = ctx->cfg.k_cap;
    const int blocks = (B + kWarpsPerBlock - 1) / kWarpsPerBlock;
    HVD_CUDA_TRY(ctx, launch_kernel(ctx->use_pdl, score_select_kernel, blocks, kWarpsPerBlock * 32, 0, stream, a));
    return HVD_OK;
}

}  // namespace hvd
