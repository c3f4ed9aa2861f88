// Payoff features, predictor and draft selection for ONE request, by one warp (Sec. 3.3, 3.4,
// App. B feature groups).  Shared by the stand-alone kernel and by the lookup kernel's fused tail.
#pragma once

#include "hvd_internal.cuh"

namespace hvd {

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
    const float* WhT;  // second hidden layer, transposed: WhT[i][j] = Wh[j][i]; NULL = one layer
    const float* bh;
    // extended feature vector only: token-class bits per vocabulary entry, optional suffix scores
    const uint8_t* cls;
    int32_t cls_V;
    const float* suffix;
    const int32_t* match_src;  // may be NULL; 1 = the match lies in the shared corpus (recency position 0)
};

constexpr int kW1StrideExt = 16;  // row stride of the first layer's weights for the extended vector
template <bool EXT>
struct NFeat { static constexpr int value = EXT ? (int)HVD_N_FEATURES_EXT : (int)HVD_N_FEATURES; };

__device__ __forceinline__ int bit_width(uint32_t x) { return 32 - __clz((int)x); }

// phi[8] of one request from its lookup results and decode state (every operation is an exact
// integer->float conversion or one correctly rounded IEEE operation).
template <int N>
__device__ __forceinline__ void payoff_features(const ScoreArgs& a, int b, int n, int d, int L, int pos, int cnt,
                                                float (&phi)[N], const hvd_req_state* state_now = nullptr,
                                                const int* prompt_now = nullptr) {
    n = max(n, 0);
    // read-only inputs go through the non-coherent path so that the compiler may issue them early
    const int P = max(prompt_now ? *prompt_now : __ldg(a.prompt_len + b), 0);
    hvd_req_state st;
    if (state_now) {  // the caller has just updated the summary itself
        st = *state_now;
    } else {
        st.sel_bits = __ldg(&a.state[b].sel_bits);
        st.acc_ring = __ldg(reinterpret_cast<const unsigned long long*>(&a.state[b].acc_ring));
    }
    cnt = max(cnt, 0);
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
}

// hidden unit j of the first layer: relu(b1[j] + sum_i W1[j][i] phi[i]), left to right.  The weights
// can be fetched ahead of the features (load_first_layer) and applied later (apply_first_layer).
template <int N>
struct FirstLayerRow {
    static constexpr int STRIDE = (N == HVD_N_FEATURES) ? HVD_N_FEATURES : kW1StrideExt;  // 32- or 64-byte rows
    float w[STRIDE];
    float bias;
};

template <int N>
__device__ __forceinline__ FirstLayerRow<N> load_first_layer(const ScoreArgs& a, int j) {
    FirstLayerRow<N> row;
    row.bias = __ldg(a.b1 + j);
    const float4* w4 = reinterpret_cast<const float4*>(a.W1 + (int64_t)j * FirstLayerRow<N>::STRIDE);
#pragma unroll
    for (int q = 0; q < FirstLayerRow<N>::STRIDE / 4; ++q) {
        const float4 v = __ldg(w4 + q);
        row.w[4 * q] = v.x; row.w[4 * q + 1] = v.y; row.w[4 * q + 2] = v.z; row.w[4 * q + 3] = v.w;
    }
    return row;
}

template <int N>
__device__ __forceinline__ float apply_first_layer(const FirstLayerRow<N>& row, const float (&phi)[N]) {
    float acc = row.bias;
#pragma unroll
    for (int i = 0; i < N; ++i) acc = __fmaf_rn(row.w[i], phi[i], acc);
    return acc > 0.0f ? acc : 0.0f;
}

template <int N>
__device__ __forceinline__ float first_layer_unit(const ScoreArgs& a, int j, const float (&phi)[N]) {
    return apply_first_layer(load_first_layer<N>(a, j), phi);
}

// Draft-structure group and suffix score of the extended vector (App. B feature groups), by one
// converged warp: the share of the draft's tokens in each of five token classes (one IEEE division
// count / d), then the caller's suffix score.  tok0 / tok1: draft tokens lane and lane + 32.
__device__ __forceinline__ void structure_features(const ScoreArgs& a, int b, int lane, int d, int tok0, int tok1,
                                                   float (&phi)[HVD_N_FEATURES_EXT]) {
    uint32_t c0 = 0, c1 = 0;
    if (lane < d && tok0 >= 0 && tok0 < a.cls_V) c0 = __ldg(a.cls + tok0);
    if (lane + 32 < d && tok1 >= 0 && tok1 < a.cls_V) c1 = __ldg(a.cls + tok1);
#pragma unroll
    for (int k = 0; k < HVD_N_TOKEN_CLASSES; ++k) {
        const int cnt = __popc(__ballot_sync(0xffffffffu, (c0 >> k) & 1u)) + __popc(__ballot_sync(0xffffffffu, (c1 >> k) & 1u));
        phi[HVD_N_FEATURES + k] = d > 0 ? __fdiv_rn((float)cnt, (float)d) : 0.0f;
    }
    phi[HVD_N_FEATURES + HVD_N_TOKEN_CLASSES] = a.suffix ? __ldg(a.suffix + b) : 0.0f;
}

// Selection rule and the selected draft, by one warp.  tok0 / tok1: cache draft tokens lane and
// lane+32 (-1 beyond the draft).  The model draft's length and tokens can be fetched ahead of the
// score (load_model_draft).
struct ModelDraft {
    int m;       // usable length of the model draft (0 without one)
    int t0, t1;  // its tokens lane and lane + 32 (-1 beyond m)
};

__device__ __forceinline__ ModelDraft load_model_draft(const ScoreArgs& a, int b, int lane) {
    ModelDraft md;
    md.m = 0; md.t0 = -1; md.t1 = -1;
    if (a.model_draft && a.model_len) {
        const int kc = a.k_cap;
        const int K = max(0, min(__ldg(a.K + b), kc));
        md.m = max(0, min(__ldg(a.model_len + b), K));
        const int32_t* src = a.model_draft + (int64_t)b * kc;
        if (lane < md.m) md.t0 = __ldg(src + lane);
        if (lane + 32 < md.m) md.t1 = __ldg(src + lane + 32);
    }
    return md;
}

__device__ __forceinline__ void select_draft(const ScoreArgs& a, int b, int lane, float y, int d, int tok0, int tok1,
                                             const ModelDraft& md) {
    const int kc = a.k_cap;
    const int sel = (d > 0 && y >= a.tau) ? 1 : 0;
    int m = d;
    if (!sel) { m = md.m; tok0 = md.t0; tok1 = md.t1; }
    if (lane < kc) a.sel_draft[(int64_t)b * kc + lane] = (lane < m) ? tok0 : -1;
    if (lane + 32 < kc) a.sel_draft[(int64_t)b * kc + lane + 32] = (lane + 32 < m) ? tok1 : -1;
    if (lane == 0) {
        a.score[b] = y;
        a.select[b] = sel;
        a.sel_len[b] = m;
    }
}

__device__ __forceinline__ void select_draft(const ScoreArgs& a, int b, int lane, float y, int d, int tok0, int tok1) {
    const int sel = (d > 0 && y >= a.tau) ? 1 : 0;
    ModelDraft md;
    md.m = 0; md.t0 = -1; md.t1 = -1;
    if (!sel) md = load_model_draft(a, b, lane);  // only fetched when it is the one verified
    select_draft(a, b, lane, y, d, tok0, tok1, md);
}

// One-hidden-layer predictor for one request by one warp.  The work is a few hundred flops per
// request, far too small and too irregular for tensor cores: lane j evaluates hidden unit j (and
// j+32, ...) with a left-to-right chain of fused multiply-adds, lane 0 then accumulates the output
// layer in unit order, so the fp32 result does not depend on the launch shape.  d, L, pos, cnt: the
// lookup results of the request; s_hid: shared memory, a.hidden floats, private to the warp.
template <bool EXT = false>
__device__ __forceinline__ void score_select_request(const ScoreArgs& a, int b, int lane, float* s_hid, int n,
                                                     int d, int L, int pos, int cnt, int tok0, int tok1,
                                                     const ModelDraft* fetched = nullptr,
                                                     const hvd_req_state* state_now = nullptr,
                                                     const int* prompt_now = nullptr) {
    constexpr int N = NFeat<EXT>::value;
    d = max(0, min(d, a.k_cap));
    float phi[N];
    payoff_features(a, b, n, d, L, pos, cnt, phi, state_now, prompt_now);
    if constexpr (EXT) structure_features(a, b, lane, d, tok0, tok1, phi);
    if (a.features && lane < N) {
        float v = phi[0];
#pragma unroll
        for (int i = 1; i < N; ++i) v = (lane == i) ? phi[i] : v;
        a.features[(int64_t)b * N + lane] = v;
    }
    for (int j = lane; j < a.hidden; j += 32) s_hid[j] = first_layer_unit(a, j, phi);
    __syncwarp();
    float y = a.b2;
    if (lane == 0) {
        for (int j = 0; j < a.hidden; ++j) y = __fmaf_rn(__ldg(a.W2 + j), s_hid[j], y);
    }
    y = __shfl_sync(0xffffffffu, y, 0);
    if (fetched) select_draft(a, b, lane, y, d, tok0, tok1, *fetched);  // the model draft was fetched ahead
    else select_draft(a, b, lane, y, d, tok0, tok1);
}

}  // namespace hvd
