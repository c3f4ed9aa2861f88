// Payoff features, predictor and draft selection (Sec. 3.3, Sec. 3.4, App. B feature groups).
//
// Stand-alone kernel: one warp per request (the per-request arithmetic is in hvd_score.cuh).
#include "hvd_score.cuh"

namespace hvd {
namespace {

constexpr int kWarpsPerBlock = 4;

template <bool EXT>
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
    int pos = a.match_pos[b];
    if (EXT && a.match_src && a.match_src[b] == 1) pos = 0;
    score_select_request<EXT>(a, b, lane, s_hid[warp], a.hist_len[b], d, a.match_len[b], pos, a.match_cnt[b], tok0, tok1);
}

// Two hidden layers (the paper's predictor shape, 2 x 256).  One CTA scores kReqPerCta (4) requests:
// the second layer's 256 KB of weights are the traffic that matters, and every request a CTA
// handles reuses the tile it has staged.  Thread j evaluates unit j of each layer, for each of the
// CTA's requests, with the same left-to-right fused multiply-add chains as the one-layer kernel
// (64 K multiply-adds per request: still far from a tensor-core shape at batch sizes of tens to
// hundreds, and a sequential order keeps the result independent of the launch).  The second
// layer's weights are stored transposed with a row stride of HVD_MAX_HIDDEN (WhT[i][j] = Wh[j][i])
// and are staged through shared memory with asynchronous 16-byte copies, two tiles of kTileRows
// rows in flight, so that the chains never wait for a global load.
constexpr int kScore2Threads = HVD_MAX_HIDDEN;
constexpr int kReqPerCta = 4;  // requests per CTA: one float4 of first-layer activations per input unit
constexpr int kTileRows = 64;
constexpr int kTileFloats = kTileRows * HVD_MAX_HIDDEN;
constexpr int kHidPad = HVD_MAX_HIDDEN + 1;  // row stride of the second-layer activations
constexpr size_t kScore2Smem = 2 * (size_t)kTileFloats * sizeof(float);  // 128 KB

__device__ __forceinline__ void copy_tile_async(float* dst, const float* src, int tid) {
    // kTileFloats floats = 4096 x 16 bytes, 16 per thread
    const uint32_t d0 = (uint32_t)__cvta_generic_to_shared(dst);
#pragma unroll
    for (int k = 0; k < kTileFloats / 4 / kScore2Threads; ++k) {
        const int v = k * kScore2Threads + tid;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d0 + v * 16), "l"(src + v * 4) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

template <bool EXT>
__global__ void __launch_bounds__(kScore2Threads) score_select2_kernel(const ScoreArgs a) {
    constexpr int N = NFeat<EXT>::value;
    extern __shared__ __align__(16) float s_tiles[];  // [2][kTileRows][HVD_MAX_HIDDEN]
    __shared__ float s_phi[kReqPerCta][N];
    __shared__ __align__(16) float s_h1[HVD_MAX_HIDDEN][kReqPerCta];  // [input unit][request]
    __shared__ float s_h2[kReqPerCta][kHidPad];
    __shared__ float s_w2[HVD_MAX_HIDDEN];
    __shared__ float s_y[kReqPerCta];
    __shared__ int s_d[kReqPerCta];
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int b0 = blockIdx.x * kReqPerCta;
    const int nreq = min(kReqPerCta, a.B - b0);
    const int kc = a.k_cap;
    const int H = a.hidden;
    const int n_tiles = (H + kTileRows - 1) / kTileRows;
    // the weights do not depend on the previous kernel: their first tiles are requested at once
    copy_tile_async(s_tiles, a.WhT, tid);
    if (n_tiles > 1) copy_tile_async(s_tiles + kTileFloats, a.WhT + kTileFloats, tid);
    if (tid < H) s_w2[tid] = __ldg(a.W2 + tid);
    pdl_trigger();
    pdl_wait();
    // features: warp r for request b0 + r
    if (warp < nreq) {
        const int b = b0 + warp;
        const int d = max(0, min(a.draft_len[b], kc));
        float phi[N];
        int pos = a.match_pos[b];
        if (EXT && a.match_src && a.match_src[b] == 1) pos = 0;
        payoff_features(a, b, a.hist_len[b], d, a.match_len[b], pos, a.match_cnt[b], phi);
        if constexpr (EXT) {
            const int32_t* src = a.draft + (int64_t)b * kc;
            structure_features(a, b, lane, d, lane < d ? src[lane] : -1, lane + 32 < d ? src[lane + 32] : -1, phi);
        }
        if (lane < N) {
            float v = phi[0];
#pragma unroll
            for (int i = 1; i < N; ++i) v = (lane == i) ? phi[i] : v;
            s_phi[warp][lane] = v;
            if (a.features) a.features[(int64_t)b * N + lane] = v;
        }
        if (lane == 0) s_d[warp] = d;
    }
    __syncthreads();
    float acc[kReqPerCta];
    if (tid < H) {
        const float bias = __ldg(a.bh + tid);
        float h1[kReqPerCta];
#pragma unroll
        for (int r = 0; r < kReqPerCta; ++r) {
            acc[r] = bias;
            h1[r] = 0.0f;
            if (r < nreq) {
                float phi[N];
#pragma unroll
                for (int i = 0; i < N; ++i) phi[i] = s_phi[r][i];
                h1[r] = first_layer_unit(a, tid, phi);
            }
        }
        *reinterpret_cast<float4*>(s_h1[tid]) = make_float4(h1[0], h1[1], h1[2], h1[3]);
    } else {
        *reinterpret_cast<float4*>(s_h1[tid]) = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    }
    for (int t = 0; t < n_tiles; ++t) {
        if (t + 1 < n_tiles) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();  // tile t has landed for every thread (and, for t = 0, s_h1 is complete)
        const float* w = s_tiles + (t & 1) * kTileFloats + tid;
        // rows beyond H hold zero weights and zero activations: adding their products changes nothing,
        // and a fixed trip count lets all the shared-memory loads of a tile be issued ahead of the chains
        if (tid < H) {
#pragma unroll 16
            for (int i = 0; i < kTileRows; ++i) {
                const float wv = w[i * HVD_MAX_HIDDEN];
                const float4 h = *reinterpret_cast<const float4*>(s_h1[t * kTileRows + i]);  // broadcast
                acc[0] = __fmaf_rn(wv, h.x, acc[0]); acc[1] = __fmaf_rn(wv, h.y, acc[1]);
                acc[2] = __fmaf_rn(wv, h.z, acc[2]); acc[3] = __fmaf_rn(wv, h.w, acc[3]);
            }
        }
        __syncthreads();  // everyone is done with this buffer
        if (t + 2 < n_tiles) copy_tile_async(s_tiles + (t & 1) * kTileFloats, a.WhT + (size_t)(t + 2) * kTileFloats, tid);
    }
    if (tid < H) {
#pragma unroll
        for (int r = 0; r < kReqPerCta; ++r) s_h2[r][tid] = acc[r] > 0.0f ? acc[r] : 0.0f;
    }
    __syncthreads();
    if (tid < nreq) {  // output layer: one sequential chain per request, operands from shared memory
        float y = a.b2;
#pragma unroll 8
        for (int j = 0; j < H; ++j) y = __fmaf_rn(s_w2[j], s_h2[tid][j], y);
        s_y[tid] = y;
    }
    __syncthreads();
    if (warp < nreq) {
        const int b = b0 + warp;
        const int d = s_d[warp];
        const int32_t* src = a.draft + (int64_t)b * kc;
        const int tok0 = lane < d ? src[lane] : -1;
        const int tok1 = lane + 32 < d ? src[lane + 32] : -1;
        select_draft(a, b, lane, s_y[warp], d, tok0, tok1);
    }
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
    a.WhT = ctx->two_layer ? ctx->d_WhT : nullptr; a.bh = ctx->d_bh;
    a.cls = nullptr; a.cls_V = 0; a.suffix = nullptr; a.match_src = nullptr;
    return a;
}

template <bool EXT>
static hvd_status launch_score_kernels(hvd_ctx* ctx, const ScoreArgs& a, int32_t B, cudaStream_t stream) {
    if (a.WhT) {
        bool& ready = EXT ? ctx->score2x_ready : ctx->score2_ready;
        if (!ready) {  // per device: the kernel needs the opt-in shared memory size
            HVD_CUDA_TRY(ctx, cudaFuncSetAttribute(score_select2_kernel<EXT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   (int)kScore2Smem));
            ready = true;
        }
        HVD_CUDA_TRY(ctx, launch_kernel(ctx->use_pdl, score_select2_kernel<EXT>, (B + kReqPerCta - 1) / kReqPerCta,
                                        kScore2Threads, kScore2Smem, stream, a));
        return HVD_OK;
    }
    const int blocks = (B + kWarpsPerBlock - 1) / kWarpsPerBlock;
    HVD_CUDA_TRY(ctx, launch_kernel(ctx->use_pdl, score_select_kernel<EXT>, blocks, kWarpsPerBlock * 32, 0, stream, a));
    return HVD_OK;
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
    return launch_score_kernels<false>(ctx, a, B, stream);
}

hvd_status launch_score_select_ext(hvd_ctx* ctx, int32_t B, const int32_t* hist_len, const int32_t* prompt_len,
                                   const hvd_req_state* state, const int32_t* K, const int32_t* draft,
                                   const int32_t* draft_len, const int32_t* match_len, const int32_t* match_pos,
                                   const int32_t* match_cnt, const int32_t* match_src, const float* suffix,
                                   const int32_t* model_draft, const int32_t* model_len, float* features, float* score,
                                   int32_t* select, int32_t* sel_draft, int32_t* sel_len, cudaStream_t stream) {
    ScoreArgs a = make_score_args(ctx, B, hist_len, prompt_len, state, K, draft, draft_len, match_len, match_pos,
                                  match_cnt, model_draft, model_len, features, score, select, sel_draft, sel_len);
    a.cls = ctx->cls; a.cls_V = ctx->cls_V; a.suffix = suffix; a.match_src = match_src;
    return launch_score_kernels<true>(ctx, a, B, stream);
}

}  // namespace hvd
