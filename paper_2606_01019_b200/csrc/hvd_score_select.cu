// Payoff features, predictor and draft selection (Sec. 3.3, Sec. 3.4, App. B feature groups).
//
// Stand-alone kernel: one warp per request (the per-request arithmetic is in hvd_score.cuh).
#include <cooperative_groups.h>

#include "hvd_score.cuh"

namespace cg = cooperative_groups;

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

// Two hidden layers (the paper's predictor shape, 2 x 256).  A thread-block cluster of four CTAs
// scores four requests (eight or sixteen for larger batches): CTA `rank` owns 64 of the second layer's 256 output units, so it stages only
// its 64 KB column slab of the weights (stored transposed with a row stride of HVD_MAX_HIDDEN:
// WhT[i][j] = Wh[j][i]) with asynchronous 16-byte copies issued before anything else; thread
// (request r, unit jj) runs one left-to-right chain of fused multiply-adds over the 256 inputs --
// the same order as the one-layer kernel and as a plain loop, so the fp32 result does not depend on
// the launch (64 K multiply-adds per request: far from a tensor-core shape at batch sizes of tens to
// hundreds).  The first layer is cheap and every CTA evaluates it for itself; the second layer's
// activations go to CTA 0 of the cluster through distributed shared memory, and after the cluster
// barrier CTA 0 runs the output layer (one sequential chain per request) and the selection.
constexpr int kScore2Threads = HVD_MAX_HIDDEN;
constexpr int kClusterSize = 4;
constexpr int kReqPerGroup = 4;  // requests that share a pass over the slab: thread (request, unit)
constexpr int kColsPerCta = HVD_MAX_HIDDEN / kClusterSize;
constexpr int kHidPad = HVD_MAX_HIDDEN + 1;  // row stride of the second-layer activations
constexpr size_t kScore2Smem = (size_t)HVD_MAX_HIDDEN * kColsPerCta * sizeof(float);  // 64 KB slab
static_assert(kScore2Threads == kReqPerGroup * kColsPerCta, "one thread per (request, unit) pair");

// G: groups of four requests per cluster (1, 2 or 4).  Larger batches take more requests per cluster so
// that a slab staged once serves more chains and the grid stays within one wave.
template <bool EXT, int G>
__global__ void __cluster_dims__(kClusterSize, 1, 1) __launch_bounds__(kScore2Threads)
score_select2_kernel(const ScoreArgs a) {
    constexpr int N = NFeat<EXT>::value;
    constexpr int REQ = kReqPerGroup * G;                  // requests per cluster
    constexpr int RW = (REQ + kScore2Threads / 32 - 1) / (kScore2Threads / 32);  // requests per warp
    extern __shared__ __align__(16) float s_w[];  // [HVD_MAX_HIDDEN inputs][kColsPerCta units]
    __shared__ float s_phi[REQ][N];
    __shared__ __align__(16) float s_h1[HVD_MAX_HIDDEN][REQ];  // [input unit][request]
    __shared__ float s_h2[REQ][kHidPad];                        // filled by the whole cluster in CTA 0
    __shared__ float s_w2[HVD_MAX_HIDDEN];
    __shared__ float s_y[REQ];
    __shared__ int s_d[REQ];
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    constexpr int NWARP = kScore2Threads / 32;
    const int b0 = (int)(blockIdx.x / kClusterSize) * REQ;
    const int nreq = min(REQ, a.B - b0);
    const int kc = a.k_cap;
    const int H = a.hidden;
    // "this CTA runs": matched by the wait in front of the stores into CTA 0's shared memory, which may only be
    // touched once every CTA of the cluster is known to have started (the arrival overlaps the slab copy)
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    // the weights do not depend on the previous kernel: this CTA's slab is requested at once
    {
        const uint32_t d0 = (uint32_t)__cvta_generic_to_shared(s_w);
        const float* src = a.WhT + rank * kColsPerCta;
#pragma unroll
        for (int k = 0; k < HVD_MAX_HIDDEN * kColsPerCta / 4 / kScore2Threads; ++k) {
            const int v = k * kScore2Threads + tid;       // 16-byte vector: row v / 16, vector v % 16 of the row
            const int row = v / (kColsPerCta / 4), c4 = v % (kColsPerCta / 4);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d0 + v * 16),
                         "l"(src + (size_t)row * HVD_MAX_HIDDEN + c4 * 4) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    if (tid < H) s_w2[tid] = __ldg(a.W2 + tid);
    // so are this thread's first-layer weights and its second-layer bias
    FirstLayerRow<N> row1;
    if (tid < H) row1 = load_first_layer<N>(a, tid);
    const int my_j = rank * kColsPerCta + tid % kColsPerCta;
    const float my_bh = (my_j < H) ? __ldg(a.bh + my_j) : 0.0f;
    // no early trigger here: with the streaming kernel resident behind it this kernel measured 2.4 us slower
    pdl_wait();
    // CTA 0 selects at the end: its warps fetch the drafts they will choose between now
    ModelDraft md[RW];
    int ctok0[RW], ctok1[RW];
#pragma unroll
    for (int k = 0; k < RW; ++k) {
        const int r = warp + k * NWARP;
        ctok0[k] = -1; ctok1[k] = -1;
        md[k].m = 0; md[k].t0 = -1; md[k].t1 = -1;
        if (rank == 0 && r < nreq) {
            const int b = b0 + r;
            md[k] = load_model_draft(a, b, lane);
            const int d = max(0, min(a.draft_len[b], kc));
            const int32_t* src = a.draft + (int64_t)b * kc;
            ctok0[k] = lane < d ? src[lane] : -1;
            ctok1[k] = lane + 32 < d ? src[lane + 32] : -1;
        }
    }
    // features: one warp per request (every CTA of the cluster needs them; CTA 0 writes them out)
    for (int r = warp; r < nreq; r += NWARP) {
        const int b = b0 + r;
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
            s_phi[r][lane] = v;
            if (a.features && rank == 0) a.features[(int64_t)b * N + lane] = v;
        }
        if (lane == 0) s_d[r] = d;
    }
    __syncthreads();
    {   // first layer: thread j evaluates unit j for every request of the cluster
#pragma unroll
        for (int r = 0; r < REQ; ++r) {
            float h1 = 0.0f;
            if (tid < H && r < nreq) {
                float phi[N];
#pragma unroll
                for (int i = 0; i < N; ++i) phi[i] = s_phi[r][i];
                h1 = apply_first_layer(row1, phi);
            }
            s_h1[tid][r] = h1;
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();  // the slab and s_h1 are complete
    {   // second layer: thread (r4, jj) -> unit j = rank * 64 + jj of requests r4, r4 + 4, ...
        const int r4 = tid / kColsPerCta, jj = tid % kColsPerCta;
        const int j = rank * kColsPerCta + jj;
        float acc[G];
#pragma unroll
        for (int g = 0; g < G; ++g) acc[g] = my_bh;
        // rows beyond H hold zero weights and zero activations: adding their products changes nothing,
        // and a fixed trip count lets the shared-memory loads be issued ahead of the chains
        const float* w = s_w + jj;
#pragma unroll 8
        for (int i = 0; i < HVD_MAX_HIDDEN; ++i) {
            const float wv = w[i * kColsPerCta];
#pragma unroll
            for (int g = 0; g < G; ++g) acc[g] = __fmaf_rn(wv, s_h1[i][r4 + kReqPerGroup * g], acc[g]);
        }
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");  // every CTA of the cluster has started
        float* dst = cluster.map_shared_rank(&s_h2[0][0], 0);  // CTA 0's copy
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const int r = r4 + kReqPerGroup * g;
            dst[r * kHidPad + j] = (j < H && r < nreq && acc[g] > 0.0f) ? acc[g] : 0.0f;
        }
    }
    cluster.sync();  // all four slabs of activations have arrived in CTA 0
    if (rank != 0) return;
    if (tid < nreq) {  // output layer: one sequential chain per request, operands from shared memory
        float y = a.b2;
#pragma unroll 8
        for (int j = 0; j < H; ++j) y = __fmaf_rn(s_w2[j], s_h2[tid][j], y);
        s_y[tid] = y;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < RW; ++k) {
        const int r = warp + k * NWARP;
        if (r < nreq) select_draft(a, b0 + r, lane, s_y[r], s_d[r], ctok0[k], ctok1[k], md[k]);
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
        if (!ready) {  // per device: the kernels need the opt-in shared memory size
            HVD_CUDA_TRY(ctx, cudaFuncSetAttribute(score_select2_kernel<EXT, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kScore2Smem));
            HVD_CUDA_TRY(ctx, cudaFuncSetAttribute(score_select2_kernel<EXT, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kScore2Smem));
            HVD_CUDA_TRY(ctx, cudaFuncSetAttribute(score_select2_kernel<EXT, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kScore2Smem));
            ready = true;
        }
        // (never launched ahead of its predecessor's end: resident early, the cluster kernel measured 4.6 us slower)
        // requests per cluster: 4, 8 or 16, the fewest that keep the grid within one CTA per SM
        const int G = B <= ctx->num_sms ? 1 : (B <= 2 * ctx->num_sms ? 2 : 4);
        const int clusters = (B + kReqPerGroup * G - 1) / (kReqPerGroup * G);
        const dim3 grid((unsigned)(clusters * kClusterSize));
        cudaError_t e;
        if (G == 1) e = launch_kernel(false, score_select2_kernel<EXT, 1>, grid, kScore2Threads, kScore2Smem, stream, a);
        else if (G == 2) e = launch_kernel(false, score_select2_kernel<EXT, 2>, grid, kScore2Threads, kScore2Smem, stream, a);
        else e = launch_kernel(false, score_select2_kernel<EXT, 4>, grid, kScore2Threads, kScore2Smem, stream, a);
        HVD_CUDA_TRY(ctx, e);
        return HVD_OK;
    }
    const int blocks = (B + kWarpsPerBlock - 1) / kWarpsPerBlock;
    HVD_CUDA_TRY(ctx, launch_kernel((ctx->pdl_mask & 8), score_select_kernel<EXT>, blocks, kWarpsPerBlock * 32, 0, stream, a));
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
