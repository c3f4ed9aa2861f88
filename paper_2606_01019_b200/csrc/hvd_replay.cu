// Payoff labels by trace replay (Sec. 3.3 "training labels"; App. B "Payoff Label Construction").
//
// Every position t of a recorded trace is a decoding state whose prefix is x[0..t).  All those
// states share one token array and differ only in their length, which is exactly the ragged batch
// the lookup kernel takes: a slice of states becomes a batch of "requests" with the same slab and
// hist_len = t.  A small kernel then counts how many draft tokens agree with the trace's own
// continuation (the label equation).  The trace is a few tens of KB and stays in L2: this path is
// bound by the lookup kernel's per-state latency chain, not by HBM.
#include "hvd_internal.cuh"

namespace hvd {
namespace {

__global__ void replay_setup_kernel(int32_t s0, int32_t count, int32_t n, int32_t K, int64_t* v_off, int32_t* v_cap,
                                    int32_t* v_len, int32_t* v_K) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= count) return;
    v_off[j] = 0;          // every state reads the same trace
    v_cap[j] = n;
    v_len[j] = s0 + j;     // prefix length of state j of the slice
    v_K[j] = K;
}

// label = max{ l <= draft_len : x[e .. e+l) == x[t .. t+l) }, the draft being x[e .. e+draft_len)
__global__ void replay_label_kernel(const int32_t* __restrict__ x, int32_t n, int32_t s0, int32_t count,
                                    const int32_t* __restrict__ draft_len, const int32_t* __restrict__ match_pos,
                                    int32_t* __restrict__ label) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= count) return;
    const int t = s0 + j;
    const int d = draft_len[j];
    const int e = match_pos[j];
    int y = 0;
    while (y < d && t + y < n && x[e + y] == x[t + y]) ++y;
    label[j] = y;
}

}  // namespace

hvd_status launch_replay(hvd_ctx* ctx, const int32_t* trace, int32_t n, int32_t K, int32_t* label, int32_t* draft_len,
                         int32_t* match_len, int32_t* match_pos, int32_t* match_cnt, cudaStream_t stream) {
    const int32_t slice = ctx->cfg.max_batch;
    for (int32_t s0 = 1; s0 <= n; s0 += slice) {
        const int32_t count = (n - s0 + 1) < slice ? (n - s0 + 1) : slice;
        const int32_t j0 = s0 - 1;  // outputs are indexed by t - 1
        replay_setup_kernel<<<(count + 255) / 256, 256, 0, stream>>>(s0, count, n, K, ctx->rp_off, ctx->rp_cap,
                                                                     ctx->rp_len, ctx->rp_K);
        HVD_CUDA_TRY(ctx, cudaGetLastError());
        const hvd_status r = launch_lookup(ctx, count, trace, ctx->rp_off, ctx->rp_cap, ctx->rp_len, ctx->rp_K,
                                           s0 + count - 1, ctx->rp_draft, draft_len + j0, match_len + j0,
                                           match_pos + j0, match_cnt + j0, nullptr, stream);
        if (r != HVD_OK) return r;
        replay_label_kernel<<<(count + 255) / 256, 256, 0, stream>>>(trace, n, s0, count, draft_len + j0,
                                                                     match_pos + j0, label + j0);
        HVD_CUDA_TRY(ctx, cudaGetLastError());
    }
    return HVD_OK;
}

}  // namespace hvd
