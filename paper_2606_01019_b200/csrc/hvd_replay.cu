// Payoff labels by trace replay (Sec. 3.3 "training labels"; App. B "Payoff Label Construction").
//
// Every position t of a recorded trace is a decoding state whose prefix is x[0..t); its cache draft
// is the lookup result on that prefix.  Looked at for all states at once, the lookup is a dynamic
// programme over (state t, distance delta): the match that ends delta tokens before the end of the
// prefix has length run(t, delta) = x[t-1] == x[t-1-delta] ? run(t-1, delta) + 1 : 0, capped at
// l_max, so one thread can follow one diagonal (fixed delta) through a segment of states with one
// compare per state, instead of every state scanning its whole prefix.  A thread starts a segment
// by counting back at most l_max tokens (the capped run needs no more).  The 32 diagonals of a warp
// are at the same state at the same time: per state the warp votes whether any of its runs reaches
// min_match, and only then sends its best (length, latest position) to that state's 64-bit maximum
// and the number of its diagonals at that length to the state's count for that length (only a
// warp's own maximum can be the state's maximum).  A second kernel per slice of states reads
// maximum and count, applies the draft-length rules, counts the draft tokens that the trace's own
// continuation confirms (the label equation) and clears the scratch.
// The trace is a few tens of KB and stays in L1/L2: this path is bound by integer throughput.
#include "hvd_internal.cuh"

namespace hvd {
namespace {

constexpr int kDiagThreads = 256;  // diagonals per CTA
constexpr int kSegStates = 256;    // states a thread follows its diagonal through
constexpr int kCntStride = HVD_MAX_L + 1;

struct ReplayArgs {
    const int32_t* x;
    int32_t n;
    int32_t ta, tb;  // states (prefix lengths) of this slice: ta <= t < tb
    int32_t K, l_max, min_match;
    float spec_factor, spec_offset;
    unsigned long long* key;  // [slice] (length << 32) | position, zero at rest
    uint32_t* cnt;            // [slice, kCntStride], zero at rest
    int32_t *label, *draft_len, *match_len, *match_pos, *match_cnt;  // indexed by t - 1
};

// One state of one diagonal: update the capped run, and let the warp report if any of its runs counts.
template <bool ALL_VALID>
__device__ __forceinline__ void walk_step(const ReplayArgs& a, int t, int delta, int lane, int warp_delta0, int mm,
                                          int32_t cur, int32_t shifted, int& c) {
    const bool valid = ALL_VALID || t >= delta + 1;
    if (valid) c = (cur == shifted) ? min(c + 1, a.l_max) : 0;
    const bool q = valid && c >= mm;
    if (__any_sync(0xffffffffu, q)) {
        const int cmax = __reduce_max_sync(0xffffffffu, q ? c : 0);
        const uint32_t top = __ballot_sync(0xffffffffu, q && c == cmax);
        if (lane == 0) {
            // the latest position among the warp's longest runs is the one with the smallest distance
            const int e = t - (warp_delta0 + __ffs(top) - 1);
            atomicMax(a.key + (t - a.ta), ((unsigned long long)(uint32_t)cmax << 32) | (uint32_t)e);
            atomicAdd(a.cnt + (int64_t)(t - a.ta) * kCntStride + cmax, (uint32_t)__popc(top));
        }
    }
}

__global__ void __launch_bounds__(kDiagThreads) replay_walk_kernel(const ReplayArgs a) {
    // tokens of the segment, staged once: s_cur[i] = x[s_lo - 1 + i] (the last token of state s_lo + i) and
    // s_sh[k] = x[s_lo - 1 - (delta0 + 255) + k], so that thread tid finds its shifted token of step i at
    // s_sh[i + 255 - tid]: consecutive lanes read consecutive words, with constant offsets once unrolled
    __shared__ int32_t s_cur[kSegStates];
    __shared__ int32_t s_sh[kSegStates + kDiagThreads];
    const int32_t* __restrict__ x = a.x;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int delta0 = 1 + blockIdx.x * kDiagThreads;  // smallest distance of the CTA
    const int delta = delta0 + tid;
    const int s_lo = a.ta + blockIdx.y * kSegStates;
    const int s_hi = min(a.tb, s_lo + kSegStates);
    if (delta0 + 1 >= s_hi) return;  // a state t has the diagonals delta <= t - 1
    const int steps = s_hi - s_lo;
    {
        if (tid < steps) s_cur[tid] = __ldg(x + s_lo - 1 + tid);
        const int base = s_lo - 1 - (delta0 + kDiagThreads - 1);
        for (int k = tid; k < steps + kDiagThreads - 1; k += kDiagThreads) s_sh[k] = (base + k >= 0) ? __ldg(x + base + k) : -1;
    }
    const int mm = max(a.min_match, 1);
    // capped run of the state before the first one this thread visits
    int c = 0;
    const int t_first = max(s_lo, delta + 1);
    if (t_first > delta + 1 && t_first < s_hi) {
        const int p = t_first - 2;  // last token of the state before
        while (c < a.l_max && p - delta - c >= 0 && __ldg(x + p - c) == __ldg(x + p - delta - c)) ++c;
    }
    __syncthreads();
    const int warp_delta0 = delta - lane;
    const int32_t* sh = s_sh + (kDiagThreads - 1 - tid);
    int i = 0;
    if (s_lo >= delta0 + kDiagThreads) {  // every diagonal of the CTA exists from the segment's first state on
        for (; i + 8 <= steps; i += 8) {
#pragma unroll
            for (int u = 0; u < 8; ++u)
                walk_step<true>(a, s_lo + i + u, delta, lane, warp_delta0, mm, s_cur[i + u], sh[i + u], c);
        }
        for (; i < steps; ++i) walk_step<true>(a, s_lo + i, delta, lane, warp_delta0, mm, s_cur[i], sh[i], c);
    } else {
        for (; i < steps; ++i) walk_step<false>(a, s_lo + i, delta, lane, warp_delta0, mm, s_cur[i], sh[i], c);
    }
}

__global__ void __launch_bounds__(256) replay_finish_kernel(const ReplayArgs a) {
    const int32_t* __restrict__ x = a.x;
    const int j0 = blockIdx.x * 256;
    const int j = j0 + threadIdx.x;
    const int t = a.ta + j;
    if (t < a.tb) {
        const unsigned long long key = a.key[j];
        int L = (int)(key >> 32);
        int e = (int)(uint32_t)(key & 0xffffffffu);
        int cnt = L ? (int)a.cnt[(int64_t)j * kCntStride + L] : 0;
        a.key[j] = 0ull;  // scratch is zero at rest
        int d = 0, y = 0;
        if (L < a.min_match || L == 0) {
            L = 0; e = -1; cnt = 0;
        } else {
            d = min(draft_limit(a.K, a.K, L, a.spec_factor, a.spec_offset), t - e);
            // label: draft tokens x[e .. e+d) that the trace's continuation x[t ..) confirms
            while (y < d && t + y < a.n && x[e + y] == x[t + y]) ++y;
        }
        a.label[t - 1] = y; a.draft_len[t - 1] = d; a.match_len[t - 1] = L; a.match_pos[t - 1] = e;
        a.match_cnt[t - 1] = cnt;
    }
    __syncthreads();  // every count of this CTA's states has been read
    const int states = min(256, a.tb - a.ta - j0);
    for (int i = threadIdx.x; i < states * kCntStride; i += 256) a.cnt[(int64_t)j0 * kCntStride + i] = 0u;
}

}  // namespace

hvd_status launch_replay(hvd_ctx* ctx, const int32_t* trace, int32_t n, int32_t K, int32_t* label, int32_t* draft_len,
                         int32_t* match_len, int32_t* match_pos, int32_t* match_cnt, cudaStream_t stream) {
    // per-state scratch for the whole trace, grown on demand (zero at rest: the finishing kernel clears it)
    if ((int64_t)n > ctx->rp_states) {
        HVD_CUDA_TRY(ctx, cudaStreamSynchronize(stream));
        cudaFree(ctx->rp_key); cudaFree(ctx->rp_cnt);
        ctx->rp_key = nullptr; ctx->rp_cnt = nullptr; ctx->rp_states = 0;
        cudaError_t e = cudaMalloc(&ctx->rp_key, (size_t)n * sizeof(unsigned long long));
        if (e == cudaSuccess) e = cudaMalloc(&ctx->rp_cnt, (size_t)n * kCntStride * sizeof(uint32_t));
        if (e == cudaSuccess) e = cudaMemsetAsync(ctx->rp_key, 0, (size_t)n * sizeof(unsigned long long), stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(ctx->rp_cnt, 0, (size_t)n * kCntStride * sizeof(uint32_t), stream);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            cudaFree(ctx->rp_key); cudaFree(ctx->rp_cnt);
            ctx->rp_key = nullptr; ctx->rp_cnt = nullptr;
            return fail(ctx, HVD_ERR_ALLOC, "hvd_replay_labels: cannot allocate the per-state scratch");
        }
        ctx->rp_states = n;
    }
    // the walk puts one segment of kSegStates states on every grid row
    if ((int64_t)n > 65535LL * kSegStates)
        return fail(ctx, HVD_ERR_UNSUPPORTED, "hvd_replay_labels: traces beyond 65535 * 256 positions are not supported");
    ReplayArgs a;
    a.x = trace; a.n = n; a.K = K; a.l_max = ctx->cfg.l_max; a.min_match = ctx->cfg.min_match;
    a.spec_factor = ctx->cfg.spec_factor; a.spec_offset = ctx->cfg.spec_offset;
    a.key = ctx->rp_key; a.cnt = ctx->rp_cnt;
    a.label = label; a.draft_len = draft_len; a.match_len = match_len; a.match_pos = match_pos; a.match_cnt = match_cnt;
    a.ta = 1; a.tb = n + 1;  // all states of the trace in one pair of launches
    if (n >= 2) {            // states below 2 have no diagonal
        const dim3 grid((unsigned)((n - 1 + kDiagThreads - 1) / kDiagThreads), (unsigned)((n + kSegStates - 1) / kSegStates));
        replay_walk_kernel<<<grid, kDiagThreads, 0, stream>>>(a);
        HVD_CUDA_TRY(ctx, cudaGetLastError());
    }
    replay_finish_kernel<<<(n + 255) / 256, 256, 0, stream>>>(a);
    HVD_CUDA_TRY(ctx, cudaGetLastError());
    return HVD_OK;
}

}  // namespace hvd
