// Commit of one cycle and the cache lookup, features, score and selection of the next one in ONE kernel
// (Algorithm 1: "append z, update C and h", then the next iteration's d_c, phi, y-hat and rule).
//
// In a decoding loop the commit of cycle i is followed at once by the lookup of cycle i + 1 on the history
// it has just extended.  As separate kernels that is a commit kernel (a chain: row keys -> compare ->
// append) and then a lookup kernel (lengths -> history -> ...).  Here one CTA per request does both: every
// thread first issues its loads of the history as it stands (the commit can only append, at most
// k_cap + 1 tokens), warp 0 commits while those loads are in flight, and after one barrier the CTA scans
// with the new tail as the query; only the vectors that overlap the appended tokens are read again
// (through the L2, where warp 0's stores are).  One launch and two dependent global round trips less
// per decoding cycle.  Requests must fit one CTA (32 K tokens); the caller falls back to the two
// separate launches otherwise.  Up to 18 K tokens the CTA has 512 threads, which fit on an SM beside the
// streaming kernel's CTAs: the loads ahead of the wait then run while the logits still stream.
#include "hvd_commit.cuh"
#include "hvd_scan.cuh"
#include "hvd_score.cuh"

namespace hvd {
namespace {

struct NextArgs {
    const int32_t* K;  // [B] draft caps of the next cycle
    int32_t n_max;     // upper bound on hist_len after the commit
    int32_t* draft;
    int32_t* draft_len;
    int32_t* match_len;
    int32_t* match_pos;
    int32_t* match_cnt;
    int32_t l_max, min_match;
    float spec_factor, spec_offset;
    int32_t n_queues, queue_stride;  // unit counters of the streaming kernel, put back to zero here
};

__device__ __forceinline__ int4 ld_hist_l2(const int4* p) { return __ldcg(p); }

template <int THREADS, int ITER>
__global__ void __launch_bounds__(THREADS, (THREADS == 1024 ? 1 : (THREADS == 512 ? 2 : 4)))
    commit_lookup_kernel(const VerifyArgs va, const NextArgs a, const ScoreArgs sa) {
    __shared__ float s_hid[HVD_MAX_HIDDEN];
    __shared__ CommitOut s_out;
    __shared__ unsigned long long s_key[THREADS / 32];
    __shared__ uint32_t s_cnt[THREADS / 32];
    const int b = blockIdx.x;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    // The streaming kernel ahead of this one waits for its own predecessor before it lets this kernel in, so
    // everything read before the wait below (the request's arrays, the history as the last cycle left it) is
    // complete.  What follows this kernel may become resident at once: it waits before it reads.
    pdl_trigger();

    // ---- before the wait: the request's scalars and the history as it stands ---------------------------
    const int n_old = va.hist_len[b];
    const int cap_b = va.hist_cap[b];
    const int64_t off_b = va.hist_off[b];
    const int K_b = a.K[b];
    const int32_t* slab = va.hist + off_b;  // this kernel also writes the slab: no read-only promise
    const int mis = (int)((reinterpret_cast<uintptr_t>(slab) >> 2) & 3);
    const int4* vbase = reinterpret_cast<const int4*>(slab - mis);
    const bool old_ok = n_old >= 0 && n_old <= cap_b;
    // the commit appends at most k_cap + 1 tokens and never beyond the slab
    int n_hi = old_ok ? min(n_old + va.k_cap + 1, cap_b) : 0;
    n_hi = min(n_hi, a.n_max);
    const int g_spec = (n_hi >= 2) ? (n_hi - 1 + mis) : 0;  // exclusive end on the aligned grid
    // Warp 0 commits (and waits for the row keys inside) while the loads of the others are in flight; its own
    // share of the history is only asked into the L2 for now, so that the commit's registers and the vectors
    // are not live together (the widest shape has 64 registers per thread).
    int4 x[ITER];
    ModelDraft md;
    md.m = 0; md.t0 = -1; md.t1 = -1;
    if (warp != 0) {
#pragma unroll
        for (int i = 0; i < ITER; ++i) {
            const int v = i * THREADS + tid;
            if (4 * v < g_spec) x[i] = ld_hist(vbase + v);
            else x[i] = make_int4(0, 0, 0, 0);
        }
    } else {
#pragma unroll
        for (int i = 0; i < ITER; ++i) {
            const int v = i * THREADS + tid;
            if (4 * v < g_spec) asm volatile("prefetch.global.L2 [%0];" ::"l"(vbase + v));
            x[i] = make_int4(0, 0, 0, 0);
        }
        md = load_model_draft(sa, b, lane);  // the next cycle's fallback draft: an input, fetched ahead
        CommitOut co;
        commit_request(va, b, lane, &co);
        if (lane == 0) s_out = co;
    }
    pdl_wait();
    if (b == 0 && tid < a.n_queues) va.next_unit[tid * a.queue_stride] = 0u;  // zero at rest
    __syncthreads();

    // ---- the next cycle's lookup on the extended history ----------------------------------------------
    const int n_raw = s_out.n;
    int n = n_raw;
    if (n < 0 || n > cap_b || n > a.n_max) n = 0;  // unusable length: empty history
    const int g_end = (n >= 2) ? (n - 1 + mis) : 0;
    if (g_end == 0) {
        if (warp == 0) {
            for (int j = lane; j < va.k_cap; j += 32) a.draft[(int64_t)b * va.k_cap + j] = -1;
            if (lane == 0) {
                a.draft_len[b] = 0; a.match_len[b] = 0; a.match_pos[b] = -1; a.match_cnt[b] = 0;
            }
            score_select_request(sa, b, lane, s_hid, n_raw, 0, 0, -1, 0, -1, -1, &md, &s_out.st);
        }
        return;
    }
    // vectors that hold appended tokens are read again, through the L2 (n > n_old only after a commit,
    // and then n_old was a valid length); warp 0 reads its share now
#pragma unroll
    for (int i = 0; i < ITER; ++i) {
        const int v = i * THREADS + tid;
        const bool again = warp == 0 || (n > n_old && 4 * v + 3 - mis >= n_old);
        if (again && 4 * v < g_end) x[i] = ld_hist_l2(vbase + v);
    }
    // query: the history's new tail.  q0 = last token; lane j keeps the tokens 1+j and 33+j back.
    const int32_t q0 = __ldcg(slab + n - 1);
    const int32_t qa = (1 + lane <= n - 1) ? __ldcg(slab + n - 2 - lane) : 0;
    const int32_t qb = (33 + lane <= n - 1) ? __ldcg(slab + n - 34 - lane) : 0;

    Best best;  // identical in all lanes of a warp
    best.key = 0; best.cnt = 0;
#pragma unroll
    for (int i = 0; i < ITER; ++i) {
        const int p0 = 4 * (i * THREADS + tid) - mis;  // position of x[i].x
        scan_vector<true>(x[i], p0, n, slab, q0, qa, qb, a.l_max, lane, [&](int L, int p) {
            Best c;
            c.key = ((unsigned long long)(uint32_t)L << 32) | (uint32_t)(p + 1);
            c.cnt = 1;
            best = combine(best, c);
        });
    }
    if (lane == 0) { s_key[warp] = best.key; s_cnt[warp] = best.cnt; }
    __syncthreads();
    if (warp != 0) return;

    Best r;
    r.key = lane < THREADS / 32 ? s_key[lane] : 0ull;
    r.cnt = lane < THREADS / 32 ? s_cnt[lane] : 0u;
    r = warp_combine(r);
    int L = (int)(r.key >> 32);
    int e = (int)(uint32_t)(r.key & 0xffffffffu);
    int cnt = (int)r.cnt;
    int d = 0;
    if (L < a.min_match || L == 0) {
        L = 0; e = -1; cnt = 0;
    } else {
        d = min(draft_limit(K_b, va.k_cap, L, a.spec_factor, a.spec_offset), n - e);
    }
    const int tok0 = lane < d ? __ldcg(slab + e + lane) : -1;
    const int tok1 = lane + 32 < d ? __ldcg(slab + e + lane + 32) : -1;
    score_select_request(sa, b, lane, s_hid, n_raw, d, L, e, cnt, tok0, tok1, &md, &s_out.st);
    if (lane < va.k_cap) a.draft[(int64_t)b * va.k_cap + lane] = tok0;
    if (lane + 32 < va.k_cap) a.draft[(int64_t)b * va.k_cap + lane + 32] = tok1;
    if (lane == 0) {
        a.draft_len[b] = d; a.match_len[b] = L; a.match_pos[b] = e; a.match_cnt[b] = cnt;
    }
}

}  // namespace

// true when the one-kernel form can take the call: every history, after the commit, fits one CTA
bool cycle_fits_one_cta(int32_t n_max) { return (int64_t)n_max + 2 <= 32768; }

hvd_status launch_commit_lookup(hvd_ctx* ctx, const VerifyArgs& va, const int32_t* K, int32_t n_max, int32_t* draft,
                                int32_t* draft_len, int32_t* match_len, int32_t* match_pos, int32_t* match_cnt,
                                const ScoreArgs& sa, cudaStream_t stream) {
    NextArgs a;
    a.K = K; a.n_max = n_max;
    a.draft = draft; a.draft_len = draft_len; a.match_len = match_len; a.match_pos = match_pos; a.match_cnt = match_cnt;
    a.l_max = ctx->cfg.l_max; a.min_match = ctx->cfg.min_match;
    a.spec_factor = ctx->cfg.spec_factor; a.spec_offset = ctx->cfg.spec_offset;
    a.n_queues = kVerifyQueues; a.queue_stride = kVerifyQueueStride;
    // one CTA per request: the smallest shape whose aligned grid covers n_max - 1 candidates plus up to
    // 3 tokens of misalignment (the same shapes as the lookup kernel's)
    // CTAs of at most 512 threads and 64 registers fit on an SM beside the streaming kernel's CTAs, so that
    // the loads ahead of the wait really run while the logits are still streaming; only the longest histories
    // take a 1024-thread CTA
    struct Shape { int threads, iter; };
    static const Shape shapes[] = {{256, 1}, {256, 2}, {512, 2}, {512, 4}, {512, 6}, {512, 8}, {512, 9}, {1024, 8}};
    int pick = -1;
    for (int k = 0; k < 8; ++k)
        if ((int64_t)shapes[k].threads * kLookupTokPerVec * shapes[k].iter >= (int64_t)n_max + 2) { pick = k; break; }
    if (pick < 0) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_verify_commit_next: history too long for one CTA");
    const bool pdl = ctx->pdl_commit;
    const dim3 grid((unsigned)va.B);
    cudaError_t e;
#define HVD_LAUNCH_CYCLE(TH, I) launch_kernel(pdl, commit_lookup_kernel<TH, I>, grid, TH, 0, stream, va, a, sa)
    switch (pick) {
        case 0: e = HVD_LAUNCH_CYCLE(256, 1); break;
        case 1: e = HVD_LAUNCH_CYCLE(256, 2); break;
        case 2: e = HVD_LAUNCH_CYCLE(512, 2); break;
        case 3: e = HVD_LAUNCH_CYCLE(512, 4); break;
        case 4: e = HVD_LAUNCH_CYCLE(512, 6); break;
        case 5: e = HVD_LAUNCH_CYCLE(512, 8); break;
        case 6: e = HVD_LAUNCH_CYCLE(512, 9); break;
        default: e = HVD_LAUNCH_CYCLE(1024, 8); break;
    }
#undef HVD_LAUNCH_CYCLE
    HVD_CUDA_TRY(ctx, e);
    return HVD_OK;
}

}  // namespace hvd
