// Frequency-weighted cache draft and suffix score (the cache score that the frequency-based hybrid
// baseline of Sec. 4.1 thresholds; drafting limits and the minimum token probability are those of
// the drafting table in App. A).
//
// The plain lookup kernel has already found, per request, the longest match length L, its latest
// occurrence and the number of occurrences.  Two more kernels follow it in the stream:
//   collect: for requests with 2 .. max_occ occurrences, scans the history again and appends every
//            position whose match length equals L to a per-request list in the context's scratch
//            (order does not matter: the walk breaks ties by position, not by list order); a
//            single occurrence is the one the lookup reported and needs no second scan;
//   walk:    one CTA per request stages the continuation tokens of all listed occurrences in shared
//            memory, then its first warp walks them step by step: the most frequent next token
//            among the occurrences still alive (ties: the token whose latest occurrence is later),
//            its share of the alive occurrences as an fp32 probability (one IEEE division), stop
//            below the minimum probability, add the probability to the score, keep the
//            occurrences that continue with that token.
// Requests with more occurrences than the list holds follow the latest occurrence only (every
// token then has probability 1), exactly like the plain lookup.
#include "hvd_scan.cuh"

namespace hvd {
namespace {

constexpr int kCollectThreads = 256;
constexpr int kCollectIter = 4;
constexpr int kCollectChunk = kCollectThreads * kLookupTokPerVec * kCollectIter;  // tokens per CTA
constexpr int kWalkThreads = HVD_FREQ_MAX_OCC;                                    // one thread per occurrence
constexpr int kSlots = HVD_FREQ_MAX_OCC / 32;
constexpr int kBatchMaxAlive = 6;   // agreement runs are looked for while at most this many occurrences are alive                                     // occurrences per lane of the walking warp

struct FreqArgs {
    const int32_t* hist;
    const int64_t* hist_off;
    const int32_t* hist_cap;
    const int32_t* hist_len;
    const int32_t* K;
    int32_t n_max;
    int32_t k_cap, l_max;
    float spec_factor, spec_offset;
    float min_prob;
    int32_t max_occ;
    float threshold;
    const int32_t* model_draft;
    const int32_t* model_len;
    // from the plain lookup
    const int32_t* match_len;
    const int32_t* match_pos;
    const int32_t* match_cnt;
    // outputs
    int32_t* draft;
    int32_t* draft_len;
    float* score;
    int32_t* select;
    int32_t* sel_draft;
    int32_t* sel_len;
    // scratch
    int32_t* occ;       // [max_batch, HVD_FREQ_MAX_OCC]
    uint32_t* occ_cnt;  // [max_batch], zero at rest
};

__device__ __forceinline__ int usable_len(const FreqArgs& a, int b) {
    const int n = a.hist_len[b];
    return (n < 0 || n > a.hist_cap[b] || n > a.n_max) ? 0 : n;
}

__global__ void __launch_bounds__(kCollectThreads) freq_collect_kernel(const FreqArgs a) {
    const int b = blockIdx.y;
    const int chunk = blockIdx.x;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    pdl_trigger();
    pdl_wait();
    const int Lstar = a.match_len[b];
    const int cnt = a.match_cnt[b];
    // nothing to merge, too many, or a single occurrence (which the lookup has already located)
    if (Lstar <= 0 || cnt > a.max_occ || cnt == 1) return;
    const int n = usable_len(a, b);
    const int32_t* __restrict__ slab = a.hist + a.hist_off[b];
    const int mis = (int)((reinterpret_cast<uintptr_t>(slab) >> 2) & 3);
    const int g_end = (n >= 2) ? (n - 1 + mis) : 0;
    if ((int64_t)chunk * kCollectChunk >= g_end) return;
    const int4* __restrict__ vbase = reinterpret_cast<const int4*>(slab - mis);
    const int v0 = chunk * (kCollectChunk / 4);

    int4 x[kCollectIter];
#pragma unroll
    for (int i = 0; i < kCollectIter; ++i) {
        const int v = v0 + i * kCollectThreads + tid;
        x[i] = (4 * v < g_end) ? ld_hist(vbase + v) : make_int4(0, 0, 0, 0);
    }
    const int32_t q0 = slab[n - 1];
    const int32_t qa = (1 + lane <= n - 1) ? slab[n - 2 - lane] : 0;
    const int32_t qb = (33 + lane <= n - 1) ? slab[n - 34 - lane] : 0;
#pragma unroll
    for (int i = 0; i < kCollectIter; ++i) {
        const int p0 = 4 * (v0 + i * kCollectThreads + tid) - mis;
        scan_vector(x[i], p0, n, slab, q0, qa, qb, a.l_max, lane, [&](int L, int p) {
            if (L == Lstar && lane == 0) {  // the continuation of the copy that ends at p starts at p + 1
                const uint32_t idx = atomicAdd(a.occ_cnt + b, 1u);
                if (idx < (uint32_t)HVD_FREQ_MAX_OCC) a.occ[(int64_t)b * HVD_FREQ_MAX_OCC + idx] = p + 1;
            }
        });
    }
}

using TokTile = int32_t[HVD_FREQ_MAX_OCC + 1];

// The walk over SLOTS * 32 listed occurrences by one warp; lane l owns occurrences l, l + 32, ...
template <int SLOTS>
__device__ __forceinline__ void walk_merged(const FreqArgs& a, const int32_t* __restrict__ slab, int n, int limit,
                                            int lane, const TokTile* s_tok, const int32_t* s_e, int32_t* s_alive,
                                            int& d, float& sc, int& tok0, int& tok1) {
    int e[SLOTS], len[SLOTS];
    bool alive[SLOTS];
    int na = 0;
#pragma unroll
    for (int j = 0; j < SLOTS; ++j) {
        e[j] = s_e[lane + 32 * j];
        alive[j] = e[j] >= 0;
        len[j] = alive[j] ? min(limit, n - e[j]) : 0;
        na += __popc(__ballot_sync(0xffffffffu, alive[j]));
    }
    bool listed = false;  // s_alive holds the indices of the alive occurrences
    while (d < limit) {
        if (na >= 2 && na <= kBatchMaxAlive && 1.0f >= a.min_prob) {
            // Steps on which every alive occurrence continues with the same token have probability 1 and
            // keep the set as it is: all of them are taken at once.  Lane l looks at draft positions l, l + 32.
            if (!listed) {
                int base = 0;
#pragma unroll
                for (int j = 0; j < SLOTS; ++j) {
                    const uint32_t mask = __ballot_sync(0xffffffffu, alive[j]);
                    if (alive[j]) s_alive[base + __popc(mask & ((1u << lane) - 1u))] = lane + 32 * j;
                    base += __popc(mask);
                }
                __syncwarp();
                listed = true;
            }
            bool ok[2];
            int t[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int q = lane + 32 * h;
                ok[h] = q >= d && q < limit;
                t[h] = -1;
                if (ok[h]) {
                    t[h] = s_tok[q][s_alive[0]];
                    for (int k = 0; k < na; ++k) {
                        const int i = s_alive[k];
                        ok[h] = ok[h] && (s_e[i] + q < n) && (s_tok[q][i] == t[h]);
                    }
                }
            }
            const unsigned long long agree = ((unsigned long long)__ballot_sync(0xffffffffu, ok[1]) << 32) |
                                             __ballot_sync(0xffffffffu, ok[0]);
            const unsigned long long miss = ~(agree >> d);  // bit r: position d + r does not agree (or is past the limit)
            const int run = miss ? __ffsll((long long)miss) - 1 : 64;
            if (run > 0) {
                if (lane >= d && lane < d + run) tok0 = t[0];
                if (lane + 32 >= d && lane + 32 < d + run) tok1 = t[1];
                for (int k = 0; k < run; ++k) sc = __fadd_rn(sc, 1.0f);  // the same additions, one by one
                d += run;
                continue;
            }
        }
        if (na == 1) {
            // one occurrence left: each further token has probability 1 until it or the limit ends
            int me = -1;
#pragma unroll
            for (int j = 0; j < SLOTS; ++j)
                if (alive[j]) me = e[j];
            const int el = __reduce_max_sync(0xffffffffu, me);
            const int r = (1.0f >= a.min_prob) ? max(0, min(limit, n - el) - d) : 0;
            if (lane >= d && lane < d + r) tok0 = slab[el + lane];
            if (lane + 32 >= d && lane + 32 < d + r) tok1 = slab[el + lane + 32];
            for (int k = 0; k < r; ++k) sc = __fadd_rn(sc, 1.0f);  // the same additions, one by one
            d += r;
            break;
        }
        int t[SLOTS];
        bool open[SLOTS];  // alive, has a token at this step, and not yet counted
        int remaining = 0;
#pragma unroll
        for (int j = 0; j < SLOTS; ++j) {
            open[j] = alive[j] && d < len[j];
            t[j] = s_tok[d][lane + 32 * j];
            remaining += __popc(__ballot_sync(0xffffffffu, open[j]));
        }
        int best_cnt = 0, best_tok = -1;
        // pivots in descending position: the first pivot of a token is that token's latest occurrence,
        // so between equal counts the earlier pivot wins
        while (remaining > best_cnt) {
            int m = -1, mt = 0;
#pragma unroll
            for (int j = 0; j < SLOTS; ++j)
                if (open[j] && e[j] > m) { m = e[j]; mt = t[j]; }
            const int pivot = __reduce_max_sync(0xffffffffu, m);
            const int owner = __ffs(__ballot_sync(0xffffffffu, m == pivot)) - 1;
            const int x = __shfl_sync(0xffffffffu, mt, owner);
            int cx = 0;
#pragma unroll
            for (int j = 0; j < SLOTS; ++j) {
                const bool hit = open[j] && t[j] == x;
                cx += __popc(__ballot_sync(0xffffffffu, hit));
                open[j] = open[j] && !hit;
            }
            remaining -= cx;
            if (cx > best_cnt) { best_cnt = cx; best_tok = x; }
        }
        if (best_cnt == 0) break;
        const float prob = __fdiv_rn((float)best_cnt, (float)na);
        if (prob < a.min_prob) break;
        if (lane == (d & 31)) { if (d < 32) tok0 = best_tok; else tok1 = best_tok; }
        sc = __fadd_rn(sc, prob);
#pragma unroll
        for (int j = 0; j < SLOTS; ++j) alive[j] = alive[j] && d < len[j] && t[j] == best_tok;
        listed = listed && best_cnt == na;  // the list stays valid only if nobody dropped out
        na = best_cnt;
        ++d;
    }
}

__global__ void __launch_bounds__(kWalkThreads) freq_walk_kernel(const FreqArgs a) {
    __shared__ int32_t s_tok[HVD_MAX_K][HVD_FREQ_MAX_OCC + 1];  // [step][occurrence]; odd stride: no bank conflicts
    __shared__ int32_t s_e[HVD_FREQ_MAX_OCC];
    __shared__ int32_t s_alive[HVD_FREQ_MAX_OCC];
    const int b = blockIdx.x;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    pdl_trigger();
    pdl_wait();
    const int kc = a.k_cap;
    const int n = usable_len(a, b);
    const int L = a.match_len[b];
    const int cnt = a.match_cnt[b];
    const int32_t* __restrict__ slab = a.hist + a.hist_off[b];

    const int limit = L > 0 ? draft_limit(a.K[b], kc, L, a.spec_factor, a.spec_offset) : 0;
    // 2 .. max_occ occurrences are merged; one occurrence, or too many, is the lookup's own draft
    const bool merged = (L > 0) && (cnt >= 2) && (cnt <= a.max_occ);
    const int c = merged ? min(cnt, HVD_FREQ_MAX_OCC) : 0;

    if (merged) {
        s_e[tid] = (tid < c) ? a.occ[(int64_t)b * HVD_FREQ_MAX_OCC + tid] : -1;
        __syncthreads();
        // all threads share the loads: consecutive threads read consecutive tokens of one occurrence
        for (int idx = tid; idx < c * limit; idx += kWalkThreads) {
            const int i = idx / limit, s = idx - i * limit;
            const int e = s_e[i];
            s_tok[s][i] = (e + s < n) ? slab[e + s] : 0;
        }
    }
    __syncthreads();
    if (tid >= 32) return;
    if (tid == 0) a.occ_cnt[b] = 0;  // scratch is zero at rest

    int d = 0;
    float sc = 0.0f;
    int tok0 = -1, tok1 = -1;  // draft tokens lane and lane + 32
    if (merged) {
        if (c <= 32) walk_merged<1>(a, slab, n, limit, lane, s_tok, s_e, s_alive, d, sc, tok0, tok1);
        else walk_merged<kSlots>(a, slab, n, limit, lane, s_tok, s_e, s_alive, d, sc, tok0, tok1);
    } else if (L > 0) {
        // one occurrence: every token has probability 1 (nothing passes a minimum above 1);
        // too many occurrences: the latest one, every token taken as certain
        const int e = a.match_pos[b];
        d = (cnt > a.max_occ || 1.0f >= a.min_prob) ? max(0, min(limit, n - e)) : 0;
        tok0 = lane < d ? slab[e + lane] : -1;
        tok1 = lane + 32 < d ? slab[e + lane + 32] : -1;
        sc = (float)d;
    }
    if (lane < kc) a.draft[(int64_t)b * kc + lane] = tok0;
    if (lane + 32 < kc) a.draft[(int64_t)b * kc + lane + 32] = tok1;
    if (lane == 0) { a.draft_len[b] = d; a.score[b] = sc; }
    if (a.select) {
        const int sel = (d > 0 && sc >= a.threshold) ? 1 : 0;
        int m = 0, o0 = -1, o1 = -1;
        if (sel) {
            m = d; o0 = tok0; o1 = tok1;
        } else if (a.model_draft) {
            m = max(0, min(a.model_len[b], kc));
            const int32_t* src = a.model_draft + (int64_t)b * kc;
            o0 = lane < m ? src[lane] : -1;
            o1 = lane + 32 < m ? src[lane + 32] : -1;
        }
        if (lane < kc) a.sel_draft[(int64_t)b * kc + lane] = o0;
        if (lane + 32 < kc) a.sel_draft[(int64_t)b * kc + lane + 32] = o1;
        if (lane == 0) { a.select[b] = sel; a.sel_len[b] = m; }
    }
}

}  // namespace

hvd_status launch_lookup_freq(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                              const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K, int32_t n_max,
                              float min_prob, int32_t max_occ, float threshold, const int32_t* model_draft,
                              const int32_t* model_len, int32_t* draft, int32_t* draft_len, float* score,
                              int32_t* match_len, int32_t* match_pos, int32_t* match_cnt, int32_t* select,
                              int32_t* sel_draft, int32_t* sel_len, cudaStream_t stream) {
    const hvd_status r = launch_lookup(ctx, B, hist, hist_off, hist_cap, hist_len, K, n_max, draft, draft_len,
                                       match_len, match_pos, match_cnt, nullptr, stream);
    if (r != HVD_OK) return r;
    FreqArgs a;
    a.hist = hist; a.hist_off = hist_off; a.hist_cap = hist_cap; a.hist_len = hist_len; a.K = K;
    a.n_max = n_max; a.k_cap = ctx->cfg.k_cap; a.l_max = ctx->cfg.l_max;
    a.spec_factor = ctx->cfg.spec_factor; a.spec_offset = ctx->cfg.spec_offset;
    a.min_prob = min_prob; a.max_occ = max_occ; a.threshold = threshold;
    a.model_draft = model_draft; a.model_len = model_len;
    a.match_len = match_len; a.match_pos = match_pos; a.match_cnt = match_cnt;
    a.draft = draft; a.draft_len = draft_len; a.score = score;
    a.select = select; a.sel_draft = sel_draft; a.sel_len = sel_len;
    a.occ = ctx->fq_occ; a.occ_cnt = ctx->fq_cnt;
    const int64_t span = (int64_t)(n_max > 1 ? n_max - 1 : 1) + 3;
    const unsigned chunks = (unsigned)((span + kCollectChunk - 1) / kCollectChunk);
    HVD_CUDA_TRY(ctx, launch_kernel(ctx->pdl_mask != 0, freq_collect_kernel, dim3(chunks, (unsigned)B), kCollectThreads, 0,
                                    stream, a));
    HVD_CUDA_TRY(ctx, launch_kernel(ctx->pdl_mask != 0, freq_walk_kernel, dim3((unsigned)B), kWalkThreads, 0, stream, a));
    return HVD_OK;
}

}  // namespace hvd
