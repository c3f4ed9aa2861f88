// Cache-draft lookup over [shared warm-up corpus, own history] (Algorithm 1: the suffix cache starts
// from warm-up traces and the prompt; lookup rule of Sec. 3.2).
//
// The corpus is one token array shared by all requests (negative entries separate traces).  The plain
// lookup kernel has already searched every request's own history; the kernel here searches the corpus
// and merges.  A CTA loads one chunk of the corpus into registers once and tests it against the
// suffixes of several requests in turn, so the corpus crosses the L2 once per group of requests and
// not once per request.  Per request the CTAs meet in three words of context scratch: a 64-bit
// (length, position) maximum, a count per match length, and an arrival counter; the CTA that
// arrives last for a request compares the corpus result with the history's (longer wins, the
// history at equal length), rewrites the outputs where the corpus wins and clears the scratch.  No
// CTA waits for another.
#include "hvd_internal.cuh"

namespace hvd {
namespace {

constexpr int kCorpusThreads = 256;
constexpr int kCorpusIter = 8;
constexpr int kCorpusChunk = kCorpusThreads * kLookupTokPerVec * kCorpusIter;  // 8192 tokens per CTA
constexpr int kCorpusMaxGroup = 16;                                            // requests per CTA
constexpr int kCorpusWarps = kCorpusThreads / 32;
constexpr int kCntStride = HVD_MAX_L + 1;  // counts by match length 0..HVD_MAX_L

struct CorpusArgs {
    const int32_t* corpus;
    int32_t m;
    int32_t n_chunks;
    int32_t group;  // requests per CTA
    int32_t B;
    const int32_t* hist;
    const int64_t* hist_off;
    const int32_t* hist_cap;
    const int32_t* hist_len;
    const int32_t* K;
    int32_t n_max;
    int32_t k_cap, l_max, min_match;
    float spec_factor, spec_offset;
    int32_t* draft;
    int32_t* draft_len;
    int32_t* match_len;
    int32_t* match_pos;
    int32_t* match_src;
    int32_t* match_cnt;
    unsigned long long* key;  // [max_batch] (length << 32) | position, zero at rest
    uint32_t* cnt;            // [max_batch, kCntStride], zero at rest
    uint32_t* arrived;        // [max_batch], zero at rest
};

__global__ void __launch_bounds__(kCorpusThreads) corpus_scan_kernel(const CorpusArgs a) {
    __shared__ unsigned long long s_key[kCorpusMaxGroup][kCorpusWarps];
    __shared__ uint32_t s_cnt[kCorpusMaxGroup][kCorpusWarps];
    __shared__ int s_last[kCorpusMaxGroup];
    __shared__ int32_t s_n[kCorpusMaxGroup];                // usable history length per request of the group
    __shared__ int32_t s_q[kCorpusMaxGroup][HVD_MAX_L];     // the history's last tokens, most recent first
    const int chunk = blockIdx.x;
    const int b0 = blockIdx.y * a.group;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int32_t* __restrict__ corpus = a.corpus;
    const int m = a.m;
    pdl_trigger();

    // this CTA's part of the corpus: candidate positions p (last token of a copy) are 0 .. m-2
    const int4* __restrict__ vbase = reinterpret_cast<const int4*>(corpus);
    const int v0 = chunk * (kCorpusChunk / 4);
    // tokens that cannot end a candidate (beyond m-2) are replaced by -1, which equals no history token
    int4 x[kCorpusIter];
#pragma unroll
    for (int i = 0; i < kCorpusIter; ++i) {
        const int p0 = 4 * (v0 + i * kCorpusThreads + tid);
        if (p0 + 3 <= m - 2) {
            x[i] = __ldg(vbase + (p0 >> 2));
        } else {  // the last vectors are read token by token
            x[i].x = (p0 + 0 <= m - 2) ? __ldg(corpus + p0 + 0) : -1;
            x[i].y = (p0 + 1 <= m - 2) ? __ldg(corpus + p0 + 1) : -1;
            x[i].z = (p0 + 2 <= m - 2) ? __ldg(corpus + p0 + 2) : -1;
            x[i].w = -1;
        }
    }
    pdl_wait();

    const int nreq = min(a.group, a.B - b0);
    // the suffixes of the group's requests, all fetched at once (one chain of dependent loads, not one per request)
    for (int r = warp; r < nreq; r += kCorpusWarps) {
        const int b = b0 + r;
        int n = a.hist_len[b];
        if (n < 0 || n > a.hist_cap[b] || n > a.n_max) n = 0;
        const int32_t* slab = a.hist + a.hist_off[b];
        s_q[r][lane] = (lane < n) ? slab[n - 1 - lane] : 0;
        s_q[r][lane + 32] = (lane + 32 < n) ? slab[n - 33 - lane] : 0;
        if (lane == 0) s_n[r] = n;
    }
    __syncthreads();
    for (int r = 0; r < nreq; ++r) {
        struct { int32_t n, q0, qa, qb; } q;
        q.n = s_n[r]; q.q0 = s_q[r][0]; q.qa = s_q[r][1 + lane]; q.qb = (lane < 31) ? s_q[r][33 + lane] : 0;
        unsigned long long best_key = 0;
        uint32_t best_cnt = 0;
        if (q.n > 0 && q.q0 >= 0) {
            // one bit per token of this thread's 8 vectors, one vote per request
            uint32_t mk = 0;
#pragma unroll
            for (int i = 0; i < kCorpusIter; ++i) {
                mk |= (x[i].x == q.q0 ? 1u : 0u) << (4 * i + 0);
                mk |= (x[i].y == q.q0 ? 1u : 0u) << (4 * i + 1);
                mk |= (x[i].z == q.q0 ? 1u : 0u) << (4 * i + 2);
                mk |= (x[i].w == q.q0 ? 1u : 0u) << (4 * i + 3);
            }
            uint32_t hits = __ballot_sync(0xffffffffu, mk != 0);
            while (hits) {
                const int src = __ffs(hits) - 1;
                hits &= hits - 1;
                uint32_t ms = __shfl_sync(0xffffffffu, mk, src);
                while (ms) {
                    const int bit = __ffs(ms) - 1;
                    ms &= ms - 1;
                    const int p = 4 * (v0 + (bit >> 2) * kCorpusThreads + (tid - lane + src)) + (bit & 3);
                    if (corpus[p + 1] < 0) continue;  // no continuation token: not a candidate (warp-uniform)
                    const int cap = min(min(a.l_max, p + 1), q.n);
                    int l = lane + 1;
                    int32_t c = (l < cap) ? corpus[p - l] : -1;
                    bool eq = (l < cap) && c >= 0 && c == q.qa;
                    uint32_t mm = __ballot_sync(0xffffffffu, !eq);
                    int L;
                    if (mm != 0) {
                        L = __ffs(mm);
                    } else {
                        l = lane + 33;
                        c = (l < cap) ? corpus[p - l] : -1;
                        eq = (l < cap) && c >= 0 && c == q.qb;
                        mm = __ballot_sync(0xffffffffu, !eq);  // lane 31 (l = 64) always fails
                        L = 32 + __ffs(mm);
                    }
                    const unsigned long long key = ((unsigned long long)(uint32_t)L << 32) | (uint32_t)(p + 1);
                    const uint32_t bl = (uint32_t)(best_key >> 32);
                    if ((uint32_t)L > bl) { best_key = key; best_cnt = 1; }
                    else if ((uint32_t)L == bl) { best_key = key > best_key ? key : best_key; ++best_cnt; }
                }
            }
        }
        if (lane == 0) { s_key[r][warp] = best_key; s_cnt[r][warp] = best_cnt; }
    }
    __syncthreads();

    // one thread per request of the group: combine the warps, publish, count the arrival
    if (tid < nreq) {
        unsigned long long key = 0;
        uint32_t cnt = 0;
        for (int w = 0; w < kCorpusWarps; ++w) {
            const unsigned long long k2 = s_key[tid][w];
            const uint32_t l1 = (uint32_t)(key >> 32), l2 = (uint32_t)(k2 >> 32);
            if (l2 > l1) { key = k2; cnt = s_cnt[tid][w]; }
            else if (l2 == l1 && l2 != 0) { key = k2 > key ? k2 : key; cnt += s_cnt[tid][w]; }
        }
        const int b = b0 + tid;
        if (key != 0) {
            atomicMax(a.key + b, key);
            atomicAdd(a.cnt + (int64_t)b * kCntStride + (key >> 32), cnt);
        }
        __threadfence();
        const uint32_t old = atomicAdd(a.arrived + b, 1u);
        s_last[tid] = (old + 1 == (uint32_t)a.n_chunks) ? 1 : 0;
    }
    __syncthreads();

    for (int r = warp; r < nreq; r += kCorpusWarps) {
        if (!s_last[r]) continue;
        const int b = b0 + r;
        __threadfence();
        const unsigned long long key = __ldcg(a.key + b);
        int Lc = (int)(key >> 32);
        const int ec = (int)(uint32_t)(key & 0xffffffffu);
        const int cc = Lc ? (int)__ldcg(a.cnt + (int64_t)b * kCntStride + Lc) : 0;
        // scratch is zero at rest
        for (int l = lane; l < kCntStride; l += 32) a.cnt[(int64_t)b * kCntStride + l] = 0;
        if (lane == 0) { a.key[b] = 0; a.arrived[b] = 0; }
        if (Lc < a.min_match) Lc = 0;
        const int Lh = a.match_len[b];
        if (Lc == 0 || Lc < Lh) {
            if (lane == 0) a.match_src[b] = 0;
        } else if (Lc == Lh) {  // the history comes first; the corpus occurrences are counted
            if (lane == 0) { a.match_src[b] = 0; a.match_cnt[b] = a.match_cnt[b] + cc; }
        } else {
            int K = max(0, min(a.K[b], a.k_cap));
            int lim = K;
            if (a.spec_factor > 0.0f) {
                const float f = __fadd_rn(__fmul_rn(a.spec_factor, (float)Lc), a.spec_offset);
                lim = max(0, (int)floorf(f));
            }
            int d = min(min(K, lim), m - ec);
            int tok0 = lane < d ? corpus[ec + lane] : 0;
            int tok1 = lane + 32 < d ? corpus[ec + lane + 32] : 0;
            // a separator ends the draft
            const uint32_t neg0 = __ballot_sync(0xffffffffu, tok0 < 0);
            const uint32_t neg1 = __ballot_sync(0xffffffffu, tok1 < 0);
            if (neg0) d = min(d, __ffs(neg0) - 1);
            else if (neg1) d = min(d, 32 + __ffs(neg1) - 1);
            if (lane >= d) tok0 = -1;
            if (lane + 32 >= d) tok1 = -1;
            if (lane < a.k_cap) a.draft[(int64_t)b * a.k_cap + lane] = tok0;
            if (lane + 32 < a.k_cap) a.draft[(int64_t)b * a.k_cap + lane + 32] = tok1;
            if (lane == 0) {
                a.draft_len[b] = d; a.match_len[b] = Lc; a.match_pos[b] = ec; a.match_src[b] = 1; a.match_cnt[b] = cc;
            }
        }
    }
}

// requests without a usable corpus: every request's match comes from its history
__global__ void corpus_none_kernel(int32_t B, int32_t* match_src) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_trigger();
    if (b < B) match_src[b] = 0;
}

}  // namespace

hvd_status launch_lookup_corpus(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                                const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K, int32_t n_max,
                                int32_t* draft, int32_t* draft_len, int32_t* match_len, int32_t* match_pos,
                                int32_t* match_src, int32_t* match_cnt, cudaStream_t stream) {
    const hvd_status r = launch_lookup(ctx, B, hist, hist_off, hist_cap, hist_len, K, n_max, draft, draft_len,
                                       match_len, match_pos, match_cnt, nullptr, stream);
    if (r != HVD_OK) return r;
    if (ctx->corpus == nullptr || ctx->corpus_len < 2) {
        HVD_CUDA_TRY(ctx, launch_kernel(ctx->use_pdl, corpus_none_kernel, dim3((unsigned)((B + 255) / 256)), 256, 0,
                                        stream, B, match_src));
        return HVD_OK;
    }
    CorpusArgs a;
    a.corpus = ctx->corpus; a.m = ctx->corpus_len;
    a.n_chunks = (int32_t)(((int64_t)a.m - 1 + kCorpusChunk - 1) / kCorpusChunk);
    // requests per CTA: as many as still leave about four CTAs per SM
    int64_t group = ((int64_t)B * a.n_chunks) / ((int64_t)ctx->num_sms * 4);
    if (group < 1) group = 1;
    if (group > kCorpusMaxGroup) group = kCorpusMaxGroup;
    a.group = (int32_t)group; a.B = B;
    a.hist = hist; a.hist_off = hist_off; a.hist_cap = hist_cap; a.hist_len = hist_len; a.K = K; a.n_max = n_max;
    a.k_cap = ctx->cfg.k_cap; a.l_max = ctx->cfg.l_max; a.min_match = ctx->cfg.min_match;
    a.spec_factor = ctx->cfg.spec_factor; a.spec_offset = ctx->cfg.spec_offset;
    a.draft = draft; a.draft_len = draft_len; a.match_len = match_len; a.match_pos = match_pos;
    a.match_src = match_src; a.match_cnt = match_cnt;
    a.key = ctx->cp_key; a.cnt = ctx->cp_cnt; a.arrived = ctx->cp_arrived;
    const dim3 grid((unsigned)a.n_chunks, (unsigned)((B + a.group - 1) / a.group));
    HVD_CUDA_TRY(ctx, launch_kernel(ctx->use_pdl, corpus_scan_kernel, grid, kCorpusThreads, 0, stream, a));
    return HVD_OK;
}

}  // namespace hvd
