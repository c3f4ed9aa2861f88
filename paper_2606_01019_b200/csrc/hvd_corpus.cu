// Cache-draft lookup over [shared warm-up corpus, own history] (Algorithm 1: the suffix cache starts
// from warm-up traces and the prompt; lookup rule of Sec. 3.2).
//
// The corpus is one token array shared by all requests (negative entries separate traces) and it does
// not change while it is registered, so it is indexed once, at registration: every position that can
// end a match (its token, the g - 1 tokens before it and the token after it are not separators;
// g = min(min_match, 2) tokens form the key) is filed under a hash of its key, and the positions are
// laid out bucket by bucket (count, exclusive scan, scatter: a counting sort).  A lookup then costs
// what the request's own suffix occurs in the corpus, not the corpus length: after the plain lookup
// kernel has searched the histories, the probe kernel reads the bucket of each request's last g
// tokens, drops the hash collisions, extends every remaining candidate backwards against the
// history's tail (eight independent loads per round) and keeps (length, position, count).  The CTAs
// of a request meet in three words of context scratch -- a 64-bit (length, position) maximum, a
// count per match length, an arrival counter; the CTA that arrives last compares the corpus result
// with the history's (longer wins, the history at equal length), rewrites the outputs where the
// corpus wins and clears the scratch.  No CTA waits for another.
#include <algorithm>

#include "hvd_scan.cuh"

namespace hvd {
namespace {

constexpr int kProbeThreads = 256;
constexpr int kProbeWarps = kProbeThreads / 32;
constexpr int kCntStride = HVD_MAX_L + 1;  // counts by match length 0..HVD_MAX_L
constexpr int kScanTile = 4096;            // entries per block of the scan
constexpr int kScanThreads = 1024;

// bucket of a key of one or two tokens (t_prev = 0 for one-token keys)
__device__ __forceinline__ uint32_t corpus_bucket(int32_t t_prev, int32_t t_last, uint32_t mask) {
    unsigned long long k = ((unsigned long long)(uint32_t)t_prev << 32) | (uint32_t)t_last;
    k ^= k >> 33; k *= 0xff51afd7ed558ccdull; k ^= k >> 33; k *= 0xc4ceb9fe1a85ec53ull; k ^= k >> 33;
    return (uint32_t)k & mask;
}

// ---- index build -------------------------------------------------------------------------------
// p is filed if it can end a match that reaches min_match and has a continuation token
__device__ __forceinline__ bool indexable(const int32_t* __restrict__ corpus, int64_t p, int64_t m, int g) {
    if (p < g - 1 || p > m - 2) return false;
    if (corpus[p] < 0 || corpus[p + 1] < 0) return false;
    return g == 1 || corpus[p - 1] >= 0;
}

__global__ void index_count_kernel(const int32_t* __restrict__ corpus, int64_t m, int g, uint32_t mask, uint32_t* cnt) {
    for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < m; p += (int64_t)gridDim.x * blockDim.x)
        if (indexable(corpus, p, m, g)) atomicAdd(cnt + corpus_bucket(g == 2 ? corpus[p - 1] : 0, corpus[p], mask), 1u);
}

__global__ void index_scatter_kernel(const int32_t* __restrict__ corpus, int64_t m, int g, uint32_t mask,
                                     const uint32_t* __restrict__ start, uint32_t* cursor, int32_t* pos) {
    for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < m; p += (int64_t)gridDim.x * blockDim.x)
        if (indexable(corpus, p, m, g)) {
            const uint32_t bk = corpus_bucket(g == 2 ? corpus[p - 1] : 0, corpus[p], mask);
            pos[start[bk] + atomicAdd(cursor + bk, 1u)] = (int32_t)p;  // order inside a bucket does not matter
        }
}

// exclusive scan of v[0..n) in three passes: tiles in place, the tile totals, then the offsets
__global__ void __launch_bounds__(kScanThreads) scan_tiles_kernel(uint32_t* v, int64_t n, uint32_t* tile_sum) {
    __shared__ uint32_t s_warp[32];
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    const int64_t i0 = (int64_t)blockIdx.x * kScanTile + 4 * t;
    uint32_t x[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) x[k] = (i0 + k < n) ? v[i0 + k] : 0u;
    const uint32_t mine = x[0] + x[1] + x[2] + x[3];
    uint32_t inc = mine;  // inclusive scan over the threads of the block
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t o = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += o;
    }
    if (lane == 31) s_warp[w] = inc;
    __syncthreads();
    if (w == 0) {
        uint32_t ws = s_warp[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t o = __shfl_up_sync(0xffffffffu, ws, off);
            if (lane >= off) ws += o;
        }
        s_warp[lane] = ws;  // inclusive over warps
    }
    __syncthreads();
    uint32_t run = inc - mine + (w ? s_warp[w - 1] : 0u);  // exclusive prefix of this thread
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        if (i0 + k < n) v[i0 + k] = run;
        run += x[k];
    }
    if (t == kScanThreads - 1) tile_sum[blockIdx.x] = s_warp[31];
}

__global__ void __launch_bounds__(kScanThreads) scan_sums_kernel(uint32_t* tile_sum, int n_tiles) {
    // one block: each thread takes a contiguous run of tile totals
    __shared__ uint32_t s_part[kScanThreads];
    const int t = threadIdx.x;
    const int per = (n_tiles + kScanThreads - 1) / kScanThreads;
    const int lo = min(t * per, n_tiles), hi = min(lo + per, n_tiles);
    uint32_t sum = 0;
    for (int i = lo; i < hi; ++i) sum += tile_sum[i];
    s_part[t] = sum;
    __syncthreads();
    if (t == 0) {
        uint32_t run = 0;
        for (int i = 0; i < kScanThreads; ++i) { const uint32_t x = s_part[i]; s_part[i] = run; run += x; }
    }
    __syncthreads();
    uint32_t run = s_part[t];
    for (int i = lo; i < hi; ++i) { const uint32_t x = tile_sum[i]; tile_sum[i] = run; run += x; }
}

__global__ void __launch_bounds__(kScanThreads) scan_add_kernel(uint32_t* v, int64_t n, const uint32_t* tile_sum) {
    const uint32_t add = tile_sum[blockIdx.x];
    const int64_t i0 = (int64_t)blockIdx.x * kScanTile + 4 * threadIdx.x;
#pragma unroll
    for (int k = 0; k < 4; ++k)
        if (i0 + k < n) v[i0 + k] += add;
}

// ---- probe ---------------------------------------------------------------------------------------
struct CorpusArgs {
    const int32_t* corpus;
    int32_t m;
    const uint32_t* start;  // [buckets + 1]
    const int32_t* pos;     // positions, bucket by bucket
    uint32_t mask;
    int32_t g;              // tokens in a key
    int32_t slices;         // CTAs per request
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

// the last CTA of a request: corpus result against the history's, by one warp
__device__ __forceinline__ void corpus_merge_request(const CorpusArgs& a, int b, int lane) {
    const int32_t* __restrict__ corpus = a.corpus;
    const int m = a.m;
    pdl_wait();  // the history lookup's result is needed from here on
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
        int d = min(draft_limit(a.K[b], a.k_cap, Lc, a.spec_factor, a.spec_offset), m - ec);
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

__global__ void __launch_bounds__(kProbeThreads) corpus_probe_kernel(const CorpusArgs a) {
    __shared__ int32_t s_q[HVD_MAX_L];  // the history's last tokens, most recent first
    __shared__ unsigned long long s_key[kProbeWarps];
    __shared__ uint32_t s_cntL[kProbeWarps];
    __shared__ int s_last;
    const int b = blockIdx.y;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int32_t* __restrict__ corpus = a.corpus;
    // Launched behind the history lookup, this kernel does not wait for it until the merge: the search of the
    // corpus reads only what was there before that lookup started (histories, lengths, the index), so the two
    // searches run side by side.
    pdl_trigger();
    int n = a.hist_len[b];
    if (n < 0 || n > a.hist_cap[b] || n > a.n_max) n = 0;
    if (tid < HVD_MAX_L) s_q[tid] = (tid < n) ? a.hist[a.hist_off[b] + n - 1 - tid] : -1;
    __syncthreads();

    Best best;  // this thread's candidates
    best.key = 0; best.cnt = 0;
    const int g = a.g;
    const int32_t q0 = s_q[0], q1 = (g == 2) ? s_q[1] : 0;
    if (n >= g && q0 >= 0 && q1 >= 0) {
        const uint32_t bk = corpus_bucket(q1, q0, a.mask);
        const uint32_t lo = __ldg(a.start + bk), hi = __ldg(a.start + bk + 1);
        for (uint32_t i = lo + blockIdx.x * kProbeThreads + tid; i < hi; i += a.slices * kProbeThreads) {
            const int p = __ldg(a.pos + i);
            if (corpus[p] != q0 || (g == 2 && corpus[p - 1] != q1)) continue;  // another key of the same bucket
            const int cap = min(min(a.l_max, p + 1), n);
            if (cap < g) continue;  // the key alone is already longer than a match may be
            int L = g;
            while (L < cap) {  // eight independent loads per round
                int32_t c[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) c[k] = (L + k < cap) ? corpus[p - L - k] : -1;
                uint32_t fail = 0;  // bit j: the token L + j back does not continue the match
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (!(L + j < cap && c[j] >= 0 && c[j] == s_q[L + j])) fail |= 1u << j;
                if (fail == 0) { L += 8; } else { L += __ffs(fail) - 1; break; }
            }
            Best c;
            c.key = ((unsigned long long)(uint32_t)L << 32) | (uint32_t)(p + 1);
            c.cnt = 1;
            best = combine(best, c);
        }
    }
    // warp, then CTA: longest length, then latest position; counts add up at equal length
    best = warp_combine(best);
    if (lane == 0) { s_key[warp] = best.key; s_cntL[warp] = best.cnt; }
    __syncthreads();
    if (tid == 0) {
        Best r;
        r.key = 0; r.cnt = 0;
        for (int w = 0; w < kProbeWarps; ++w) {
            Best o;
            o.key = s_key[w]; o.cnt = s_cntL[w];
            r = combine(r, o);
        }
        const unsigned long long key = r.key;
        const uint32_t cnt = r.cnt;
        if (key != 0) {
            atomicMax(a.key + b, key);
            atomicAdd(a.cnt + (int64_t)b * kCntStride + (key >> 32), cnt);
        }
        __threadfence();
        const uint32_t old = atomicAdd(a.arrived + b, 1u);
        s_last = (old + 1 == (uint32_t)a.slices) ? 1 : 0;
    }
    __syncthreads();
    if (s_last && warp == 0) corpus_merge_request(a, b, lane);
}

// requests without a usable corpus: every request's match comes from its history
__global__ void corpus_none_kernel(int32_t B, int32_t* match_src) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_trigger();
    if (b < B) match_src[b] = 0;
}

}  // namespace

void release_corpus_index(hvd_ctx* ctx) {
    cudaFree(ctx->cp_start); cudaFree(ctx->cp_pos);
    ctx->cp_start = nullptr; ctx->cp_pos = nullptr; ctx->cp_mask = 0;
    ctx->corpus = nullptr; ctx->corpus_len = 0;
}

// Builds the index of a newly registered corpus on the default stream and waits for it.
hvd_status build_corpus_index(hvd_ctx* ctx, const int32_t* corpus, int64_t m) {
    release_corpus_index(ctx);
    if (corpus == nullptr || m < 2) return HVD_OK;  // fewer than two tokens: no position has a continuation
    uint64_t buckets = 1024;
    while (buckets < 2 * (uint64_t)m && buckets < (1ull << 26)) buckets <<= 1;
    const int64_t n_scan = (int64_t)buckets + 1;
    const int n_tiles = (int)((n_scan + kScanTile - 1) / kScanTile);
    uint32_t *start = nullptr, *cursor = nullptr, *tile_sum = nullptr;
    int32_t* pos = nullptr;
    cudaError_t e = cudaMalloc(&start, n_scan * sizeof(uint32_t));
    if (e == cudaSuccess) e = cudaMalloc(&cursor, buckets * sizeof(uint32_t));
    if (e == cudaSuccess) e = cudaMalloc(&tile_sum, (size_t)n_tiles * sizeof(uint32_t));
    if (e == cudaSuccess) e = cudaMalloc(&pos, (size_t)m * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemsetAsync(start, 0, n_scan * sizeof(uint32_t), 0);
    if (e == cudaSuccess) e = cudaMemsetAsync(cursor, 0, buckets * sizeof(uint32_t), 0);
    if (e == cudaSuccess) {
        const int g = ctx->cfg.min_match >= 2 ? 2 : 1;
        const uint32_t mask = (uint32_t)(buckets - 1);
        const int blocks = (int)std::min<int64_t>((m + 255) / 256, (int64_t)ctx->num_sms * 16);
        index_count_kernel<<<blocks, 256>>>(corpus, m, g, mask, start);
        scan_tiles_kernel<<<n_tiles, kScanThreads>>>(start, n_scan, tile_sum);
        scan_sums_kernel<<<1, kScanThreads>>>(tile_sum, n_tiles);
        scan_add_kernel<<<n_tiles, kScanThreads>>>(start, n_scan, tile_sum);
        index_scatter_kernel<<<blocks, 256>>>(corpus, m, g, mask, start, cursor, pos);
        e = cudaGetLastError();
        if (e == cudaSuccess) e = cudaStreamSynchronize(0);
        ctx->cp_g = g; ctx->cp_mask = mask;
    }
    cudaFree(cursor); cudaFree(tile_sum);
    if (e != cudaSuccess) {
        cudaFree(start); cudaFree(pos);
        return cuda_fail(ctx, e, "hvd_set_corpus: index build");
    }
    ctx->cp_start = start; ctx->cp_pos = pos;
    ctx->corpus = corpus; ctx->corpus_len = (int32_t)m;
    return HVD_OK;
}

hvd_status launch_lookup_corpus(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                                const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K, int32_t n_max,
                                int32_t* draft, int32_t* draft_len, int32_t* match_len, int32_t* match_pos,
                                int32_t* match_src, int32_t* match_cnt, cudaStream_t stream) {
    const hvd_status r = launch_lookup(ctx, B, hist, hist_off, hist_cap, hist_len, K, n_max, draft, draft_len,
                                       match_len, match_pos, match_cnt, nullptr, stream, ctx->cp_start != nullptr);
    if (r != HVD_OK) return r;
    if (ctx->cp_start == nullptr) {
        HVD_CUDA_TRY(ctx, launch_kernel(false, corpus_none_kernel, dim3((unsigned)((B + 255) / 256)), 256, 0,
                                        stream, B, match_src));
        return HVD_OK;
    }
    CorpusArgs a;
    a.corpus = ctx->corpus; a.m = ctx->corpus_len;
    a.start = ctx->cp_start; a.pos = ctx->cp_pos; a.mask = ctx->cp_mask; a.g = ctx->cp_g;
    // CTAs per request: enough to fill the GPU a few times over, so that a long bucket is shared out
    int slices = (ctx->num_sms * 4 + B - 1) / B;
    a.slices = slices < 1 ? 1 : (slices > 8 ? 8 : slices);
    a.hist = hist; a.hist_off = hist_off; a.hist_cap = hist_cap; a.hist_len = hist_len; a.K = K; a.n_max = n_max;
    a.k_cap = ctx->cfg.k_cap; a.l_max = ctx->cfg.l_max; a.min_match = ctx->cfg.min_match;
    a.spec_factor = ctx->cfg.spec_factor; a.spec_offset = ctx->cfg.spec_offset;
    a.draft = draft; a.draft_len = draft_len; a.match_len = match_len; a.match_pos = match_pos;
    a.match_src = match_src; a.match_cnt = match_cnt;
    a.key = ctx->cp_key; a.cnt = ctx->cp_cnt; a.arrived = ctx->cp_arrived;
    HVD_CUDA_TRY(ctx, launch_kernel(ctx->pdl_mask != 0, corpus_probe_kernel, dim3((unsigned)a.slices, (unsigned)B),
                                    kProbeThreads, 0, stream, a));
    return HVD_OK;
}

}  // namespace hvd
