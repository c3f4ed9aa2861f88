// Cache-draft lookup (Sec. 3.2): longest match of the history's own suffix inside the history.
//
// One CTA scans a request's history (histories longer than 32 K tokens are cut into chunks of 8 K
// tokens, one CTA each) with 128-bit loads, all issued up front, looking for the last token of the
// history.  Every hit is a candidate end position; the warp that found it extends the match
// backwards cooperatively (one compared token per lane, ballot + find-first-set gives the match
// length).  Each CTA leaves one partial (best length, latest position, count) in
// the context's scratch; the CTA that arrives last for a request combines the partials, applies the
// minimum-length and draft-length rules and copies the draft -- and, in the fused form, goes
// straight on to the payoff features, the predictor and the draft selection of that request
// (one kernel and one global round trip less per decoding step).  No CTA waits for another.
#include "hvd_scan.cuh"
#include "hvd_score.cuh"

namespace hvd {
namespace {

// How many tokens of a slab to ask the L2 for ahead of the wait for the previous kernel.  The length is read
// while that kernel may still be about to raise it (a commit appends at most k_cap + 1 tokens), so it is only a hint:
// it sizes a prefetch and nothing else, and whatever it holds, the range stays inside the slab.
__device__ __forceinline__ int length_ahead(const LookupArgs& a, int b, int cap_b) {
    const int hint = *reinterpret_cast<const volatile int32_t*>(a.hist_len + b);
    return (int)min((int64_t)min(cap_b, a.n_max), (int64_t)max(hint, 0) + a.k_cap + 1);
}

template <int THREADS, int ITER, bool FUSED>
__global__ void __launch_bounds__(THREADS, (THREADS == 1024 ? 1 : (THREADS == 512 ? 2 : 4))) lookup_kernel(const LookupArgs a, const ScoreArgs sa) {
    __shared__ float s_hid[FUSED ? HVD_MAX_HIDDEN : 1];
    // requests run fastest: with ragged lengths the CTAs of the low chunks, which every request has, are
    // dispatched first and the empty ones come last (chunks move to x when they outgrow the y range)
    const int b = a.chunks_on_x ? blockIdx.y : blockIdx.x;
    const int chunk = a.chunks_on_x ? blockIdx.x : blockIdx.y;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    // The next kernel may come in at once when it does nothing ahead of its own wait.  A successor that does
    // (the corpus probe reads the histories there) must not start before this kernel's predecessor, which may
    // have written them, is known to be complete: then the wait comes first.
    const bool late = !FUSED && a.successor_works_ahead;  // the fused form is never followed by such a kernel
    if (!late) pdl_trigger();
    constexpr int CHUNK = THREADS * kLookupTokPerVec * ITER;  // tokens of the aligned grid per CTA
    // The request's scalars are fetched together, before any of them is looked at: the kernel is a chain of
    // dependent round trips and this keeps them to one.  The shapes for one request per SM (8 K to 32 K tokens)
    // split that round trip: where the slab lies and how long it can get is never written by a kernel of this
    // library, so it is read ahead of the wait for the previous kernel, and the L2 is asked for the slab; when the
    // previous kernel is still running, the scan finds its tokens in the L2 (step of 64 x 16 K tokens 47.1 -> 46.5 us, of
    // 128 x 32 K tokens 159.0 -> 157.5 us).  When it is not, the second round trip costs up to 0.7 us; the shapes for
    // short histories and for more than one request per SM gained nothing in a step and do not do this.
    constexpr bool AHEAD = THREADS == 1024 && ITER >= 4;
    int n_raw, cap_b, K_b;
    int64_t off_b;
    if constexpr (AHEAD) {
        cap_b = a.hist_cap[b];
        off_b = a.hist_off[b];
        K_b = a.K[b];
        if (warp == 0) {
            const int32_t* first = a.hist + off_b;
            const int skip = (int)((4 - ((reinterpret_cast<uintptr_t>(first) >> 2) & 3)) & 3);
            prefetch_history_l2(first + skip + chunk * CHUNK, min(CHUNK, length_ahead(a, b, cap_b) - skip - chunk * CHUNK), lane);
        }
        pdl_wait();
        if (late) pdl_trigger();
        n_raw = a.hist_len[b];
    } else {
        pdl_wait();
        if (late) pdl_trigger();
        n_raw = a.hist_len[b];
        cap_b = a.hist_cap[b];
        off_b = a.hist_off[b];
        K_b = a.K[b];
    }
    const int32_t* __restrict__ slab = a.hist + off_b;
    // 128-bit loads run on the 16-byte grid, which starts at the first 16-byte boundary inside the slab: the
    // `head` (0 to 3) tokens in front of it are looked at one by one, by the first warp of the first chunk, so
    // that a history of 2^k tokens takes 2^k / CHUNK chunks whatever its alignment
    const int head = (int)((4 - ((reinterpret_cast<uintptr_t>(slab) >> 2) & 3)) & 3);
    int n = n_raw;
    if (n < 0 || n > cap_b || n > a.n_max) n = 0;  // unusable length: empty history
    // candidate positions p (index of the matched copy's last token) are 0 .. n-2; grid position g is p - head
    const int g_end = (n >= 2) ? max(n - 1 - head, 0) : 0;  // exclusive end on the aligned grid
    const int n_chunks = (n >= 2) ? max((g_end + CHUNK - 1) / CHUNK, 1) : 0;

    if (n_chunks == 0) {
        if (chunk == 0 && warp == 0) {
            for (int j = lane; j < a.k_cap; j += 32) a.draft[(int64_t)b * a.k_cap + j] = -1;
            if (lane == 0) {
                a.draft_len[b] = 0; a.match_len[b] = 0; a.match_pos[b] = -1; a.match_cnt[b] = 0;
            }
            if (FUSED) score_select_request(sa, b, lane, s_hid, n_raw, 0, 0, -1, 0, -1, -1);
        }
        return;
    }
    if (chunk >= n_chunks) return;

    const int4* __restrict__ vbase = reinterpret_cast<const int4*>(slab + head);
    const int v0 = chunk * (CHUNK / 4);

    // At most DEPTH vectors per thread are in flight: with more than that to scan, the register that a vector has
    // just left takes the load DEPTH vectors ahead (a ring; the indices are static once unrolled).  Shapes of up
    // to 8 loads issue them all up front.  The 16-load shape (batches above one request per SM) keeps 4 in
    // flight: all 16 at once spilled registers and filled the load/store unit's queues (C3 lookup 12.0 us; ring
    // of 12: 11.0, 8: 10.7, 6 and 4: 10.0, 3: 10.1, 2: 10.5).
    constexpr int DEPTH = ITER > 8 ? 4 : ITER;
    auto load_vec = [&](int i) -> int4 {
        const int v = v0 + i * THREADS + tid;
        // (bounds-checked builds: the last aligned vector may reach up to 3 tokens past the slab's end)
        if (4 * v < g_end && HVD_IN_BOUNDS(a.dev_error, 4 * v + head, 0, (int64_t)cap_b + 1)) return ld_hist(vbase + v);
        return make_int4(0, 0, 0, 0);
    };
    int4 x[DEPTH];
#pragma unroll
    for (int i = 0; i < DEPTH; ++i) x[i] = load_vec(i);
    // query: the history's own tail.  q0 = last token; lane j keeps the tokens 1+j and 33+j back.
    const int32_t q0 = HVD_IN_BOUNDS(a.dev_error, n - 1, 0, cap_b) ? slab[n - 1] : 0;
    const int32_t qa = (1 + lane <= n - 1 && HVD_IN_BOUNDS(a.dev_error, n - 2 - lane, 0, cap_b)) ? slab[n - 2 - lane] : 0;
    const int32_t qb = (33 + lane <= n - 1 && HVD_IN_BOUNDS(a.dev_error, n - 34 - lane, 0, cap_b)) ? slab[n - 34 - lane] : 0;

    Best best;  // identical in all lanes of a warp
    best.key = 0; best.cnt = 0;

#pragma unroll
    for (int i = 0; i < ITER; ++i) {
        const int p0 = 4 * (v0 + i * THREADS + tid) + head;  // position of x[i].x
        const int4 xi = x[i % DEPTH];
        if (i + DEPTH < ITER) x[i % DEPTH] = load_vec(i + DEPTH);
        scan_vector(xi, p0, n, slab, q0, qa, qb, a.l_max, lane, [&](int L, int p) {
            Best c;
            c.key = ((unsigned long long)(uint32_t)L << 32) | (uint32_t)(p + 1);
            c.cnt = 1;
            best = combine(best, c);
        }, a.dev_error);
    }
    if (chunk == 0 && warp == 0 && head > 0) {
        // the tokens in front of the grid: positions 0 .. head - 1, as one more vector in lane 0
        int4 xh = make_int4(0, 0, 0, 0);
        if (lane == 0) {
            if (0 < head && 0 <= n - 2) xh.x = slab[0];
            if (1 < head && 1 <= n - 2) xh.y = slab[1];
            if (2 < head && 2 <= n - 2) xh.z = slab[2];
        }
        scan_vector(xh, lane == 0 ? 0 : -8, n, slab, q0, qa, qb, a.l_max, lane, [&](int L, int p) {
            Best c;
            c.key = ((unsigned long long)(uint32_t)L << 32) | (uint32_t)(p + 1);
            c.cnt = 1;
            best = combine(best, c);
        }, a.dev_error, head - 1);
    }

    __shared__ unsigned long long s_key[THREADS / 32];
    __shared__ uint32_t s_cnt[THREADS / 32];
    if (lane == 0) { s_key[warp] = best.key; s_cnt[warp] = best.cnt; }
    __syncthreads();
    if (warp != 0) return;

    Best r;
    r.key = lane < THREADS / 32 ? s_key[lane] : 0ull;
    r.cnt = lane < THREADS / 32 ? s_cnt[lane] : 0u;
    r = warp_combine(r);

    uint32_t last = 0;
    if (lane == 0) {
        if (n_chunks > 1) {
            LookupPartial* slot = a.partial + (int64_t)b * a.max_chunks + chunk;
            if (HVD_IN_BOUNDS(a.dev_error, chunk, 0, a.max_chunks)) { slot->key = r.key; slot->cnt = r.cnt; }
            __threadfence();
            const uint32_t old = atomicAdd(a.req_cnt + b, 1u);
            last = (old + 1 == (uint32_t)n_chunks) ? 1u : 0u;
        } else {
            last = 1;
        }
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (!last) return;

    if (n_chunks > 1) {
        __threadfence();
        Best t; t.key = 0; t.cnt = 0;
        const LookupPartial* slots = a.partial + (int64_t)b * a.max_chunks;
        for (int c = lane; c < n_chunks; c += 32) {
            Best o;
            o.key = __ldcg(&slots[c].key);
            o.cnt = __ldcg(&slots[c].cnt);
            t = combine(t, o);
        }
        r = warp_combine(t);
        if (lane == 0) a.req_cnt[b] = 0;  // scratch is zero at rest
    }

    int L = (int)(r.key >> 32);
    int e = (int)(uint32_t)(r.key & 0xffffffffu);
    int cnt = (int)r.cnt;
    int d = 0;
    if (L < a.min_match || L == 0) {
        L = 0; e = -1; cnt = 0;
    } else {
        d = min(draft_limit(K_b, a.k_cap, L, a.spec_factor, a.spec_offset), n - e);
    }
    const int tok0 = (lane < d && HVD_IN_BOUNDS(a.dev_error, e + lane, 0, n)) ? slab[e + lane] : -1;
    const int tok1 = (lane + 32 < d && HVD_IN_BOUNDS(a.dev_error, e + lane + 32, 0, n)) ? slab[e + lane + 32] : -1;
    if (FUSED) {
        // everything the scoring reads is requested before the lookup's own results are stored (a store
        // would hold back the loads behind it): draft tokens, decode state and model draft in one round trip
        const ModelDraft md = load_model_draft(sa, b, lane);
        score_select_request(sa, b, lane, s_hid, n_raw, d, L, e, cnt, tok0, tok1, &md);
    }
    if (lane < a.k_cap) a.draft[(int64_t)b * a.k_cap + lane] = tok0;
    if (lane + 32 < a.k_cap) a.draft[(int64_t)b * a.k_cap + lane + 32] = tok1;
    if (lane == 0) {
        a.draft_len[b] = d; a.match_len[b] = L; a.match_pos[b] = e; a.match_cnt[b] = cnt;
    }
}


// ---------------------------------------------------------------------------------------------------
// Cluster form of the chunked scan, for batches of long histories that fit the GPU in one wave: the chunk
// CTAs of a request (2 to 16 of them, 256 or 512 threads x 8 loads each) are one thread-block cluster, every CTA
// stores its partial result into the first CTA's shared memory (distributed shared memory) and one cluster
// barrier takes the place of partial -> fence -> arrival counter -> partials read again, i.e. of three
// dependent global round trips at the end of every request.  The hardware releases the barrier: nothing
// spins.  A cluster's CTAs are placed together and stay until the barrier, so this form is only taken when all
// clusters of the batch are resident at once (the launch code asks the occupancy calculator).
constexpr int kClusterIter = 8;
constexpr int kMaxClusterSize = 16;

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

template <int THREADS, bool FUSED>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? 4 : 2) lookup_cluster_kernel(const LookupArgs a, const ScoreArgs sa) {
    constexpr int ITER = kClusterIter, CHUNK = THREADS * kLookupTokPerVec * ITER;
    __shared__ float s_hid[FUSED ? HVD_MAX_HIDDEN : 1];
    __shared__ LookupPartial s_part[kMaxClusterSize];  // in the cluster's first CTA: one slot per CTA
    __shared__ unsigned long long s_key[THREADS / 32];
    __shared__ uint32_t s_cnt[THREADS / 32];
    const int b = blockIdx.y;
    const int chunk = blockIdx.x;  // = rank in the cluster: gridDim.x is the cluster size
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    cluster_arrive();  // "this CTA runs": matched by the wait in front of the store into the first CTA
    const bool late = !FUSED && a.successor_works_ahead;
    if (!late) pdl_trigger();
    // where the slab lies and how long it can get is never written by a kernel of this library: read ahead of the
    // wait for the previous kernel, and the L2 is asked for this CTA's part of the slab, so that the scan finds its
    // tokens there when the previous kernel is still running (C4 step 72.8 -> 71.6 us; a call that does not
    // overlap its predecessor pays 0.25 us for the second round trip)
    const int cap_b = a.hist_cap[b];
    const int64_t off_b = a.hist_off[b];
    const int K_b = a.K[b];
    const int32_t* __restrict__ slab = a.hist + off_b;
    const int head = (int)((4 - ((reinterpret_cast<uintptr_t>(slab) >> 2) & 3)) & 3);
    constexpr int CHUNK_AHEAD = THREADS * kLookupTokPerVec * kClusterIter;
    if (warp == 0)
        prefetch_history_l2(slab + head + chunk * CHUNK_AHEAD, min(CHUNK_AHEAD, length_ahead(a, b, cap_b) - head - chunk * CHUNK_AHEAD), lane);
    pdl_wait();
    if (late) pdl_trigger();
    const int n_raw = a.hist_len[b];
    int n = n_raw;
    if (n < 0 || n > cap_b || n > a.n_max) n = 0;  // unusable length: empty history
    const int g_end = (n >= 2) ? max(n - 1 - head, 0) : 0;
    const int n_chunks = (n >= 2) ? max((g_end + CHUNK - 1) / CHUNK, 1) : 0;
    const bool has_work = chunk < n_chunks;  // a CTA without work still goes through both barriers

    Best best;
    best.key = 0; best.cnt = 0;
    // the first CTA finishes the request: what the scoring reads is asked for half-way through its scan
    ModelDraft md;
    md.m = 0; md.t0 = -1; md.t1 = -1;
    hvd_req_state st_ahead;
    st_ahead.sel_bits = 0; st_ahead.acc_ring = 0;
    int prompt_ahead = 0;
    const bool ahead = FUSED && chunk == 0 && warp == 0;
    if (ahead && !has_work) {
        md = load_model_draft(sa, b, lane);
        st_ahead.sel_bits = __ldg(&sa.state[b].sel_bits);
        st_ahead.acc_ring = __ldg(reinterpret_cast<const unsigned long long*>(&sa.state[b].acc_ring));
        prompt_ahead = __ldg(sa.prompt_len + b);
    }
    if (has_work) {
        const int4* __restrict__ vbase = reinterpret_cast<const int4*>(slab + head);
        const int v0 = chunk * (CHUNK / 4);
        constexpr int DEPTH = THREADS == 512 ? 4 : ITER;  // vectors in flight per thread (C4: 8 -> 6.86 us, 4 -> 6.76, 2 -> 6.96)
        auto load_vec = [&](int i) -> int4 {
            const int v = v0 + i * THREADS + tid;
            if (4 * v < g_end && HVD_IN_BOUNDS(a.dev_error, 4 * v + head, 0, (int64_t)cap_b + 1)) return ld_hist(vbase + v);
            return make_int4(0, 0, 0, 0);
        };
        int4 x[DEPTH];
#pragma unroll
        for (int i = 0; i < DEPTH; ++i) x[i] = load_vec(i);
        const int32_t q0 = HVD_IN_BOUNDS(a.dev_error, n - 1, 0, cap_b) ? slab[n - 1] : 0;
        const int32_t qa = (1 + lane <= n - 1 && HVD_IN_BOUNDS(a.dev_error, n - 2 - lane, 0, cap_b)) ? slab[n - 2 - lane] : 0;
        const int32_t qb = (33 + lane <= n - 1 && HVD_IN_BOUNDS(a.dev_error, n - 34 - lane, 0, cap_b)) ? slab[n - 34 - lane] : 0;
        auto take = [&](int L, int p) {
            Best c;
            c.key = ((unsigned long long)(uint32_t)L << 32) | (uint32_t)(p + 1);
            c.cnt = 1;
            best = combine(best, c);
        };
#pragma unroll
        for (int i = 0; i < ITER; ++i) {
            if (FUSED && i == ITER / 2 && ahead) {
                md = load_model_draft(sa, b, lane);
                st_ahead.sel_bits = __ldg(&sa.state[b].sel_bits);
                st_ahead.acc_ring = __ldg(reinterpret_cast<const unsigned long long*>(&sa.state[b].acc_ring));
                prompt_ahead = __ldg(sa.prompt_len + b);
            }
            const int p0 = 4 * (v0 + i * THREADS + tid) + head;
            const int4 xi = x[i % DEPTH];
            if (i + DEPTH < ITER) x[i % DEPTH] = load_vec(i + DEPTH);
            scan_vector(xi, p0, n, slab, q0, qa, qb, a.l_max, lane, take, a.dev_error);
        }
        if (chunk == 0 && warp == 0 && head > 0) {  // the tokens in front of the grid, as one more vector in lane 0
            int4 xh = make_int4(0, 0, 0, 0);
            if (lane == 0) {
                if (0 < head && 0 <= n - 2) xh.x = slab[0];
                if (1 < head && 1 <= n - 2) xh.y = slab[1];
                if (2 < head && 2 <= n - 2) xh.z = slab[2];
            }
            scan_vector(xh, lane == 0 ? 0 : -8, n, slab, q0, qa, qb, a.l_max, lane, take, a.dev_error, head - 1);
        }
    }
    if (lane == 0) { s_key[warp] = best.key; s_cnt[warp] = best.cnt; }
    __syncthreads();
    Best r;
    r.key = 0; r.cnt = 0;
    if (warp == 0) {
        r.key = lane < THREADS / 32 ? s_key[lane] : 0ull;
        r.cnt = lane < THREADS / 32 ? s_cnt[lane] : 0u;
        r = warp_combine(r);
    }
    cluster_wait();  // every CTA of the cluster runs: the first one's shared memory may be written
    if (warp == 0 && lane == 0) {
        const uint32_t local = (uint32_t)__cvta_generic_to_shared(&s_part[chunk]);
        uint32_t remote;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(0));
        asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(remote), "l"(r.key) : "memory");
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(remote + 8u), "r"(r.cnt) : "memory");
    }
    cluster_arrive();
    cluster_wait();
    if (chunk != 0 || warp != 0) return;

    const int cs = (int)gridDim.x;
    Best t;
    t.key = 0; t.cnt = 0;
    if (lane < cs) { t.key = s_part[lane].key; t.cnt = s_part[lane].cnt; }
    r = warp_combine(t);
    int L = (int)(r.key >> 32);
    int e = (int)(uint32_t)(r.key & 0xffffffffu);
    int cnt = (int)r.cnt;
    int d = 0;
    if (L < a.min_match || L == 0) {
        L = 0; e = -1; cnt = 0;
    } else {
        d = min(draft_limit(K_b, a.k_cap, L, a.spec_factor, a.spec_offset), n - e);
    }
    const int tok0 = (lane < d && HVD_IN_BOUNDS(a.dev_error, e + lane, 0, n)) ? slab[e + lane] : -1;
    const int tok1 = (lane + 32 < d && HVD_IN_BOUNDS(a.dev_error, e + lane + 32, 0, n)) ? slab[e + lane + 32] : -1;
    if (FUSED) score_select_request(sa, b, lane, s_hid, n_raw, d, L, e, cnt, tok0, tok1, &md, &st_ahead, &prompt_ahead);
    if (lane < a.k_cap) a.draft[(int64_t)b * a.k_cap + lane] = tok0;
    if (lane + 32 < a.k_cap) a.draft[(int64_t)b * a.k_cap + lane + 32] = tok1;
    if (lane == 0) {
        a.draft_len[b] = d; a.match_len[b] = L; a.match_pos[b] = e; a.match_cnt[b] = cnt;
    }
}

template <int THREADS, bool FUSED>
cudaError_t launch_cluster(bool pdl, int cs, int B, cudaStream_t stream, const LookupArgs& a, const ScoreArgs& sa) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)cs, (unsigned)B); cfg.blockDim = dim3(THREADS); cfg.dynamicSmemBytes = 0; cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, lookup_cluster_kernel<THREADS, FUSED>, a, sa);
}

template <int THREADS, bool FUSED>
int resident_clusters(int cs) {
    if (cs > 8 && cudaFuncSetAttribute(lookup_cluster_kernel<THREADS, FUSED>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)cs, 1024u); cfg.blockDim = dim3(THREADS);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, lookup_cluster_kernel<THREADS, FUSED>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return n;
}

}  // namespace

// How many clusters of 2, 4, 8 and 16 CTAs of the cluster kernel are resident together on this device (0: that
// size cannot be launched): asked once per context.
void lookup_cluster_setup(hvd_ctx* ctx) {
    for (int k = 0; k < 4; ++k) {
        const int cs = 2 << k;
        const int n0 = resident_clusters<256, false>(cs), n1 = resident_clusters<256, true>(cs);
        ctx->lk_clusters[0][k] = n0 < n1 ? n0 : n1;
        const int m0 = resident_clusters<512, false>(cs), m1 = resident_clusters<512, true>(cs);
        ctx->lk_clusters[1][k] = m0 < m1 ? m0 : m1;
    }
}

hvd_status launch_lookup(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                         const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K,
                         int32_t n_max, int32_t* draft, int32_t* draft_len, int32_t* match_len,
                         int32_t* match_pos, int32_t* match_cnt, const ScoreArgs* fused, cudaStream_t stream,
                         bool successor_works_ahead) {
    LookupArgs a;
    a.B = B;
    a.dev_error = ctx->dev_error;
    a.successor_works_ahead = successor_works_ahead;
    a.hist = hist; a.hist_off = hist_off; a.hist_cap = hist_cap; a.hist_len = hist_len; a.K = K;
    a.n_max = n_max;
    a.draft = draft; a.draft_len = draft_len; a.match_len = match_len; a.match_pos = match_pos;
    a.match_cnt = match_cnt;
    a.partial = ctx->lk_partial; a.req_cnt = ctx->lk_cnt; a.max_chunks = ctx->lk_max_chunks;
    a.k_cap = ctx->cfg.k_cap; a.l_max = ctx->cfg.l_max; a.min_match = ctx->cfg.min_match;
    a.spec_factor = ctx->cfg.spec_factor; a.spec_offset = ctx->cfg.spec_offset;

    // aligned-grid tokens to cover: at most n_max - 1 candidates (the tokens in front of a slab's first 16-byte
    // boundary are not on the grid)
    const int64_t span = (int64_t)(n_max > 1 ? n_max - 1 : 1);
    // The kernel is a chain of dependent global round trips, and a request that fits one CTA skips
    // two of them (no partials, no last-arrival counter): take the smallest CTA shape that covers
    // the candidate positions, up to 32 K tokens (128 KB in flight).  Longer histories are cut into chunks of
    // 8 K tokens (256 threads x 8 loads, four CTAs per SM).
    struct Shape { int threads, iter; };
    // single-CTA shapes by size class (wide CTAs with few loads per thread finish soonest), then
    // the chunk shape for longer histories
    static const Shape shapes[] = {{256, 1}, {256, 2}, {512, 2}, {1024, 2}, {1024, 4}, {1024, 8}, {512, 16}, {256, 8}};
    int pick = 7;
    for (int k = 0; k < 6; ++k)
        if ((int64_t)shapes[k].threads * kLookupTokPerVec * shapes[k].iter >= n_max - 1) { pick = k; break; }
    // 32 K tokens: one 1024-thread CTA per SM; with more requests than SMs, two 512-thread CTAs per SM
    if (pick == 5 && B > ctx->num_sms) pick = 6;
    const int64_t chunk = (int64_t)shapes[pick].threads * kLookupTokPerVec * shapes[pick].iter;
    const int64_t chunks = (span + chunk - 1) / chunk;
    if (chunks > ctx->lk_max_chunks) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_lookup: n_max exceeds max_hist_len");
    if (pick == 7 && chunks > 1 && ctx->lk_cluster_mode != 0) {
        // a request's chunks as one cluster, when every cluster of the batch is resident at once: chunks of 8 K
        // tokens (256 threads) if that many clusters fit, else of 16 K tokens (512 threads, half as many CTAs)
        for (int t = 0; t < 2; ++t) {
            const int64_t c = (span + (chunk << t) - 1) / (chunk << t);
            if (c < 2 || c > kMaxClusterSize) continue;
            int k = 0;
            while ((2 << k) < c) ++k;
            if (B > ctx->lk_clusters[t][k]) continue;
            a.chunks_on_x = true;
            const ScoreArgs sa = fused ? *fused : ScoreArgs();
            const bool pdl = (ctx->pdl_mask & 2) != 0;
            cudaError_t e;
            if (t == 0) e = fused ? launch_cluster<256, true>(pdl, 2 << k, B, stream, a, sa) : launch_cluster<256, false>(pdl, 2 << k, B, stream, a, sa);
            else e = fused ? launch_cluster<512, true>(pdl, 2 << k, B, stream, a, sa) : launch_cluster<512, false>(pdl, 2 << k, B, stream, a, sa);
            HVD_CUDA_TRY(ctx, e);
            return HVD_OK;
        }
    }
    a.chunks_on_x = chunks > 65535;
    const dim3 grid = a.chunks_on_x ? dim3((unsigned)chunks, (unsigned)B) : dim3((unsigned)B, (unsigned)chunks);
    cudaError_t e;
    const ScoreArgs sa = fused ? *fused : ScoreArgs();
#define HVD_LAUNCH_LOOKUP(TH, I)                                                                       \
    (fused ? launch_kernel((ctx->pdl_mask & 2), lookup_kernel<TH, I, true>, grid, TH, 0, stream, a, sa)      \
           : launch_kernel((ctx->pdl_mask & 2), lookup_kernel<TH, I, false>, grid, TH, 0, stream, a, sa))
    switch (pick) {
        case 0: e = HVD_LAUNCH_LOOKUP(256, 1); break;
        case 1: e = HVD_LAUNCH_LOOKUP(256, 2); break;
        case 2: e = HVD_LAUNCH_LOOKUP(512, 2); break;
        case 3: e = HVD_LAUNCH_LOOKUP(1024, 2); break;
        case 4: e = HVD_LAUNCH_LOOKUP(1024, 4); break;
        case 5: e = HVD_LAUNCH_LOOKUP(1024, 8); break;
        case 6: e = HVD_LAUNCH_LOOKUP(512, 16); break;
        default: e = HVD_LAUNCH_LOOKUP(256, 8); break;
    }
#undef HVD_LAUNCH_LOOKUP
    HVD_CUDA_TRY(ctx, e);
    return HVD_OK;
}

}  // namespace hvd
