// Greedy verification and commit (Sec. 3.1 Verify, Sec. 3.4, Algorithm 1), as two kernels.
//
// verify_stream_kernel: a bandwidth-bound stream over the logits rows that are actually needed
// (rows 0..sel_len of each request).  Under that stream every other global access takes
// microseconds, so the streaming warps touch global memory for nothing but the logits, one
// counter fetch that is issued two units before its answer is needed, and fire-and-forget atomic
// maxima:
//  * Phase 0 (once per CTA): the number of needed rows per request, its prefix over requests and
//    the first logits row of each request go to shared memory.  The needed rows, laid end to
//    end, are cut into batches of 32*kVerifyUnroll 128-bit vectors (4 KB: what one warp loads with
//    all its loads in flight) and into units of kVerifyUnitBatches batches.
//  * Warps draw units from kVerifyQueues global counters (unit numbers interleaved over the
//    queues; one counter cannot serve more than one fetch per ~1.5 ns under load), so SMs that
//    get less DRAM bandwidth take fewer units (per-SM rates differ by up to 2x on this part, and
//    static splits lose a third of the bandwidth to the slowest SMs).  A warp whose queue runs
//    dry tries the next queue once.
//  * A lane keeps, for each of its packed element slots, the running maximum and the load that
//    raised it (three instructions per two bf16 logits); one warp reduction per batch gives the
//    exact (maximum, lowest index), which is folded into the row's 64-bit key in global scratch
//    with an atomic max whose result nobody waits for.
// verify_commit_kernel: one warp per request reads the row keys (the kernel boundary orders them
// after every atomic), turns them into target tokens, compares them with the draft, commits, and
// puts the scratch back to zero.
// verify_small_kernel: the streaming kernel for logits of up to 160 MB (one warp per batch, no queues).
// No warp waits for another.
#include <cuda_bf16.h>

#include <algorithm>

#include "hvd_commit.cuh"

namespace hvd {
namespace {

constexpr int T = kVerifyThreads;
constexpr int NW = T / 32;
constexpr int U = kVerifyUnroll;
constexpr int UB = kVerifyUnitBatches;
constexpr int Q = kVerifyQueues;
constexpr int kQueueStride = kVerifyQueueStride;
static_assert(NW % Q == 0, "every CTA must serve every queue equally");
constexpr int kBatchVec = 32 * U;  // vectors a warp loads per batch
constexpr uint32_t kFull = 0xffffffffu;
static_assert(U <= 8, "the load number must fit the packed 16-bit tracking");

// order-preserving map float -> uint32 with -0.0 folded onto +0.0 (0 is never produced by a
// non-NaN value, so 0 can stand for "nothing")
__device__ __forceinline__ uint32_t ord32(float f) {
    uint32_t b = __float_as_uint(f);
    if ((b << 1) == 0) b = 0;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// The logits are read once and are larger than the L2: they bypass the L1 and are marked to leave the
// L2 first, so that what the other kernels of a step reuse (histories, per-request arrays, predictor
// weights) is still there when the stream has passed.
__device__ __forceinline__ unsigned long long stream_policy() {
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p, unsigned long long pol) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(pol));
    return v;
}

// Per-lane argmax over the (up to) U vectors of one batch.  best(): order key of the maximum and
// the offset, inside the batch, of its first occurrence: (load u * 32 + lane) * kPerVec + k.
template <typename E>
struct Tracker;

template <>
struct Tracker<float> {
    static constexpr int kPerVec = 4;
    float v[4];
    int u[4];
    __device__ static __forceinline__ float scalar(const void* row, int64_t i) {
        return static_cast<const float*>(row)[i];
    }
    __device__ __forceinline__ void init(const uint4& x) {
        v[0] = __uint_as_float(x.x); v[1] = __uint_as_float(x.y);
        v[2] = __uint_as_float(x.z); v[3] = __uint_as_float(x.w);
        u[0] = u[1] = u[2] = u[3] = 0;
    }
    __device__ __forceinline__ void fold(const uint4& x, int load) {
        const float y[4] = {__uint_as_float(x.x), __uint_as_float(x.y), __uint_as_float(x.z), __uint_as_float(x.w)};
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (y[k] > v[k]) { v[k] = y[k]; u[k] = load; }
    }
    __device__ __forceinline__ void best(int lane, uint32_t& ord, uint32_t& off) const {
        ord = 0u; off = 0xffffffffu;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t o = ord32(v[k]);
            const uint32_t f = (uint32_t)((u[k] * 32 + lane) * 4 + k);
            if (o > ord || (o == ord && f < off)) { ord = o; off = f; }
        }
    }
};

template <>
struct Tracker<__nv_bfloat16> {
    static constexpr int kPerVec = 8;
    uint32_t v[4];  // packed maxima: element 2c in the low half of v[c], 2c+1 in the high half
    uint32_t u[4];  // packed load numbers, same layout
    __device__ static __forceinline__ float scalar(const void* row, int64_t i) {
        return __uint_as_float((uint32_t)static_cast<const uint16_t*>(row)[i] << 16);  // widening is exact
    }
    __device__ static __forceinline__ uint32_t max2(uint32_t a, uint32_t b) {
        uint32_t d;
        asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
        return d;
    }
    __device__ static __forceinline__ uint32_t gt2(uint32_t a, uint32_t b) {  // 0xffff per half with a > b
        uint32_t d;
        asm("set.gt.u32.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
        return d;
    }
    __device__ __forceinline__ void init(const uint4& x) {
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
        u[0] = u[1] = u[2] = u[3] = 0u;
    }
    __device__ __forceinline__ void fold(const uint4& x, int load) {
        const uint32_t y[4] = {x.x, x.y, x.z, x.w};
        const uint32_t tag = (uint32_t)load * 0x00010001u;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint32_t m = gt2(y[c], v[c]);
            v[c] = max2(v[c], y[c]);
            u[c] = (u[c] & ~m) | (tag & m);
        }
    }
    __device__ static __forceinline__ uint32_t eq2(uint32_t a, uint32_t b) {  // 0xffff per equal half
        uint32_t d;
        asm("set.eq.u32.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
        return d;
    }
    __device__ static __forceinline__ uint32_t minu2(uint32_t a, uint32_t b) {
        uint32_t d;
        asm("min.u16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
        return d;
    }
    // all in packed form: the lane maximum, then the smallest (load, slot) among the slots equal to it
    __device__ __forceinline__ void best(int lane, uint32_t& ord, uint32_t& off) const {
        const uint32_t m = max2(max2(v[0], v[1]), max2(v[2], v[3]));
        const float vmax = fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xffff0000u));
        const uint32_t h = __float_as_uint(vmax) >> 16;
        const uint32_t mm = h | (h << 16);
        uint32_t cand = 0xffffffffu;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint32_t e = eq2(v[c], mm);
            const uint32_t k = (u[c] << 3) | (uint32_t)(((2 * c + 1) << 16) | (2 * c));  // (load << 3 | slot) per half
            cand = minu2(cand, (k & e) | ~e);
        }
        const uint32_t b16 = min(cand & 0xffffu, cand >> 16);
        ord = ord32(vmax);
        off = ((b16 >> 3) * 32u + (uint32_t)lane) * 8u + (b16 & 7u);
    }
};

// Commit of one request whose draft is a token TREE (node i: token sel_draft[i], parent[i] in
// {-1, 0..i-1}; logits row 0 follows the prefix, row i+1 follows node i), by one warp.  The walk
// starts at the prefix; at each node the target's token is the argmax of that node's row; the first
// child that carries it is accepted, else the walk stops and that token is the last one committed.
__device__ __forceinline__ void commit_tree_request(const VerifyArgs& a, int b, int lane) {
    const int kc = a.k_cap;
    const int32_t* d = a.sel_draft + (int64_t)b * kc;
    const int32_t* par = a.parent + (int64_t)b * kc;
    int dt[2], pr[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {  // nodes lane, lane+32 (k_cap <= 64)
        const int node = lane + 32 * k;
        dt[k] = node < kc ? d[node] : -1;
        pr[k] = node < kc ? par[node] : -2;
    }
    const int64_t hoff = a.hist_off[b];
    const int sel = a.select[b];
    hvd_req_state st = a.state[b];
    const int n = a.hist_len[b];
    const int cap = a.hist_cap[b];
    const Req q = load_req(a, b);
    int32_t* z = a.committed + (int64_t)b * (kc + 1);
    if (q.nr == 0) {
        for (int j = lane; j <= kc; j += 32) z[j] = -1;
        if (a.target_tok)
            for (int64_t r = q.r0 + lane; r < q.r1; r += 32)
                if (HVD_IN_BOUNDS(a.dev_error, r, 0, a.total_rows)) a.target_tok[r] = -1;
        if (lane == 0) { a.accepted[b] = 0; a.n_commit[b] = 0; a.status[b] = HVD_REQ_BAD_LEN; }
        return;
    }
    const int m = q.nr - 1;
    pdl_wait();
    int tok[3];  // target tokens of rows lane, lane+32, lane+64
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        const int i = lane + 32 * k;
        tok[k] = 0;
        if (i <= m) {
            const unsigned long long key = read_row_key(a, q.r0 + i);
            const int t = (int)(~(uint32_t)(key & 0xffffffffu));
            tok[k] = (int)min((int64_t)max(t, 0), a.V - 1);
            if (a.target_tok && HVD_IN_BOUNDS(a.dev_error, q.r0 + i, 0, a.total_rows)) a.target_tok[q.r0 + i] = tok[k];
        }
    }
    if (a.target_tok)
        for (int64_t r = q.r0 + q.nr + lane; r < q.r1; r += 32)
            if (HVD_IN_BOUNDS(a.dev_error, r, 0, a.total_rows)) a.target_tok[r] = -1;
    int zr[3] = {-1, -1, -1};  // committed tokens lane, lane+32, lane+64
    int acc = 0, cur = -1;
    for (;;) {
        const int row = cur + 1;
        const int t0 = __shfl_sync(kFull, tok[0], row & 31);
        const int t1 = __shfl_sync(kFull, tok[1], row & 31);
        const int t2 = __shfl_sync(kFull, tok[2], row & 31);
        const int want = row < 32 ? t0 : (row < 64 ? t1 : t2);  // the target's token after the current node
        if ((acc & 31) == lane) zr[acc >> 5] = want;             // accepted tokens equal the target's tokens
        const bool ok0 = lane < m && lane > cur && pr[0] == cur && dt[0] == want;
        const bool ok1 = lane + 32 < m && lane + 32 > cur && pr[1] == cur && dt[1] == want;
        const uint32_t b0 = __ballot_sync(kFull, ok0), b1 = __ballot_sync(kFull, ok1);
        if ((b0 | b1) == 0u) break;
        cur = b0 ? __ffs(b0) - 1 : 32 + __ffs(b1) - 1;
        ++acc;
    }
    const int room = cap - n;
    const int w = min(acc + 1, room);
    int32_t* h = a.hist + hoff;
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        const int j = lane + 32 * k;
        if (j <= kc) {
            const int tk = j <= acc ? zr[k] : -1;
            z[j] = tk;
            if (j < w && HVD_IN_BOUNDS(a.dev_error, n + j, 0, cap)) h[n + j] = tk;
        }
    }
    if (lane == 0) {
        a.hist_len[b] = n + w;
        a.n_commit[b] = w;
        a.accepted[b] = acc;
        a.status[b] = (w < acc + 1) ? HVD_REQ_CAPACITY : HVD_REQ_OK;
        st.sel_bits = (st.sel_bits << 1) | (sel ? 1u : 0u);
        st.acc_ring = (st.acc_ring << 8) | (unsigned long long)(acc & 0xff);
        a.state[b] = st;
    }
}

constexpr int kCommitWarps = 4;

__global__ void __launch_bounds__(kCommitWarps * 32) verify_commit_kernel(const VerifyArgs a) {
    const int b = blockIdx.x * kCommitWarps + (threadIdx.x >> 5);
    pdl_trigger();
    // launched ahead of the streaming kernel's end when the launch allows it: the request's own data is
    // fetched at once, the wait for the row keys sits inside the commit
    if (b < a.B) {
        if (a.parent) commit_tree_request(a, b, threadIdx.x & 31);
        else commit_request(a, b, threadIdx.x & 31);
    }
    pdl_wait();
    if (b == 0 && (threadIdx.x & 31) < Q) a.next_unit[(threadIdx.x & 31) * kQueueStride] = 0u;  // zero at rest
}

// Row keys of one vocabulary shard, for a reduction across ranks: indices become global (v_offset),
// the order becomes that of signed 64-bit integers (so that a plain MAX all-reduce picks the larger
// value and, among equal values, the lower global index), rows that were not read become the
// smallest integer; the unit counters go back to zero.
__global__ void keys_finish_kernel(unsigned long long* row_key, long long* keys, int64_t total_rows, int64_t v_offset,
                                   uint32_t* next_unit) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    pdl_trigger();
    pdl_wait();
    if (r < Q) next_unit[r * kQueueStride] = 0u;
    if (r >= total_rows) return;
    unsigned long long key = row_key[r];
    row_key[r] = 0ull;  // scratch is zero at rest
    if (key != 0ull) {
        const uint32_t idx = ~(uint32_t)(key & 0xffffffffu);
        key = (key & 0xffffffff00000000ull) | (uint32_t)(~(idx + (uint32_t)v_offset));
    }
    keys[r] = (long long)(key ^ kKeySign);
}

// Commit from row keys the caller hands in (reduced over the vocabulary shards of several ranks).
__global__ void __launch_bounds__(kCommitWarps * 32) commit_keys_kernel(const VerifyArgs a) {
    const int b = blockIdx.x * kCommitWarps + (threadIdx.x >> 5);
    pdl_trigger();
    pdl_wait();
    if (b < a.B) commit_request(a, b, threadIdx.x & 31);
}

// Prefix verification, between two streaming launches: one warp per request looks at the row keys of the window
// that has just been streamed (they stay in place for the commit) and decides whether the request goes on: every
// row of the window must carry its draft token, and rows must be left beyond the window.  A request that has
// met its first rejected token, or has used up its draft, is dead for all later windows.
__global__ void __launch_bounds__(kCommitWarps * 32) prefix_gate_kernel(const VerifyArgs a) {
    const int b = blockIdx.x * kCommitWarps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    pdl_trigger();
    bool go = false;
    if (b < a.B) {
        const Req q = load_req(a, b);
        const int m = q.nr - 1;
        const int lo = a.win_lo, hi = a.win_hi;
        const int32_t* d = a.sel_draft + (int64_t)b * a.k_cap;
        const int i0 = lo + lane, i1 = lo + lane + 32;  // a window has at most 64 rows
        const int d0 = (i0 < hi && i0 < m) ? d[i0] : -1;
        const int d1 = (i1 < hi && i1 < m) ? d[i1] : -1;
        pdl_wait();  // the row keys come from the streaming kernel, the flags from the gate before it
        const bool was = q.nr > 0 && hi <= m && (lo == 0 || a.alive[b] != 0);  // hi <= m: rows are left beyond the window
        // the target's token of a row, exactly as the commit reads it (inside the vocabulary whatever the data)
        auto token = [&](int i) {
            if (!HVD_IN_BOUNDS(a.dev_error, q.r0 + i, 0, a.total_rows)) return -2;
            const int t = (int)(~(uint32_t)(a.row_key[q.r0 + i] & 0xffffffffu));
            return (int)min((int64_t)max(t, 0), a.V - 1);
        };
        bool ok = true;
        if (was) {
            if (i0 < hi) ok = ok && token(i0) == d0;
            if (i1 < hi) ok = ok && token(i1) == d1;
        }
        go = was && __all_sync(0xffffffffu, ok);
        if (lane == 0) a.alive[b] = go ? 1 : 0;
    } else {
        pdl_wait();
    }
    if (b == 0 && lane < Q) a.next_unit[lane * kQueueStride] = 0u;  // the next launch draws its units from zero
}

struct Smem {
    long long* row0;  // [B] first logits row of each request
    int* pref;        // [B+1] exclusive prefix of needed rows over requests
    __device__ __forceinline__ Smem(unsigned char* base, int B) {
        row0 = reinterpret_cast<long long*>(base);
        pref = reinterpret_cast<int*>(base + (size_t)B * 8);
    }
};


template <typename E>
__global__ void __launch_bounds__(T, HVD_VERIFY_MIN_BLOCKS) verify_stream_kernel(const VerifyArgs a) {
    extern __shared__ __align__(16) unsigned char s_raw[];
    __shared__ int s_wsum[NW];
    __shared__ int s_carry;
    const Smem sm(s_raw, a.B);

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    constexpr int EPV = Tracker<E>::kPerVec;
    constexpr int ESZ = 16 / EPV;
    // wait first, then let the commit kernel in: it reads the selection before its own wait, so it must not
    // start before the kernel that wrote the selection (this kernel's predecessor) is known to be complete
    pdl_wait();
    pdl_trigger();

    // Unit u belongs to queue u % Q.  The first unit of a warp is the one with its own number
    // (queue warp % Q); the next one is requested now and its answer is looked at after the first
    // unit has been streamed.
    const uint32_t n_warps = gridDim.x * (uint32_t)NW;
    uint32_t cur = blockIdx.x * (uint32_t)NW + (uint32_t)warp;
    int queue = warp % Q;
    int tries = 0;  // queues found dry so far
    auto fetch = [&](int q) { return (n_warps / Q + atomicAdd(a.next_unit + q * kQueueStride, 1u)) * Q + (uint32_t)q; };
    uint32_t nxt = 0;
    if (lane == 0) nxt = fetch(queue);

    // ---- phase 0: rows needed per request (device data), prefix over requests ----------------------
    if (tid == 0) { s_carry = 0; sm.pref[0] = 0; }
    __syncthreads();
    for (int base = 0; base < a.B; base += T) {
        const int b = base + tid;
        int nr = 0;
        if (b < a.B) {
            const Req q = load_req(a, b);
            int64_t first;
            nr = streamed_rows(a, q, b, first);
            sm.row0[b] = first;
        }
        int v = nr;  // inclusive scan of nr over the tile
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(kFull, v, off);
            if (lane >= off) v += o;
        }
        if (lane == 31) s_wsum[warp] = v;
        __syncthreads();
        int wbase = 0;
#pragma unroll
        for (int k = 0; k < NW; ++k) wbase += (k < warp) ? s_wsum[k] : 0;
        const int carry = s_carry;
        if (b < a.B) sm.pref[b + 1] = carry + wbase + v;
        __syncthreads();
        if (tid == T - 1) s_carry = carry + wbase + v;
        __syncthreads();
    }

    const int nbr = a.n_batch_row;
    const int64_t total = (int64_t)sm.pref[a.B] * nbr;  // batches of all needed rows
    if (a.rows_read && !a.rows_in_commit && blockIdx.x == 0 && tid == 0) atomicAdd(a.rows_read, (unsigned long long)sm.pref[a.B]);
    // all but the last 1/2^HVD_VERIFY_ENDGAME_SHIFT (1/64) of the batches go out in units of UB, the rest one by one:
    // near the end a warp on a slow SM should not sit on more than it can finish quickly
    const uint32_t n_big = (uint32_t)((total - (total >> HVD_VERIFY_ENDGAME_SHIFT)) / UB);
    const uint32_t n_units = n_big + (uint32_t)(total - (int64_t)n_big * UB);
    const char* base_ptr = static_cast<const char*>(a.logits);
    const unsigned long long pol = stream_policy();

    // ---- phase 1: units of batches -------------------------------------------------------------------
    while (cur < n_units) {
        // `nxt` was requested a unit ago; the one after it is requested now, a whole unit before it is
        // needed (in the end game too: holding one single-batch unit back costs less than waiting for every
        // answer: measured 1.3 us per C2 launch, 17 us on C3)
        uint32_t nn = 0;
        nxt = __shfl_sync(kFull, nxt, 0);
        if (nxt >= n_units && tries == 0) {  // own queue is dry: one look at the neighbour queue
            tries = 1;
            queue = (queue + 1) % Q;
            if (lane == 0) nxt = fetch(queue);
            nxt = __shfl_sync(kFull, nxt, 0);
        }
        if (nxt < n_units) { if (lane == 0) nn = fetch(queue); }
        else nn = nxt;  // nothing left, stays so

        const int64_t c0 = cur < n_big ? (int64_t)cur * UB : (int64_t)n_big * UB + (cur - n_big);
        const int64_t c1 = cur < n_big ? c0 + UB : c0 + 1;
        int r = (int)(c0 / nbr);                // needed-row number of the batch
        int gb = (int)(c0 - (int64_t)r * nbr);  // batch number inside that row
        unsigned long long ukey = 0ull;         // best of the unit's batches in the current row
        int64_t grow = -1;
        // 128-bit grid inside the current row: `head` leading elements, n_vec full vectors, a tail
        const char* row = nullptr;
        const uint4* vrow = nullptr;
        int head = 0, n_vec = 0, tail = 0;
        int geom_r = -1;
#pragma unroll 1
        for (int64_t p = c0; p < c1; ++p, ++gb) {
            if (gb >= nbr) { gb -= nbr; ++r; }
            if (r != geom_r) {
                if (lane == 0 && ukey != 0ull && grow >= 0) atomicMax(a.row_key + grow, ukey);
                ukey = 0ull;
                geom_r = r;
                int lo = 0, hi = a.B;  // request of the row: largest b with pref[b] <= r
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (sm.pref[mid] <= r) lo = mid; else hi = mid;
                }
                grow = sm.row0[lo] + (r - sm.pref[lo]);
                if (!HVD_IN_BOUNDS(a.dev_error, grow, 0, a.total_rows)) { grow = -1; head = 0; n_vec = 0; tail = 0; continue; }
                row = base_ptr + grow * a.V * ESZ;
                const int head_bytes = (int)((16 - (reinterpret_cast<uintptr_t>(row) & 15)) & 15);
                head = (int)min((int64_t)(head_bytes / ESZ), a.V);
                n_vec = (int)((a.V - head) / EPV);
                tail = (int)(a.V - head - (int64_t)n_vec * EPV);
                vrow = reinterpret_cast<const uint4*>(row + (int64_t)head * ESZ);
            }
            const int left = n_vec - gb * kBatchVec;  // vectors of the row from this batch on
            const uint4* ptr = vrow + (int64_t)gb * kBatchVec + lane;

            uint32_t lord = 0u, loff = 0xffffffffu;  // this lane's maximum and its element index in the row
            // Every load of the batch is issued before any is used, in a full batch and in the ragged last
            // batch of a row alike (there the loads beyond the row are left out).  One code path with a
            // warp-uniform switch: two paths with a register array each spilled, and a ragged path that
            // loaded and folded in turn cost 2 us per C2 launch (one batch in 63 is ragged there).
            const bool full = left >= kBatchVec;
            if (full || lane < left) {
                uint4 x[U];
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (full || u * 32 + lane < left) x[u] = ld_stream(ptr + u * 32, pol);
                Tracker<E> t;
                t.init(x[0]);
#pragma unroll
                for (int u = 1; u < U; ++u)
                    if (full || u * 32 + lane < left) t.fold(x[u], u);
                t.best(lane, lord, loff);
                loff += (uint32_t)(head + gb * kBatchVec * EPV);
            }
            // the ragged edges of the row (at most 2*(EPV-1) elements) ride along with batch 0
            if (gb == 0 && lane < head + tail) {
                const int idx = lane < head ? lane : head + n_vec * EPV + (lane - head);
                const uint32_t eord = ord32(Tracker<E>::scalar(row, idx));
                if (eord > lord || (eord == lord && (uint32_t)idx < loff)) { lord = eord; loff = (uint32_t)idx; }
            }
            const uint32_t word = __reduce_max_sync(kFull, lord);
            const uint32_t widx = __reduce_min_sync(kFull, lord == word ? loff : 0xffffffffu);
            if (word != 0u && widx != 0xffffffffu) {
                const unsigned long long key = ((unsigned long long)word << 32) | (uint32_t)(~widx);
                ukey = key > ukey ? key : ukey;
            }
        }
        if (lane == 0 && ukey != 0ull && grow >= 0) atomicMax(a.row_key + grow, ukey);
        cur = nxt;
        nxt = nn;
    }
}

}  // namespace

// Small calls (a few requests, a few MB of logits): the time of the streaming kernel above is then its chain
// of dependent round trips (unit counters, per-request prefix, logits, atomic), not bandwidth.  Here one warp
// takes one 4 KB batch of one logits row, known from its block and warp number alone, and issues its loads at
// once; whether the row is needed at all (row <= sel_len of its request) is looked up while they are in
// flight, and only needed rows publish their maximum.  Rows beyond the selected draft are read in vain,
// which at these sizes costs less than finding out first.  Same keys, same result as the kernel above.
constexpr int kSmallWarps = 4;

template <typename E, bool SPEC>
__global__ void __launch_bounds__(kSmallWarps * 32) verify_small_kernel(const VerifyArgs a) {
    constexpr int EPV = Tracker<E>::kPerVec;
    constexpr int ESZ = 16 / EPV;
    const int lane = threadIdx.x & 31;
    const int gb = blockIdx.x * kSmallWarps + (threadIdx.x >> 5);  // batch inside the row
    const int64_t r = blockIdx.y;                                  // logits row
    if (!HVD_IN_BOUNDS(a.dev_error, r, 0, a.total_rows)) return;   // warp-uniform
    // wait first, then let the commit kernel in (it reads the selection before its own wait)
    pdl_wait();
    pdl_trigger();
    if (gb >= a.n_batch_row) return;

    const char* row = static_cast<const char*>(a.logits) + r * a.V * ESZ;
    const int head_bytes = (int)((16 - (reinterpret_cast<uintptr_t>(row) & 15)) & 15);
    const int head = (int)min((int64_t)(head_bytes / ESZ), a.V);
    const int n_vec = (int)((a.V - head) / EPV);
    const int tail = (int)(a.V - head - (int64_t)n_vec * EPV);
    const uint4* vrow = reinterpret_cast<const uint4*>(row + (int64_t)head * ESZ);
    const int left = n_vec - gb * kBatchVec;
    const uint4* ptr = vrow + (int64_t)gb * kBatchVec + lane;
    const unsigned long long pol = stream_policy();

    uint32_t lord = 0u, loff = 0xffffffffu;
    const bool full = left >= kBatchVec;
    uint4 x[U];
    if (SPEC && (full || lane < left)) {
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (full || u * 32 + lane < left) x[u] = ld_stream(ptr + u * 32, pol);
    }
    // the row's request and whether it needs the row (with SPEC: while the loads are in flight)
    bool needed = false;
    if (a.row_off && a.B <= 1024) {
        // Lane j fetches everything about request base + j in one round trip and the lane whose request owns
        // the row decides.  With more than 32 requests a first round trip over 32 evenly spaced entries of
        // row_off finds the block of (B + 31) / 32 <= 32 requests, from `base` on, that holds the row's owner.
        int base = 0;
        if (a.B > 32) {
            const int stride = (a.B + 31) / 32;
            const int j = min(lane * stride, a.B);
            const uint32_t below = __ballot_sync(kFull, a.row_off[j] <= r);  // lanes 0..s (row_off is sorted)
            base = below ? (31 - __clz((int)below)) * stride : 0;  // the owner is one of the next `stride` requests
        }
        const int jb = base + lane;
        const bool in = jb < a.B && lane < ((a.B > 32) ? (a.B + 31) / 32 : 32);
        const int64_t lo = in ? a.row_off[jb] : 0;
        const int64_t hi = in ? a.row_off[jb + 1] : 0;
        const int n = in ? a.hist_len[jb] : -1;
        const int cap = in ? a.hist_cap[jb] : 0;
        const int sl = in ? a.sel_len[jb] : 0;
        bool mine = in && lo <= r && r < hi;
        if (mine) {
            int nr = 0;
            if (n >= 0 && n <= cap && lo >= 0 && hi <= a.total_rows) {  // the rule of load_req
                int m = max(0, min(sl, a.k_cap));
                if ((int64_t)m > hi - lo - 1) m = (int)(hi - lo - 1);
                nr = m + 1;
            }
            mine = r - lo < nr;
        }
        needed = __any_sync(kFull, mine);
    } else {
        int b;
        if (a.row_off) {
            int lo = 0, hi = a.B;  // largest b with row_off[b] <= r
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (a.row_off[mid] <= r) lo = mid; else hi = mid;
            }
            b = (a.row_off[lo] <= r && r < a.row_off[lo + 1]) ? lo : -1;
        } else {
            b = (int)(r / (a.k_uniform + 1));
            if (b >= a.B) b = -1;
        }
        if (b >= 0) {
            const Req q = load_req(a, b);
            needed = r - q.r0 < q.nr;
        }
    }
    if (!SPEC) {
        if (!needed) return;  // warp-uniform
        if (full || lane < left) {
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (full || u * 32 + lane < left) x[u] = ld_stream(ptr + u * 32, pol);
        }
    }
    if (full || lane < left) {
        Tracker<E> t;
        t.init(x[0]);
#pragma unroll
        for (int u = 1; u < U; ++u)
            if (full || u * 32 + lane < left) t.fold(x[u], u);
        t.best(lane, lord, loff);
        loff += (uint32_t)(head + gb * kBatchVec * EPV);
    }
    if (gb == 0 && lane < head + tail) {  // the ragged edges of the row ride along with batch 0
        const int idx = lane < head ? lane : head + n_vec * EPV + (lane - head);
        const uint32_t eord = ord32(Tracker<E>::scalar(row, idx));
        if (eord > lord || (eord == lord && (uint32_t)idx < loff)) { lord = eord; loff = (uint32_t)idx; }
    }
    const uint32_t word = __reduce_max_sync(kFull, lord);
    const uint32_t widx = __reduce_min_sync(kFull, lord == word ? loff : 0xffffffffu);
    if (needed && lane == 0 && word != 0u && widx != 0xffffffffu)
        atomicMax(a.row_key + r, ((unsigned long long)word << 32) | (uint32_t)(~widx));
}

namespace {

// Prefix verification, early windows: while (nearly) every request is still alive, a window's rows are known from
// the grid alone -- block z is the request, block y the row inside the window, and one warp takes one 4 KB batch of
// that row, as in the kernel above.  The warp looks its request up (one round trip), leaves if the request is dead
// or has no such row, and streams its batch.  No work list, no queues: a launch of up to 160 MB starts and ends
// sooner than the persistent kernel (whose start and end game cost 8 to 10 us).
template <typename E>
__global__ void __launch_bounds__(kSmallWarps * 32) verify_window_kernel(const VerifyArgs a) {
    constexpr int EPV = Tracker<E>::kPerVec;
    constexpr int ESZ = 16 / EPV;
    const int lane = threadIdx.x & 31;
    const int gb = blockIdx.x * kSmallWarps + (threadIdx.x >> 5);  // batch inside the row
    const int b = blockIdx.z;
    pdl_wait();
    pdl_trigger();
    if (gb >= a.n_batch_row) return;
    const Req q = load_req(a, b);
    int64_t first;
    const int rows = streamed_rows(a, q, b, first);
    if ((int)blockIdx.y >= rows) return;  // warp-uniform
    const int64_t r = first + blockIdx.y;
    if (!HVD_IN_BOUNDS(a.dev_error, r, 0, a.total_rows)) return;

    const char* row = static_cast<const char*>(a.logits) + r * a.V * ESZ;
    const int head_bytes = (int)((16 - (reinterpret_cast<uintptr_t>(row) & 15)) & 15);
    const int head = (int)min((int64_t)(head_bytes / ESZ), a.V);
    const int n_vec = (int)((a.V - head) / EPV);
    const int tail = (int)(a.V - head - (int64_t)n_vec * EPV);
    const uint4* vrow = reinterpret_cast<const uint4*>(row + (int64_t)head * ESZ);
    const int left = n_vec - gb * kBatchVec;
    const uint4* ptr = vrow + (int64_t)gb * kBatchVec + lane;
    const unsigned long long pol = stream_policy();

    uint32_t lord = 0u, loff = 0xffffffffu;
    const bool full = left >= kBatchVec;
    if (full || lane < left) {
        uint4 x[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (full || u * 32 + lane < left) x[u] = ld_stream(ptr + u * 32, pol);
        Tracker<E> t;
        t.init(x[0]);
#pragma unroll
        for (int u = 1; u < U; ++u)
            if (full || u * 32 + lane < left) t.fold(x[u], u);
        t.best(lane, lord, loff);
        loff += (uint32_t)(head + gb * kBatchVec * EPV);
    }
    if (gb == 0 && lane < head + tail) {  // the ragged edges of the row ride along with batch 0
        const int idx = lane < head ? lane : head + n_vec * EPV + (lane - head);
        const uint32_t eord = ord32(Tracker<E>::scalar(row, idx));
        if (eord > lord || (eord == lord && (uint32_t)idx < loff)) { lord = eord; loff = (uint32_t)idx; }
    }
    const uint32_t word = __reduce_max_sync(kFull, lord);
    const uint32_t widx = __reduce_min_sync(kFull, lord == word ? loff : 0xffffffffu);
    if (lane == 0 && word != 0u && widx != 0xffffffffu)
        atomicMax(a.row_key + r, ((unsigned long long)word << 32) | (uint32_t)(~widx));
    if (a.rows_read && !a.rows_in_commit && gb == 0 && blockIdx.y == 0 && lane == 0) atomicAdd(a.rows_read, (unsigned long long)rows);
}

}  // namespace

size_t verify_dyn_smem(int32_t B) { return (size_t)B * 8 + (size_t)(B + 1) * 4; }

int verify_occupancy(hvd_dtype dtype, size_t dyn_smem) {
    int n = 0;
    cudaError_t e = cudaSuccess;
    {
        // Large batches need the opt-in shared memory size for the per-request tables.  The attribute belongs to
        // the device, not to a context: always opt in to the size of the largest batch a context can have, so
        // that a later context (or the allocation-free entry point) never lowers what an earlier one relies on.
        const int most = (int)verify_dyn_smem(8192);
        e = dtype == HVD_F32 ? cudaFuncSetAttribute(verify_stream_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, most)
                             : cudaFuncSetAttribute(verify_stream_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    }
    if (dtype == HVD_F32)
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, verify_stream_kernel<float>, T, dyn_smem);
    else
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, verify_stream_kernel<__nv_bfloat16>, T, dyn_smem);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return n;
}

hvd_status launch_verify_keys(hvd_ctx* ctx, VerifyArgs a, hvd_dtype dtype, long long* keys, int64_t v_offset,
                              cudaStream_t stream) {
    // the maxima gather in the context's row keys (zero at rest); the finishing kernel moves them out
    const hvd_status r = launch_verify(ctx, a, dtype, stream, false);
    if (r != HVD_OK) return r;
    const int64_t n = a.total_rows > Q ? a.total_rows : Q;
    HVD_CUDA_TRY(ctx, launch_kernel(ctx->pdl_mask != 0, keys_finish_kernel, dim3((unsigned)((n + 255) / 256)), 256, 0, stream,
                                    a.row_key, keys, a.total_rows, v_offset, a.next_unit));
    return HVD_OK;
}

hvd_status launch_commit_keys(hvd_ctx* ctx, VerifyArgs a, cudaStream_t stream) {
    HVD_CUDA_TRY(ctx, launch_kernel(false, commit_keys_kernel, (a.B + kCommitWarps - 1) / kCommitWarps,
                                    kCommitWarps * 32, 0, stream, a));
    return HVD_OK;
}

// Windows of prefix verification: needed rows [e[j], e[j+1]) are streamed by launch j.  A boundary between two
// windows costs what about 64 MiB of streaming costs (the tail of one launch, the gate, the start of the next:
// 8 to 10 us measured), so the first window takes at least that much of the batch (at least two rows), windows
// double from there (no request reads more than twice what it needs plus the first window), and no further
// boundary is set once what is left cannot repay it even if half of the requests die per window.  Small calls
// end up with one window: the plain verification.
static int prefix_edges(int k_cap, int64_t bytes_per_row_index, int64_t boundary, int* e) {
    int n = 0;
    e[n++] = 0;
    const int64_t per_row = bytes_per_row_index > 0 ? bytes_per_row_index : 1;
    const int64_t w0 = std::max<int64_t>(2, (boundary + per_row - 1) / per_row);
    int j = 1;
    for (int64_t x = w0; x < k_cap; x *= 2, ++j) {
        e[n++] = (int)x;
        if ((((int64_t)(k_cap + 1) - x) * per_row >> j) < 2 * boundary) break;
    }
    e[n++] = k_cap + 1;
    return n - 1;  // number of windows
}

int prefix_window_edges(const hvd_ctx* ctx, const VerifyArgs& a, hvd_dtype dtype, int* e) {
    return prefix_edges(a.k_cap, (int64_t)a.B * a.V * (dtype == HVD_F32 ? 4 : 2), ctx->vf_boundary_bytes, e);
}

// Window j of n_win: the streaming launch over rows [e[j], e[j+1]) of the requests still alive and, unless it is
// the last window, the gate that decides who goes on (flags in the context's scratch).
hvd_status launch_prefix_window(hvd_ctx* ctx, VerifyArgs a, hvd_dtype dtype, const int* e, int j, int n_win, cudaStream_t stream) {
    a.target_tok = nullptr;
    a.alive = ctx->vf_alive;
    a.win_lo = e[j]; a.win_hi = e[j + 1]; a.win_index = j;
    VerifyArgs s = a;
    if (j == 0) s.alive = nullptr;  // every request starts alive (the flags are written by the first gate)
    const hvd_status r = launch_verify(ctx, s, dtype, stream, false);
    if (r != HVD_OK) return r;
    if (j + 1 < n_win)
        HVD_CUDA_TRY(ctx, launch_kernel(ctx->pdl_commit, prefix_gate_kernel, (a.B + kCommitWarps - 1) / kCommitWarps,
                                        kCommitWarps * 32, 0, stream, a));
    return HVD_OK;
}

hvd_status launch_prefix_commit(hvd_ctx* ctx, VerifyArgs a, cudaStream_t stream) {
    a.target_tok = nullptr;
    a.win_lo = 0; a.win_hi = 0x7fffffff; a.alive = nullptr;
    HVD_CUDA_TRY(ctx, launch_kernel(ctx->pdl_commit, verify_commit_kernel, (a.B + kCommitWarps - 1) / kCommitWarps,
                                    kCommitWarps * 32, 0, stream, a));
    return HVD_OK;
}

hvd_status launch_verify_prefix(hvd_ctx* ctx, VerifyArgs a, hvd_dtype dtype, cudaStream_t stream) {
    int e[16];
    const int n_win = prefix_window_edges(ctx, a, dtype, e);
    a.target_tok = nullptr;
    if (n_win == 1) {  // the plain verification, whichever streaming kernel it takes; the commit counts the rows
        a.rows_in_commit = true;
        return launch_verify(ctx, a, dtype, stream, true);
    }
    for (int j = 0; j < n_win; ++j) {
        const hvd_status r = launch_prefix_window(ctx, a, dtype, e, j, n_win, stream);
        if (r != HVD_OK) return r;
    }
    return launch_prefix_commit(ctx, a, stream);
}

hvd_status launch_verify(hvd_ctx* ctx, VerifyArgs a, hvd_dtype dtype, cudaStream_t stream, bool with_commit) {
    const int per_sm = ctx->vf_blocks_per_sm[dtype == HVD_F32 ? 0 : 1];
    int grid = ctx->num_sms * (per_sm > 0 ? per_sm : 1);
    const int64_t esz = dtype == HVD_F32 ? 4 : 2;
    a.n_batch_row = (int32_t)((a.V * esz / 16 + kBatchVec - 1) / kBatchVec);
    if (a.n_batch_row < 1) a.n_batch_row = 1;
    // a small call gets no more warps than it can have units, but at least one CTA for every second SM
    // (measured on 36 rows of 32 000 floats: 74 to 96 CTAs 6.5 us, the full 592 CTAs 7.5 us, 72 CTAs 7.3 us,
    // 37 CTAs 9.4 us)
    const bool windowed = a.win_lo != 0 || a.win_hi != 0x7fffffff;
    const int64_t rows_upper = windowed ? std::min<int64_t>(a.total_rows, (int64_t)a.B * (a.win_hi - a.win_lo)) : a.total_rows;
    const int64_t units_upper = (rows_upper * (int64_t)a.n_batch_row + UB - 1) / UB;
    const int64_t want = std::max<int64_t>((units_upper + NW - 1) / NW, (ctx->num_sms + 1) / 2);
    if (want < grid) grid = (int)want;
    // unit numbers are 32-bit
    if (a.total_rows * (int64_t)a.n_batch_row / UB + 4 * (int64_t)grid * NW >= 0x7fffffffLL)
        return fail(ctx, HVD_ERR_UNSUPPORTED, "hvd_verify_commit: too many batches");
    const size_t smem = verify_dyn_smem(a.B);
    // By the full size of the logits (the needed part is only known on the device): up to 8 MB one warp per
    // batch with loads issued before the row is known to be needed, up to vf_small_bytes (160 MB) one warp
    // per batch that checks first, beyond that the persistent streaming kernel.  Measured, verify call with
    // about half the rows needed, bf16 rows of 128 256 (persistent kernel -> warp per batch): 4.4 MB 6.3 -> 3.8 us,
    // 17 MB 7.5 -> 5.5, 70 MB 11.2 -> 9.0, 140 MB 17.6 -> 14.5, 279 MB 27.8 -> 26.4; with (nearly) all rows
    // needed the persistent kernel is ahead from about 150 MB on (279 MB: 41.7 against 50.7 us).
    // Between vf_small_bytes and four times that (160 to 640 MB), when the row blocks are of about equal height, a
    // grid of (batch, row of the block, request) is hardly larger than the logits, and the kernel with that grid (a
    // warp knows its request and row from its block numbers, looks the request up and streams its batch: no work
    // list, no queues) starts and ends sooner than the persistent kernel.  Measured, step in us, persistent ->
    // grid: 209 MB 38.0 -> 35.8, 257 MB (C2) 46.4 -> 45.3, 397 MB 66.5 -> 63.9, 428 MB with a fifth of the rows not
    // needed (C4) 70.9 -> 71.1, 515 MB 81.8 -> 81.6; below 160 MB it equals the warp-per-batch kernels (17 MB 11.7 ->
    // 11.6, 70 MB 19.5 -> 19.1, 140 MB 27.5 -> 27.5), at 2.1 GB the persistent kernel is 6 us ahead, and on ragged
    // blocks the grid wastes its CTAs (C5: 345 against 321 us for the verify call).
    // Prefix verification: the first two windows (most requests still alive) of up to 640 MB take the grid kernel
    // over the window's rows; later windows the persistent kernel, whose work list leaves out the dead requests.
    // Measured, prefix step with the persistent kernel for every window -> with the grid kernel for the first two:
    // C2 37.9 -> 34.4 us, C3 141.0 -> 132.5, C4 70.6 -> 65.6 (windows of 74 to 156 MB), C5 168.1 -> 159.9 (262 MB).
    const int64_t full_bytes = a.total_rows * a.V * esz;
    const bool spec = full_bytes <= kVerifySpecBytes;
    bool by_grid = false;
    if (windowed) {
        by_grid = a.win_index < 2;
    } else if (!spec) {
        const int64_t block_rows = (a.row_off ? a.k_cap : a.k_uniform) + 1;  // rows of the tallest block
        by_grid = (int64_t)a.B * block_rows * 4 <= a.total_rows * 5 &&      // grid rows <= 1.25 x the rows there are
                  (int64_t)a.B * block_rows * a.V * esz > ctx->vf_small_bytes;
        if (by_grid) { a.win_lo = 0; a.win_hi = (int32_t)block_rows; a.win_index = 0; a.alive = nullptr; }
    }
    if (by_grid && a.B <= 65535 && a.win_hi - a.win_lo <= 65535 &&
        (int64_t)a.B * (a.win_hi - a.win_lo) * a.V * esz <= 4 * ctx->vf_small_bytes) {
        const dim3 wgrid((unsigned)((a.n_batch_row + kSmallWarps - 1) / kSmallWarps), (unsigned)(a.win_hi - a.win_lo), (unsigned)a.B);
        const bool pdl = (ctx->pdl_mask & 4);
        HVD_CUDA_TRY(ctx, dtype == HVD_F32 ? launch_kernel(pdl, verify_window_kernel<float>, wgrid, kSmallWarps * 32, 0, stream, a)
                                           : launch_kernel(pdl, verify_window_kernel<__nv_bfloat16>, wgrid, kSmallWarps * 32, 0, stream, a));
        if (with_commit)
            HVD_CUDA_TRY(ctx, launch_kernel(ctx->pdl_commit, verify_commit_kernel, (a.B + kCommitWarps - 1) / kCommitWarps,
                                            kCommitWarps * 32, 0, stream, a));
        return HVD_OK;
    }
    if (!windowed) { a.win_lo = 0; a.win_hi = 0x7fffffff; }
    const bool small = !windowed && a.total_rows <= 65535 && full_bytes <= ctx->vf_small_bytes;
    if (small) {
        const dim3 sgrid((unsigned)((a.n_batch_row + kSmallWarps - 1) / kSmallWarps), (unsigned)a.total_rows);
        const bool pdl = (ctx->pdl_mask & 4);
        cudaError_t e;
        if (dtype == HVD_F32)
            e = spec ? launch_kernel(pdl, verify_small_kernel<float, true>, sgrid, kSmallWarps * 32, 0, stream, a)
                     : launch_kernel(pdl, verify_small_kernel<float, false>, sgrid, kSmallWarps * 32, 0, stream, a);
        else
            e = spec ? launch_kernel(pdl, verify_small_kernel<__nv_bfloat16, true>, sgrid, kSmallWarps * 32, 0, stream, a)
                     : launch_kernel(pdl, verify_small_kernel<__nv_bfloat16, false>, sgrid, kSmallWarps * 32, 0, stream, a);
        HVD_CUDA_TRY(ctx, e);
    } else if (dtype == HVD_F32)
        HVD_CUDA_TRY(ctx, launch_kernel((ctx->pdl_mask & 4), verify_stream_kernel<float>, grid, T, smem, stream, a));
    else
        HVD_CUDA_TRY(ctx, launch_kernel((ctx->pdl_mask & 4), verify_stream_kernel<__nv_bfloat16>, grid, T, smem, stream, a));
    if (with_commit)
        HVD_CUDA_TRY(ctx, launch_kernel(ctx->pdl_commit, verify_commit_kernel, (a.B + kCommitWarps - 1) / kCommitWarps,
                                        kCommitWarps * 32, 0, stream, a));
    return HVD_OK;
}

}  // namespace hvd
