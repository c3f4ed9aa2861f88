// Greedy verification and commit (Sec. 3.1 Verify, Sec. 3.4, Algorithm 1).
//
// The step is a bandwidth-bound stream over the logits rows that are actually needed
// (rows 0..sel_len of each request).  Those rows are cut into work items of kVerifyVecPerItem
// 128-bit vectors (32 KB); persistent CTAs draw items from a counter, so SMs that get less DRAM
// bandwidth simply take fewer items.  Per item every thread issues all its loads at once, keeps a
// packed running maximum, and the CTA reduces (value, lowest index) to one 64-bit key that it
// leaves in scratch.  The CTA that delivers the last item of a request turns the keys into target
// tokens, compares them with the draft, and commits.  No CTA waits for another.
#include <cuda_bf16.h>

#include "hvd_internal.cuh"

namespace hvd {
namespace {

constexpr int T = kVerifyThreads;
constexpr int U = kVerifyUnroll;
constexpr uint32_t kFull = 0xffffffffu;

// order-preserving map float -> uint32 with -0.0 folded onto +0.0
__device__ __forceinline__ uint32_t ord32(float f) {
    uint32_t b = __float_as_uint(f);
    if ((b << 1) == 0) b = 0;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

template <typename E>
struct Elem;

template <>
struct Elem<float> {
    static constexpr int kPerVec = 4;
    static constexpr uint32_t kFillWord = 0xff800000u;  // -inf
    __device__ static __forceinline__ float scalar(const void* row, int64_t i) {
        return static_cast<const float*>(row)[i];
    }
    __device__ static __forceinline__ float get(const uint4& v, int k) {
        const uint32_t w = k == 0 ? v.x : k == 1 ? v.y : k == 2 ? v.z : v.w;
        return __uint_as_float(w);
    }
    // maximum of the U vectors held by one thread
    __device__ static __forceinline__ float thread_max(const uint4 (&x)[U]) {
        float m0 = __uint_as_float(x[0].x), m1 = __uint_as_float(x[0].y);
        float m2 = __uint_as_float(x[0].z), m3 = __uint_as_float(x[0].w);
#pragma unroll
        for (int u = 1; u < U; ++u) {
            m0 = fmaxf(m0, __uint_as_float(x[u].x)); m1 = fmaxf(m1, __uint_as_float(x[u].y));
            m2 = fmaxf(m2, __uint_as_float(x[u].z)); m3 = fmaxf(m3, __uint_as_float(x[u].w));
        }
        return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
    }
};

template <>
struct Elem<__nv_bfloat16> {
    static constexpr int kPerVec = 8;
    static constexpr uint32_t kFillWord = 0xff80ff80u;  // two bf16 -inf
    __device__ static __forceinline__ float scalar(const void* row, int64_t i) {
        return __uint_as_float((uint32_t)static_cast<const uint16_t*>(row)[i] << 16);
    }
    __device__ static __forceinline__ float get(const uint4& v, int k) {
        const uint32_t w = (k >> 1) == 0 ? v.x : (k >> 1) == 1 ? v.y : (k >> 1) == 2 ? v.z : v.w;
        return __uint_as_float((k & 1) ? (w & 0xffff0000u) : (w << 16));  // widening is exact
    }
    __device__ static __forceinline__ uint32_t max2(uint32_t a, uint32_t b) {
        uint32_t d;
        asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
        return d;
    }
    __device__ static __forceinline__ float thread_max(const uint4 (&x)[U]) {
        uint32_t m0 = x[0].x, m1 = x[0].y, m2 = x[0].z, m3 = x[0].w;
#pragma unroll
        for (int u = 1; u < U; ++u) {
            m0 = max2(m0, x[u].x); m1 = max2(m1, x[u].y);
            m2 = max2(m2, x[u].z); m3 = max2(m3, x[u].w);
        }
        const uint32_t m = max2(max2(m0, m1), max2(m2, m3));
        return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xffff0000u));
    }
};

// number of needed rows of request b (0 = request skipped) and its first logits row
__device__ __forceinline__ int needed_rows(const VerifyArgs& a, int b, int64_t* r0_out) {
    int64_t r0, r1;
    if (a.row_off) { r0 = a.row_off[b]; r1 = a.row_off[b + 1]; }
    else { r0 = (int64_t)b * (a.k_uniform + 1); r1 = r0 + a.k_uniform + 1; }
    *r0_out = r0;
    const int n = a.hist_len[b];
    if (n < 0 || n > a.hist_cap[b] || r1 <= r0) return 0;
    int m = a.sel_len[b];
    m = max(0, min(m, a.k_cap));
    if ((int64_t)m > r1 - r0 - 1) m = (int)(r1 - r0 - 1);
    return m + 1;
}

// Commit of one request by one warp, after all its row partials are in scratch.
__device__ void commit_request(const VerifyArgs& a, int b, int pref_b, int nr, int lane) {
    int64_t r0;
    (void)needed_rows(a, b, &r0);
    const int64_t r1 = a.row_off ? a.row_off[b + 1] : r0 + a.k_uniform + 1;
    const int m = nr - 1;
    const int kc = a.k_cap;
    const int32_t* d = a.sel_draft + (int64_t)b * kc;
    int acc = -1;
    int t_acc = 0;
    // rows in rounds of 32: lane handles row i, finds its target token and compares with the draft
    for (int base = 0; base <= m; base += 32) {
        const int i = base + lane;
        int t = 0;
        bool stop = true;
        if (i <= m) {
            unsigned long long key = 0;
            const unsigned long long* p = a.partial + (int64_t)(pref_b + i) * a.n_seg;
            for (int s = 0; s < a.n_seg; ++s) {
                const unsigned long long k = __ldcg(p + s);
                key = k > key ? k : key;
            }
            t = (int)(~(uint32_t)(key & 0xffffffffu));
            t = (int)min((int64_t)max(t, 0), a.V - 1);  // stays inside the vocabulary whatever the data
            if (a.target_tok) a.target_tok[r0 + i] = t;
            stop = (i >= m) || (d[i] != t);
        }
        const uint32_t stops = __ballot_sync(kFull, stop);
        if (acc < 0 && stops != 0) {
            const int j = __ffs(stops) - 1;
            acc = base + j;
            t_acc = __shfl_sync(kFull, t, j);
        }
    }
    // acc <= m always (row m stops).  Rows beyond m were not read.
    if (a.target_tok)
        for (int64_t r = r0 + nr + lane; r < r1; r += 32) a.target_tok[r] = -1;
    int32_t* z = a.committed + (int64_t)b * (kc + 1);
    const int n = a.hist_len[b];
    const int room = a.hist_cap[b] - n;
    const int w = min(acc + 1, room);
    int32_t* h = a.hist + a.hist_off[b];
    for (int j = lane; j <= kc; j += 32) {
        const int tok = (j < acc) ? d[j] : (j == acc ? t_acc : -1);
        z[j] = tok;
        if (j < w) h[n + j] = tok;
    }
    if (lane == 0) {
        a.hist_len[b] = n + w;
        a.n_commit[b] = w;
        a.accepted[b] = acc;
        a.status[b] = (w < acc + 1) ? HVD_REQ_CAPACITY : HVD_REQ_OK;
        hvd_req_state st = a.state[b];
        st.sel_bits = (st.sel_bits << 1) | (a.select[b] ? 1u : 0u);
        st.acc_ring = (st.acc_ring << 8) | (unsigned long long)(acc & 0xff);
        a.state[b] = st;
        a.req_cnt[b] = 0;  // scratch is zero at rest
    }
}

template <typename E>
__global__ void __launch_bounds__(T) verify_commit_kernel(const VerifyArgs a) {
    extern __shared__ int s_pref[];  // [B+1] exclusive prefix of needed rows
    __shared__ uint32_t s_wmax[T / 32];
    __shared__ uint32_t s_minidx;
    __shared__ uint32_t s_next;
    __shared__ int s_carry;

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    constexpr int EPV = Elem<E>::kPerVec;
    constexpr int ESZ = 16 / EPV;

    // ---- phase 0: which rows are needed (device data), prefix over requests -----------------
    if (tid == 0) { s_carry = 0; s_pref[0] = 0; }
    __syncthreads();
    for (int base = 0; base < a.B; base += T) {
        const int b = base + tid;
        int64_t r0 = 0;
        const int nr = (b < a.B) ? needed_rows(a, b, &r0) : 0;
        if (b < a.B && nr == 0 && blockIdx.x == 0) {
            // skipped request: neutral outputs, nothing else touched
            const int64_t r1 = a.row_off ? a.row_off[b + 1] : r0 + a.k_uniform + 1;
            a.accepted[b] = 0; a.n_commit[b] = 0; a.status[b] = HVD_REQ_BAD_LEN;
            for (int j = 0; j <= a.k_cap; ++j) a.committed[(int64_t)b * (a.k_cap + 1) + j] = -1;
            if (a.target_tok) for (int64_t r = r0; r < r1; ++r) a.target_tok[r] = -1;
        }
        // inclusive scan of nr over the tile
        int v = nr;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(kFull, v, off);
            if (lane >= off) v += o;
        }
        __shared__ int s_wsum[T / 32];
        if (lane == 31) s_wsum[warp] = v;
        __syncthreads();
        int wbase = 0;
#pragma unroll
        for (int k = 0; k < T / 32; ++k) wbase += (k < warp) ? s_wsum[k] : 0;
        const int carry = s_carry;
        if (b < a.B) s_pref[b + 1] = carry + wbase + v;
        __syncthreads();
        if (tid == T - 1) s_carry = carry + wbase + v;
        __syncthreads();
    }
    const int total_rows = s_pref[a.B];
    const uint32_t total_items = (uint32_t)total_rows * (uint32_t)a.n_seg;

    if (tid == 0) s_next = atomicAdd(&a.ctrl->next_item, 1u);
    __syncthreads();
    uint32_t cur = s_next;

    const int64_t row_bytes = a.V * ESZ;
    const char* base_ptr = static_cast<const char*>(a.logits);

    while (cur < total_items) {
        uint32_t nxt = 0;
        if (tid == 0) nxt = atomicAdd(&a.ctrl->next_item, 1u);  // overlaps with this item's loads

        // ---- decode the item -> (request b, row i, segment s) ------------------------------
        const int r = (int)(cur / (uint32_t)a.n_seg);
        const int s = (int)(cur - (uint32_t)r * (uint32_t)a.n_seg);
        int lo = 0, hi = a.B;  // largest b with s_pref[b] <= r
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_pref[mid] <= r) lo = mid; else hi = mid;
        }
        const int b = lo;
        const int i = r - s_pref[b];
        const int64_t row0 = a.row_off ? a.row_off[b] : (int64_t)b * (a.k_uniform + 1);
        const char* row = base_ptr + (row0 + i) * row_bytes;

        // 128-bit grid inside the row: `head` leading elements, then n_vec full vectors, then a tail
        const int head_bytes = (int)((16 - (reinterpret_cast<uintptr_t>(row) & 15)) & 15);
        const int head = (int)min((int64_t)(head_bytes / ESZ), a.V);
        const int64_t n_vec = (a.V - head) / EPV;
        const int tail = (int)(a.V - head - n_vec * EPV);
        const uint4* vrow = reinterpret_cast<const uint4*>(row + (int64_t)head * ESZ);
        const int64_t vbeg = (int64_t)s * kVerifyVecPerItem;
        const int64_t nv = min((int64_t)kVerifyVecPerItem, n_vec - vbeg);  // may be <= 0

        uint4 x[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int vi = u * T + tid;
            if (vi < nv) x[u] = ld_stream(vrow + vbeg + vi);
            else x[u] = make_uint4(Elem<E>::kFillWord, Elem<E>::kFillWord, Elem<E>::kFillWord, Elem<E>::kFillWord);
        }
        // ragged edges of the row (at most 2*(EPV-1) elements) ride along with segment 0
        float edge = 0.0f;
        int edge_idx = -1;
        if (s == 0 && tid < head + tail) {
            edge_idx = tid < head ? tid : (int)(head + n_vec * EPV + (tid - head));
            edge = Elem<E>::scalar(row, edge_idx);
        }

        float tmax = Elem<E>::thread_max(x);
        uint32_t tord = (tid < nv) ? ord32(tmax) : 0u;  // a thread without a vector holds nothing
        if (edge_idx >= 0) tord = max(tord, ord32(edge));
        const uint32_t word = __reduce_max_sync(kFull, tord);
        if (lane == 0) s_wmax[warp] = word;
        if (tid == 0) { s_minidx = 0xffffffffu; s_next = nxt; }
        __syncthreads();  // A
        uint32_t bord = s_wmax[0];
#pragma unroll
        for (int k = 1; k < T / 32; ++k) bord = max(bord, s_wmax[k]);
        nxt = s_next;
        if (tord == bord && bord != 0u) {
            // this thread holds a maximum: find its lowest index (rare path)
            uint32_t best = 0xffffffffu;
            if (edge_idx >= 0 && ord32(edge) == bord) best = (uint32_t)edge_idx;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int vi = u * T + tid;
                if (vi < nv) {
#pragma unroll
                    for (int k = 0; k < EPV; ++k) {
                        if (ord32(Elem<E>::get(x[u], k)) == bord) {
                            const uint32_t idx = (uint32_t)(head + (vbeg + vi) * EPV + k);
                            best = min(best, idx);
                        }
                    }
                }
            }
            atomicMin(&s_minidx, best);
        }
        __syncthreads();  // B

        // ---- warp 0: publish the partial, count the item, commit if the request is complete ----
        if (warp == 0) {
            const int nr = s_pref[b + 1] - s_pref[b];
            uint32_t last = 0;
            if (lane == 0) {
                const uint32_t idx = s_minidx;
                const unsigned long long key =
                    (bord == 0u || idx == 0xffffffffu) ? 0ull : (((unsigned long long)bord << 32) | (uint32_t)(~idx));
                a.partial[(int64_t)r * a.n_seg + s] = key;
                __threadfence();
                const uint32_t old = atomicAdd(a.req_cnt + b, 1u);
                last = (old + 1 == (uint32_t)nr * (uint32_t)a.n_seg) ? 1u : 0u;
            }
            last = __shfl_sync(kFull, last, 0);
            if (last) {
                __threadfence();
                commit_request(a, b, s_pref[b], nr, lane);
            }
        }
        cur = nxt;
    }

    // ---- the last CTA to leave resets the work counter for the next call -----------------------
    if (tid == 0) {
        const uint32_t old = atomicAdd(&a.ctrl->blocks_exited, 1u);
        if (old + 1 == gridDim.x) {
            a.ctrl->next_item = 0;
            a.ctrl->blocks_exited = 0;
        }
    }
}

}  // namespace

size_t verify_dyn_smem(int32_t B) { return (size_t)(B + 1) * sizeof(int); }

int verify_occupancy(hvd_dtype dtype, size_t dyn_smem) {
    int n = 0;
    cudaError_t e;
    if (dtype == HVD_F32)
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, verify_commit_kernel<float>, T, dyn_smem);
    else
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, verify_commit_kernel<__nv_bfloat16>, T, dyn_smem);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return n;
}

hvd_status launch_verify(hvd_ctx* ctx, const VerifyArgs& a, hvd_dtype dtype, cudaStream_t stream) {
    const size_t smem = verify_dyn_smem(a.B);
    const int per_sm = ctx->vf_blocks_per_sm[dtype == HVD_F32 ? 0 : 1];
    const int grid = ctx->num_sms * (per_sm > 0 ? per_sm : 1);
    if (dtype == HVD_F32)
        verify_commit_kernel<float><<<grid, T, smem, stream>>>(a);
    else
        verify_commit_kernel<__nv_bfloat16><<<grid, T, smem, stream>>>(a);
    HVD_CUDA_TRY(ctx, cudaGetLastError());
    return HVD_OK;
}

}  // namespace hvd
