// The inner step of the history scan, shared by the lookup kernel and by the kernel that collects the
// occurrences of the longest match: one 128-bit vector of history tokens per lane, candidates are the
// positions that hold the history's last token, and the warp that finds one extends the match backwards
// together (lane j compares the token j + 1 back; ballot + find-first-set gives the length, a second
// round covers lengths 33 to 64).
#pragma once

#include "hvd_internal.cuh"

namespace hvd {

// Arguments of the lookup kernels (the one-CTA / chunk form and the tiled form).
struct LookupArgs {
    int32_t B;
    const int32_t* hist;
    const int64_t* hist_off;
    const int32_t* hist_cap;
    const int32_t* hist_len;
    const int32_t* K;
    int32_t n_max;
    int32_t* draft;
    int32_t* draft_len;
    int32_t* match_len;
    int32_t* match_pos;
    int32_t* match_cnt;
    LookupPartial* partial;
    uint32_t* req_cnt;
    int32_t max_chunks;
    int32_t k_cap, l_max, min_match;
    float spec_factor, spec_offset;
    bool successor_works_ahead;
    bool chunks_on_x;
    int* dev_error;   // device status word of the context (set when a bounded wait runs out)
};

// Best match seen so far: the longest length, then the latest position; the count is the number of
// positions that reach that length.
struct Best {
    unsigned long long key;  // (L << 32) | e ; 0 = nothing found
    uint32_t cnt;
};

__device__ __forceinline__ Best combine(Best a, Best b) {
    const uint32_t la = (uint32_t)(a.key >> 32), lb = (uint32_t)(b.key >> 32);
    if (la > lb) return a;
    if (lb > la) return b;
    Best r;
    r.key = a.key > b.key ? a.key : b.key;
    r.cnt = a.cnt + b.cnt;
    return r;
}

__device__ __forceinline__ Best warp_combine(Best v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Best o;
        o.key = __shfl_xor_sync(0xffffffffu, v.key, off);
        o.cnt = __shfl_xor_sync(0xffffffffu, v.cnt, off);
        v = combine(v, o);
    }
    return v;
}

__device__ __forceinline__ int4 ld_hist(const int4* p) {
    int4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Asks the L2 for `tokens` history tokens from p (16-byte aligned) on: 32 bulk prefetches, one per lane of the
// calling warp.  Nothing is waited for and nothing arrives in the SM: a later load finds the line in the L2 or
// on its way there.  Used ahead of the wait for the previous kernel: the L2 is the point of coherence, so a
// line fetched early still shows what that kernel writes afterwards.
__device__ __forceinline__ void prefetch_history_l2(const int32_t* p, int tokens, int lane) {
    const int bytes = (tokens >> 2) << 4;
    if (bytes <= 0) return;
    const int seg = (((bytes + 31) >> 5) + 127) & ~127;
    const int at = lane * seg;
    if (at < bytes) {
        const uint32_t size = (uint32_t)min(seg, bytes - at);
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(reinterpret_cast<const char*>(p) + at), "r"(size) : "memory");
    }
}

// x: this lane's four tokens at positions p0 .. p0 + 3 of a history of n tokens (slab); q0 its last token,
// qa / qb the tokens 1 + lane and 33 + lane back.  Calls on_match(L, p), in every lane of the warp with the
// same arguments, for every candidate p in [0, n - 2] of the warp's 32 vectors: p holds q0 and L >= 1 is the
// match length of the copy that ends there (capped at l_max and at the slab start).
// COHERENT: the tokens compared during the extension are read through the L2 (for a kernel that has itself
// appended to the history it scans).  p_last: candidates beyond this position are left to another call
// (default: none are).
template <bool COHERENT = false, class OnMatch>
__device__ __forceinline__ void scan_vector(const int4 x, int p0, int n, const int32_t* __restrict__ slab, int32_t q0,
                                            int32_t qa, int32_t qb, int l_max, int lane, OnMatch&& on_match,
                                            int* status_word = nullptr, int p_last = 0x7fffffff) {
    const int last = min(n - 2, p_last);
    uint32_t m = 0;
    m |= (x.x == q0 && p0 + 0 >= 0 && p0 + 0 <= last) ? 1u : 0u;
    m |= (x.y == q0 && p0 + 1 >= 0 && p0 + 1 <= last) ? 2u : 0u;
    m |= (x.z == q0 && p0 + 2 >= 0 && p0 + 2 <= last) ? 4u : 0u;
    m |= (x.w == q0 && p0 + 3 >= 0 && p0 + 3 <= last) ? 8u : 0u;
    uint32_t hits = __ballot_sync(0xffffffffu, m != 0);
    while (hits) {
        const int src = __ffs(hits) - 1;
        hits &= hits - 1;
        uint32_t ms = __shfl_sync(0xffffffffu, m, src);
        const int ps = __shfl_sync(0xffffffffu, p0, src);
        while (ms) {
            const int k = __ffs(ms) - 1;
            ms &= ms - 1;
            const int p = ps + k;
            // match length of the copy ending at p (>= 1 already); limit: l_max and the slab start
            const int cap = min(l_max, p + 1);
            int l = lane + 1;
            bool eq = (l < cap) && HVD_IN_BOUNDS(status_word, p - l, 0, n) && ((COHERENT ? __ldcg(slab + p - l) : slab[p - l]) == qa);
            uint32_t mm = __ballot_sync(0xffffffffu, !eq);
            int L;
            if (mm != 0) {
                L = __ffs(mm);  // first failing lane j: lengths 1..j hold, so L = 1 + j
            } else {
                l = lane + 33;
                eq = (l < cap) && HVD_IN_BOUNDS(status_word, p - l, 0, n) && ((COHERENT ? __ldcg(slab + p - l) : slab[p - l]) == qb);
                mm = __ballot_sync(0xffffffffu, !eq);  // lane 31 (l = 64) always fails
                L = 32 + __ffs(mm);
            }
            on_match(L, p);
        }
    }
}

}  // namespace hvd
