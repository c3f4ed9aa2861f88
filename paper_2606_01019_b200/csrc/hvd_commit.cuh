// Commit of one request by one warp (Sec. 3.1 Verify, Sec. 3.4, Algorithm 1 "append z, update h"),
// shared by the commit kernels and by the kernel that goes straight on to the next cycle's lookup.
#pragma once

#include "hvd_internal.cuh"

namespace hvd {

struct Req {
    int64_t r0, r1;  // logits rows of the request
    int nr;          // rows needed = sel_len + 1 (0: request skipped)
};

__device__ __forceinline__ Req load_req(const VerifyArgs& a, int b) {
    Req q;
    if (a.row_off) { q.r0 = a.row_off[b]; q.r1 = a.row_off[b + 1]; }
    else { q.r0 = (int64_t)b * (a.k_uniform + 1); q.r1 = q.r0 + a.k_uniform + 1; }
    // every input is fetched before any is looked at: one round trip, not a chain of three
    const int n = a.hist_len[b];
    const int cap = a.hist_cap[b];
    const int sl = a.sel_len[b];
    q.nr = 0;
    // rows outside the logits array (a row_off entry below 0 or beyond total_rows): the request is skipped and
    // its row range emptied, so that neither the logits nor the row keys nor target_tok are touched there
    if (q.r0 < 0 || q.r1 > a.total_rows || q.r1 < q.r0) { q.r0 = 0; q.r1 = 0; }
    if (n >= 0 && n <= cap && q.r1 > q.r0) {
        int m = max(0, min(sl, a.k_cap));
        if ((int64_t)m > q.r1 - q.r0 - 1) m = (int)(q.r1 - q.r0 - 1);
        q.nr = m + 1;
    }
    return q;
}

// The part of a request's needed rows that the current launch streams: all of them, or (prefix verification)
// rows [win_lo, win_hi) of a request that is still alive.  Returns the number of rows, `first` = the first one.
__device__ __forceinline__ int streamed_rows(const VerifyArgs& a, const Req& q, int b, int64_t& first) {
    const int lo = min(a.win_lo, q.nr);
    int hi = min(a.win_hi, q.nr);
    if (a.alive && hi > lo && a.alive[b] == 0) hi = lo;
    first = q.r0 + lo;
    return hi - lo;
}

constexpr unsigned long long kKeySign = 0x8000000000000000ull;

// The (value, ~index) key of a logits row.  Context scratch is put back to zero as it is read; keys
// handed in by the caller (hvd_commit_keys) are in signed order and are left alone.
__device__ __forceinline__ unsigned long long read_row_key(const VerifyArgs& a, int64_t r) {
    if (!HVD_IN_BOUNDS(a.dev_error, r, 0, a.total_rows)) return 0ull;
    if (a.ext_keys) return (unsigned long long)a.ext_keys[r] ^ kKeySign;  // "row not read" becomes 0
    const unsigned long long key = a.row_key[r];
    a.row_key[r] = 0ull;  // scratch is zero at rest
    return key;
}

// Commit of one request by one warp, after all its needed rows are folded into the row keys.
// Every load that does not depend on another is issued up front: the kernel is a short chain of
// global round trips at the end of every decoding step.
// What the commit leaves behind, identical in every lane: the request's history length and recent-history
// summary after the call (as read, when the request was skipped).
struct CommitOut {
    int n;
    hvd_req_state st;
};

__device__ __forceinline__ void commit_request(const VerifyArgs& a, int b, int lane, CommitOut* out = nullptr) {
    const int kc = a.k_cap;
    const int32_t* d = a.sel_draft + (int64_t)b * kc;
    const int d0 = lane < kc ? d[lane] : -1;            // draft tokens lane, lane+32 (k_cap <= 64)
    const int d1 = lane + 32 < kc ? d[lane + 32] : -1;
    const int64_t hoff = a.hist_off[b];
    const int sel = a.select[b];
    hvd_req_state st = a.state[b];
    const int n = a.hist_len[b];
    const int cap = a.hist_cap[b];
    const Req q = load_req(a, b);
    int32_t* z = a.committed + (int64_t)b * (kc + 1);
    if (q.nr == 0) {
        // skipped request: neutral outputs, nothing else touched
        for (int j = lane; j <= kc; j += 32) z[j] = -1;
        if (a.target_tok)
            for (int64_t r = q.r0 + lane; r < q.r1; r += 32)
                if (HVD_IN_BOUNDS(a.dev_error, r, 0, a.total_rows)) a.target_tok[r] = -1;
        if (lane == 0) { a.accepted[b] = 0; a.n_commit[b] = 0; a.status[b] = HVD_REQ_BAD_LEN; }
        if (out) { out->n = n; out->st = st; }
        return;
    }
    const int m = q.nr - 1;
    if (a.rows_in_commit && a.rows_read && lane == 0) atomicAdd(a.rows_read, (unsigned long long)q.nr);
    pdl_wait();  // everything above was the request's own data; the row keys come from the streaming kernel
    // rows lane, lane+32, lane+64 (at most 65 rows): target tokens from the row keys
    unsigned long long key[3];
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        const int i = lane + 32 * k;
        key[k] = 0ull;
        if (i <= m) {
            key[k] = read_row_key(a, q.r0 + i);
        }
    }
    int acc = -1;
    int t_acc = 0;
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        const int i = lane + 32 * k;
        int t = (int)(~(uint32_t)(key[k] & 0xffffffffu));
        t = (int)min((int64_t)max(t, 0), a.V - 1);  // inside the vocabulary whatever the data
        bool stop = true;
        if (i <= m) {
            if (a.target_tok && HVD_IN_BOUNDS(a.dev_error, q.r0 + i, 0, a.total_rows)) a.target_tok[q.r0 + i] = t;
            const int di = k == 0 ? d0 : (k == 1 ? d1 : -1);
            stop = (i >= m) || (di != t);
        }
        const uint32_t stops = __ballot_sync(0xffffffffu, stop);
        if (acc < 0 && stops != 0 && 32 * k <= m) {
            const int j = __ffs(stops) - 1;
            acc = 32 * k + j;
            t_acc = __shfl_sync(0xffffffffu, t, j);
        }
    }
    // acc <= m always (row m stops).  Rows beyond m were not read.
    if (a.target_tok)
        for (int64_t r = q.r0 + q.nr + lane; r < q.r1; r += 32)
            if (HVD_IN_BOUNDS(a.dev_error, r, 0, a.total_rows)) a.target_tok[r] = -1;
    const int room = cap - n;
    const int w = min(acc + 1, room);
    int32_t* h = a.hist + hoff;
    for (int j = lane; j <= kc; j += 32) {
        const int dj = j < 32 ? d0 : d1;
        const int tok = (j < acc) ? dj : (j == acc ? t_acc : -1);
        z[j] = tok;
        if (j < w && HVD_IN_BOUNDS(a.dev_error, n + j, 0, cap)) h[n + j] = tok;
    }
    st.sel_bits = (st.sel_bits << 1) | (sel ? 1u : 0u);
    st.acc_ring = (st.acc_ring << 8) | (unsigned long long)(acc & 0xff);
    if (lane == 0) {
        a.hist_len[b] = n + w;
        a.n_commit[b] = w;
        a.accepted[b] = acc;
        a.status[b] = (w < acc + 1) ? HVD_REQ_CAPACITY : HVD_REQ_OK;
        a.state[b] = st;
    }
    if (out) { out->n = n + w; out->st = st; }
}

}  // namespace hvd
