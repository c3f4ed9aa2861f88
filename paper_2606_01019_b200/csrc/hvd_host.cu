// Host-buffer form of one decoding cycle: stage inputs on the device, run the three kernels,
// bring the results back.  The arithmetic is entirely in the device entry points; this file only
// moves bytes and appends the committed block to the caller's host histories.
#include <string.h>

#include "hvd_internal.cuh"

using namespace hvd;

namespace {

struct Carver {
    char* base;
    size_t off;
    template <typename P>
    P* take(size_t count) {
        off = (off + 255) & ~(size_t)255;
        P* p = base ? reinterpret_cast<P*>(base + off) : nullptr;
        off += count * sizeof(P);
        return p;
    }
};

struct Staging {
    int32_t *hist, *hist_cap, *hist_len, *K, *prompt_len, *model_draft, *model_len;
    int64_t *hist_off, *row_off;
    hvd_req_state* state;
    char* logits;
    int32_t *draft, *draft_len, *match_len, *match_pos, *match_cnt;
    float* score;
    int32_t *select, *sel_draft, *sel_len, *accepted, *committed, *n_commit, *status;
};

size_t carve(Carver& c, Staging& s, const hvd_host_step_args& a, int k_cap) {
    const size_t B = (size_t)a.B;
    const size_t esz = a.dtype == HVD_F32 ? 4 : 2;
    s.hist = c.take<int32_t>((size_t)a.hist_words);
    s.hist_off = c.take<int64_t>(B);
    s.hist_cap = c.take<int32_t>(B);
    s.hist_len = c.take<int32_t>(B);
    s.K = c.take<int32_t>(B);
    s.prompt_len = c.take<int32_t>(B);
    s.state = c.take<hvd_req_state>(B);
    s.model_draft = c.take<int32_t>(B * k_cap);
    s.model_len = c.take<int32_t>(B);
    s.row_off = c.take<int64_t>(B + 1);
    s.logits = c.take<char>((size_t)a.total_rows * (size_t)a.V * esz);
    s.draft = c.take<int32_t>(B * k_cap);
    s.draft_len = c.take<int32_t>(B);
    s.match_len = c.take<int32_t>(B);
    s.match_pos = c.take<int32_t>(B);
    s.match_cnt = c.take<int32_t>(B);
    s.score = c.take<float>(B);
    s.select = c.take<int32_t>(B);
    s.sel_draft = c.take<int32_t>(B * k_cap);
    s.sel_len = c.take<int32_t>(B);
    s.accepted = c.take<int32_t>(B);
    s.committed = c.take<int32_t>(B * (k_cap + 1));
    s.n_commit = c.take<int32_t>(B);
    s.status = c.take<int32_t>(B);
    return (c.off + 255) & ~(size_t)255;
}

}  // namespace

extern "C" hvd_status hvd_step_host(hvd_ctx* ctx, const hvd_host_step_args* args, void* stream) {
    if (!ctx) return HVD_ERR_INVALID_ARG;
    if (!args) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_step_host: NULL args");
    const hvd_host_step_args& a = *args;
    if (a.B < 1 || a.B > ctx->cfg.max_batch) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_step_host: B outside [1, max_batch]");
    if (a.dtype != HVD_F32 && a.dtype != HVD_BF16) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_step_host: unknown dtype");
    if (a.hist_words < 1 || a.total_rows < 1 || a.V < 1) return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_step_host: empty array");
    if (!a.hist || !a.hist_off || !a.hist_cap || !a.hist_len || !a.K || !a.prompt_len || !a.state ||
        !a.logits || !a.score || !a.select || !a.sel_draft || !a.sel_len || !a.accepted || !a.committed ||
        !a.n_commit || !a.status)
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_step_host: NULL pointer");
    if ((a.model_draft == nullptr) != (a.model_len == nullptr))
        return fail(ctx, HVD_ERR_INVALID_ARG, "hvd_step_host: model_draft and model_len go together");

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int kc = ctx->cfg.k_cap;
    const size_t B = (size_t)a.B;
    Staging s;
    Carver sizing{nullptr, 0};
    const size_t need = carve(sizing, s, a, kc);
    if (need > ctx->host_ws_bytes) {
        HVD_CUDA_TRY(ctx, cudaStreamSynchronize(st));
        if (ctx->host_ws) HVD_CUDA_TRY(ctx, cudaFree(ctx->host_ws));
        ctx->host_ws = nullptr;
        ctx->host_ws_bytes = 0;
        if (cudaMalloc(reinterpret_cast<void**>(&ctx->host_ws), need) != cudaSuccess) {
            (void)cudaGetLastError();
            return fail(ctx, HVD_ERR_ALLOC, "hvd_step_host: cannot allocate the device staging area");
        }
        ctx->host_ws_bytes = need;
    }
    Carver c{ctx->host_ws, 0};
    carve(c, s, a, kc);

    const size_t esz = a.dtype == HVD_F32 ? 4 : 2;
#define H2D(dst, src, bytes) HVD_CUDA_TRY(ctx, cudaMemcpyAsync((dst), (src), (bytes), cudaMemcpyHostToDevice, st))
#define D2H(dst, src, bytes) HVD_CUDA_TRY(ctx, cudaMemcpyAsync((dst), (src), (bytes), cudaMemcpyDeviceToHost, st))
    H2D(s.hist, a.hist, (size_t)a.hist_words * 4);
    H2D(s.hist_off, a.hist_off, B * 8);
    H2D(s.hist_cap, a.hist_cap, B * 4);
    H2D(s.hist_len, a.hist_len, B * 4);
    H2D(s.K, a.K, B * 4);
    H2D(s.prompt_len, a.prompt_len, B * 4);
    H2D(s.state, a.state, B * sizeof(hvd_req_state));
    if (a.model_draft) {
        H2D(s.model_draft, a.model_draft, B * kc * 4);
        H2D(s.model_len, a.model_len, B * 4);
    }
    if (a.row_off) H2D(s.row_off, a.row_off, (B + 1) * 8);

    hvd_status r = hvd_lookup(ctx, a.B, s.hist, s.hist_off, s.hist_cap, s.hist_len, s.K, a.n_max, s.draft,
                              s.draft_len, s.match_len, s.match_pos, s.match_cnt, st);
    if (r != HVD_OK) return r;
    r = hvd_score_select(ctx, a.B, s.hist_len, s.prompt_len, s.state, s.K, s.draft, s.draft_len, s.match_len,
                         s.match_pos, s.match_cnt, a.model_draft ? s.model_draft : nullptr,
                         a.model_draft ? s.model_len : nullptr, nullptr, s.score, s.select, s.sel_draft,
                         s.sel_len, st);
    if (r != HVD_OK) return r;

    // The logits are the bulk of the bytes that cross the bus, and verification reads as hvd_verify_commit_prefix
    // does (this entry point has no target_tok): only rows up to the window of a request's first rejected draft
    // token.
    D2H(a.sel_len, s.sel_len, B * 4);
    const hvd_dtype dtype = (hvd_dtype)a.dtype;
    auto verify_args = [&](const void* logits, VerifyArgs* va) {
        return make_verify_args(ctx, a.B, logits, dtype, a.V, a.row_off ? s.row_off : nullptr, a.k_uniform, a.total_rows,
                                s.sel_draft, s.sel_len, s.select, s.hist, s.hist_off, s.hist_cap, s.hist_len, s.state,
                                s.accepted, s.committed, s.n_commit, s.status, va);
    };

    // Logits in page-locked host memory (cudaHostAlloc, cudaHostRegister, a pinned tensor) are read where they
    // lie: the streaming kernels load every needed row once, straight over the bus; nothing is staged and the
    // host waits for nothing in between.
    auto verify_in_place = [&](const void* device_view) -> hvd_status {
        VerifyArgs va;
        const hvd_status e = verify_args(device_view, &va);
        return e != HVD_OK ? e : launch_verify_prefix(ctx, va, dtype, st);
    };

    // Pageable logits: the selection comes back first, then the needed rows are copied and verified window by
    // window (adjacent ranges in one copy each); the flags of who is still alive come back to the host after
    // every window but the last and decide the next window's copies.
    auto verify_staged = [&]() -> hvd_status {
        HVD_CUDA_TRY(ctx, cudaStreamSynchronize(st));
        const size_t row_bytes = (size_t)a.V * esz;
        auto copy_rows = [&](int lo, int hi, const int32_t* alive) -> hvd_status {  // rows [lo, hi) of the needed rows
            int64_t run0 = 0, run1 = 0;  // pending range of rows
            for (int32_t b = 0; b <= a.B; ++b) {
                int64_t r0 = 0, r1 = 0;
                if (b < a.B) {
                    const int64_t first = a.row_off ? a.row_off[b] : (int64_t)b * (a.k_uniform + 1);
                    const int64_t rend = a.row_off ? a.row_off[b + 1] : first + a.k_uniform + 1;
                    const bool ok = a.hist_len[b] >= 0 && a.hist_len[b] <= a.hist_cap[b] && rend > first && first >= 0 &&
                                    rend <= a.total_rows && (!alive || alive[b] != 0);
                    int64_t m = a.sel_len[b] < 0 ? 0 : (a.sel_len[b] > kc ? kc : a.sel_len[b]);
                    if (m > rend - first - 1) m = rend - first - 1;
                    const int64_t nr = ok ? m + 1 : 0;  // needed rows of the request
                    r0 = first + (lo < nr ? lo : nr);
                    r1 = first + (hi < nr ? hi : nr);
                }
                if (b < a.B && r1 > r0 && r0 == run1 && run1 > run0) { run1 = r1; continue; }  // extends the pending range
                if (run1 > run0)
                    H2D(s.logits + (size_t)run0 * row_bytes, static_cast<const char*>(a.logits) + (size_t)run0 * row_bytes,
                        (size_t)(run1 - run0) * row_bytes);
                run0 = r0; run1 = r1;
            }
            return HVD_OK;
        };
        VerifyArgs va;
        hvd_status e = verify_args(s.logits, &va);
        if (e != HVD_OK) return e;
        int edges[16];
        const int n_win = prefix_window_edges(ctx, va, dtype, edges);
        if (n_win == 1) {  // a small call: all needed rows at once
            e = copy_rows(0, 0x7fffffff, nullptr);
            return e != HVD_OK ? e : launch_verify_prefix(ctx, va, dtype, st);
        }
        int32_t* alive = nullptr;  // host copy of the flags: the caller's `accepted` array serves until the results arrive
        for (int j = 0; j < n_win; ++j) {
            e = copy_rows(edges[j], edges[j + 1], alive);
            if (e != HVD_OK) return e;
            e = launch_prefix_window(ctx, va, dtype, edges, j, n_win, st);
            if (e != HVD_OK) return e;
            if (j + 1 < n_win) {
                alive = a.accepted;
                D2H(alive, ctx->vf_alive, B * 4);
                HVD_CUDA_TRY(ctx, cudaStreamSynchronize(st));
            }
        }
        return launch_prefix_commit(ctx, va, st);
    };

    cudaPointerAttributes at;
    const bool page_locked = cudaPointerGetAttributes(&at, a.logits) == cudaSuccess && at.type == cudaMemoryTypeHost &&
                             at.devicePointer != nullptr;
    if (!page_locked) (void)cudaGetLastError();
    r = page_locked ? verify_in_place(at.devicePointer) : verify_staged();
    if (r != HVD_OK) return r;

    D2H(a.score, s.score, B * 4);
    D2H(a.select, s.select, B * 4);
    D2H(a.sel_draft, s.sel_draft, B * kc * 4);
    D2H(a.accepted, s.accepted, B * 4);
    D2H(a.committed, s.committed, B * (kc + 1) * 4);
    D2H(a.n_commit, s.n_commit, B * 4);
    D2H(a.status, s.status, B * 4);
    D2H(a.hist_len, s.hist_len, B * 4);
    D2H(a.state, s.state, B * sizeof(hvd_req_state));
#undef H2D
#undef D2H
    HVD_CUDA_TRY(ctx, cudaStreamSynchronize(st));

    // mirror the device-side append on the host histories (the device copy is only staging)
    for (int32_t b = 0; b < a.B; ++b) {
        const int32_t w = a.n_commit[b];
        if (w <= 0) continue;
        const int32_t n_after = a.hist_len[b];
        memcpy(a.hist + a.hist_off[b] + (n_after - w), a.committed + (size_t)b * (kc + 1), (size_t)w * 4);
    }
    return HVD_OK;
}
