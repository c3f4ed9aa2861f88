// Internal declarations shared by the translation units of the CUDA library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "hvd.h"

namespace hvd {

// One partial result of the history scan: best match seen by one chunk of one request.
struct LookupPartial {
    unsigned long long key;  // (match length << 32) | position of the first continuation token
    uint32_t cnt;            // positions in the chunk reaching that length
    uint32_t pad;
};

constexpr int kLookupThreads = 256;
constexpr int kLookupTokPerVec = 4;
constexpr int kLookupMinChunk = kLookupThreads * kLookupTokPerVec;  // tokens: sizes the partial scratch

// tunables of the verify kernel (overridable at compile time for experiments)
#ifndef HVD_VERIFY_THREADS
#define HVD_VERIFY_THREADS 256
#endif
#ifndef HVD_VERIFY_UNROLL
#define HVD_VERIFY_UNROLL 8
#endif
#ifndef HVD_VERIFY_MIN_BLOCKS
#define HVD_VERIFY_MIN_BLOCKS 4
#endif
constexpr int kVerifyThreads = HVD_VERIFY_THREADS;
constexpr int kVerifyUnroll = HVD_VERIFY_UNROLL;      // 128-bit loads in flight per lane
#ifndef HVD_VERIFY_UNIT_BATCHES
#define HVD_VERIFY_UNIT_BATCHES 2
#endif
constexpr int kVerifyUnitBatches = HVD_VERIFY_UNIT_BATCHES;  // 4 KB batches per unit drawn by a warp
#ifndef HVD_VERIFY_ENDGAME_SHIFT
#define HVD_VERIFY_ENDGAME_SHIFT 6
#endif
#ifndef HVD_VERIFY_QUEUES
#define HVD_VERIFY_QUEUES 8
#endif
constexpr int kVerifyQueues = HVD_VERIFY_QUEUES;  // unit counters
constexpr int kVerifyQueueStride = 32;           // ... on separate 128-byte lines (in 32-bit words)
constexpr long long kVerifySmallBytes = 160LL << 20;  // logits up to this size: one warp per 4 KB batch
constexpr long long kPrefixBoundaryBytes = 64LL << 20;  // prefix verification: a window boundary costs what streaming this much costs
constexpr long long kVerifySpecBytes = 8LL << 20;     // ... and up to this size: loads before the need is known


}  // namespace hvd

struct hvd_ctx {
    hvd_config cfg;
    int device;
    int num_sms;
    // predictor
    float* d_W1;
    float* d_b1;
    float* d_W2;
    float* d_WhT;  // second hidden layer, transposed [hidden, hidden]
    float* d_bh;
    float b2, tau;
    bool has_predictor;      // a predictor on the 8 base features is stored
    bool has_predictor_ext;  // a predictor on the extended feature vector is stored (same buffers)
    bool two_layer;
    bool score2_ready;  // the two-layer kernel's shared-memory size has been opted in on this device
    bool score2x_ready; // the same for its extended-feature instance
    const uint8_t* cls; // token-class bits per vocabulary entry (caller-owned), NULL = none
    int32_t cls_V;
    // lookup scratch
    hvd::LookupPartial* lk_partial;  // [max_batch, lk_max_chunks]
    uint32_t* lk_cnt;                // [max_batch], zero at rest
    int lk_max_chunks;
    int lk_clusters[2][4];           // clusters of 2, 4, 8, 16 CTAs of the cluster lookup kernel (256, 512 threads) resident together
    int lk_cluster_mode;             // 0: never take the cluster form (HVD_LOOKUP_CLUSTER=0; tests run both forms)
    // occurrence lists of the frequency-weighted draft
    int32_t* fq_occ;    // [max_batch, HVD_FREQ_MAX_OCC]
    uint32_t* fq_cnt;   // [max_batch], zero at rest
    // shared warm-up corpus (caller-owned); cp_key / cp_cnt / cp_arrived: scratch in which the CTAs of a corpus
    // probe, or the diagonals of a trace replay, meet per request or state; zero at rest
    const int32_t* corpus;
    int32_t corpus_len;
    uint32_t* cp_start;  // index of the corpus: bucket boundaries [buckets + 1] ...
    int32_t* cp_pos;     // ... and the indexed positions, bucket by bucket
    uint32_t cp_mask;    // buckets - 1
    int cp_g;            // tokens in a key (min(min_match, 2))
    unsigned long long* cp_key;  // [max_batch]
    uint32_t* cp_cnt;            // [max_batch, HVD_MAX_L + 1]
    uint32_t* cp_arrived;        // [max_batch]
    // trace replay: per-state maximum and counts for a whole trace, grown on demand, zero at rest
    unsigned long long* rp_key;  // [rp_states]
    uint32_t* rp_cnt;            // [rp_states, HVD_MAX_L + 1]
    int64_t rp_states;
    // verify scratch
    unsigned long long* vf_row_key;  // [max_rows], zero at rest
    uint32_t* vf_next_unit;          // zero at rest
    int32_t* vf_alive;               // [max_batch] prefix verification: request still accepted through the last window
    int* dev_error;                  // device status word
    int vf_blocks_per_sm[2];         // per dtype
    long long vf_small_bytes;        // size limit of the warp-per-batch kernels (HVD_VERIFY_SMALL_BYTES; 0 = never)
    long long vf_boundary_bytes;     // prefix verification: streamed bytes that one window boundary is worth (HVD_PREFIX_BOUNDARY_BYTES)
    // device staging of the host-buffer entry point (grown on demand)
    int pdl_mask;     // ... for the three kernels of a step: bit 0 commit, 1 lookup, 2 stream, 3 one-layer scoring (default all)
    bool pdl_commit;  // bit 0 of the mask
    char* host_ws;
    size_t host_ws_bytes;
    char last_error[256];
};

namespace hvd {

inline hvd_status fail(hvd_ctx* ctx, hvd_status s, const char* msg) {
    if (ctx) snprintf(ctx->last_error, sizeof(ctx->last_error), "%s", msg);
    return s;
}

inline hvd_status cuda_fail(hvd_ctx* ctx, cudaError_t e, const char* where) {
    if (ctx) snprintf(ctx->last_error, sizeof(ctx->last_error), "%s: %s", where, cudaGetErrorString(e));
    return HVD_ERR_CUDA;
}

#define HVD_CUDA_TRY(ctx, call)                                          \
    do {                                                                 \
        cudaError_t e_ = (call);                                         \
        if (e_ != cudaSuccess) return hvd::cuda_fail((ctx), e_, #call);  \
    } while (0)

// Bounds-checked builds (-DHVD_DEBUG_BOUNDS; the stand-in for a memory checker where none can be run): every
// index into a history slab, the logits, the row keys and the per-row / per-request outputs is tested before
// the access.  A violation sets the device status word to HVD_DEV_OUT_OF_BOUNDS and the access is skipped:
// nothing traps.  In the normal build the test is the constant `true` and costs nothing.
#if defined(__CUDACC__) && defined(HVD_DEBUG_BOUNDS)
__device__ __forceinline__ bool index_in_bounds(int* status_word, long long i, long long lo, long long hi) {
    if (i >= lo && i < hi) return true;
    if (status_word) atomicExch(status_word, (int)HVD_DEV_OUT_OF_BOUNDS);
    return false;
}
#define HVD_IN_BOUNDS(status_word, i, lo, hi) hvd::index_in_bounds((status_word), (long long)(i), (long long)(lo), (long long)(hi))
#else
#define HVD_IN_BOUNDS(status_word, i, lo, hi) true
#endif

// Programmatic dependent launch: every kernel of the path lets its successor in the stream be
// scheduled early (pdl_trigger) and waits for its predecessor's memory (pdl_wait) before it reads
// anything a predecessor wrote.  Both are no-ops for a launch without the attribute.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Draft-length limit of a match of length L (App. A drafting table: draft cap, speculative factor and
// offset): min(K, floor(factor * L + offset)) with K clamped to [0, k_cap]; the product and the sum are two
// separately rounded fp32 operations; a factor <= 0 disables the second limit.
__device__ __forceinline__ int draft_limit(int K, int k_cap, int L, float spec_factor, float spec_offset) {
    int lim = max(0, min(K, k_cap));
    if (spec_factor > 0.0f) {
        const float f = __fadd_rn(__fmul_rn(spec_factor, (float)L), spec_offset);
        lim = min(lim, max(0, (int)floorf(f)));
    }
    return lim;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

struct ScoreArgs;  // hvd_score.cuh

// `fused` != NULL: the CTA that finishes a request also scores it and selects its draft
hvd_status launch_lookup(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                         const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K,
                         int32_t n_max, int32_t* draft, int32_t* draft_len, int32_t* match_len,
                         int32_t* match_pos, int32_t* match_cnt, const ScoreArgs* fused, cudaStream_t stream,
                         bool successor_works_ahead = false);


void lookup_cluster_setup(hvd_ctx* ctx);

ScoreArgs make_score_args(hvd_ctx* ctx, int32_t B, const int32_t* hist_len, const int32_t* prompt_len,
                          const hvd_req_state* state, const int32_t* K, const int32_t* draft,
                          const int32_t* draft_len, const int32_t* match_len, const int32_t* match_pos,
                          const int32_t* match_cnt, const int32_t* model_draft, const int32_t* model_len,
                          float* features, float* score, int32_t* select, int32_t* sel_draft, int32_t* sel_len);

hvd_status launch_score_select(hvd_ctx* ctx, int32_t B, const int32_t* hist_len,
                               const int32_t* prompt_len, const hvd_req_state* state, const int32_t* K,
                               const int32_t* draft, const int32_t* draft_len, const int32_t* match_len,
                               const int32_t* match_pos, const int32_t* match_cnt,
                               const int32_t* model_draft, const int32_t* model_len, float* features,
                               float* score, int32_t* select, int32_t* sel_draft, int32_t* sel_len,
                               cudaStream_t stream);

hvd_status launch_score_select_ext(hvd_ctx* ctx, int32_t B, const int32_t* hist_len, const int32_t* prompt_len,
                                   const hvd_req_state* state, const int32_t* K, const int32_t* draft,
                                   const int32_t* draft_len, const int32_t* match_len, const int32_t* match_pos,
                                   const int32_t* match_cnt, const int32_t* match_src, const float* suffix,
                                   const int32_t* model_draft, const int32_t* model_len, float* features, float* score,
                                   int32_t* select, int32_t* sel_draft, int32_t* sel_len, cudaStream_t stream);

hvd_status launch_replay(hvd_ctx* ctx, const int32_t* trace, int32_t n, int32_t K, int32_t* label, int32_t* draft_len,
                         int32_t* match_len, int32_t* match_pos, int32_t* match_cnt, cudaStream_t stream);

hvd_status launch_lookup_freq(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                              const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K, int32_t n_max,
                              float min_prob, int32_t max_occ, float threshold, const int32_t* model_draft,
                              const int32_t* model_len, int32_t* draft, int32_t* draft_len, float* score,
                              int32_t* match_len, int32_t* match_pos, int32_t* match_cnt, int32_t* select,
                              int32_t* sel_draft, int32_t* sel_len, cudaStream_t stream);

hvd_status launch_lookup_corpus(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                                const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K, int32_t n_max,
                                int32_t* draft, int32_t* draft_len, int32_t* match_len, int32_t* match_pos,
                                int32_t* match_src, int32_t* match_cnt, cudaStream_t stream);

hvd_status build_corpus_index(hvd_ctx* ctx, const int32_t* corpus, int64_t m);
void release_corpus_index(hvd_ctx* ctx);

struct VerifyArgs {
    int32_t B;
    const void* logits;
    int64_t V;
    const int64_t* row_off;
    int32_t k_uniform;
    const int32_t* sel_draft;
    const int32_t* sel_len;
    const int32_t* parent;  // NULL: the draft is a chain; else parent[b, i] of tree node i
    const int32_t* select;
    int32_t* hist;
    const int64_t* hist_off;
    const int32_t* hist_cap;
    int32_t* hist_len;
    hvd_req_state* state;
    int32_t* accepted;
    int32_t* committed;
    int32_t* n_commit;
    int32_t* target_tok;
    int32_t* status;
    int32_t k_cap;
    // scratch
    unsigned long long* row_key;  // [total_rows] (value, ~index) key per logits row, zero at rest
    const long long* ext_keys;    // NULL, or row keys in signed order handed in by the caller (commit only)
    int64_t total_rows;
    uint32_t* next_unit;   // unit counter, zero at rest
    int* dev_error;        // device status word (no kernel sets it at present)
    int32_t n_batch_row;   // 4 KB batches per row
    // prefix verification: only the needed rows [win_lo, win_hi) of a request are streamed, and only while the
    // request is alive (alive == NULL: every request is); the defaults stream every needed row
    int32_t win_lo = 0, win_hi = 0x7fffffff;
    int32_t win_index = 0;
    int32_t* alive = nullptr;
    unsigned long long* rows_read = nullptr;  // optional: += logits rows streamed by the call
    bool rows_in_commit = false;              // ... counted by the commit (one window: any streaming kernel) or by the streaming launches
};

hvd_status launch_verify(hvd_ctx* ctx, VerifyArgs a, hvd_dtype dtype, cudaStream_t stream, bool with_commit = true);
// the same result (without target tokens) from the rows up to the first rejected draft token only
hvd_status launch_verify_prefix(hvd_ctx* ctx, VerifyArgs a, hvd_dtype dtype, cudaStream_t stream);
// ... and its pieces, for the host-buffer entry point, which copies a window's rows between two launches:
// the window edges e[0..n] (returns n), window j (streaming launch and gate), the commit
int prefix_window_edges(const hvd_ctx* ctx, const VerifyArgs& a, hvd_dtype dtype, int* e);
hvd_status launch_prefix_window(hvd_ctx* ctx, VerifyArgs a, hvd_dtype dtype, const int* e, int j, int n_win, cudaStream_t stream);
hvd_status launch_prefix_commit(hvd_ctx* ctx, VerifyArgs a, cudaStream_t stream);
// the checked arguments of a verification call (hvd_api.cu), without launching anything
hvd_status make_verify_args(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V, const int64_t* row_off,
                            int32_t k_uniform, int64_t total_rows, const int32_t* sel_draft, const int32_t* sel_len,
                            const int32_t* select, int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                            int32_t* hist_len, hvd_req_state* state, int32_t* accepted, int32_t* committed,
                            int32_t* n_commit, int32_t* status, VerifyArgs* out);
// commit and the next cycle's lookup + scoring in one kernel (after launch_verify without its commit)
bool cycle_fits_one_cta(int32_t n_max);
hvd_status launch_commit_lookup(hvd_ctx* ctx, const VerifyArgs& va, const int32_t* K, int32_t n_max, int32_t* draft,
                                int32_t* draft_len, int32_t* match_len, int32_t* match_pos, int32_t* match_cnt,
                                const ScoreArgs& sa, cudaStream_t stream);
hvd_status launch_verify_keys(hvd_ctx* ctx, VerifyArgs a, hvd_dtype dtype, long long* keys, int64_t v_offset,
                              cudaStream_t stream);
hvd_status launch_commit_keys(hvd_ctx* ctx, VerifyArgs a, cudaStream_t stream);
int verify_occupancy(hvd_dtype dtype, size_t dyn_smem);
size_t verify_dyn_smem(int32_t B);

}  // namespace hvd
