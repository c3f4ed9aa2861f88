/*
 * hvd.h -- C ABI of the B200 (sm_100a) library for the per-step path of
 * Hybrid Verified Decoding: cache-draft lookup, payoff scoring and draft
 * selection, greedy verification and commit.
 *
 * One decoding cycle (Algorithm 1 of the paper) maps to three calls:
 *
 *     d_c          <- D_C(x; C)                      hvd_lookup
 *     phi, y       <- Phi(x, d_c, C, h), g_theta     hvd_score_select
 *     d            <- d_c if y >= tau else D_m(x)    hvd_score_select
 *     (target forward on x || d: the caller's job, gives the logits)
 *     a, z         <- Verify(x, d; M)                hvd_verify_commit
 *     x <- x || z, update C and h                    hvd_verify_commit
 *
 * Conventions
 *  - Unless an argument is marked HOST, every pointer is a DEVICE pointer owned
 *    by the caller.  The library never frees caller memory and keeps no
 *    reference to it after the call returns; the two registration calls
 *    (hvd_set_corpus, hvd_set_token_classes) say so where they do.
 *  - Device entry points only enqueue work on `stream` (a cudaStream_t passed
 *    as void*, NULL = default stream) and never synchronise.  The set-up calls
 *    (hvd_create, hvd_set_predictor*, hvd_set_corpus), hvd_step_host and the
 *    first hvd_replay_labels call for a longer trace do wait, and say so.
 *  - Variants of the three steps (two-layer and extended predictors, token
 *    trees, frequency-weighted drafts, a shared warm-up corpus, vocabulary
 *    shards, trace replay) are declared next to the step they vary.
 *  - Errors the host can see (NULL pointer, sizes outside the limits given at
 *    hvd_create, unknown dtype, misaligned base pointer) are returned at once
 *    and nothing is enqueued.  Data-dependent problems are reported per
 *    request in `status[b]` by the device; nothing is ever written out of
 *    bounds and no kernel traps or waits on another.
 *  - A context belongs to one device.  Calls on one context must not overlap
 *    on the GPU (they share the context's scratch memory): use one stream per
 *    context, or one context per concurrent stream.
 *  - Token histories are ragged: request b owns the slab
 *    hist[hist_off[b] .. hist_off[b] + hist_cap[b]) of which the first
 *    hist_len[b] tokens are valid (prompt followed by committed tokens).
 *  - Consecutive kernels of a context are joined by programmatic dependent
 *    launch: a kernel may be resident while its predecessor on the stream
 *    still runs, and waits on the device before it reads anything the
 *    predecessor writes.  What no call of this library writes (hist_off,
 *    hist_cap, K, the predictor) may be read before that wait, and the
 *    lookup asks the L2 for the history slabs there.  A caller's own kernel
 *    that writes those arrays is complete before a kernel of the library
 *    starts, unless it signals programmatic launch completion itself: then it
 *    must have written them before it does.
 *    Results do not depend on it.  One environment
 *    variable, read once by hvd_create, changes it: HVD_PDL_MASK (a bit per
 *    kernel pair: 1 commit, 2 lookup, 4 verify stream, 8 scoring; default 15,
 *    0 = plain launches).  It exists for the tests, which run the parity
 *    cases with and without the overlap.
 *  - hvd_verify_commit and its variants stream the logits with one of two
 *    kernels, chosen by the size of the logits: one warp per 4 KB batch of a
 *    row up to 160 MB, a persistent kernel with work queues beyond that.
 *    HVD_VERIFY_SMALL_BYTES (read once by hvd_create) moves the limit, 0 =
 *    always the persistent kernel: it exists for the tests, which run both
 *    kernels over the same cases.  Results do not depend on it.
 *  - hvd_lookup and its variants scan a history that does not fit one CTA
 *    in chunks of 8 K or 16 K tokens, one CTA each.  When every request's
 *    chunk CTAs can be resident at once they form one thread-block cluster
 *    per request and meet in distributed shared memory, else they meet
 *    through the context's scratch.  HVD_LOOKUP_CLUSTER=0 (read once by
 *    hvd_create) turns the cluster form off: it exists for the tests, which
 *    run both.  Results do not depend on it.
 *  - hvd_verify_commit_prefix cuts the rows of a request into windows whose
 *    sizes follow from the size of the call; HVD_PREFIX_BOUNDARY_BYTES (read
 *    once by hvd_create; default 64 MiB, what one more streaming launch is
 *    worth in streamed bytes) moves them: it exists for the tests, which set
 *    it to 1 to get every window on small inputs.  Results do not depend on
 *    it.  Nothing else is read from the environment by the product path.
 */
#ifndef HVD_H
#define HVD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define HVD_API __attribute__((visibility("default")))
#else
#define HVD_API
#endif

typedef struct hvd_ctx hvd_ctx;

typedef enum {
    HVD_OK = 0,
    HVD_ERR_INVALID_ARG = 1,
    HVD_ERR_CUDA = 2,
    HVD_ERR_UNSUPPORTED = 3,
    HVD_ERR_ALLOC = 4
} hvd_status;

typedef enum { HVD_F32 = 0, HVD_BF16 = 1 } hvd_dtype;

/* written per request, on the device, by hvd_verify_commit */
typedef enum {
    HVD_REQ_OK = 0,
    HVD_REQ_CAPACITY = 1, /* slab too small: commit clamped to the free space */
    HVD_REQ_BAD_LEN = 2   /* hist_len outside [0, hist_cap] or no logits rows: request skipped */
} hvd_req_status;

/* values of the device status word (hvd_device_status) */
typedef enum {
    HVD_DEV_OK = 0,
    HVD_DEV_WAIT_EXPIRED = 1, /* a kernel gave up a bounded wait for its own copies: outputs incomplete */
    HVD_DEV_OUT_OF_BOUNDS = 2 /* bounds-checked builds only: an index left its array; the access was skipped */
} hvd_dev_status;

/* Recent-history summary h of one request (Sec. 3.3; Algorithm 1 "update C and h").
   bit j of sel_bits = 1 if the cache draft was verified j steps ago;
   byte j of acc_ring = accepted length j steps ago. */
typedef struct {
    uint32_t sel_bits;
    uint32_t pad;
    uint64_t acc_ring;
} hvd_req_state;

enum { HVD_N_FEATURES = 8, HVD_MAX_K = 64, HVD_MAX_L = 64, HVD_MAX_HIDDEN = 256 };
/* Longest history a context accepts: positions and the rounded-up scan range stay inside int32. */
enum { HVD_MAX_HIST_LEN = 0x7fffffff - (1 << 20) };
enum { HVD_N_TOKEN_CLASSES = 5, HVD_N_FEATURES_EXT = 14 };

typedef struct {
    int32_t max_batch;    /* largest B of any call, 1..8192 */
    int32_t k_cap;        /* row length of every draft array, 1..64 (suffix cache "maximum draft tokens") */
    int32_t l_max;        /* longest suffix match looked for, 1..64 (suffix cache "maximum tree depth") */
    int32_t min_match;    /* shorter matches count as no match, >= 1 */
    float spec_factor;    /* draft_len <= floor(spec_factor*match_len + spec_offset); <= 0 disables the limit */
    float spec_offset;    /* ("maximum speculative factor / offset" of the suffix cache: 1.0 / 0.0) */
    int32_t hidden;       /* hidden units of the payoff MLP, 1..256 */
    int32_t max_hist_len; /* largest hist_len of any request, in [1, HVD_MAX_HIST_LEN] */
    int64_t max_rows;     /* largest total number of logits rows of any call */
    int64_t max_vocab;    /* largest V of any call */
} hvd_config;

/* Creates a context on the current CUDA device and allocates its scratch
   memory (a few MB; sized from cfg).  *out is NULL on failure. */
HVD_API hvd_status hvd_create(hvd_ctx** out, const hvd_config* cfg);
HVD_API hvd_status hvd_destroy(hvd_ctx* ctx);
HVD_API const char* hvd_status_string(hvd_status s);
/* text of the last error recorded on this context ("" if none) */
HVD_API const char* hvd_last_error(const hvd_ctx* ctx);

/* Device-side status of the context: *code = 0 if every kernel ran to completion, 1 if a kernel
   gave up a bounded wait (its outputs are then incomplete).  Waits for the device (HOST pointer). */
HVD_API hvd_status hvd_device_status(hvd_ctx* ctx, int32_t* code);

/* Payoff predictor g_theta (Sec. 3.3): y = b2 + sum_j W2[j] * relu(b1[j] + sum_i W1[j][i] * phi[i]),
   fp32, accumulated left to right with fused multiply-adds, and the threshold tau of Sec. 3.4.
   W1 [hidden, 8] row-major, b1 [hidden], W2 [hidden]: HOST pointers, copied before returning. */
HVD_API hvd_status hvd_set_predictor(hvd_ctx* ctx, const float* W1, const float* b1, const float* W2,
                             float b2, float tau, void* stream);

/* The same predictor with two hidden ReLU layers, the shape the paper trains (App. B, table "Payoff
   predictor training configuration": 2 hidden layers of 256 units):
   h1 = relu(W1 phi + b1), h2 = relu(Wh h1 + bh), y = b2 + W2 . h2, same accumulation rule.
   Wh [hidden, hidden] row-major (row j = inputs of unit j), bh [hidden]: HOST pointers, copied before
   returning.  Afterwards hvd_score_select and hvd_lookup_score_select use this predictor (the
   latter then runs as two kernels); hvd_set_predictor switches back to one layer. */
HVD_API hvd_status hvd_set_predictor2(hvd_ctx* ctx, const float* W1, const float* b1, const float* Wh,
                                      const float* bh, const float* W2, float b2, float tau, void* stream);

/*
 * Cache-based drafting D_C (Sec. 3.2), with the request's own history as the cache.
 * For every request: among the positions e in [1, n-1], find the longest l <= l_max such that
 * hist[e-l .. e) equals the last l tokens hist[n-l .. n)  (n = hist_len[b]; e = n, the suffix
 * itself, is left out; occurrences may overlap the suffix).
 *   match_len[b] = that l (0 if it is shorter than min_match)
 *   match_pos[b] = the largest e reaching it (-1 if none): the most recent occurrence
 *   match_cnt[b] = how many e reach it (lengths are capped at l_max before counting)
 *   draft[b, 0..d) = hist[e .. e+d),  d = draft_len[b] = min(K[b], floor(spec_factor*l + spec_offset), n - e);
 *   draft[b, d..k_cap) = -1
 * K[b] is clamped to [0, k_cap].  A request whose hist_len is outside [0, min(hist_cap, n_max)]
 * is treated as an empty history (no match).
 *
 * hist      int32, 16-byte aligned base; slabs should start on 16-byte boundaries (any start works)
 * hist_off  int64 [B], hist_cap int32 [B], hist_len int32 [B], K int32 [B]
 * n_max     HOST value: upper bound on hist_len[b] of this call (sizes the launch), <= max_hist_len
 * outputs   draft int32 [B, k_cap]; draft_len, match_len, match_pos, match_cnt int32 [B]
 */
HVD_API hvd_status hvd_lookup(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                      const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K,
                      int32_t n_max, int32_t* draft, int32_t* draft_len, int32_t* match_len,
                      int32_t* match_pos, int32_t* match_cnt, void* stream);

/*
 * Payoff features Phi, predictor g_theta and the selection rule (Sec. 3.3, Sec. 3.4, App. B):
 *   phi0 = match_len, phi1 = draft_len, phi2 = bit_width(match_cnt),
 *   phi3 = (n - match_pos) / n (0 without a match),
 *   phi4 = bit_width(prompt_len), phi5 = (n - prompt_len) / n (0 for n = 0),
 *   phi6 = popcount(sel_bits & 0xFF) / 8, phi7 = (sum of the 8 bytes of acc_ring) / 8,
 *   score = g_theta(phi);   select = 1 (verify the cache draft) iff draft_len > 0 and score >= tau,
 *   sel_draft/sel_len = the cache draft if select, else the first min(model_len, K) model tokens.
 * model_draft [B, k_cap] / model_len [B] may both be NULL (no model drafter: empty draft).
 * features [B, 8] may be NULL.  Outputs: score fp32 [B], select int32 [B], sel_draft int32
 * [B, k_cap] (-1 beyond sel_len), sel_len int32 [B].  Needs hvd_set_predictor first.
 */
HVD_API hvd_status hvd_score_select(hvd_ctx* ctx, int32_t B, const int32_t* hist_len,
                            const int32_t* prompt_len, const hvd_req_state* state, const int32_t* K,
                            const int32_t* draft, const int32_t* draft_len, const int32_t* match_len,
                            const int32_t* match_pos, const int32_t* match_cnt,
                            const int32_t* model_draft, const int32_t* model_len, float* features,
                            float* score, int32_t* select, int32_t* sel_draft, int32_t* sel_len,
                            void* stream);

/*
 * The same step on the extended feature vector (App. B feature-group table, all four groups):
 * features 0..7 as in hvd_score_select; 8..12 the draft-structure group, for each of
 * HVD_N_TOKEN_CLASSES token classes (bit 0 whitespace, 1 punctuation, 2 line break, 3 bracket,
 * 4 delimiter-like) the share of the cache draft's tokens that carry the class, count / draft_len as
 * one IEEE division (0 for an empty draft; tokens outside [0, V) carry no class); 13 the suffix
 * score of the cache match (suffix_score float [B], DEVICE, e.g. hvd_lookup_freq's score; NULL: 0).
 * match_src (int32 [B], DEVICE, hvd_lookup_corpus's output; may be NULL): where it is 1 the match lies
 * in the shared corpus and feature 3 (recency) is taken at position 0, i.e. older than the history.
 *
 * hvd_set_token_classes registers the class bits: cls uint8 [V], DEVICE, owned by the caller and kept
 * alive while registered (NULL or V = 0 unregisters).  hvd_set_predictor_ext stores a predictor that
 * takes the 14 features: W1 [hidden, 14] row-major, b1 [hidden], optional second layer Wh [hidden,
 * hidden] / bh [hidden] (both NULL: one hidden layer), W2 [hidden], HOST pointers, copied before the
 * call returns; it replaces the predictor of hvd_set_predictor / hvd_set_predictor2 and vice versa
 * (hvd_score_select then fails until its own predictor is set again).  Evaluation order as in
 * hvd_score_select, over 14 inputs.  features float [B, 14] or NULL.  Everything else as in
 * hvd_score_select.
 */
HVD_API hvd_status hvd_set_token_classes(hvd_ctx* ctx, const uint8_t* cls, int64_t V);
HVD_API hvd_status hvd_set_predictor_ext(hvd_ctx* ctx, const float* W1, const float* b1, const float* Wh,
                                         const float* bh, const float* W2, float b2, float tau, void* stream);
HVD_API hvd_status hvd_score_select_ext(hvd_ctx* ctx, int32_t B, const int32_t* hist_len, const int32_t* prompt_len,
                                        const hvd_req_state* state, const int32_t* K, const int32_t* draft,
                                        const int32_t* draft_len, const int32_t* match_len,
                                        const int32_t* match_pos, const int32_t* match_cnt,
                                        const int32_t* match_src, const float* suffix_score,
                                        const int32_t* model_draft, const int32_t* model_len, float* features,
                                        float* score, int32_t* select, int32_t* sel_draft, int32_t* sel_len,
                                        void* stream);

/*
 * hvd_lookup and hvd_score_select in one launch (Alg. 1: draft, score and select are consecutive
 * and per request): the thread block that finishes a request's history scan goes straight on to
 * its features, score and selection.  Arguments and every output exactly as in the two separate
 * calls; all lookup outputs are still written.
 */
HVD_API hvd_status hvd_lookup_score_select(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                                           const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K,
                                           int32_t n_max, const int32_t* prompt_len, const hvd_req_state* state,
                                           const int32_t* model_draft, const int32_t* model_len, int32_t* draft,
                                           int32_t* draft_len, int32_t* match_len, int32_t* match_pos,
                                           int32_t* match_cnt, float* features, float* score, int32_t* select,
                                           int32_t* sel_draft, int32_t* sel_len, void* stream);

/*
 * Shared warm-up corpus (Algorithm 1: the suffix cache is initialised from cache-warmup traces and
 * the prompt; App. C: warm-up prompts of the same dataset).  hvd_set_corpus registers one token
 * array shared by all requests: corpus int32 [m], DEVICE, 16-byte aligned, owned by the caller and
 * kept alive and unchanged while registered; a negative entry separates two traces (it is never
 * part of a match and ends a draft); m (HOST value) in [0, 2^31 - 2]; corpus = NULL or m = 0
 * unregisters.  Registration builds an index of the corpus (device memory of about 12 bytes per
 * token, kernels on the default stream) and returns when it is ready: a set-up call, not for the
 * decoding loop and not under stream capture; no hvd_lookup_corpus call of this context may be in
 * flight.  Takes effect for later hvd_lookup_corpus calls on any stream.  The index is keyed on the
 * last min(min_match, 2) tokens of a match.  Errors: HVD_ERR_INVALID_ARG (alignment, m),
 * HVD_ERR_CUDA (allocation or build failed: no corpus is registered afterwards).
 *
 * hvd_lookup_corpus is hvd_lookup over [corpus, own history].  Candidates are the history positions
 * of hvd_lookup and the corpus positions e in [1, m-1] whose token corpus[e] is not a separator,
 * with match length l <= min(l_max, e, n) and no separator inside the match.  The longest match
 * wins; at equal length the history comes before the corpus, and within a source the latest
 * position.  match_src int32 [B] (DEVICE output): 0 = history (or no match), 1 = corpus; match_pos
 * is the position in that source; match_cnt counts both sources; a corpus draft is
 * corpus[e .. e + d), d = min(K, floor(spec_factor * L + spec_offset), m - e), cut before the first
 * separator.  Everything else as in hvd_lookup.  hvd_score_select_ext takes match_src for the payoff
 * features of corpus matches.
 * Uses context scratch: one call at a time per context.
 */
HVD_API hvd_status hvd_set_corpus(hvd_ctx* ctx, const int32_t* corpus, int64_t m);
HVD_API hvd_status hvd_lookup_corpus(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                                     const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K,
                                     int32_t n_max, int32_t* draft, int32_t* draft_len, int32_t* match_len,
                                     int32_t* match_pos, int32_t* match_src, int32_t* match_cnt, void* stream);

/*
 * Frequency-weighted cache draft, suffix score and the score-threshold selection (Sec. 4.1
 * "Frequency-Based Hybrid Decoding": same cache-first structure, the decision taken on the
 * frequency-derived cache score; App. A drafting table: speculation limits and the minimum token
 * probability).  Steps, per request:
 *   1. hvd_lookup's search: longest match length L, its latest occurrence, the number c of
 *      occurrences (match_len / match_pos / match_cnt exactly as hvd_lookup writes them).
 *   2. limit = min(K, floor(spec_factor * L + spec_offset)) as in hvd_lookup.  If c <= max_occ all c
 *      occurrences are merged: starting with all of them alive, step s takes the token that most
 *      alive occurrences continue with at offset s (ties: the token whose latest such occurrence is
 *      later; occurrences that run into the end of the history have no token), p = count / alive in
 *      fp32 (one IEEE division); the walk stops when p < min_prob, at `limit` tokens, or when no alive
 *      occurrence has a token left; otherwise the token joins the draft, p is added to the score
 *      (fp32, in step order) and only the occurrences that continue with it stay alive.
 *      If c > max_occ the draft is hvd_lookup's (latest occurrence only) and score = draft_len.
 *   3. optional (select, sel_draft, sel_len all non-NULL): select = (draft_len > 0 && score >= threshold);
 *      sel_draft / sel_len as in hvd_score_select (the model draft, or an empty draft, otherwise).
 * draft int32 [B, k_cap] (-1 beyond draft_len), draft_len int32 [B], score float [B]: DEVICE outputs.
 * min_prob, max_occ (1 .. HVD_FREQ_MAX_OCC), threshold: HOST values.  Everything else as in hvd_lookup.
 * Uses context scratch: one call at a time per context.
 */
enum { HVD_FREQ_MAX_OCC = 128 };
HVD_API hvd_status hvd_lookup_freq(hvd_ctx* ctx, int32_t B, const int32_t* hist, const int64_t* hist_off,
                                   const int32_t* hist_cap, const int32_t* hist_len, const int32_t* K,
                                   int32_t n_max, float min_prob, int32_t max_occ, float threshold,
                                   const int32_t* model_draft, const int32_t* model_len, int32_t* draft,
                                   int32_t* draft_len, float* score, int32_t* match_len, int32_t* match_pos,
                                   int32_t* match_cnt, int32_t* select, int32_t* sel_draft, int32_t* sel_len,
                                   void* stream);

/*
 * Payoff labels by trace replay (Sec. 3.3, "We derive training labels ..."; App. B "Payoff Label
 * Construction").  Every position t = 1..n of a recorded trace x[0..n) is a decoding state with prefix
 * x[0..t): its cache draft is the hvd_lookup result on that prefix (same rules, K for every state),
 * and its label is y_t = max{ l <= draft_len : draft[0..l) == x[t .. t+l) }, the number of draft tokens
 * the trace's own continuation confirms.  Outputs (int32 [n], index t-1): label, draft_len, match_len,
 * match_pos, match_cnt.  trace: DEVICE, 16-byte aligned; n (HOST value) <= max_hist_len.  The first
 * call, and any call with a longer trace than before, allocates per-state scratch (268 bytes per
 * position) after waiting for the stream: not for use under stream capture.  These are the
 * regression targets of the payoff predictor; the recent-history features depend on the decoding
 * loop and are not produced here.  Uses context scratch: one call at a time per context.
 */
HVD_API hvd_status hvd_replay_labels(hvd_ctx* ctx, const int32_t* trace, int32_t n, int32_t K, int32_t* label,
                                     int32_t* draft_len, int32_t* match_len, int32_t* match_pos,
                                     int32_t* match_cnt, void* stream);

/*
 * Greedy verification and commit (Sec. 3.1 Verify; Sec. 3.4; Algorithm 1; the accepted length is
 * the label equation of Sec. 3.3).  Request b owns logits rows [r0, r1): r0 = row_off[b],
 * r1 = row_off[b+1], or r0 = b*(k_uniform+1), r1 = r0 + k_uniform + 1 when row_off is NULL.  Row r
 * holds V values of `dtype`, densely packed at logits + r*V.  Row r0+i is the target model's
 * output after the prefix extended by the first i draft tokens.  With m = min(sel_len[b], r1-r0-1):
 *   t_i = argmax of row r0+i, i = 0..m   (lowest index among equal maxima; -0.0 equals +0.0; the
 *         logits must not contain NaN)
 *   a   = largest l <= m with sel_draft[b, j] == t_j for all j < l         -> accepted[b]
 *   z   = sel_draft[b, 0..a) followed by t_a  (always a+1 tokens)          -> committed[b, 0..a], -1 after
 *   the first w = min(a+1, hist_cap - n) tokens of z are appended to the history,
 *   hist_len[b] += w, n_commit[b] = w, status[b] = HVD_REQ_CAPACITY if w < a+1;
 *   state[b].sel_bits = sel_bits << 1 | select[b];  state[b].acc_ring = acc_ring << 8 | a.
 * Rows beyond m are not read.  target_tok (may be NULL) receives t_i for the rows read, -1 for
 * the others.
 *
 * logits     16-byte aligned base recommended (any alignment of the element type works)
 * total_rows HOST value: number of rows in `logits` (= row_off[B]); <= max_rows
 * in/out     hist, hist_len [B], state [B];   outputs accepted, n_commit, status int32 [B],
 *            committed int32 [B, k_cap+1], target_tok int32 [total_rows] or NULL
 */
HVD_API hvd_status hvd_verify_commit(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V,
                             const int64_t* row_off, int32_t k_uniform, int64_t total_rows,
                             const int32_t* sel_draft, const int32_t* sel_len, const int32_t* select,
                             int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                             int32_t* hist_len, hvd_req_state* state, int32_t* accepted,
                             int32_t* committed, int32_t* n_commit, int32_t* target_tok,
                             int32_t* status, void* stream);

/*
 * hvd_verify_commit without target_tok, reading the logits only as far as the result depends on them
 * (Sec. 3.1: Verify returns the accepted length a and the tokens z; rows behind the first rejected draft
 * token enter neither).  The needed rows of a request are streamed window by window, one streaming launch
 * per window over all requests that are still alive: a request goes on to its next window only if every row
 * so far carried its draft token and rows are left.  The first window holds at least 64 MiB of the batch
 * (B * V * element size per row index) and at least two rows, the windows double from there, and no further
 * boundary is set once the rows left, halved per window so far, weigh less than 128 MiB: on a large call
 * rows [0,2), [2,4), [4,8), [8,16), [16, k_cap]; on a small one a single window, i.e. hvd_verify_commit.
 * accepted, committed, n_commit, status, the histories and the state come out exactly as from
 * hvd_verify_commit; a request reads at most twice the rows its result needs, plus the first window.
 * It pays when accepted lengths are short against the drafts (the paper's runs: a few tokens on average,
 * Sec. 5.4 execution breakdown) and the logits are large; when most drafts are accepted to the end the
 * extra launches are paid for nothing (8 to 10 us each).  Chain drafts only (no token trees).
 *
 * rows_read  device uint64, 8-byte aligned, or NULL: the number of needed logits rows streamed is ADDED to it
 * all else   as hvd_verify_commit
 */
HVD_API hvd_status hvd_verify_commit_prefix(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V,
                                    const int64_t* row_off, int32_t k_uniform, int64_t total_rows,
                                    const int32_t* sel_draft, const int32_t* sel_len, const int32_t* select,
                                    int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                                    int32_t* hist_len, hvd_req_state* state, int32_t* accepted,
                                    int32_t* committed, int32_t* n_commit, uint64_t* rows_read,
                                    int32_t* status, void* stream);

/*
 * hvd_verify_commit, then at once the NEXT cycle's hvd_lookup_score_select on the histories it has just
 * extended (Algorithm 1: the end of one iteration and the start of the next).  In a decoding loop the two
 * are adjacent, and one kernel does the commit and the lookup: a launch and two dependent global round
 * trips less per cycle.  Results are exactly those of the two calls one after the other.
 * The verification arguments are hvd_verify_commit's.  `next` (a HOST struct of DEVICE pointers, read
 * before the call returns) holds hvd_lookup_score_select's remaining arguments:
 *   K, prompt_len, model_draft, model_len (or both NULL)   inputs of the next cycle
 *   n_max            HOST value: upper bound on hist_len[b] AFTER this commit (<= max_hist_len)
 *   draft .. match_cnt, features (or NULL), score          outputs as in hvd_lookup / hvd_score_select
 *   select, sel_draft, sel_len                             the next selection; these may be the very
 *                    arrays the commit reads (a request's old entries are read before its new ones are written)
 * hist, hist_off, hist_cap, hist_len and state are the ones of the verification.  The one-kernel form
 * needs n_max + 2 <= 32768 and the one-layer predictor; otherwise the call enqueues the same kernels
 * as the two separate calls.  Needs hvd_set_predictor first.
 */
typedef struct {
    const int32_t* K;
    int32_t n_max;
    const int32_t* prompt_len;
    const int32_t* model_draft;
    const int32_t* model_len;
    int32_t* draft;
    int32_t* draft_len;
    int32_t* match_len;
    int32_t* match_pos;
    int32_t* match_cnt;
    float* features;
    float* score;
    int32_t* select;
    int32_t* sel_draft;
    int32_t* sel_len;
} hvd_next_cycle;
HVD_API hvd_status hvd_verify_commit_next(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V,
                                          const int64_t* row_off, int32_t k_uniform, int64_t total_rows,
                                          const int32_t* sel_draft, const int32_t* sel_len, const int32_t* select,
                                          int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                                          int32_t* hist_len, hvd_req_state* state, int32_t* accepted,
                                          int32_t* committed, int32_t* n_commit, int32_t* target_tok,
                                          int32_t* status, const hvd_next_cycle* next, void* stream);

/*
 * Greedy verification of a token TREE and commit.  The paper's model drafter (EAGLE3) proposes a
 * tree (App. A "Drafting configuration": 32 draft tokens, depth 8, top-k 4); the verification rule is
 * unchanged (Sec. 3.1, Sec. 3.4).  Node i of request b has token sel_draft[b, i] and parent
 * parent[b, i] in {-1, 0..i-1} (-1: the node follows the prefix directly; any other value makes the
 * node unreachable); sel_len[b] = number of nodes.  Row r0 of the request's logits is the target's
 * output after the prefix, row r0+i+1 its output after node i.  The walk starts at the prefix: the
 * target's token at the current node is the argmax of that node's row; the first child (lowest
 * index) that carries this token is accepted and the walk goes on there; otherwise it stops.
 * accepted[b] = number of accepted nodes, committed[b] = their tokens followed by the target's token
 * at the last node.  Everything else (rows, ties, append, capacity, state, target_tok, status) is as
 * in hvd_verify_commit, which is the special case parent[b, i] = i-1.
 */
HVD_API hvd_status hvd_verify_commit_tree(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V,
                                          const int64_t* row_off, int32_t k_uniform, int64_t total_rows,
                                          const int32_t* sel_draft, const int32_t* sel_len,
                                          const int32_t* parent /*[B, k_cap]*/, const int32_t* select,
                                          int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                                          int32_t* hist_len, hvd_req_state* state, int32_t* accepted,
                                          int32_t* committed, int32_t* n_commit, int32_t* target_tok,
                                          int32_t* status, void* stream);

/*
 * The same decoding cycle with HOST buffers: one call copies the step's inputs to the device,
 * runs hvd_lookup, hvd_score_select and hvd_verify_commit there, copies the results back, waits
 * for the stream, and appends the committed tokens to the host histories.  Every pointer in the
 * struct is a HOST pointer (pinned memory makes the copies asynchronous and faster; pageable
 * memory works).  Arrays have the shapes documented at the three device entry points.
 * Of the logits only rows that verification reads cross the bus, and verification reads as
 * hvd_verify_commit_prefix does (there is no target_tok here): with accepted lengths of a few tokens most
 * of the logits stay on the host.  Logits in page-locked memory (cudaHostAlloc, cudaHostRegister, a pinned
 * tensor) are read in place: the streaming kernels load the rows they need straight from the host buffer,
 * nothing is staged, and the call waits for the stream once, before it returns.  Pageable logits are staged:
 * the call waits for the selection, then copies and verifies the needed rows window by window, waiting after
 * every window but the last for the flags of which requests are still accepted so far (a small call, one
 * window, copies rows 0..sel_len of every valid request at once).
 * The context keeps a device staging area that it (re)allocates when a call needs more than any
 * earlier one (a synchronous cudaMalloc: not for use inside stream capture).
 */
typedef struct {
    int32_t B;
    int32_t n_max;            /* upper bound on hist_len[b] */
    int64_t hist_words;       /* length of the hist array in int32 words (all slabs) */
    int32_t* hist;            /* in/out: committed tokens are appended */
    const int64_t* hist_off;  /* [B] */
    const int32_t* hist_cap;  /* [B] */
    int32_t* hist_len;        /* [B] in/out */
    const int32_t* K;         /* [B] */
    const int32_t* prompt_len; /* [B] */
    hvd_req_state* state;     /* [B] in/out */
    const int32_t* model_draft; /* [B, k_cap] or NULL */
    const int32_t* model_len; /* [B] or NULL */
    const void* logits;       /* [total_rows, V] of dtype */
    int32_t dtype;            /* hvd_dtype */
    int32_t k_uniform;        /* used when row_off is NULL */
    int64_t V;
    const int64_t* row_off;   /* [B+1] or NULL */
    int64_t total_rows;
    /* outputs */
    float* score;             /* [B] */
    int32_t* select;          /* [B] */
    int32_t* sel_draft;       /* [B, k_cap] */
    int32_t* sel_len;         /* [B] */
    int32_t* accepted;        /* [B] */
    int32_t* committed;       /* [B, k_cap+1] */
    int32_t* n_commit;        /* [B] */
    int32_t* status;          /* [B] */
} hvd_host_step_args;

HVD_API hvd_status hvd_step_host(hvd_ctx* ctx, const hvd_host_step_args* args, void* stream);

/*
 * Verification with the vocabulary sharded over several ranks (a vocabulary-parallel output layer:
 * every rank holds, for all rows, the logits of its own V_shard consecutive vocabulary entries
 * starting at v_offset).  The argmax of Sec. 3.1's Verify splits into a per-shard part and a
 * reduction:
 *   hvd_verify_keys   streams this rank's shard (rows of V_shard values, same row layout and the same
 *                     needed-row rule as hvd_verify_commit: rows beyond sel_len are not read) and
 *                     writes one key per row, keys int64 [total_rows] (DEVICE output): larger key =
 *                     larger logit, and among equal logits the lower GLOBAL index; a row that was
 *                     not read gets the smallest int64.  Nothing else is written.
 *   (caller)          element-wise MAX of the keys over the ranks (e.g. an all-reduce with MAX on
 *                     int64: 8 bytes per row cross the links instead of the logits).
 *   hvd_commit_keys   hvd_verify_commit's accepted length, commit, append and state update, with the
 *                     row maxima taken from the reduced keys; V is the whole vocabulary size.  Every
 *                     rank that holds the request's history runs it and gets identical results.
 * Together the two calls give exactly hvd_verify_commit's outputs on the concatenated logits.
 * hvd_verify_keys uses context scratch: one call at a time per context.
 */
HVD_API hvd_status hvd_verify_keys(hvd_ctx* ctx, int32_t B, const void* logits, hvd_dtype dtype, int64_t V_shard,
                                   int64_t v_offset, const int64_t* row_off, int32_t k_uniform, int64_t total_rows,
                                   const int32_t* sel_len, const int32_t* hist_len, const int32_t* hist_cap,
                                   int64_t* keys, void* stream);
HVD_API hvd_status hvd_commit_keys(hvd_ctx* ctx, int32_t B, const int64_t* keys, int64_t V, const int64_t* row_off,
                                   int32_t k_uniform, int64_t total_rows, const int32_t* sel_draft,
                                   const int32_t* sel_len, const int32_t* select, int32_t* hist,
                                   const int64_t* hist_off, const int32_t* hist_cap, int32_t* hist_len,
                                   hvd_req_state* state, int32_t* accepted, int32_t* committed, int32_t* n_commit,
                                   int32_t* target_tok, int32_t* status, void* stream);

/*
 * Greedy verification and commit without a context and without any allocation.  (The paper has
 * no counterpart: this is a packaging variant of hvd_verify_commit.)
 *
 * For callers that cannot allocate device memory where the decoding step runs: an engine whose
 * memory pool owns the whole device, a call made while a stream is being captured, a plugin that
 * may only touch the tensors it is handed.  Arguments, layouts and results are those of
 * hvd_verify_commit, with k_cap (row length of sel_draft, committed has k_cap+1) passed directly.
 * The kernels' scratch memory is a static device array inside the library (about 129 KB, held by
 * every GPU that loads the library until the process exits), so:
 *   - B <= HVD_NOALLOC_MAX_BATCH and total_rows <= HVD_NOALLOC_MAX_ROWS; larger calls are
 *     rejected with HVD_ERR_INVALID_ARG (hvd_noalloc_last_error() says which limit);
 *   - all calls on a device share the array: two calls that overlap on the GPU (different
 *     streams, or threads launching at once) race and give wrong results; serialise them;
 *   - the array keeps the previous call's contents; each call first clears, on `stream`, the part
 *     it will read;
 *   - the first call on each device looks up the array's device address and the launch shape
 *     (queries only); make that first call outside of any stream capture.
 * It calls no cudaMalloc, cudaFree or allocating library routine.
 */
enum { HVD_NOALLOC_MAX_ROWS = 16384, HVD_NOALLOC_MAX_BATCH = 2048 };
HVD_API hvd_status hvd_verify_commit_noalloc(int32_t B, int32_t k_cap, const void* logits, hvd_dtype dtype,
                                             int64_t V, const int64_t* row_off, int32_t k_uniform,
                                             int64_t total_rows, const int32_t* sel_draft,
                                             const int32_t* sel_len, const int32_t* select, int32_t* hist,
                                             const int64_t* hist_off, const int32_t* hist_cap,
                                             int32_t* hist_len, hvd_req_state* state, int32_t* accepted,
                                             int32_t* committed, int32_t* n_commit, int32_t* target_tok,
                                             int32_t* status, void* stream);
/* text of the last error of hvd_verify_commit_noalloc on the calling thread ("" if none) */
HVD_API const char* hvd_noalloc_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* HVD_H */
