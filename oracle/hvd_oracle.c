/*
 * CPU oracle for the per-step path of Hybrid Verified Decoding.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition of what
 * the CUDA library must compute.  It shares no code, header, table or helper
 * with the CUDA path, and the CUDA path never calls it.  Only the tests, the
 * smoke check and the benchmark's CPU-baseline leg load it.
 *
 * Every function works on host pointers.  Requests are independent; the
 * batch entry points may spread requests over `nthreads` POSIX threads (a
 * plain parallel-for over b, nothing else is parallel).
 *
 * What is pinned by the CPU tests (brute-force enumeration on tiny inputs,
 * constructed cases, invariants, library special cases):
 *   - longest suffix match length, its count and the draft      (Sec. 3.2)
 *   - MLP score closed forms and the >= rule                    (Sec. 3.3, 3.4)
 *   - first-maximum argmax, accepted length, committed block    (Sec. 3.1, label eq. of Sec. 3.3)
 * Parity unpinned by the paper (the paper is silent; self-consistency only):
 *   - most-recent-occurrence tie-break among equally long matches,
 *   - the exact formulas of the eight payoff features (the paper names only
 *     feature groups, App. B table "Payoff predictor feature groups"),
 *   - the layout of the recent-history summary h,
 *   - the draft-structure features (shares of the draft's tokens per token
 *     class; the paper lists the classes, not the formula),
 *   - how warm-up traces and the own history share the cache (history before
 *     corpus at equal match length; separators between traces),
 *   - the frequency-weighted continuation and its score (the paper names the
 *     baseline's "frequency-derived cache score" without defining it; pinned
 *     to an independent restatement and hand-worked cases only).
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    uint32_t sel_bits; /* bit j = 1 if the cache draft was selected j steps ago */
    uint32_t pad;
    uint64_t acc_ring; /* byte j = accepted length j steps ago */
} oracle_req_state;

enum { ORACLE_REQ_OK = 0, ORACLE_REQ_CAPACITY = 1, ORACLE_REQ_BAD_LEN = 2 };
enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };
enum { ORACLE_N_FEATURES = 8 };

/* ------------------------------------------------------------------ */
/* parallel-for over requests                                          */
/* ------------------------------------------------------------------ */
typedef void (*req_fn)(int32_t b, void* arg);
typedef struct {
    req_fn fn;
    void* arg;
    int32_t B, tid, nthreads;
} worker_t;

static void* worker_main(void* p) {
    worker_t* w = (worker_t*)p;
    for (int32_t b = w->tid; b < w->B; b += w->nthreads) w->fn(b, w->arg);
    return NULL;
}

static void for_each_request(int32_t B, int32_t nthreads, req_fn fn, void* arg) {
    if (nthreads > B) nthreads = B;
    if (nthreads <= 1) {
        for (int32_t b = 0; b < B; ++b) fn(b, arg);
        return;
    }
    pthread_t* th = (pthread_t*)malloc(sizeof(pthread_t) * (size_t)nthreads);
    worker_t* ws = (worker_t*)malloc(sizeof(worker_t) * (size_t)nthreads);
    for (int32_t t = 0; t < nthreads; ++t) {
        ws[t].fn = fn; ws[t].arg = arg; ws[t].B = B; ws[t].tid = t; ws[t].nthreads = nthreads;
        pthread_create(&th[t], NULL, worker_main, &ws[t]);
    }
    for (int32_t t = 0; t < nthreads; ++t) pthread_join(th[t], NULL);
    free(ws);
    free(th);
}

/* ------------------------------------------------------------------ */
/* Step 1: cache draft = continuation of the longest suffix match      */
/* (Sec. 3.2; suffix-cache limits from the "Drafting configuration"    */
/* table: depth l_max, draft cap K, speculative factor and offset).    */
/* ------------------------------------------------------------------ */
void oracle_lookup_one(const int32_t* h, int32_t n, int32_t K, int32_t k_cap, int32_t l_max,
                       int32_t min_match, float spec_factor, float spec_offset,
                       int32_t* draft /*[k_cap]*/, int32_t* draft_len, int32_t* match_len,
                       int32_t* match_pos, int32_t* match_cnt) {
    int32_t best_L = 0, best_e = -1, cnt = 0;
    if (K < 0) K = 0;
    if (K > k_cap) K = k_cap;
    /* e = index of the first continuation token of a candidate occurrence.
       e = n would be the suffix matching itself and is left out. */
    for (int32_t e = 1; e <= n - 1; ++e) {
        int32_t l = 0;
        while (l < l_max && l < e && h[e - 1 - l] == h[n - 1 - l]) ++l;
        if (l > best_L) {
            best_L = l; best_e = e; cnt = 1;
        } else if (l == best_L && l > 0) {
            best_e = e; /* the latest occurrence wins among equals */
            ++cnt;
        }
    }
    for (int32_t j = 0; j < k_cap; ++j) draft[j] = -1;
    if (best_L < min_match || best_L == 0) {
        *match_len = 0; *match_pos = -1; *match_cnt = 0; *draft_len = 0;
        return;
    }
    int32_t cap = K;
    if (spec_factor > 0.0f) {
        float prod = spec_factor * (float)best_L; /* two roundings: multiply, then add */
        float lim = prod + spec_offset;
        cap = (int32_t)floorf(lim);
        if (cap < 0) cap = 0;
    }
    int32_t d = K;
    if (cap < d) d = cap;
    if (n - best_e < d) d = n - best_e;
    for (int32_t j = 0; j < d; ++j) draft[j] = h[best_e + j];
    *match_len = best_L; *match_pos = best_e; *match_cnt = cnt; *draft_len = d;
}

typedef struct {
    const int32_t* hist; const int64_t* hist_off; const int32_t* hist_cap; const int32_t* hist_len;
    const int32_t* K; int32_t k_cap, l_max, min_match; float spec_factor, spec_offset;
    int32_t *draft, *draft_len, *match_len, *match_pos, *match_cnt;
} lookup_args;

static void lookup_req(int32_t b, void* p) {
    lookup_args* a = (lookup_args*)p;
    int32_t n = a->hist_len[b];
    if (n < 0 || n > a->hist_cap[b]) n = 0; /* unusable length: behaves as an empty history */
    oracle_lookup_one(a->hist + a->hist_off[b], n, a->K[b], a->k_cap, a->l_max, a->min_match,
                      a->spec_factor, a->spec_offset, a->draft + (int64_t)b * a->k_cap,
                      a->draft_len + b, a->match_len + b, a->match_pos + b, a->match_cnt + b);
}

void oracle_lookup(int32_t B, const int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                   const int32_t* hist_len, const int32_t* K, int32_t k_cap, int32_t l_max,
                   int32_t min_match, float spec_factor, float spec_offset, int32_t* draft,
                   int32_t* draft_len, int32_t* match_len, int32_t* match_pos, int32_t* match_cnt,
                   int32_t nthreads) {
    lookup_args a = {hist, hist_off, hist_cap, hist_len, K, k_cap, l_max, min_match, spec_factor,
                     spec_offset, draft, draft_len, match_len, match_pos, match_cnt};
    for_each_request(B, nthreads, lookup_req, &a);
}

/* ------------------------------------------------------------------ */
/* Step 1 with a shared warm-up corpus (Algorithm 1, "Initialize C from */
/* cache-warmup traces and the input prompt"; App. C: warm-up prompts  */
/* of the same dataset initialise the suffix cache).  The cache of a   */
/* request is then [corpus, own history]: the corpus is one token      */
/* array shared by all requests; a negative entry separates two        */
/* traces, is never part of a match and ends a draft.  Candidates:     */
/*   history e in [1, n-1] as in oracle_lookup_one;                    */
/*   corpus  e in [1, m-1] with corpus[e] >= 0 (a continuation token    */
/*   exists), match length l <= min(l_max, e, n).                       */
/* The longest match wins; among equally long ones the history comes   */
/* before the corpus, and within a source the latest position.         */
/* match_src = 0 (history) or 1 (corpus); match_pos is the position in  */
/* that source; match_cnt counts both sources.                         */
/* ------------------------------------------------------------------ */
void oracle_lookup_corpus_one(const int32_t* h, int32_t n, const int32_t* corpus, int32_t m, int32_t K,
                              int32_t k_cap, int32_t l_max, int32_t min_match, float spec_factor,
                              float spec_offset, int32_t* draft /*[k_cap]*/, int32_t* draft_len,
                              int32_t* match_len, int32_t* match_pos, int32_t* match_src, int32_t* match_cnt) {
    int32_t best_L = 0, best_e = -1, best_src = 0, cnt = 0;
    if (K < 0) K = 0;
    if (K > k_cap) K = k_cap;
    /* corpus first, history second: with ">=" on ties the later candidate of this order wins */
    for (int32_t e = 1; e <= m - 1; ++e) {
        if (corpus[e] < 0) continue;
        int32_t l = 0;
        while (l < l_max && l < e && l < n && corpus[e - 1 - l] >= 0 && corpus[e - 1 - l] == h[n - 1 - l]) ++l;
        if (l == 0) continue;
        if (l > best_L) { best_L = l; best_e = e; best_src = 1; cnt = 1; }
        else if (l == best_L) { best_e = e; best_src = 1; ++cnt; }
    }
    for (int32_t e = 1; e <= n - 1; ++e) {
        int32_t l = 0;
        while (l < l_max && l < e && h[e - 1 - l] == h[n - 1 - l]) ++l;
        if (l == 0) continue;
        if (l > best_L) { best_L = l; best_e = e; best_src = 0; cnt = 1; }
        else if (l == best_L) { best_e = e; best_src = 0; ++cnt; }
    }
    for (int32_t j = 0; j < k_cap; ++j) draft[j] = -1;
    if (best_L < min_match || best_L == 0) {
        *match_len = 0; *match_pos = -1; *match_src = 0; *match_cnt = 0; *draft_len = 0;
        return;
    }
    int32_t d = K;
    if (spec_factor > 0.0f) {
        float prod = spec_factor * (float)best_L;
        float lim = prod + spec_offset;
        int32_t cap = (int32_t)floorf(lim);
        if (cap < 0) cap = 0;
        if (cap < d) d = cap;
    }
    if (best_src == 0) {
        if (n - best_e < d) d = n - best_e;
        for (int32_t j = 0; j < d; ++j) draft[j] = h[best_e + j];
    } else {
        if (m - best_e < d) d = m - best_e;
        int32_t j = 0;
        while (j < d && corpus[best_e + j] >= 0) { draft[j] = corpus[best_e + j]; ++j; } /* a separator ends the draft */
        d = j;
    }
    *match_len = best_L; *match_pos = best_e; *match_src = best_src; *match_cnt = cnt; *draft_len = d;
}

typedef struct {
    lookup_args l; const int32_t* corpus; int32_t m; int32_t* match_src;
} lookup_corpus_args;

static void lookup_corpus_req(int32_t b, void* p) {
    lookup_corpus_args* ca = (lookup_corpus_args*)p;
    lookup_args* a = &ca->l;
    int32_t n = a->hist_len[b];
    if (n < 0 || n > a->hist_cap[b]) n = 0;
    oracle_lookup_corpus_one(a->hist + a->hist_off[b], n, ca->corpus, ca->m, a->K[b], a->k_cap, a->l_max,
                             a->min_match, a->spec_factor, a->spec_offset, a->draft + (int64_t)b * a->k_cap,
                             a->draft_len + b, a->match_len + b, a->match_pos + b, ca->match_src + b,
                             a->match_cnt + b);
}

void oracle_lookup_corpus(int32_t B, const int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                          const int32_t* hist_len, const int32_t* K, const int32_t* corpus, int32_t m,
                          int32_t k_cap, int32_t l_max, int32_t min_match, float spec_factor, float spec_offset,
                          int32_t* draft, int32_t* draft_len, int32_t* match_len, int32_t* match_pos,
                          int32_t* match_src, int32_t* match_cnt, int32_t nthreads) {
    lookup_corpus_args ca = {{hist, hist_off, hist_cap, hist_len, K, k_cap, l_max, min_match, spec_factor,
                              spec_offset, draft, draft_len, match_len, match_pos, match_cnt}, corpus, m, match_src};
    for_each_request(B, nthreads, lookup_corpus_req, &ca);
}

/* ------------------------------------------------------------------ */
/* Frequency-weighted continuation and the suffix score (the cache     */
/* drafter of the paper follows SuffixDecoding, Sec. 3.2; its limits   */
/* are in App. A "Drafting configuration": speculative factor/offset,  */
/* minimum token probability 0.1; the Frequency-Based Hybrid baseline  */
/* of Sec. 4.2 thresholds "the frequency-derived cache score").        */
/* All occurrences of the longest matched suffix are merged: the walk  */
/* starts with the set of their end positions; at each step the next   */
/* token carried by most of the occurrences still alive is taken (ties:*/
/* the token whose latest alive occurrence is latest), with            */
/* probability count / alive; the walk stops when that probability is  */
/* below min_prob or the draft limit is reached; the score is the sum  */
/* of the probabilities.  With more than max_occ occurrences only the  */
/* latest one is followed (probability 1 per token).                   */
/* ------------------------------------------------------------------ */
void oracle_lookup_freq_one(const int32_t* h, int32_t n, int32_t K, int32_t k_cap, int32_t l_max,
                            int32_t min_match, float spec_factor, float spec_offset, float min_prob,
                            int32_t max_occ, int32_t* draft /*[k_cap]*/, int32_t* draft_len, float* score,
                            int32_t* match_len, int32_t* match_pos, int32_t* match_cnt) {
    int32_t plain[64];
    int32_t plain_len;
    oracle_lookup_one(h, n, K, k_cap, l_max, min_match, spec_factor, spec_offset, plain, &plain_len, match_len,
                      match_pos, match_cnt);
    for (int32_t j = 0; j < k_cap; ++j) draft[j] = -1;
    *draft_len = 0;
    *score = 0.0f;
    const int32_t L = *match_len;
    if (L == 0) return;
    if (K < 0) K = 0;
    if (K > k_cap) K = k_cap;
    int32_t limit = K;
    if (spec_factor > 0.0f) {
        float lim = spec_factor * (float)L;
        lim = lim + spec_offset;
        int32_t cap = (int32_t)floorf(lim);
        if (cap < 0) cap = 0;
        if (cap < limit) limit = cap;
    }
    if (*match_cnt > max_occ) { /* too many to merge: follow the latest occurrence only */
        for (int32_t j = 0; j < plain_len; ++j) { draft[j] = plain[j]; *score = *score + 1.0f; }
        *draft_len = plain_len;
        return;
    }
    /* the occurrences: every e whose (capped) match length equals L */
    int32_t* alive = (int32_t*)malloc(sizeof(int32_t) * (size_t)(*match_cnt > 0 ? *match_cnt : 1));
    int32_t na = 0;
    for (int32_t e = 1; e <= n - 1; ++e) {
        int32_t l = 0;
        while (l < l_max && l < e && h[e - 1 - l] == h[n - 1 - l]) ++l;
        if (l == L) alive[na++] = e;
    }
    int32_t d = 0;
    float sc = 0.0f;
    while (d < limit) {
        /* best next token among the alive occurrences */
        int32_t best_tok = -1, best_cnt = 0, best_last = -1;
        for (int32_t i = 0; i < na; ++i) {
            if (alive[i] + d >= n) continue;
            const int32_t x = h[alive[i] + d];
            int32_t c = 0, last = -1;
            for (int32_t j = 0; j < na; ++j)
                if (alive[j] + d < n && h[alive[j] + d] == x) { ++c; if (alive[j] > last) last = alive[j]; }
            if (c > best_cnt || (c == best_cnt && last > best_last)) { best_cnt = c; best_tok = x; best_last = last; }
        }
        if (best_cnt == 0) break;
        const float prob = (float)best_cnt / (float)na;
        if (prob < min_prob) break;
        draft[d] = best_tok;
        sc = sc + prob;
        int32_t nb = 0;
        for (int32_t i = 0; i < na; ++i)
            if (alive[i] + d < n && h[alive[i] + d] == best_tok) alive[nb++] = alive[i];
        na = nb;
        ++d;
    }
    free(alive);
    *draft_len = d;
    *score = sc;
}

typedef struct {
    lookup_args l; float min_prob; int32_t max_occ; float* score;
} lookup_freq_args;

static void lookup_freq_req(int32_t b, void* p) {
    lookup_freq_args* fa = (lookup_freq_args*)p;
    lookup_args* a = &fa->l;
    int32_t n = a->hist_len[b];
    if (n < 0 || n > a->hist_cap[b]) n = 0;
    oracle_lookup_freq_one(a->hist + a->hist_off[b], n, a->K[b], a->k_cap, a->l_max, a->min_match, a->spec_factor,
                           a->spec_offset, fa->min_prob, fa->max_occ, a->draft + (int64_t)b * a->k_cap,
                           a->draft_len + b, fa->score + b, a->match_len + b, a->match_pos + b, a->match_cnt + b);
}

void oracle_lookup_freq(int32_t B, const int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                        const int32_t* hist_len, const int32_t* K, int32_t k_cap, int32_t l_max,
                        int32_t min_match, float spec_factor, float spec_offset, float min_prob, int32_t max_occ,
                        int32_t* draft, int32_t* draft_len, float* score, int32_t* match_len,
                        int32_t* match_pos, int32_t* match_cnt, int32_t nthreads) {
    lookup_freq_args fa = {{hist, hist_off, hist_cap, hist_len, K, k_cap, l_max, min_match, spec_factor,
                            spec_offset, draft, draft_len, match_len, match_pos, match_cnt}, min_prob, max_occ,
                           score};
    for_each_request(B, nthreads, lookup_freq_req, &fa);
}

/* Selection of the frequency-based hybrid rule (Sec. 4.1): verify the cache draft when it is not
   empty and its frequency score reaches the threshold, the model draft otherwise. */
void oracle_freq_select(int32_t B, int32_t k_cap, const int32_t* draft, const int32_t* draft_len,
                        const float* score, float threshold, const int32_t* model_draft /*may be NULL*/,
                        const int32_t* model_len, int32_t* select, int32_t* sel_draft, int32_t* sel_len) {
    for (int32_t b = 0; b < B; ++b) {
        const int32_t s = (draft_len[b] > 0 && score[b] >= threshold) ? 1 : 0;
        const int32_t* src = NULL;
        int32_t m = 0;
        if (s) { src = draft + (int64_t)b * k_cap; m = draft_len[b]; }
        else if (model_draft) {
            src = model_draft + (int64_t)b * k_cap; m = model_len[b];
            if (m < 0) m = 0;
            if (m > k_cap) m = k_cap;
        }
        select[b] = s;
        sel_len[b] = m;
        for (int32_t j = 0; j < k_cap; ++j) sel_draft[(int64_t)b * k_cap + j] = j < m ? src[j] : -1;
    }
}

/* ------------------------------------------------------------------ */
/* Payoff labels by trace replay (Sec. 3.3 "training labels"; App. B   */
/* "Payoff Label Construction"): every position t of a recorded trace  */
/* is a decoding state with prefix x[0..t); its cache draft comes from */
/* the lookup above on that prefix; the label is the number of draft   */
/* tokens that agree with the trace's own continuation x[t..).         */
/* Outputs are indexed by t-1, t = 1..n.                               */
/* ------------------------------------------------------------------ */
typedef struct {
    const int32_t* x; int32_t n, K, k_cap, l_max, min_match; float spec_factor, spec_offset;
    int32_t *label, *draft_len, *match_len, *match_pos, *match_cnt;
} replay_args;

static void replay_state(int32_t j, void* p) {
    replay_args* a = (replay_args*)p;
    const int32_t t = j + 1;
    int32_t draft[64];
    oracle_lookup_one(a->x, t, a->K, a->k_cap, a->l_max, a->min_match, a->spec_factor, a->spec_offset, draft,
                      a->draft_len + j, a->match_len + j, a->match_pos + j, a->match_cnt + j);
    int32_t y = 0;
    while (y < a->draft_len[j] && t + y < a->n && draft[y] == a->x[t + y]) ++y;
    a->label[j] = y;
}

void oracle_replay_labels(const int32_t* x, int32_t n, int32_t K, int32_t k_cap, int32_t l_max, int32_t min_match,
                          float spec_factor, float spec_offset, int32_t* label, int32_t* draft_len,
                          int32_t* match_len, int32_t* match_pos, int32_t* match_cnt, int32_t nthreads) {
    replay_args a = {x, n, K, k_cap, l_max, min_match, spec_factor, spec_offset, label, draft_len, match_len,
                     match_pos, match_cnt};
    for_each_request(n, nthreads, replay_state, &a);
}

/* ------------------------------------------------------------------ */
/* Step 2: payoff features (Sec. 3.3; App. B feature-group table).     */
/* Every operation is an exact integer->float conversion or a single   */
/* correctly rounded IEEE operation.                                   */
/* ------------------------------------------------------------------ */
static int32_t bit_width_u32(uint32_t x) {
    int32_t w = 0;
    while (x) { ++w; x >>= 1; }
    return w;
}

void oracle_features_one(int32_t n, int32_t prompt_len, oracle_req_state st, int32_t draft_len,
                         int32_t match_len, int32_t match_pos, int32_t match_cnt, float* phi /*[8]*/) {
    if (n < 0) n = 0;
    if (prompt_len < 0) prompt_len = 0;
    if (match_cnt < 0) match_cnt = 0;
    /* cache match group */
    phi[0] = (float)match_len;
    phi[1] = (float)draft_len;
    phi[2] = (float)bit_width_u32((uint32_t)match_cnt);
    phi[3] = (match_pos < 0 || n == 0) ? 0.0f : (float)(n - match_pos) / (float)n;
    /* decode state group */
    phi[4] = (float)bit_width_u32((uint32_t)prompt_len);
    phi[5] = (n == 0) ? 0.0f : (float)(n - prompt_len) / (float)n;
    /* recent history group: last 8 steps */
    int32_t sel_count = 0;
    for (int j = 0; j < 8; ++j) sel_count += (int32_t)((st.sel_bits >> j) & 1u);
    phi[6] = (float)sel_count / 8.0f;
    int32_t acc_sum = 0;
    for (int j = 0; j < 8; ++j) acc_sum += (int32_t)((st.acc_ring >> (8 * j)) & 0xFFu);
    phi[7] = (float)acc_sum / 8.0f;
}

/* Extended feature vector (App. B feature-group table, all four groups): the eight features above,
   then the draft-structure group -- for each of five token classes (bit 0 whitespace, 1 punctuation,
   2 line break, 3 bracket, 4 delimiter-like; one byte of class bits per vocabulary entry, supplied
   by the caller from its tokenizer) the share of the cache draft's tokens that carry the class, one
   IEEE division count / draft_len (0 for an empty draft; tokens outside [0, V) carry no class) --
   and last the cache-match group's suffix score (the frequency score of oracle_lookup_freq; 0 when
   the caller has none). */
enum { ORACLE_N_FEATURES_EXT = 14, ORACLE_N_TOKEN_CLASSES = 5 };

void oracle_features_ext_one(int32_t n, int32_t prompt_len, oracle_req_state st, int32_t draft_len,
                             int32_t match_len, int32_t match_pos, int32_t match_cnt, const int32_t* draft,
                             const uint8_t* cls, int32_t cls_V, float suffix_score, float* phi /*[14]*/) {
    oracle_features_one(n, prompt_len, st, draft_len, match_len, match_pos, match_cnt, phi);
    for (int k = 0; k < ORACLE_N_TOKEN_CLASSES; ++k) {
        int32_t c = 0;
        for (int32_t j = 0; j < draft_len; ++j) {
            const int32_t t = draft[j];
            if (t >= 0 && t < cls_V && ((cls[t] >> k) & 1u)) ++c;
        }
        phi[ORACLE_N_FEATURES + k] = draft_len > 0 ? (float)c / (float)draft_len : 0.0f;
    }
    phi[ORACLE_N_FEATURES + ORACLE_N_TOKEN_CLASSES] = suffix_score;
}

/* ------------------------------------------------------------------ */
/* Step 3: payoff score y = g_theta(phi) and the rule y >= tau          */
/* (Sec. 3.3 predictor; Sec. 3.4 selection equation; Algorithm 1).     */
/* One hidden ReLU layer; fp32 with a fixed left-to-right fused         */
/* multiply-add chain, plus an fp64 evaluation of the same network.    */
/* ------------------------------------------------------------------ */
float oracle_mlp_f32(const float* phi, int32_t F, int32_t H, const float* W1 /*[H,F]*/,
                     const float* b1, const float* W2, float b2) {
    float y = b2;
    for (int32_t j = 0; j < H; ++j) {
        float acc = b1[j];
        for (int32_t i = 0; i < F; ++i) acc = fmaf(W1[(int64_t)j * F + i], phi[i], acc);
        float hid = acc > 0.0f ? acc : 0.0f;
        y = fmaf(W2[j], hid, y);
    }
    return y;
}

double oracle_mlp_f64(const float* phi, int32_t F, int32_t H, const float* W1, const float* b1,
                      const float* W2, float b2) {
    double y = (double)b2;
    for (int32_t j = 0; j < H; ++j) {
        double acc = (double)b1[j];
        for (int32_t i = 0; i < F; ++i) acc += (double)W1[(int64_t)j * F + i] * (double)phi[i];
        double hid = acc > 0.0 ? acc : 0.0;
        y += (double)W2[j] * hid;
    }
    return y;
}

/* The same predictor with a second hidden ReLU layer (the paper's trained predictor has two hidden
   layers of 256 units: App. B, table "Payoff predictor training configuration"):
   h1 = relu(W1 phi + b1), h2 = relu(Wh h1 + bh), y = b2 + W2 . h2; same left-to-right fmaf chains. */
float oracle_mlp2_f32(const float* phi, int32_t F, int32_t H, const float* W1 /*[H,F]*/, const float* b1,
                      const float* Wh /*[H,H]*/, const float* bh, const float* W2, float b2) {
    float h1[1024];
    for (int32_t j = 0; j < H; ++j) {
        float acc = b1[j];
        for (int32_t i = 0; i < F; ++i) acc = fmaf(W1[(int64_t)j * F + i], phi[i], acc);
        h1[j] = acc > 0.0f ? acc : 0.0f;
    }
    float y = b2;
    for (int32_t j = 0; j < H; ++j) {
        float acc = bh[j];
        for (int32_t i = 0; i < H; ++i) acc = fmaf(Wh[(int64_t)j * H + i], h1[i], acc);
        float hid = acc > 0.0f ? acc : 0.0f;
        y = fmaf(W2[j], hid, y);
    }
    return y;
}

double oracle_mlp2_f64(const float* phi, int32_t F, int32_t H, const float* W1, const float* b1,
                       const float* Wh, const float* bh, const float* W2, float b2) {
    double h1[1024];
    for (int32_t j = 0; j < H; ++j) {
        double acc = (double)b1[j];
        for (int32_t i = 0; i < F; ++i) acc += (double)W1[(int64_t)j * F + i] * (double)phi[i];
        h1[j] = acc > 0.0 ? acc : 0.0;
    }
    double y = (double)b2;
    for (int32_t j = 0; j < H; ++j) {
        double acc = (double)bh[j];
        for (int32_t i = 0; i < H; ++i) acc += (double)Wh[(int64_t)j * H + i] * h1[i];
        y += (double)W2[j] * (acc > 0.0 ? acc : 0.0);
    }
    return y;
}

typedef struct {
    const int32_t *hist_len, *prompt_len; const oracle_req_state* state; const int32_t* K;
    const int32_t *draft, *draft_len, *match_len, *match_pos, *match_cnt;
    const int32_t *model_draft, *model_len; int32_t k_cap, H;
    const float *W1, *b1, *W2; float b2, tau;
    float *features, *score; double* score64; int32_t *select, *sel_draft, *sel_len;
    const float *Wh, *bh; /* second hidden layer, NULL for the one-layer predictor */
    const uint8_t* cls; int32_t cls_V; const float* suffix; /* cls != NULL: the extended feature vector */
    const int32_t* match_src; /* extended only, may be NULL: 1 = the match lies in the shared corpus */
} score_args;

static void score_req(int32_t b, void* p) {
    score_args* a = (score_args*)p;
    float phi[ORACLE_N_FEATURES_EXT];
    int32_t kc = a->k_cap;
    int32_t K = a->K[b];
    if (K < 0) K = 0;
    if (K > kc) K = kc;
    int32_t d = a->draft_len[b];
    if (d < 0) d = 0;
    if (d > kc) d = kc;
    int32_t F = ORACLE_N_FEATURES;
    if (a->cls) {
        F = ORACLE_N_FEATURES_EXT;
        /* a match in the shared corpus is older than every history token: position 0 for the recency feature */
        const int32_t pos = (a->match_src && a->match_src[b] == 1) ? 0 : a->match_pos[b];
        oracle_features_ext_one(a->hist_len[b], a->prompt_len[b], a->state[b], d, a->match_len[b], pos,
                                a->match_cnt[b], a->draft + (int64_t)b * kc, a->cls, a->cls_V,
                                a->suffix ? a->suffix[b] : 0.0f, phi);
    } else {
        oracle_features_one(a->hist_len[b], a->prompt_len[b], a->state[b], d, a->match_len[b],
                            a->match_pos[b], a->match_cnt[b], phi);
    }
    if (a->features) memcpy(a->features + (int64_t)b * F, phi, sizeof(float) * (size_t)F);
    float y = a->Wh ? oracle_mlp2_f32(phi, F, a->H, a->W1, a->b1, a->Wh, a->bh, a->W2, a->b2)
                    : oracle_mlp_f32(phi, F, a->H, a->W1, a->b1, a->W2, a->b2);
    a->score[b] = y;
    if (a->score64)
        a->score64[b] = a->Wh ? oracle_mlp2_f64(phi, F, a->H, a->W1, a->b1, a->Wh, a->bh, a->W2, a->b2)
                              : oracle_mlp_f64(phi, F, a->H, a->W1, a->b1, a->W2, a->b2);
    /* cache draft is verified iff it exists and its predicted payoff reaches the threshold */
    int32_t sel = (d > 0 && y >= a->tau) ? 1 : 0;
    a->select[b] = sel;
    int32_t* out = a->sel_draft + (int64_t)b * kc;
    for (int32_t j = 0; j < kc; ++j) out[j] = -1;
    if (sel) {
        for (int32_t j = 0; j < d; ++j) out[j] = a->draft[(int64_t)b * kc + j];
        a->sel_len[b] = d;
    } else {
        int32_t m = 0;
        if (a->model_draft && a->model_len) {
            m = a->model_len[b];
            if (m < 0) m = 0;
            if (m > K) m = K;
            for (int32_t j = 0; j < m; ++j) out[j] = a->model_draft[(int64_t)b * kc + j];
        }
        a->sel_len[b] = m;
    }
}

void oracle_score_select(int32_t B, const int32_t* hist_len, const int32_t* prompt_len,
                         const oracle_req_state* state, const int32_t* K, const int32_t* draft,
                         const int32_t* draft_len, const int32_t* match_len, const int32_t* match_pos,
                         const int32_t* match_cnt, const int32_t* model_draft, const int32_t* model_len,
                         int32_t k_cap, int32_t H, const float* W1, const float* b1, const float* W2,
                         float b2, float tau, float* features, float* score, double* score64,
                         int32_t* select, int32_t* sel_draft, int32_t* sel_len, int32_t nthreads) {
    score_args a = {hist_len, prompt_len, state, K, draft, draft_len, match_len, match_pos, match_cnt,
                    model_draft, model_len, k_cap, H, W1, b1, W2, b2, tau, features, score, score64,
                    select, sel_draft, sel_len, NULL, NULL, NULL, 0, NULL, NULL};
    for_each_request(B, nthreads, score_req, &a);
}

void oracle_score_select2(int32_t B, const int32_t* hist_len, const int32_t* prompt_len,
                          const oracle_req_state* state, const int32_t* K, const int32_t* draft,
                          const int32_t* draft_len, const int32_t* match_len, const int32_t* match_pos,
                          const int32_t* match_cnt, const int32_t* model_draft, const int32_t* model_len,
                          int32_t k_cap, int32_t H, const float* W1, const float* b1, const float* Wh,
                          const float* bh, const float* W2, float b2, float tau, float* features, float* score,
                          double* score64, int32_t* select, int32_t* sel_draft, int32_t* sel_len,
                          int32_t nthreads) {
    score_args a = {hist_len, prompt_len, state, K, draft, draft_len, match_len, match_pos, match_cnt,
                    model_draft, model_len, k_cap, H, W1, b1, W2, b2, tau, features, score, score64,
                    select, sel_draft, sel_len, Wh, bh, NULL, 0, NULL, NULL};
    for_each_request(B, nthreads, score_req, &a);
}

/* The same step on the extended feature vector: W1 is [H, 14]; Wh / bh NULL for one hidden layer;
   features [B, 14]; suffix (float [B]) and match_src (int32 [B], from oracle_lookup_corpus) may be NULL. */
void oracle_score_select_ext(int32_t B, const int32_t* hist_len, const int32_t* prompt_len,
                             const oracle_req_state* state, const int32_t* K, const int32_t* draft,
                             const int32_t* draft_len, const int32_t* match_len, const int32_t* match_pos,
                             const int32_t* match_cnt, const int32_t* match_src, const float* suffix,
                             const uint8_t* cls, int32_t cls_V, const int32_t* model_draft, const int32_t* model_len, int32_t k_cap, int32_t H,
                             const float* W1, const float* b1, const float* Wh, const float* bh, const float* W2,
                             float b2, float tau, float* features, float* score, double* score64,
                             int32_t* select, int32_t* sel_draft, int32_t* sel_len, int32_t nthreads) {
    score_args a = {hist_len, prompt_len, state, K, draft, draft_len, match_len, match_pos, match_cnt,
                    model_draft, model_len, k_cap, H, W1, b1, W2, b2, tau, features, score, score64,
                    select, sel_draft, sel_len, Wh, bh, cls, cls_V, suffix, match_src};
    for_each_request(B, nthreads, score_req, &a);
}

/* ------------------------------------------------------------------ */
/* Step 4: greedy verification and commit (Sec. 3.1 Verify; Sec. 3.4;  */
/* Algorithm 1 verify/append/update lines; accepted length = the label */
/* equation of Sec. 3.3).                                              */
/* ------------------------------------------------------------------ */
static float widen_bf16(uint16_t u) {
    uint32_t bits = (uint32_t)u << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

/* index of the first maximum: scan ascending, replace only on strictly greater */
int32_t oracle_argmax_row(const void* row, int32_t dtype, int64_t V) {
    int64_t best = 0;
    if (dtype == ORACLE_BF16) {
        const uint16_t* r = (const uint16_t*)row;
        float bv = widen_bf16(r[0]);
        for (int64_t v = 1; v < V; ++v) {
            float x = widen_bf16(r[v]);
            if (x > bv) { bv = x; best = v; }
        }
    } else {
        const float* r = (const float*)row;
        float bv = r[0];
        for (int64_t v = 1; v < V; ++v) {
            if (r[v] > bv) { bv = r[v]; best = v; }
        }
    }
    return (int32_t)best;
}

typedef struct {
    const void* logits; int32_t dtype; int64_t V; const int64_t* row_off; int32_t k_uniform;
    const int32_t *sel_draft, *sel_len, *select; int32_t k_cap;
    int32_t* hist; const int64_t* hist_off; const int32_t* hist_cap; int32_t* hist_len;
    oracle_req_state* state;
    int32_t *accepted, *committed, *n_commit, *target_tok, *status;
} verify_args;

static void verify_req(int32_t b, void* p) {
    verify_args* a = (verify_args*)p;
    int32_t kc = a->k_cap;
    int64_t r0 = a->row_off ? a->row_off[b] : (int64_t)b * (a->k_uniform + 1);
    int64_t r1 = a->row_off ? a->row_off[b + 1] : r0 + (a->k_uniform + 1);
    int64_t rows = r1 - r0;
    size_t elt = a->dtype == ORACLE_BF16 ? 2 : 4;
    int32_t* z = a->committed + (int64_t)b * (kc + 1);
    for (int32_t j = 0; j <= kc; ++j) z[j] = -1;
    if (a->target_tok)
        for (int64_t i = 0; i < rows; ++i) a->target_tok[r0 + i] = -1;
    int32_t n = a->hist_len[b];
    if (n < 0 || n > a->hist_cap[b] || rows <= 0) {
        a->status[b] = ORACLE_REQ_BAD_LEN; a->accepted[b] = 0; a->n_commit[b] = 0;
        return;
    }
    int32_t m = a->sel_len[b];
    if (m < 0) m = 0;
    if (m > kc) m = kc;
    if (m > rows - 1) m = (int32_t)(rows - 1);
    int32_t t[65 + 1];
    for (int32_t i = 0; i <= m; ++i) {
        const char* row = (const char*)a->logits + (size_t)(r0 + i) * (size_t)a->V * elt;
        t[i] = oracle_argmax_row(row, a->dtype, a->V);
        if (a->target_tok) a->target_tok[r0 + i] = t[i];
    }
    const int32_t* d = a->sel_draft + (int64_t)b * kc;
    int32_t acc = 0;
    while (acc < m && d[acc] == t[acc]) ++acc;
    for (int32_t j = 0; j < acc; ++j) z[j] = d[j];
    z[acc] = t[acc]; /* the target's own token after the accepted prefix: always committed */
    int32_t room = a->hist_cap[b] - n;
    int32_t w = acc + 1;
    int32_t st = ORACLE_REQ_OK;
    if (w > room) { w = room; st = ORACLE_REQ_CAPACITY; }
    int32_t* h = a->hist + a->hist_off[b];
    for (int32_t j = 0; j < w; ++j) h[n + j] = z[j];
    a->hist_len[b] = n + w;
    a->n_commit[b] = w;
    a->accepted[b] = acc;
    a->status[b] = st;
    oracle_req_state s = a->state[b];
    s.sel_bits = (s.sel_bits << 1) | (uint32_t)(a->select[b] ? 1 : 0);
    s.acc_ring = (s.acc_ring << 8) | (uint64_t)(uint8_t)acc;
    a->state[b] = s;
}

void oracle_verify_commit(int32_t B, const void* logits, int32_t dtype, int64_t V,
                          const int64_t* row_off, int32_t k_uniform, const int32_t* sel_draft,
                          const int32_t* sel_len, const int32_t* select, int32_t k_cap, int32_t* hist,
                          const int64_t* hist_off, const int32_t* hist_cap, int32_t* hist_len,
                          oracle_req_state* state, int32_t* accepted, int32_t* committed,
                          int32_t* n_commit, int32_t* target_tok, int32_t* status, int32_t nthreads) {
    verify_args a = {logits, dtype, V, row_off, k_uniform, sel_draft, sel_len, select, k_cap, hist,
                     hist_off, hist_cap, hist_len, state, accepted, committed, n_commit, target_tok,
                     status};
    for_each_request(B, nthreads, verify_req, &a);
}

/* ------------------------------------------------------------------ */
/* Verification of a token TREE (the model drafter of the paper,       */
/* EAGLE3, proposes a tree: App. A "Drafting configuration": 32 draft  */
/* tokens, depth 8, top-k 4).  Node i has token d[i] and parent        */
/* par[i] in {-1, 0..i-1} (-1: it follows the prefix directly).  Row 0 */
/* of the request's logits is the target's output after the prefix,    */
/* row i+1 its output after node i.  Greedy verification (Sec. 3.1,    */
/* Sec. 3.4) walks down from the prefix: the target's token at the     */
/* current node is the argmax of that node's row; if a child carries   */
/* that token (the first such child) it is accepted and the walk goes  */
/* on there, else the walk stops and the target's token is committed   */
/* as the last token.  A chain (par[i] = i-1) gives exactly            */
/* oracle_verify_commit.                                               */
/* ------------------------------------------------------------------ */
typedef struct {
    verify_args v;
    const int32_t* parent;
} verify_tree_args;

static void verify_tree_req(int32_t b, void* p) {
    verify_tree_args* ta = (verify_tree_args*)p;
    verify_args* a = &ta->v;
    int32_t kc = a->k_cap;
    int64_t r0 = a->row_off ? a->row_off[b] : (int64_t)b * (a->k_uniform + 1);
    int64_t r1 = a->row_off ? a->row_off[b + 1] : r0 + (a->k_uniform + 1);
    int64_t rows = r1 - r0;
    size_t elt = a->dtype == ORACLE_BF16 ? 2 : 4;
    int32_t* z = a->committed + (int64_t)b * (kc + 1);
    for (int32_t j = 0; j <= kc; ++j) z[j] = -1;
    if (a->target_tok)
        for (int64_t i = 0; i < rows; ++i) a->target_tok[r0 + i] = -1;
    int32_t n = a->hist_len[b];
    if (n < 0 || n > a->hist_cap[b] || rows <= 0) {
        a->status[b] = ORACLE_REQ_BAD_LEN; a->accepted[b] = 0; a->n_commit[b] = 0;
        return;
    }
    int32_t m = a->sel_len[b];
    if (m < 0) m = 0;
    if (m > kc) m = kc;
    if (m > rows - 1) m = (int32_t)(rows - 1);
    int32_t t[65 + 1];
    for (int32_t i = 0; i <= m; ++i) {
        const char* row = (const char*)a->logits + (size_t)(r0 + i) * (size_t)a->V * elt;
        t[i] = oracle_argmax_row(row, a->dtype, a->V);
        if (a->target_tok) a->target_tok[r0 + i] = t[i];
    }
    const int32_t* d = a->sel_draft + (int64_t)b * kc;
    const int32_t* par = ta->parent + (int64_t)b * kc;
    int32_t acc = 0, cur = -1;
    for (;;) {
        int32_t want = t[cur + 1]; /* the target's token after the current node */
        int32_t next = -1;
        for (int32_t c = cur + 1; c < m; ++c)
            if (par[c] == cur && d[c] == want) { next = c; break; }
        if (next < 0) { z[acc] = want; break; }
        z[acc++] = d[next];
        cur = next;
    }
    int32_t room = a->hist_cap[b] - n;
    int32_t w = acc + 1;
    int32_t st = ORACLE_REQ_OK;
    if (w > room) { w = room; st = ORACLE_REQ_CAPACITY; }
    int32_t* h = a->hist + a->hist_off[b];
    for (int32_t j = 0; j < w; ++j) h[n + j] = z[j];
    a->hist_len[b] = n + w;
    a->n_commit[b] = w;
    a->accepted[b] = acc;
    a->status[b] = st;
    oracle_req_state s = a->state[b];
    s.sel_bits = (s.sel_bits << 1) | (uint32_t)(a->select[b] ? 1 : 0);
    s.acc_ring = (s.acc_ring << 8) | (uint64_t)(uint8_t)acc;
    a->state[b] = s;
}

void oracle_verify_commit_tree(int32_t B, const void* logits, int32_t dtype, int64_t V,
                               const int64_t* row_off, int32_t k_uniform, const int32_t* sel_draft,
                               const int32_t* sel_len, const int32_t* parent, const int32_t* select,
                               int32_t k_cap, int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                               int32_t* hist_len, oracle_req_state* state, int32_t* accepted,
                               int32_t* committed, int32_t* n_commit, int32_t* target_tok, int32_t* status,
                               int32_t nthreads) {
    verify_tree_args ta = {{logits, dtype, V, row_off, k_uniform, sel_draft, sel_len, select, k_cap, hist,
                            hist_off, hist_cap, hist_len, state, accepted, committed, n_commit, target_tok,
                            status}, parent};
    for_each_request(B, nthreads, verify_tree_req, &ta);
}
