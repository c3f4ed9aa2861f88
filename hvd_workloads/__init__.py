"""Seeded synthetic inputs for the per-step path of Hybrid Verified Decoding.

This module only DRAWS inputs: token histories with repeated spans, decode
state, predictor weights, model-drafter tokens, logits noise and the planted
agreement between logits and a given draft.  It contains none of the method's
arithmetic (no suffix search, no scoring, no argmax): where an input depends on
an earlier step's result (the selected draft that the logits agree with, the
scores a threshold is calibrated on) that result is passed in by the caller.

The paper evaluates on public datasets with real models; these inputs stand in
for them and take only their structure from the paper's description: repeated
tool-call / edit spans with re-randomised arguments, long contexts, accepted
lengths of a few tokens on average (Sec. 4, App. C aggregate tables).
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass
from typing import Optional, Tuple, Union

import numpy as np

BASE_SEED = 260601019 * 10**4
# stream ids
S_TEMPLATES, S_HIST, S_TAIL, S_STATE, S_WEIGHTS, S_MODEL, S_AGREE, S_LOGITS, S_PLANT, S_TREE, S_CORPUS = range(11)

GUARD_WORDS = 64          # canary words either side of every history slab
GUARD_VALUE = -1515870811  # 0xA5A5A5A5 as int32
FREE_VALUE = -7            # fills the free tail of a slab (beyond hist_len)
PLANT_VALUE = 32.0         # planted maximum; noise is clipped to +-CLIP < PLANT_VALUE
CLIP = 30.0

STATE_DTYPE = np.dtype([("sel_bits", "<u4"), ("pad", "<u4"), ("acc_ring", "<u8")])


def stream_seed(config_index: int, stream_id: int, extra: int = 0) -> int:
    return BASE_SEED + 100 * config_index + stream_id + 1000003 * extra


def _rng(config_index: int, stream_id: int, extra: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(stream_seed(config_index, stream_id, extra)))


IntOrRange = Union[int, Tuple[int, int]]


@dataclass(frozen=True)
class Workload:
    name: str
    index: int                      # seeds derive from it
    B: int
    n: IntOrRange                   # history length, or (lo, hi) log-uniform
    V: int
    K: IntOrRange                   # draft cap, or (lo, hi) uniform per request
    k_cap: int
    n_templates: int
    template_len: IntOrRange        # fixed, or (lo, hi) log-uniform
    rep: Union[float, Tuple[float, float]]   # template mass fraction (or per-request uniform range)
    mutation: float                 # per-token mutation probability of a template copy
    zipf: bool                      # template popularity ~ 1/(i+1) instead of uniform
    json_like: bool                 # alternate fixed structural runs and re-randomised argument fields
    q_tail: Optional[float]         # fraction of requests whose tail re-enters an earlier span (None: = rep_b)
    tail_T: Tuple[int, int]
    dtype: str                      # "f32" | "bf16"
    sigma: float
    agree: Tuple                    # ("geom", p) | ("uniform",) | ("geom_per_req", lo, hi)
    tau: float
    b2: float
    calibrate_cache_frac: Optional[float] = None   # tau := score quantile so this fraction selects cache
    hidden: int = 32
    hidden_layers: int = 1          # 2: the paper's predictor shape (two hidden layers)
    min_match: int = 2
    l_max: int = 64
    filler_run: Tuple[int, int] = (16, 256)

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)

    @property
    def elt(self) -> int:
        return 4 if self.dtype == "f32" else 2


CONFIGS = {
    "C1": Workload("C1", 0, B=4, n=2048, V=32000, K=8, k_cap=8, n_templates=16, template_len=64,
                   rep=1.0, mutation=0.10, zipf=False, json_like=False, q_tail=0.5, tail_T=(2, 80),
                   dtype="f32", sigma=1.0, agree=("geom", 0.3), tau=2.0, b2=2.0),
    "C2": Workload("C2", 1, B=64, n=16384, V=128256, K=16, k_cap=16, n_templates=256, template_len=128,
                   rep=0.40, mutation=0.05, zipf=True, json_like=False, q_tail=1.0, tail_T=(2, 80),
                   dtype="bf16", sigma=2.0, agree=("geom", 0.25), tau=6.0, b2=6.0,
                   calibrate_cache_frac=0.5),
    "C3": Workload("C3", 2, B=256, n=32768, V=151936, K=32, k_cap=32, n_templates=128,
                   template_len=(32, 512), rep=0.70, mutation=0.0, zipf=False, json_like=True,
                   q_tail=0.6, tail_T=(2, 80), dtype="bf16", sigma=1.0, agree=("geom", 0.15),
                   tau=6.0, b2=6.0, calibrate_cache_frac=0.35),
    "C4": Workload("C4", 3, B=32, n=131072, V=128256, K=64, k_cap=64, n_templates=64, template_len=1024,
                   rep=0.85, mutation=0.02, zipf=False, json_like=False, q_tail=0.75, tail_T=(2, 96),
                   dtype="bf16", sigma=2.0, agree=("uniform",), tau=6.0, b2=6.0, calibrate_cache_frac=0.5),
    "C5": Workload("C5", 4, B=512, n=(512, 65536), V=128256, K=(4, 32), k_cap=32, n_templates=256,
                   template_len=128, rep=(0.0, 0.9), mutation=0.05, zipf=True, json_like=False,
                   q_tail=None, tail_T=(2, 80), dtype="bf16", sigma=2.0,
                   agree=("geom_per_req", 0.05, 0.5), tau=6.0, b2=6.0, calibrate_cache_frac=0.25),
}


@dataclass
class Requests:
    """Host-side request batch.  `hist` is one flat int32 array holding every slab and its guards."""
    hist: np.ndarray        # int32 [total]
    hist_off: np.ndarray    # int64 [B]   first token of slab b
    hist_cap: np.ndarray    # int32 [B]   slab capacity in tokens
    hist_len: np.ndarray    # int32 [B]
    K: np.ndarray           # int32 [B]
    prompt_len: np.ndarray  # int32 [B]
    state: np.ndarray       # STATE_DTYPE [B]
    model_draft: np.ndarray  # int32 [B, k_cap]
    model_len: np.ndarray   # int32 [B]
    row_off: np.ndarray     # int64 [B+1]  logits row blocks of K_b+1 rows
    guard_mask: np.ndarray  # bool [total]  True on canary words

    @property
    def B(self) -> int:
        return len(self.hist_len)

    def copy(self) -> "Requests":
        return Requests(**{f.name: getattr(self, f.name).copy() for f in dataclasses.fields(self)})

    def slab(self, b: int) -> np.ndarray:
        o = int(self.hist_off[b])
        return self.hist[o:o + int(self.hist_cap[b])]

    def history(self, b: int) -> np.ndarray:
        o = int(self.hist_off[b])
        return self.hist[o:o + int(self.hist_len[b])]


def _draw_int(rng, spec: IntOrRange, size=None, log=False):
    if isinstance(spec, tuple):
        lo, hi = spec
        if log:
            return np.floor(np.exp(rng.uniform(math.log(lo), math.log(hi), size))).astype(np.int64)
        return rng.integers(lo, hi + 1, size)
    return np.full(size, spec, dtype=np.int64) if size is not None else spec


def make_templates(w: Workload):
    """Returns a list of (tokens int32[len], arg_mask bool[len]); arg positions are redrawn per copy."""
    rng = _rng(w.index, S_TEMPLATES)
    lens = _draw_int(rng, w.template_len, w.n_templates, log=True)
    out = []
    struct_vocab = min(1024, w.V)
    for L in lens:
        L = int(L)
        if not w.json_like:
            out.append((rng.integers(0, w.V, L).astype(np.int32), np.zeros(L, bool)))
            continue
        toks = np.empty(L, np.int32)
        mask = np.zeros(L, bool)
        p = 0
        fixed = True
        while p < L:
            run = int(rng.integers(4, 25)) if fixed else int(rng.integers(1, 9))
            run = min(run, L - p)
            if fixed:
                toks[p:p + run] = rng.integers(0, struct_vocab, run)
            else:
                toks[p:p + run] = 0
                mask[p:p + run] = True
            p += run
            fixed = not fixed
        out.append((toks, mask))
    return out


def _template_probs(w: Workload) -> np.ndarray:
    if w.zipf:
        p = 1.0 / (np.arange(w.n_templates) + 1.0)
    else:
        p = np.ones(w.n_templates)
    return p / p.sum()


def _one_history(w: Workload, rng, templates, tprobs, n: int, rep: float):
    """Token array of length n and a mask of positions that came from template copies."""
    mean_t = float(sum(len(t[0]) * p for t, p in zip(templates, tprobs)))
    mean_f = 0.5 * (w.filler_run[0] + w.filler_run[1])
    if rep >= 1.0:
        q = 1.0
    elif rep <= 0.0:
        q = 0.0
    else:
        q = rep * mean_f / (mean_t * (1.0 - rep) + rep * mean_f)
    pieces, masks, total = [], [], 0
    # random phase: start somewhere inside the first piece
    first = True
    while total < n:
        if rng.random() < q:
            toks, amask = templates[int(rng.choice(len(templates), p=tprobs))]
            piece = toks.copy()
            if amask.any():
                piece[amask] = rng.integers(0, w.V, int(amask.sum()))
            if w.mutation > 0.0:
                mut = rng.random(len(piece)) < w.mutation
                if mut.any():
                    piece[mut] = rng.integers(0, w.V, int(mut.sum()))
            m = np.ones(len(piece), bool)
        else:
            run = int(rng.integers(w.filler_run[0], w.filler_run[1] + 1))
            piece = rng.integers(0, w.V, run).astype(np.int32)
            m = np.zeros(run, bool)
        if first:
            cut = int(rng.integers(0, len(piece)))
            piece, m = piece[cut:], m[cut:]
            first = False
        pieces.append(piece)
        masks.append(m)
        total += len(piece)
    h = np.concatenate(pieces)[:n].astype(np.int32)
    tm = np.concatenate(masks)[:n]
    return h, tm


def make_requests(w: Workload) -> Requests:
    templates = make_templates(w)
    tprobs = _template_probs(w)
    r_hist = _rng(w.index, S_HIST)
    r_tail = _rng(w.index, S_TAIL)
    r_state = _rng(w.index, S_STATE)
    r_model = _rng(w.index, S_MODEL)
    B = w.B
    n_all = np.asarray(_draw_int(r_hist, w.n, B, log=True), dtype=np.int64)
    K_all = np.asarray(_draw_int(r_hist, w.K, B), dtype=np.int64)
    K_all = np.minimum(K_all, w.k_cap)
    if isinstance(w.rep, tuple):
        rep_all = r_hist.uniform(w.rep[0], w.rep[1], B)
    else:
        rep_all = np.full(B, float(w.rep))
    hists = []
    for b in range(B):
        n = int(n_all[b])
        h, tm = _one_history(w, r_hist, templates, tprobs, n, float(rep_all[b]))
        q_tail = float(rep_all[b]) if w.q_tail is None else w.q_tail
        if r_tail.random() < q_tail:
            T = int(r_tail.integers(w.tail_T[0], w.tail_T[1] + 1))
            K = int(K_all[b])
            lo, hi = T + 1, n - T - K
            if hi > lo:
                cand = np.nonzero(tm[lo:hi])[0]
                e0 = lo + (int(cand[r_tail.integers(0, len(cand))]) if len(cand) else
                           int(r_tail.integers(0, hi - lo)))
                h[n - T:n] = h[e0 - T:e0]
        hists.append(h)
    cap = (n_all + 4 * (K_all + 1)).astype(np.int64)
    u = r_state.uniform(0.25, 0.9, B)
    prompt_len = np.floor(n_all * u).astype(np.int32)
    state = np.zeros(B, STATE_DTYPE)
    state["sel_bits"] = r_state.integers(0, 256, B).astype(np.uint32)
    ring = np.zeros(B, np.uint64)
    for j in range(8):
        ring |= (r_state.integers(0, K_all + 1).astype(np.uint64) << np.uint64(8 * j))
    state["acc_ring"] = ring
    model_draft = np.full((B, w.k_cap), -1, np.int32)
    for b in range(B):
        model_draft[b, :int(K_all[b])] = r_model.integers(0, w.V, int(K_all[b]))
    return pack_requests(hists, K_all, cap, prompt_len, state, model_draft, K_all.astype(np.int32))


def make_corpus(w: Workload, n_traces: int = 16, trace_len: IntOrRange = (1024, 8192), rep: float = 0.6,
                separator: int = -1) -> np.ndarray:
    """Shared warm-up corpus: `n_traces` recorded traces drawn from the workload's own template family
    (so that requests of the workload find some of their suffixes in it), joined by a negative
    separator.  Stands in for the warm-up prompts of the paper's datasets."""
    templates = make_templates(w)
    tprobs = _template_probs(w)
    rng = _rng(w.index, S_CORPUS)
    parts = []
    for t in range(n_traces):
        n = int(_draw_int(rng, trace_len, log=True))
        h, _ = _one_history(w, rng, templates, tprobs, n, rep)
        if t:
            parts.append(np.array([separator], np.int32))
        parts.append(h)
    return np.concatenate(parts).astype(np.int32) if parts else np.zeros(0, np.int32)


def pack_requests(hists, K, cap, prompt_len, state, model_draft, model_len, hist_len=None,
                  misalign=None) -> Requests:
    """Lays token lists out as guarded slabs: [64 canary words][slab, start aligned to 128 bytes]...
    `hist_len` may override the true lengths (to build invalid requests); `misalign[b]` shifts slab
    b by that many words off the 128-byte boundary."""
    B = len(hists)
    K = np.asarray(K, np.int64)
    cap = np.asarray(cap, np.int64)
    off = np.empty(B, np.int64)
    p = 0
    for b in range(B):
        p += GUARD_WORDS
        p = (p + 31) // 32 * 32
        if misalign is not None:
            p += int(misalign[b])
        off[b] = p
        p += int(cap[b])
    p += GUARD_WORDS
    total = (p + 31) // 32 * 32
    hist = np.full(total, GUARD_VALUE, np.int32)
    guard = np.ones(total, bool)
    for b in range(B):
        o, c, n = int(off[b]), int(cap[b]), len(hists[b])
        hist[o:o + c] = FREE_VALUE
        hist[o:o + n] = hists[b]
        guard[o:o + c] = False
    row_off = np.zeros(B + 1, np.int64)
    row_off[1:] = np.cumsum(K + 1)
    n_all = np.asarray([len(h) for h in hists], np.int32) if hist_len is None else np.asarray(hist_len, np.int32)
    return Requests(hist, off, cap.astype(np.int32), n_all, K.astype(np.int32),
                    np.asarray(prompt_len, np.int32), np.ascontiguousarray(state, STATE_DTYPE),
                    np.ascontiguousarray(model_draft, np.int32), np.asarray(model_len, np.int32),
                    row_off, guard)


def subset_requests(rq: Requests, lo: int, hi: int) -> Requests:
    """Requests [lo, hi) of a batch.  The flat history array is shared (offsets stay valid); logits
    row offsets are rebased to the first kept row, so pass logits[row_off[lo]:row_off[hi]] along."""
    keep = slice(lo, hi)
    return Requests(rq.hist, rq.hist_off[keep].copy(), rq.hist_cap[keep].copy(), rq.hist_len[keep].copy(),
                    rq.K[keep].copy(), rq.prompt_len[keep].copy(), rq.state[keep].copy(),
                    rq.model_draft[keep].copy(), rq.model_len[keep].copy(),
                    rq.row_off[lo:hi + 1] - rq.row_off[lo], rq.guard_mask)


def make_predictor(w: Workload):
    """W1 [H,8], b1 [H], W2 [H] ~ N(0, 0.1^2) fp32 drawn in that order; b2 and tau from the config."""
    rng = _rng(w.index, S_WEIGHTS)
    H = w.hidden
    W1 = rng.normal(0.0, 0.1, (H, 8)).astype(np.float32)
    b1 = rng.normal(0.0, 0.1, H).astype(np.float32)
    W2 = rng.normal(0.0, 0.1, H).astype(np.float32)
    return W1, b1, W2, float(np.float32(w.b2)), float(np.float32(w.tau))


def make_second_layer(w: Workload):
    """Wh [H,H], bh [H] ~ N(0, 0.1^2) fp32 of the second hidden layer (drawn after W1, b1, W2 from the
    same stream, so the one-layer weights do not change)."""
    rng = _rng(w.index, S_WEIGHTS)
    H = w.hidden
    rng.normal(0.0, 0.1, (H, 8)); rng.normal(0.0, 0.1, H); rng.normal(0.0, 0.1, H)
    Wh = rng.normal(0.0, 0.1, (H, H)).astype(np.float32)
    bh = rng.normal(0.0, 0.1, H).astype(np.float32)
    return Wh, bh


def calibrate_tau(scores: np.ndarray, eligible: np.ndarray, frac: float) -> float:
    """Threshold halfway between two neighbouring scores so that `frac` of ALL requests (taken from
    the eligible ones, highest scores first) reach it.  Input generation only: the scores come from
    whoever ran the scoring step."""
    s = np.sort(np.asarray(scores, np.float64)[np.asarray(eligible, bool)])[::-1]
    k = int(round(frac * len(scores)))
    if len(s) == 0 or k <= 0:
        return float("inf")
    if k >= len(s):
        return float(np.float32(s[-1] - 1.0))
    return float(np.float32(0.5 * (s[k - 1] + s[k])))


def make_agreement(w: Workload, sel_len: np.ndarray) -> np.ndarray:
    """Planted accepted length A_b in [0, sel_len_b].  'geom' uses p as the per-token stop
    probability: P(A = a) = (1-p)^a p, clipped to the draft length."""
    rng = _rng(w.index, S_AGREE)
    B = len(sel_len)
    kind = w.agree[0]
    if kind == "uniform":
        A = rng.integers(0, w.k_cap + 1, B)
    else:
        if kind == "geom":
            p = np.full(B, w.agree[1])
        else:
            p = rng.uniform(w.agree[1], w.agree[2], B)
        A = rng.geometric(p) - 1
    return np.minimum(A, np.asarray(sel_len)).astype(np.int32)


def make_logits(w: Workload, total_rows: int, device="cpu", salt: int = 0):
    """[total_rows, V] logits ~ N(0, sigma^2), clipped to +-CLIP, in the workload's dtype, drawn with
    a seeded torch generator on `device` (the stream differs between cpu and cuda; the consumer on
    the other side always gets a copy of this very tensor)."""
    import torch
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(stream_seed(w.index, S_LOGITS, salt))
    dt = torch.float32 if w.dtype == "f32" else torch.bfloat16
    out = torch.empty((total_rows, w.V), dtype=dt, device=dev)
    step = max(1, (1 << 26) // w.V)
    for r in range(0, total_rows, step):
        blk = torch.randn((min(step, total_rows - r), w.V), generator=g, device=dev, dtype=torch.float32)
        out[r:r + blk.shape[0]] = blk.mul_(w.sigma).clamp_(-CLIP, CLIP).to(dt)
    return out


def plant_agreement(w: Workload, logits, row_off: np.ndarray, sel_draft: np.ndarray,
                    sel_len: np.ndarray, A: np.ndarray, tie_frac: float = 0.10,
                    trap_frac: float = 0.25, salt: int = 0) -> np.ndarray:
    """Overwrite single logits (a torch tensor [rows, V], any device) so that the row maxima agree
    with `sel_draft` for exactly the first A_b rows of request b:
      rows i < A_b        : PLANT_VALUE at column sel_draft[b, i]  (strict maximum)
      row  i = A_b < m_b  : PLANT_VALUE at a different column      (forces the rejection)
      rows i > A_b        : with probability trap_frac the draft token is planted again (a row that
                            would agree, after the rejection point: must not be counted)
    and, on a fraction tie_frac of requests, one agreeing row gets a SECOND PLANT_VALUE at another
    column (an exact tie at the maximum, so the lowest-index rule decides).  Returns a bool [B] mask
    of the requests that were planted strictly (no tie row), on which accepted == A_b must hold."""
    import torch
    rng = _rng(w.index, S_PLANT, salt)
    rows, cols = [], []
    B = len(sel_len)
    strict = np.ones(B, bool)
    for b in range(B):
        m, a, r0 = int(sel_len[b]), int(A[b]), int(row_off[b])
        d = sel_draft[b]
        for i in range(a):
            rows.append(r0 + i); cols.append(int(d[i]))
        if a < m:
            rows.append(r0 + a); cols.append((int(d[a]) + 1 + int(rng.integers(0, w.V - 1))) % w.V
                                             if w.V > 1 else 0)
            for i in range(a + 1, m):
                if rng.random() < trap_frac:
                    rows.append(r0 + i); cols.append(int(d[i]))
        if a > 0 and w.V > 1 and rng.random() < tie_frac:
            i = int(rng.integers(0, a))
            other = (int(d[i]) + 1 + int(rng.integers(0, w.V - 1))) % w.V
            rows.append(r0 + i); cols.append(other)
            strict[b] = False
    if rows:
        ri = torch.as_tensor(np.asarray(rows, np.int64), device=logits.device)
        ci = torch.as_tensor(np.asarray(cols, np.int64), device=logits.device)
        logits[ri, ci] = PLANT_VALUE
    return strict


def logits_to_numpy(logits) -> np.ndarray:
    """Host copy for the CPU side: float32 array, or uint16 bit patterns for bfloat16."""
    import torch
    t = logits.detach().to("cpu").contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def make_tree_drafts(w: Workload, K: np.ndarray, max_nodes: int = 32, max_depth: int = 8, top_k: int = 4):
    """Model-drafter token trees in the shape the paper's drafter uses (App. A: 32 draft tokens, depth 8,
    top-k 4): per request up to min(max_nodes, K_b) nodes; node i hangs under a uniformly drawn earlier
    node (or under the prefix, parent -1) that is shallower than max_depth and has fewer than top_k
    children; sibling tokens are distinct.  Returns (tokens [B,k_cap], parent [B,k_cap], n_nodes [B])."""
    rng = _rng(w.index, S_TREE)
    B = len(K)
    tok = np.full((B, w.k_cap), -1, np.int32)
    par = np.full((B, w.k_cap), -2, np.int32)
    cnt = np.zeros(B, np.int32)
    for b in range(B):
        m = int(min(max_nodes, K[b], w.k_cap))
        depth, kids = {-1: 0}, {-1: []}
        for i in range(m):
            open_nodes = [p for p in depth if depth[p] < max_depth and len(kids[p]) < top_k]
            p = open_nodes[int(rng.integers(0, len(open_nodes)))]
            t = int(rng.integers(0, w.V))
            while t in [int(tok[b, c]) for c in kids[p]] and w.V > top_k:
                t = int(rng.integers(0, w.V))
            tok[b, i], par[b, i] = t, p
            kids[p].append(i); kids[i] = []; depth[i] = depth[p] + 1
        cnt[b] = m
    return tok, par, cnt


def plant_tree_agreement(w: Workload, logits, row_off: np.ndarray, tok: np.ndarray, par: np.ndarray,
                         n_nodes: np.ndarray, A: np.ndarray, salt: int = 0) -> np.ndarray:
    """Plants PLANT_VALUE so that greedy verification walks a random root path of (up to) A_b nodes and
    then stops: row(cur) gets its maximum at the chosen child's token; the row of the last node gets it
    at a token none of its children carries.  Returns the planted path lengths."""
    import torch
    rng = _rng(w.index, S_PLANT, 7919 + salt)
    rows, cols = [], []
    depth = np.zeros(len(n_nodes), np.int32)
    for b in range(len(n_nodes)):
        m, r0 = int(n_nodes[b]), int(row_off[b])
        cur, a = -1, 0
        while a < int(A[b]):
            kids = [c for c in range(m) if par[b, c] == cur]
            if not kids:
                break
            c = kids[int(rng.integers(0, len(kids)))]
            rows.append(r0 + cur + 1); cols.append(int(tok[b, c]))
            cur, a = c, a + 1
        kid_toks = {int(tok[b, c]) for c in range(m) if par[b, c] == cur}
        t = int(rng.integers(0, w.V))
        while t in kid_toks and w.V > len(kid_toks):
            t = int(rng.integers(0, w.V))
        rows.append(r0 + cur + 1); cols.append(t)
        depth[b] = a
    ri = torch.as_tensor(np.asarray(rows, np.int64), device=logits.device)
    ci = torch.as_tensor(np.asarray(cols, np.int64), device=logits.device)
    logits[ri, ci] = PLANT_VALUE
    return depth
