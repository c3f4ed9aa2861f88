"""ctypes front end of the CPU oracle (test infrastructure only).

Loads ``libhvd_oracle.so`` built from ``hvd_oracle.c`` and exposes the three
steps on numpy arrays.  Nothing here is imported by the CUDA package; only the
tests, the smoke check and the benchmark's CPU-baseline leg use it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hvd_oracle.c")
_LIB = os.path.join(_HERE, "libhvd_oracle.so")

F32, BF16 = 0, 1
REQ_OK, REQ_CAPACITY, REQ_BAD_LEN = 0, 1, 2
N_FEATURES = 8

STATE_DTYPE = np.dtype([("sel_bits", "<u4"), ("pad", "<u4"), ("acc_ring", "<u8")])


def build(force: bool = False) -> str:
    """Compile the oracle with gcc; contraction off so every fp32 step rounds as written."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared", "-pthread",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_argmax_row.restype = C.c_int32
        _lib.oracle_mlp_f32.restype = C.c_float
        _lib.oracle_mlp_f64.restype = C.c_double
        _lib.oracle_mlp2_f32.restype = C.c_float
        _lib.oracle_mlp2_f64.restype = C.c_double
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


@dataclass
class LookupOut:
    draft: np.ndarray
    draft_len: np.ndarray
    match_len: np.ndarray
    match_pos: np.ndarray
    match_cnt: np.ndarray


def lookup(hist, hist_off, hist_cap, hist_len, K, *, k_cap, l_max=64, min_match=2,
           spec_factor=1.0, spec_offset=0.0, nthreads=1) -> LookupOut:
    B = len(hist_len)
    hist = _i32(hist); hist_len = _i32(hist_len); hist_cap = _i32(hist_cap); K = _i32(K)
    hist_off = np.ascontiguousarray(hist_off, dtype=np.int64)
    out = LookupOut(np.empty((B, k_cap), np.int32), np.empty(B, np.int32), np.empty(B, np.int32),
                    np.empty(B, np.int32), np.empty(B, np.int32))
    lib().oracle_lookup(C.c_int32(B), _p(hist), _p(hist_off), _p(hist_cap), _p(hist_len), _p(K),
                        C.c_int32(k_cap), C.c_int32(l_max), C.c_int32(min_match),
                        C.c_float(spec_factor), C.c_float(spec_offset), _p(out.draft),
                        _p(out.draft_len), _p(out.match_len), _p(out.match_pos), _p(out.match_cnt),
                        C.c_int32(nthreads))
    return out


@dataclass
class CorpusOut(LookupOut):
    match_src: np.ndarray = None


def lookup_corpus(hist, hist_off, hist_cap, hist_len, K, corpus, *, k_cap, l_max=64, min_match=2, spec_factor=1.0,
                  spec_offset=0.0, nthreads=1) -> CorpusOut:
    """Cache draft from [shared warm-up corpus, own history]; negative corpus entries separate traces."""
    B = len(hist_len)
    hist = _i32(hist); hist_len = _i32(hist_len); hist_cap = _i32(hist_cap); K = _i32(K); corpus = _i32(corpus)
    hist_off = np.ascontiguousarray(hist_off, dtype=np.int64)
    out = CorpusOut(np.empty((B, k_cap), np.int32), np.empty(B, np.int32), np.empty(B, np.int32),
                    np.empty(B, np.int32), np.empty(B, np.int32), np.empty(B, np.int32))
    lib().oracle_lookup_corpus(C.c_int32(B), _p(hist), _p(hist_off), _p(hist_cap), _p(hist_len), _p(K), _p(corpus),
                               C.c_int32(len(corpus)), C.c_int32(k_cap), C.c_int32(l_max), C.c_int32(min_match),
                               C.c_float(spec_factor), C.c_float(spec_offset), _p(out.draft), _p(out.draft_len),
                               _p(out.match_len), _p(out.match_pos), _p(out.match_src), _p(out.match_cnt),
                               C.c_int32(nthreads))
    return out


@dataclass
class FreqOut(LookupOut):
    score: np.ndarray = None


def lookup_freq(hist, hist_off, hist_cap, hist_len, K, *, k_cap, l_max=64, min_match=2, spec_factor=1.0,
                spec_offset=0.0, min_prob=0.1, max_occ=256, nthreads=1) -> FreqOut:
    """Frequency-weighted cache draft and its suffix score (merging all occurrences of the longest match)."""
    B = len(hist_len)
    hist = _i32(hist); hist_len = _i32(hist_len); hist_cap = _i32(hist_cap); K = _i32(K)
    hist_off = np.ascontiguousarray(hist_off, dtype=np.int64)
    out = FreqOut(np.empty((B, k_cap), np.int32), np.empty(B, np.int32), np.empty(B, np.int32),
                  np.empty(B, np.int32), np.empty(B, np.int32), np.empty(B, np.float32))
    lib().oracle_lookup_freq(C.c_int32(B), _p(hist), _p(hist_off), _p(hist_cap), _p(hist_len), _p(K),
                             C.c_int32(k_cap), C.c_int32(l_max), C.c_int32(min_match), C.c_float(spec_factor),
                             C.c_float(spec_offset), C.c_float(min_prob), C.c_int32(max_occ), _p(out.draft),
                             _p(out.draft_len), _p(out.score), _p(out.match_len), _p(out.match_pos),
                             _p(out.match_cnt), C.c_int32(nthreads))
    return out


def freq_select(out: FreqOut, threshold, model_draft=None, model_len=None):
    """The frequency-based hybrid rule on lookup_freq's result: (select, sel_draft, sel_len)."""
    B, k_cap = out.draft.shape
    select = np.empty(B, np.int32); sel_len = np.empty(B, np.int32); sel_draft = np.empty((B, k_cap), np.int32)
    md = None if model_draft is None else _i32(model_draft)
    ml = None if model_len is None else _i32(model_len)
    lib().oracle_freq_select(C.c_int32(B), C.c_int32(k_cap), _p(out.draft), _p(out.draft_len), _p(out.score),
                             C.c_float(threshold), None if md is None else _p(md), None if ml is None else _p(ml),
                             _p(select), _p(sel_draft), _p(sel_len))
    return select, sel_draft, sel_len


@dataclass
class ReplayOut:
    label: np.ndarray
    draft_len: np.ndarray
    match_len: np.ndarray
    match_pos: np.ndarray
    match_cnt: np.ndarray


def replay_labels(trace, K, *, k_cap=None, l_max=64, min_match=2, spec_factor=1.0, spec_offset=0.0,
                  nthreads=1) -> ReplayOut:
    """Labels y_t for every prefix length t = 1..n of one trace (arrays indexed by t-1)."""
    x = _i32(trace)
    n = len(x)
    k_cap = k_cap or max(K, 1)
    out = ReplayOut(*(np.empty(n, np.int32) for _ in range(5)))
    lib().oracle_replay_labels(_p(x), C.c_int32(n), C.c_int32(K), C.c_int32(k_cap), C.c_int32(l_max),
                               C.c_int32(min_match), C.c_float(spec_factor), C.c_float(spec_offset),
                               _p(out.label), _p(out.draft_len), _p(out.match_len), _p(out.match_pos),
                               _p(out.match_cnt), C.c_int32(nthreads))
    return out


@dataclass
class ScoreOut:
    features: np.ndarray
    score: np.ndarray
    score64: np.ndarray
    select: np.ndarray
    sel_draft: np.ndarray
    sel_len: np.ndarray


def score_select(hist_len, prompt_len, state, K, lk: LookupOut, model_draft, model_len, *, k_cap,
                 W1, b1, W2, b2, tau, nthreads=1, Wh=None, bh=None) -> ScoreOut:
    """Wh [H,H], bh [H]: optional second hidden layer (between W1/b1 and the output weights W2/b2)."""
    B = len(hist_len)
    H = int(np.asarray(W2).shape[0])
    W1 = np.ascontiguousarray(W1, np.float32); b1 = np.ascontiguousarray(b1, np.float32)
    W2 = np.ascontiguousarray(W2, np.float32)
    assert W1.shape == (H, N_FEATURES)
    if Wh is not None:
        Wh = np.ascontiguousarray(Wh, np.float32); bh = np.ascontiguousarray(bh, np.float32)
        assert Wh.shape == (H, H) and bh.shape == (H,) and H <= 1024
    state = np.ascontiguousarray(state, dtype=STATE_DTYPE)
    hist_len = _i32(hist_len); prompt_len = _i32(prompt_len); K = _i32(K)
    md = None if model_draft is None else _i32(model_draft)
    ml = None if model_len is None else _i32(model_len)
    out = ScoreOut(np.empty((B, N_FEATURES), np.float32), np.empty(B, np.float32),
                   np.empty(B, np.float64), np.empty(B, np.int32), np.empty((B, k_cap), np.int32),
                   np.empty(B, np.int32))
    head = (C.c_int32(B), _p(hist_len), _p(prompt_len), _p(state), _p(K),
            _p(_i32(lk.draft)), _p(_i32(lk.draft_len)), _p(_i32(lk.match_len)),
            _p(_i32(lk.match_pos)), _p(_i32(lk.match_cnt)), _p(md), _p(ml),
            C.c_int32(k_cap), C.c_int32(H), _p(W1), _p(b1))
    tail = (_p(W2), C.c_float(b2), C.c_float(tau), _p(out.features), _p(out.score), _p(out.score64),
            _p(out.select), _p(out.sel_draft), _p(out.sel_len), C.c_int32(nthreads))
    if Wh is None:
        lib().oracle_score_select(*head, *tail)
    else:
        lib().oracle_score_select2(*head, _p(Wh), _p(bh), *tail)
    return out


N_FEATURES_EXT = 14
N_TOKEN_CLASSES = 5


def score_select_ext(hist_len, prompt_len, state, K, lk: LookupOut, suffix, cls, model_draft, model_len, *, k_cap,
                     W1, b1, W2, b2, tau, nthreads=1, Wh=None, bh=None, match_src=None) -> ScoreOut:
    """score_select on the extended feature vector: cls uint8 [V] token-class bits, suffix float [B] or None,
    W1 [H, 14]."""
    B = len(hist_len)
    H = int(np.asarray(W2).shape[0])
    W1 = np.ascontiguousarray(W1, np.float32); b1 = np.ascontiguousarray(b1, np.float32)
    W2 = np.ascontiguousarray(W2, np.float32)
    assert W1.shape == (H, N_FEATURES_EXT)
    if Wh is not None:
        Wh = np.ascontiguousarray(Wh, np.float32); bh = np.ascontiguousarray(bh, np.float32)
        assert Wh.shape == (H, H) and bh.shape == (H,)
    cls = np.ascontiguousarray(cls, np.uint8)
    sfx = None if suffix is None else np.ascontiguousarray(suffix, np.float32)
    state = np.ascontiguousarray(state, dtype=STATE_DTYPE)
    hist_len = _i32(hist_len); prompt_len = _i32(prompt_len); K = _i32(K)
    md = None if model_draft is None else _i32(model_draft)
    ml = None if model_len is None else _i32(model_len)
    out = ScoreOut(np.empty((B, N_FEATURES_EXT), np.float32), np.empty(B, np.float32), np.empty(B, np.float64),
                   np.empty(B, np.int32), np.empty((B, k_cap), np.int32), np.empty(B, np.int32))
    lib().oracle_score_select_ext(
        C.c_int32(B), _p(hist_len), _p(prompt_len), _p(state), _p(K), _p(_i32(lk.draft)), _p(_i32(lk.draft_len)),
        _p(_i32(lk.match_len)), _p(_i32(lk.match_pos)), _p(_i32(lk.match_cnt)),
        None if match_src is None else _p(_i32(match_src)), _p(sfx), _p(cls),
        C.c_int32(len(cls)), _p(md), _p(ml), C.c_int32(k_cap), C.c_int32(H), _p(W1), _p(b1), _p(Wh), _p(bh), _p(W2),
        C.c_float(b2), C.c_float(tau), _p(out.features), _p(out.score), _p(out.score64), _p(out.select),
        _p(out.sel_draft), _p(out.sel_len), C.c_int32(nthreads))
    return out


def features_ext_one(n, prompt_len, sel_bits, acc_ring, draft, match_len, match_pos, match_cnt, cls, suffix_score=0.0):
    class St(C.Structure):
        _fields_ = [("sel_bits", C.c_uint32), ("pad", C.c_uint32), ("acc_ring", C.c_uint64)]
    phi = np.empty(N_FEATURES_EXT, np.float32)
    draft = _i32(draft); cls = np.ascontiguousarray(cls, np.uint8)
    lib().oracle_features_ext_one(C.c_int32(n), C.c_int32(prompt_len), St(sel_bits, 0, acc_ring),
                                  C.c_int32(len(draft)), C.c_int32(match_len), C.c_int32(match_pos),
                                  C.c_int32(match_cnt), _p(draft), _p(cls), C.c_int32(len(cls)),
                                  C.c_float(suffix_score), _p(phi))
    return phi


@dataclass
class VerifyOut:
    accepted: np.ndarray
    committed: np.ndarray
    n_commit: np.ndarray
    target_tok: np.ndarray
    status: np.ndarray


def verify_commit(logits, dtype, V, row_off, k_uniform, sel_draft, sel_len, select, *, k_cap, hist,
                  hist_off, hist_cap, hist_len, state, nthreads=1, parent=None) -> VerifyOut:
    """`parent` (int32 [B, k_cap]) makes the draft a token tree.
    `hist`, `hist_len` and `state` are updated IN PLACE (they must be writable, contiguous
    int32 / int32 / STATE_DTYPE arrays).  `logits` is a contiguous float32 array (dtype F32) or a
    uint16 array of bfloat16 bit patterns (dtype BF16), rows of V."""
    B = len(hist_len)
    assert hist.dtype == np.int32 and hist.flags.c_contiguous and hist.flags.writeable
    assert hist_len.dtype == np.int32 and hist_len.flags.c_contiguous
    assert state.dtype == STATE_DTYPE and state.flags.c_contiguous
    assert logits.flags.c_contiguous
    assert logits.dtype == (np.float32 if dtype == F32 else np.uint16)
    hist_off = np.ascontiguousarray(hist_off, dtype=np.int64)
    hist_cap = _i32(hist_cap)
    if row_off is not None:
        row_off = np.ascontiguousarray(row_off, dtype=np.int64)
        total_rows = int(row_off[B])
    else:
        total_rows = B * (k_uniform + 1)
    assert logits.size >= total_rows * V
    out = VerifyOut(np.empty(B, np.int32), np.empty((B, k_cap + 1), np.int32), np.empty(B, np.int32),
                    np.empty(total_rows, np.int32), np.empty(B, np.int32))
    tail = (_p(_i32(select)), C.c_int32(k_cap), _p(hist), _p(hist_off), _p(hist_cap), _p(hist_len), _p(state),
            _p(out.accepted), _p(out.committed), _p(out.n_commit), _p(out.target_tok), _p(out.status),
            C.c_int32(nthreads))
    head = (C.c_int32(B), _p(logits), C.c_int32(dtype), C.c_int64(V), _p(row_off), C.c_int32(k_uniform),
            _p(_i32(sel_draft)), _p(_i32(sel_len)))
    if parent is None:
        lib().oracle_verify_commit(*head, *tail)
    else:       # the draft is a token tree: parent[b, i] in {-1, 0..i-1}
        lib().oracle_verify_commit_tree(*head, _p(_i32(parent)), *tail)
    return out


PREFIX_BOUNDARY_BYTES = 64 << 20


def prefix_windows(k_cap: int, bytes_per_row_index: int, boundary_bytes: int = PREFIX_BOUNDARY_BYTES) -> list:
    """Row windows of the prefix verification: needed rows [e[j], e[j+1]) of every request form window j.
    bytes_per_row_index = B * V * element size: what one row of every request weighs.  The first window holds at
    least boundary_bytes (64 MiB) of the batch and at least two rows, windows double from there, and no boundary
    is set once the rows left, halved once per window so far, weigh less than twice that; the last window ends
    at row k_cap (a block has k_cap + 1 rows)."""
    per_row = max(int(bytes_per_row_index), 1)
    e, x, j = [0], max(2, -(-boundary_bytes // per_row)), 1
    while x < k_cap:
        e.append(x)
        if ((k_cap + 1 - x) * per_row) // (1 << j) < 2 * boundary_bytes:
            break
        x *= 2
        j += 1
    e.append(k_cap + 1)
    return e


@dataclass
class PrefixOut:
    accepted: np.ndarray
    committed: np.ndarray
    n_commit: np.ndarray
    status: np.ndarray
    rows_read: int          # logits rows looked at, whole windows counted
    rows_needed: int        # rows the results depend on: sum of accepted + 1


def verify_commit_prefix(logits, dtype, V, row_off, k_uniform, sel_draft, sel_len, select, *, k_cap, hist,
                         hist_off, hist_cap, hist_len, state, boundary_bytes=PREFIX_BOUNDARY_BYTES) -> PrefixOut:
    """Verify (Sec. 3.1) and commit (Sec. 3.4, Algorithm 1) of a chain draft, walking the rows of each request in
    order and looking at no row behind the first rejected draft token: (a, z) depend on rows 0..a only.  Rows
    are taken window by window (prefix_windows); a request goes on to its next window only if every row so far
    carried its draft token and rows are left.  Plain Python over requests and rows; the argmax of a row is the
    scalar first-maximum scan of the C oracle.  `hist`, `hist_len`, `state` are updated IN PLACE."""
    B = len(hist_len)
    edges = prefix_windows(k_cap, B * V * (4 if dtype == F32 else 2), boundary_bytes)
    out = PrefixOut(np.zeros(B, np.int32), np.full((B, k_cap + 1), -1, np.int32), np.zeros(B, np.int32),
                    np.zeros(B, np.int32), 0, 0)
    rows2d = logits.reshape(-1, V)
    for b in range(B):
        r0 = int(row_off[b]) if row_off is not None else b * (k_uniform + 1)
        r1 = int(row_off[b + 1]) if row_off is not None else r0 + k_uniform + 1
        n, cap = int(hist_len[b]), int(hist_cap[b])
        if n < 0 or n > cap or r1 - r0 <= 0:
            out.status[b] = REQ_BAD_LEN
            continue
        m = min(max(int(sel_len[b]), 0), k_cap, r1 - r0 - 1)
        d = sel_draft[b]
        a, t_a = None, None
        for lo, hi in zip(edges[:-1], edges[1:]):
            if lo > m:
                break
            top = min(hi, m + 1)
            out.rows_read += top - lo                      # the whole window is looked at
            for i in range(lo, top):
                t = argmax_row(rows2d[r0 + i], dtype)
                if a is None and (i == m or int(d[i]) != t):
                    a, t_a = i, t                          # first rejected position (or the draft's end)
            if a is not None:
                break                                      # nothing behind this window is looked at
        out.rows_needed += a + 1
        z = [int(x) for x in d[:a]] + [t_a]
        w = min(a + 1, cap - n)
        out.committed[b, :a + 1] = z
        o = int(hist_off[b])
        hist[o + n:o + n + w] = z[:w]
        hist_len[b] = n + w
        out.n_commit[b] = w
        out.accepted[b] = a
        out.status[b] = REQ_CAPACITY if w < a + 1 else REQ_OK
        state["sel_bits"][b] = np.uint32(((int(state["sel_bits"][b]) << 1) | (1 if select[b] else 0)) & 0xffffffff)
        state["acc_ring"][b] = np.uint64(((int(state["acc_ring"][b]) << 8) | (a & 0xff)) & 0xffffffffffffffff)
    return out


def argmax_row(row: np.ndarray, dtype: int) -> int:
    row = np.ascontiguousarray(row)
    return int(lib().oracle_argmax_row(_p(row), C.c_int32(dtype), C.c_int64(row.size)))


def mlp_f32(phi, W1, b1, W2, b2) -> float:
    phi = np.ascontiguousarray(phi, np.float32); W1 = np.ascontiguousarray(W1, np.float32)
    b1 = np.ascontiguousarray(b1, np.float32); W2 = np.ascontiguousarray(W2, np.float32)
    return float(lib().oracle_mlp_f32(_p(phi), C.c_int32(phi.size), C.c_int32(W2.size), _p(W1), _p(b1),
                                      _p(W2), C.c_float(b2)))


def mlp_f64(phi, W1, b1, W2, b2) -> float:
    phi = np.ascontiguousarray(phi, np.float32); W1 = np.ascontiguousarray(W1, np.float32)
    b1 = np.ascontiguousarray(b1, np.float32); W2 = np.ascontiguousarray(W2, np.float32)
    return float(lib().oracle_mlp_f64(_p(phi), C.c_int32(phi.size), C.c_int32(W2.size), _p(W1), _p(b1),
                                      _p(W2), C.c_float(b2)))


def mlp2_f32(phi, W1, b1, Wh, bh, W2, b2) -> float:
    a = [np.ascontiguousarray(x, np.float32) for x in (phi, W1, b1, Wh, bh, W2)]
    return float(lib().oracle_mlp2_f32(_p(a[0]), C.c_int32(a[0].size), C.c_int32(a[5].size), _p(a[1]), _p(a[2]),
                                       _p(a[3]), _p(a[4]), _p(a[5]), C.c_float(b2)))


def mlp2_f64(phi, W1, b1, Wh, bh, W2, b2) -> float:
    a = [np.ascontiguousarray(x, np.float32) for x in (phi, W1, b1, Wh, bh, W2)]
    return float(lib().oracle_mlp2_f64(_p(a[0]), C.c_int32(a[0].size), C.c_int32(a[5].size), _p(a[1]), _p(a[2]),
                                       _p(a[3]), _p(a[4]), _p(a[5]), C.c_float(b2)))


def features_one(n, prompt_len, sel_bits, acc_ring, draft_len, match_len, match_pos, match_cnt):
    class St(C.Structure):
        _fields_ = [("sel_bits", C.c_uint32), ("pad", C.c_uint32), ("acc_ring", C.c_uint64)]
    phi = np.empty(N_FEATURES, np.float32)
    lib().oracle_features_one(C.c_int32(n), C.c_int32(prompt_len), St(sel_bits, 0, acc_ring),
                              C.c_int32(draft_len), C.c_int32(match_len), C.c_int32(match_pos),
                              C.c_int32(match_cnt), _p(phi))
    return phi
