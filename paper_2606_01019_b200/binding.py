"""ctypes binding of the C ABI declared in ``include/hvd.h``: same names, marshalling only.

Tensors are torch CUDA tensors (device memory and streams are all torch is used for); each method
passes raw device pointers and the current CUDA stream to the library.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

F32, BF16 = 0, 1
REQ_OK, REQ_CAPACITY, REQ_BAD_LEN = 0, 1, 2
N_FEATURES = 8
STATE_DTYPE = np.dtype([("sel_bits", "<u4"), ("pad", "<u4"), ("acc_ring", "<u8")])

_vp, _i32, _i64, _f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float


class HvdError(RuntimeError):
    pass


class HvdConfig(C.Structure):
    _fields_ = [("max_batch", _i32), ("k_cap", _i32), ("l_max", _i32), ("min_match", _i32),
                ("spec_factor", _f32), ("spec_offset", _f32), ("hidden", _i32),
                ("max_hist_len", _i32), ("max_rows", _i64), ("max_vocab", _i64)]


class NextCycle(C.Structure):
    """hvd_next_cycle: the next cycle's lookup / score / select arguments of hvd_verify_commit_next."""
    _fields_ = [("K", _vp), ("n_max", _i32), ("prompt_len", _vp), ("model_draft", _vp), ("model_len", _vp),
                ("draft", _vp), ("draft_len", _vp), ("match_len", _vp), ("match_pos", _vp), ("match_cnt", _vp),
                ("features", _vp), ("score", _vp), ("select", _vp), ("sel_draft", _vp), ("sel_len", _vp)]


class HvdHostStepArgs(C.Structure):
    _fields_ = [("B", _i32), ("n_max", _i32), ("hist_words", _i64), ("hist", _vp), ("hist_off", _vp),
                ("hist_cap", _vp), ("hist_len", _vp), ("K", _vp), ("prompt_len", _vp), ("state", _vp),
                ("model_draft", _vp), ("model_len", _vp), ("logits", _vp), ("dtype", _i32),
                ("k_uniform", _i32), ("V", _i64), ("row_off", _vp), ("total_rows", _i64),
                ("score", _vp), ("select", _vp), ("sel_draft", _vp), ("sel_len", _vp), ("accepted", _vp),
                ("committed", _vp), ("n_commit", _vp), ("status", _vp)]


_SIGNATURES = {
    "hvd_create": (_i32, [C.POINTER(_vp), C.POINTER(HvdConfig)]),
    "hvd_destroy": (_i32, [_vp]),
    "hvd_status_string": (C.c_char_p, [_i32]),
    "hvd_last_error": (C.c_char_p, [_vp]),
    "hvd_device_status": (_i32, [_vp, C.POINTER(_i32)]),
    "hvd_set_predictor": (_i32, [_vp, _vp, _vp, _vp, _f32, _f32, _vp]),
    "hvd_set_predictor2": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _f32, _f32, _vp]),
    "hvd_lookup": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "hvd_lookup_score_select": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _i32] + [_vp] * 14 + [_vp]),
    "hvd_set_token_classes": (_i32, [_vp, _vp, _i64]),
    "hvd_set_predictor_ext": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _f32, _f32, _vp]),
    "hvd_score_select_ext": (_i32, [_vp, _i32] + [_vp] * 18 + [_vp]),
    "hvd_set_corpus": (_i32, [_vp, _vp, _i64]),
    "hvd_lookup_corpus": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "hvd_lookup_freq": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _i32, _f32, _i32, _f32] + [_vp] * 11 + [_vp]),
    "hvd_replay_labels": (_i32, [_vp, _vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "hvd_score_select": (_i32, [_vp, _i32] + [_vp] * 16 + [_vp]),
    "hvd_verify_commit": (_i32, [_vp, _i32, _vp, _i32, _i64, _vp, _i32, _i64] + [_vp] * 13 + [_vp]),
    "hvd_verify_commit_prefix": (_i32, [_vp, _i32, _vp, _i32, _i64, _vp, _i32, _i64] + [_vp] * 13 + [_vp]),
    "hvd_verify_commit_next": (_i32, [_vp, _i32, _vp, _i32, _i64, _vp, _i32, _i64] + [_vp] * 13 + [_vp, _vp]),
    "hvd_verify_commit_tree": (_i32, [_vp, _i32, _vp, _i32, _i64, _vp, _i32, _i64] + [_vp] * 14 + [_vp]),
    "hvd_verify_keys": (_i32, [_vp, _i32, _vp, _i32, _i64, _i64, _vp, _i32, _i64, _vp, _vp, _vp, _vp, _vp]),
    "hvd_commit_keys": (_i32, [_vp, _i32, _vp, _i64, _vp, _i32, _i64] + [_vp] * 13 + [_vp]),
    "hvd_step_host": (_i32, [_vp, C.POINTER(HvdHostStepArgs), _vp]),
    "hvd_verify_commit_noalloc": (_i32, [_i32, _i32, _vp, _i32, _i64, _vp, _i32, _i64] + [_vp] * 13 + [_vp]),
    "hvd_noalloc_last_error": (C.c_char_p, []),
}

_lib = None


def library_path() -> str:
    return _build.LIB


def exported_symbols():
    return sorted(_SIGNATURES)


def load_library(build: bool = True):
    """Loads (building first if the sources are newer) the shared library.  Fails loudly if it
    cannot be built or loaded: there is no other implementation to fall back to."""
    global _lib
    if _lib is None:
        if build:
            _build.build()
        if not os.path.exists(_build.LIB):
            raise HvdError(f"{_build.LIB} is missing: run paper_2606_01019_b200/build.py")
        lib = C.CDLL(_build.LIB)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def _ptr(t):
    return None if t is None else t.data_ptr()


def _hptr(a):
    """Address of a host array: a torch CPU tensor (pinned or not) or a numpy array."""
    if a is None:
        return None
    return a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data


def _stream():
    import torch
    return torch.cuda.current_stream().cuda_stream


NOALLOC_MAX_ROWS, NOALLOC_MAX_BATCH = 16384, 2048
FREQ_MAX_OCC = 128   # HVD_FREQ_MAX_OCC
N_FEATURES_EXT, N_TOKEN_CLASSES = 14, 5


def hvd_verify_commit_noalloc(B, k_cap, logits, dtype, V, row_off, k_uniform, total_rows, sel_draft, sel_len,
                              select, hist, hist_off, hist_cap, hist_len, state, accepted, committed, n_commit,
                              target_tok, status):
    """Verification and commit for callers that cannot allocate: no context, scratch memory is a
    static array inside the library (limits NOALLOC_MAX_ROWS / NOALLOC_MAX_BATCH).  Calls on one
    device must not overlap.  Enqueues on the current CUDA stream."""
    lib = load_library()
    st = lib.hvd_verify_commit_noalloc(B, k_cap, _ptr(logits), dtype, V, _ptr(row_off), k_uniform, total_rows,
                                       _ptr(sel_draft), _ptr(sel_len), _ptr(select), _ptr(hist), _ptr(hist_off),
                                       _ptr(hist_cap), _ptr(hist_len), _ptr(state), _ptr(accepted),
                                       _ptr(committed), _ptr(n_commit), _ptr(target_tok), _ptr(status), _stream())
    if st != 0:
        raise HvdError(f"hvd_verify_commit_noalloc: {lib.hvd_status_string(st).decode()}: "
                       f"{lib.hvd_noalloc_last_error().decode()}")


class Context:
    """One library context on the current CUDA device (see ``hvd_create``)."""

    def __init__(self, *, max_batch, k_cap, max_hist_len, max_rows, max_vocab, l_max=64, min_match=2,
                 spec_factor=1.0, spec_offset=0.0, hidden=32):
        import torch
        if not torch.cuda.is_available():
            raise HvdError("no CUDA device: the HVD path runs only in its sm_100a kernels")
        self._lib = load_library()
        self.cfg = HvdConfig(max_batch, k_cap, l_max, min_match, spec_factor, spec_offset, hidden,
                             max_hist_len, max_rows, max_vocab)
        self._h = _vp()
        st = self._lib.hvd_create(C.byref(self._h), C.byref(self.cfg))
        if st != 0:
            raise HvdError(f"hvd_create: {self._lib.hvd_status_string(st).decode()}")
        self.k_cap = k_cap
        self.hidden = hidden

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.hvd_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st, what):
        if st != 0:
            raise HvdError(f"{what}: {self._lib.hvd_status_string(st).decode()}: "
                           f"{self._lib.hvd_last_error(self._h).decode()}")

    def hvd_device_status(self) -> int:
        code = _i32(0)
        self._check(self._lib.hvd_device_status(self._h, C.byref(code)), "hvd_device_status")
        return int(code.value)

    def hvd_set_predictor(self, W1, b1, W2, b2, tau):
        W1 = np.ascontiguousarray(W1, np.float32); b1 = np.ascontiguousarray(b1, np.float32)
        W2 = np.ascontiguousarray(W2, np.float32)
        if W1.shape != (self.hidden, N_FEATURES) or b1.shape != (self.hidden,) or W2.shape != (self.hidden,):
            raise HvdError("hvd_set_predictor: weight shapes do not match the context")
        self._check(self._lib.hvd_set_predictor(self._h, W1.ctypes.data, b1.ctypes.data, W2.ctypes.data,
                                                float(b2), float(tau), _stream()), "hvd_set_predictor")

    def hvd_set_predictor2(self, W1, b1, Wh, bh, W2, b2, tau):
        H = self.hidden
        W1 = np.ascontiguousarray(W1, np.float32); b1 = np.ascontiguousarray(b1, np.float32)
        Wh = np.ascontiguousarray(Wh, np.float32); bh = np.ascontiguousarray(bh, np.float32)
        W2 = np.ascontiguousarray(W2, np.float32)
        if W1.shape != (H, N_FEATURES) or b1.shape != (H,) or Wh.shape != (H, H) or bh.shape != (H,) or W2.shape != (H,):
            raise HvdError("hvd_set_predictor2: weight shapes do not match the context")
        self._check(self._lib.hvd_set_predictor2(self._h, W1.ctypes.data, b1.ctypes.data, Wh.ctypes.data,
                                                 bh.ctypes.data, W2.ctypes.data, float(b2), float(tau), _stream()),
                    "hvd_set_predictor2")

    def hvd_set_token_classes(self, cls):
        """Registers a device uint8 tensor of class bits per vocabulary entry (None unregisters); the
        context keeps a reference so that the tensor stays alive while registered."""
        self._cls = cls
        self._check(self._lib.hvd_set_token_classes(self._h, _ptr(cls), 0 if cls is None else int(cls.numel())),
                    "hvd_set_token_classes")

    def hvd_set_predictor_ext(self, W1, b1, W2, b2, tau, Wh=None, bh=None):
        H = self.hidden
        W1 = np.ascontiguousarray(W1, np.float32); b1 = np.ascontiguousarray(b1, np.float32)
        W2 = np.ascontiguousarray(W2, np.float32)
        if W1.shape != (H, N_FEATURES_EXT) or b1.shape != (H,) or W2.shape != (H,):
            raise HvdError("hvd_set_predictor_ext: weight shapes do not match the context")
        if Wh is not None:
            Wh = np.ascontiguousarray(Wh, np.float32); bh = np.ascontiguousarray(bh, np.float32)
            if Wh.shape != (H, H) or bh.shape != (H,):
                raise HvdError("hvd_set_predictor_ext: second-layer shapes do not match the context")
        self._check(self._lib.hvd_set_predictor_ext(self._h, W1.ctypes.data, b1.ctypes.data,
                                                    None if Wh is None else Wh.ctypes.data,
                                                    None if Wh is None else bh.ctypes.data, W2.ctypes.data,
                                                    float(b2), float(tau), _stream()), "hvd_set_predictor_ext")

    def hvd_score_select_ext(self, B, hist_len, prompt_len, state, K, draft, draft_len, match_len, match_pos,
                             match_cnt, suffix_score, model_draft, model_len, features, score, select, sel_draft,
                             sel_len, match_src=None):
        self._check(self._lib.hvd_score_select_ext(self._h, B, _ptr(hist_len), _ptr(prompt_len), _ptr(state),
                                                   _ptr(K), _ptr(draft), _ptr(draft_len), _ptr(match_len),
                                                   _ptr(match_pos), _ptr(match_cnt), _ptr(match_src), _ptr(suffix_score),
                                                   _ptr(model_draft), _ptr(model_len), _ptr(features), _ptr(score),
                                                   _ptr(select), _ptr(sel_draft), _ptr(sel_len), _stream()),
                    "hvd_score_select_ext")

    def hvd_lookup(self, B, hist, hist_off, hist_cap, hist_len, K, n_max, draft, draft_len, match_len,
                   match_pos, match_cnt):
        self._check(self._lib.hvd_lookup(self._h, B, _ptr(hist), _ptr(hist_off), _ptr(hist_cap),
                                         _ptr(hist_len), _ptr(K), n_max, _ptr(draft), _ptr(draft_len),
                                         _ptr(match_len), _ptr(match_pos), _ptr(match_cnt), _stream()),
                    "hvd_lookup")

    def hvd_lookup_score_select(self, B, hist, hist_off, hist_cap, hist_len, K, n_max, prompt_len, state,
                                model_draft, model_len, draft, draft_len, match_len, match_pos, match_cnt,
                                features, score, select, sel_draft, sel_len):
        self._check(self._lib.hvd_lookup_score_select(
            self._h, B, _ptr(hist), _ptr(hist_off), _ptr(hist_cap), _ptr(hist_len), _ptr(K), n_max,
            _ptr(prompt_len), _ptr(state), _ptr(model_draft), _ptr(model_len), _ptr(draft), _ptr(draft_len),
            _ptr(match_len), _ptr(match_pos), _ptr(match_cnt), _ptr(features), _ptr(score), _ptr(select),
            _ptr(sel_draft), _ptr(sel_len), _stream()), "hvd_lookup_score_select")

    def hvd_set_corpus(self, corpus, m=None):
        """Registers a device int32 tensor as the shared warm-up corpus (None unregisters); the context
        keeps a reference so that the tensor stays alive while registered."""
        self._corpus = corpus
        n = 0 if corpus is None else (int(corpus.numel()) if m is None else int(m))
        self._check(self._lib.hvd_set_corpus(self._h, _ptr(corpus), n), "hvd_set_corpus")

    def hvd_lookup_corpus(self, B, hist, hist_off, hist_cap, hist_len, K, n_max, draft, draft_len, match_len,
                          match_pos, match_src, match_cnt):
        self._check(self._lib.hvd_lookup_corpus(self._h, B, _ptr(hist), _ptr(hist_off), _ptr(hist_cap),
                                                _ptr(hist_len), _ptr(K), n_max, _ptr(draft), _ptr(draft_len),
                                                _ptr(match_len), _ptr(match_pos), _ptr(match_src),
                                                _ptr(match_cnt), _stream()), "hvd_lookup_corpus")

    def hvd_lookup_freq(self, B, hist, hist_off, hist_cap, hist_len, K, n_max, min_prob, max_occ, threshold,
                        model_draft, model_len, draft, draft_len, score, match_len, match_pos, match_cnt,
                        select=None, sel_draft=None, sel_len=None):
        self._check(self._lib.hvd_lookup_freq(
            self._h, B, _ptr(hist), _ptr(hist_off), _ptr(hist_cap), _ptr(hist_len), _ptr(K), n_max, min_prob,
            max_occ, threshold, _ptr(model_draft), _ptr(model_len), _ptr(draft), _ptr(draft_len), _ptr(score),
            _ptr(match_len), _ptr(match_pos), _ptr(match_cnt), _ptr(select), _ptr(sel_draft), _ptr(sel_len),
            _stream()), "hvd_lookup_freq")

    def hvd_replay_labels(self, trace, n, K, label, draft_len, match_len, match_pos, match_cnt):
        self._check(self._lib.hvd_replay_labels(self._h, _ptr(trace), n, K, _ptr(label), _ptr(draft_len),
                                                _ptr(match_len), _ptr(match_pos), _ptr(match_cnt), _stream()),
                    "hvd_replay_labels")

    def hvd_score_select(self, B, hist_len, prompt_len, state, K, draft, draft_len, match_len, match_pos,
                         match_cnt, model_draft, model_len, features, score, select, sel_draft, sel_len):
        self._check(self._lib.hvd_score_select(self._h, B, _ptr(hist_len), _ptr(prompt_len), _ptr(state),
                                               _ptr(K), _ptr(draft), _ptr(draft_len), _ptr(match_len),
                                               _ptr(match_pos), _ptr(match_cnt), _ptr(model_draft),
                                               _ptr(model_len), _ptr(features), _ptr(score), _ptr(select),
                                               _ptr(sel_draft), _ptr(sel_len), _stream()),
                    "hvd_score_select")

    def hvd_verify_commit(self, B, logits, dtype, V, row_off, k_uniform, total_rows, sel_draft, sel_len,
                          select, hist, hist_off, hist_cap, hist_len, state, accepted, committed,
                          n_commit, target_tok, status):
        self._check(self._lib.hvd_verify_commit(self._h, B, _ptr(logits), dtype, V, _ptr(row_off),
                                                k_uniform, total_rows, _ptr(sel_draft), _ptr(sel_len),
                                                _ptr(select), _ptr(hist), _ptr(hist_off), _ptr(hist_cap),
                                                _ptr(hist_len), _ptr(state), _ptr(accepted),
                                                _ptr(committed), _ptr(n_commit), _ptr(target_tok),
                                                _ptr(status), _stream()),
                    "hvd_verify_commit")

    def hvd_verify_commit_prefix(self, B, logits, dtype, V, row_off, k_uniform, total_rows, sel_draft, sel_len,
                                 select, hist, hist_off, hist_cap, hist_len, state, accepted, committed,
                                 n_commit, rows_read, status):
        self._check(self._lib.hvd_verify_commit_prefix(self._h, B, _ptr(logits), dtype, V, _ptr(row_off),
                                                       k_uniform, total_rows, _ptr(sel_draft), _ptr(sel_len),
                                                       _ptr(select), _ptr(hist), _ptr(hist_off), _ptr(hist_cap),
                                                       _ptr(hist_len), _ptr(state), _ptr(accepted),
                                                       _ptr(committed), _ptr(n_commit), _ptr(rows_read),
                                                       _ptr(status), _stream()),
                    "hvd_verify_commit_prefix")

    def hvd_verify_commit_next(self, B, logits, dtype, V, row_off, k_uniform, total_rows, sel_draft, sel_len,
                               select, hist, hist_off, hist_cap, hist_len, state, accepted, committed,
                               n_commit, target_tok, status, *, K, n_max, prompt_len, model_draft, model_len,
                               draft, draft_len, match_len, match_pos, match_cnt, features, score,
                               next_select, next_sel_draft, next_sel_len):
        nxt = NextCycle(_ptr(K), int(n_max), _ptr(prompt_len), _ptr(model_draft), _ptr(model_len), _ptr(draft),
                        _ptr(draft_len), _ptr(match_len), _ptr(match_pos), _ptr(match_cnt), _ptr(features),
                        _ptr(score), _ptr(next_select), _ptr(next_sel_draft), _ptr(next_sel_len))
        self._check(self._lib.hvd_verify_commit_next(self._h, B, _ptr(logits), dtype, V, _ptr(row_off),
                                                     k_uniform, total_rows, _ptr(sel_draft), _ptr(sel_len),
                                                     _ptr(select), _ptr(hist), _ptr(hist_off), _ptr(hist_cap),
                                                     _ptr(hist_len), _ptr(state), _ptr(accepted),
                                                     _ptr(committed), _ptr(n_commit), _ptr(target_tok),
                                                     _ptr(status), C.byref(nxt), _stream()),
                    "hvd_verify_commit_next")

    def hvd_verify_keys(self, B, logits, dtype, V_shard, v_offset, row_off, k_uniform, total_rows, sel_len, hist_len,
                        hist_cap, keys):
        self._check(self._lib.hvd_verify_keys(self._h, B, _ptr(logits), dtype, V_shard, v_offset, _ptr(row_off),
                                              k_uniform, total_rows, _ptr(sel_len), _ptr(hist_len), _ptr(hist_cap),
                                              _ptr(keys), _stream()), "hvd_verify_keys")

    def hvd_commit_keys(self, B, keys, V, row_off, k_uniform, total_rows, sel_draft, sel_len, select, hist, hist_off,
                        hist_cap, hist_len, state, accepted, committed, n_commit, target_tok, status):
        self._check(self._lib.hvd_commit_keys(self._h, B, _ptr(keys), V, _ptr(row_off), k_uniform, total_rows,
                                              _ptr(sel_draft), _ptr(sel_len), _ptr(select), _ptr(hist), _ptr(hist_off),
                                              _ptr(hist_cap), _ptr(hist_len), _ptr(state), _ptr(accepted),
                                              _ptr(committed), _ptr(n_commit), _ptr(target_tok), _ptr(status),
                                              _stream()), "hvd_commit_keys")

    def hvd_verify_commit_tree(self, B, logits, dtype, V, row_off, k_uniform, total_rows, sel_draft, sel_len,
                               parent, select, hist, hist_off, hist_cap, hist_len, state, accepted, committed,
                               n_commit, target_tok, status):
        self._check(self._lib.hvd_verify_commit_tree(
            self._h, B, _ptr(logits), dtype, V, _ptr(row_off), k_uniform, total_rows, _ptr(sel_draft),
            _ptr(sel_len), _ptr(parent), _ptr(select), _ptr(hist), _ptr(hist_off), _ptr(hist_cap),
            _ptr(hist_len), _ptr(state), _ptr(accepted), _ptr(committed), _ptr(n_commit), _ptr(target_tok),
            _ptr(status), _stream()), "hvd_verify_commit_tree")

    def hvd_step_host(self, *, B, n_max, hist, hist_off, hist_cap, hist_len, K, prompt_len, state,
                      model_draft, model_len, logits, dtype, V, row_off, k_uniform, total_rows, score,
                      select, sel_draft, sel_len, accepted, committed, n_commit, status):
        """All arrays are HOST arrays (torch CPU tensors, ideally pinned, or numpy arrays)."""
        hist_words = hist.numel() if hasattr(hist, "numel") else hist.size
        args = HvdHostStepArgs(B, n_max, hist_words, _hptr(hist), _hptr(hist_off), _hptr(hist_cap),
                               _hptr(hist_len), _hptr(K), _hptr(prompt_len), _hptr(state),
                               _hptr(model_draft), _hptr(model_len), _hptr(logits), dtype, k_uniform, V,
                               _hptr(row_off), total_rows, _hptr(score), _hptr(select), _hptr(sel_draft),
                               _hptr(sel_len), _hptr(accepted), _hptr(committed), _hptr(n_commit),
                               _hptr(status))
        self._check(self._lib.hvd_step_host(self._h, C.byref(args), _stream()), "hvd_step_host")
