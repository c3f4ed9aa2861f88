"""Device-side plumbing for one request batch: uploads host arrays into torch CUDA tensors, holds
the output tensors, and calls the three library entry points.  No step of the method is computed
here; every call goes to the CUDA library."""
from __future__ import annotations

import numpy as np

from .binding import BF16, F32, STATE_DTYPE, Context


class DeviceBatch:
    def __init__(self, ctx: Context, *, hist, hist_off, hist_cap, hist_len, K, prompt_len, state,
                 model_draft, model_len, row_off, V, dtype, uniform_rows=False, device="cuda"):
        import torch
        self.torch = torch
        self.ctx = ctx
        self.dev = torch.device(device)
        self.B = int(len(hist_len))
        self.V = int(V)
        self.dtype = F32 if dtype in ("f32", F32) else BF16
        kc = ctx.k_cap
        up = lambda a, dt: torch.as_tensor(np.ascontiguousarray(a, dt), device=self.dev)
        self.hist = up(hist, np.int32)
        self.hist_off = up(hist_off, np.int64)
        self.hist_cap = up(hist_cap, np.int32)
        self.hist_len = up(hist_len, np.int32)
        self.K = up(K, np.int32)
        self.prompt_len = up(prompt_len, np.int32)
        self.state = torch.as_tensor(np.ascontiguousarray(state, STATE_DTYPE).view(np.int64).reshape(self.B, 2),
                                     device=self.dev)
        self.model_draft = None if model_draft is None else up(model_draft, np.int32)
        self.model_len = None if model_len is None else up(model_len, np.int32)
        self.total_rows = int(row_off[-1])
        self.k_uniform = int(row_off[1] - row_off[0]) - 1 if uniform_rows else 0
        self.row_off = None if uniform_rows else up(row_off, np.int64)
        # host-side upper bound on hist_len: the longest valid history now, raised by every commit
        self.cap_max = int(max(0, np.max(hist_cap))) if len(hist_cap) else 0
        hl = np.asarray(hist_len, np.int64)
        ok = (hl >= 0) & (hl <= np.asarray(hist_cap, np.int64))
        self.n_max = int(hl[ok].max()) if ok.any() else 0
        B = self.B
        i32 = lambda *s: torch.full(s, -12345, dtype=torch.int32, device=self.dev)
        self.draft, self.draft_len = i32(B, kc), i32(B)
        self.match_len, self.match_pos, self.match_cnt = i32(B), i32(B), i32(B)
        self.features = torch.full((B, 8), float("nan"), dtype=torch.float32, device=self.dev)
        # outputs of the variants: frequency score, source of a corpus match, the extended feature vector
        self.freq_score = torch.full((B,), float("nan"), dtype=torch.float32, device=self.dev)
        self.match_src = i32(B)
        self.features_ext = torch.full((B, 14), float("nan"), dtype=torch.float32, device=self.dev)
        self.score = torch.full((B,), float("nan"), dtype=torch.float32, device=self.dev)
        self.select, self.sel_draft, self.sel_len = i32(B), i32(B, kc), i32(B)
        self.accepted, self.committed, self.n_commit = i32(B), i32(B, kc + 1), i32(B)
        self.target_tok, self.status = i32(max(self.total_rows, 1)), i32(B)

    def lookup(self):
        self.ctx.hvd_lookup(self.B, self.hist, self.hist_off, self.hist_cap, self.hist_len, self.K,
                            self.n_max, self.draft, self.draft_len, self.match_len, self.match_pos,
                            self.match_cnt)

    def score_select(self):
        self.ctx.hvd_score_select(self.B, self.hist_len, self.prompt_len, self.state, self.K, self.draft,
                                  self.draft_len, self.match_len, self.match_pos, self.match_cnt,
                                  self.model_draft, self.model_len, self.features, self.score,
                                  self.select, self.sel_draft, self.sel_len)

    def lookup_score_select(self):
        self.ctx.hvd_lookup_score_select(self.B, self.hist, self.hist_off, self.hist_cap, self.hist_len, self.K,
                                         self.n_max, self.prompt_len, self.state, self.model_draft,
                                         self.model_len, self.draft, self.draft_len, self.match_len,
                                         self.match_pos, self.match_cnt, self.features, self.score,
                                         self.select, self.sel_draft, self.sel_len)

    def lookup_freq(self, min_prob=0.1, max_occ=128, threshold=None):
        """Frequency-weighted draft and score; with a threshold also the score-threshold selection."""
        sel = (self.select, self.sel_draft, self.sel_len) if threshold is not None else (None, None, None)
        self.ctx.hvd_lookup_freq(self.B, self.hist, self.hist_off, self.hist_cap, self.hist_len, self.K, self.n_max,
                                 float(min_prob), int(max_occ), float(threshold or 0.0), self.model_draft,
                                 self.model_len, self.draft, self.draft_len, self.freq_score, self.match_len,
                                 self.match_pos, self.match_cnt, *sel)

    def lookup_corpus(self):
        self.ctx.hvd_lookup_corpus(self.B, self.hist, self.hist_off, self.hist_cap, self.hist_len, self.K, self.n_max,
                                   self.draft, self.draft_len, self.match_len, self.match_pos, self.match_src,
                                   self.match_cnt)

    def score_select_ext(self, suffix=False, src=False):
        self.ctx.hvd_score_select_ext(self.B, self.hist_len, self.prompt_len, self.state, self.K, self.draft,
                                      self.draft_len, self.match_len, self.match_pos, self.match_cnt,
                                      self.freq_score if suffix else None, self.model_draft, self.model_len,
                                      self.features_ext, self.score, self.select, self.sel_draft, self.sel_len,
                                      match_src=self.match_src if src else None)

    def verify_commit(self, logits, target_tok=True):
        self.ctx.hvd_verify_commit(self.B, logits, self.dtype, self.V, self.row_off, self.k_uniform,
                                   self.total_rows, self.sel_draft, self.sel_len, self.select, self.hist,
                                   self.hist_off, self.hist_cap, self.hist_len, self.state,
                                   self.accepted, self.committed, self.n_commit,
                                   self.target_tok if target_tok else None, self.status)
        self.n_max = min(self.cap_max, self.n_max + self.ctx.k_cap + 1)

    def verify_commit_prefix(self, logits, rows_read=None):
        """Verification and commit that read the logits only up to the first rejected draft token
        (no target_tok); rows_read: optional uint64 device scalar that the rows streamed are added to."""
        self.ctx.hvd_verify_commit_prefix(self.B, logits, self.dtype, self.V, self.row_off, self.k_uniform,
                                          self.total_rows, self.sel_draft, self.sel_len, self.select, self.hist,
                                          self.hist_off, self.hist_cap, self.hist_len, self.state,
                                          self.accepted, self.committed, self.n_commit, rows_read, self.status)
        self.n_max = min(self.cap_max, self.n_max + self.ctx.k_cap + 1)

    def verify_commit_next(self, logits, target_tok=True, K=None, model_draft=None, model_len=None):
        """Verification and commit of this cycle, then the next cycle's lookup, score and selection (on the
        histories just extended) in the same call.  K / model_draft / model_len: the next cycle's inputs
        (default: this cycle's arrays)."""
        n_max = min(self.cap_max, self.n_max + self.ctx.k_cap + 1)
        self.ctx.hvd_verify_commit_next(self.B, logits, self.dtype, self.V, self.row_off, self.k_uniform,
                                        self.total_rows, self.sel_draft, self.sel_len, self.select, self.hist,
                                        self.hist_off, self.hist_cap, self.hist_len, self.state,
                                        self.accepted, self.committed, self.n_commit,
                                        self.target_tok if target_tok else None, self.status,
                                        K=self.K if K is None else K, n_max=n_max, prompt_len=self.prompt_len,
                                        model_draft=self.model_draft if model_draft is None else model_draft,
                                        model_len=self.model_len if model_len is None else model_len,
                                        draft=self.draft, draft_len=self.draft_len, match_len=self.match_len,
                                        match_pos=self.match_pos, match_cnt=self.match_cnt,
                                        features=self.features, score=self.score, next_select=self.select,
                                        next_sel_draft=self.sel_draft, next_sel_len=self.sel_len)
        self.n_max = n_max

    def step(self, logits, target_tok=True, fused=False):
        if fused:
            self.lookup_score_select()
        else:
            self.lookup()
            self.score_select()
        self.verify_commit(logits, target_tok)

    def download(self) -> dict:
        """Host copies of every output and in/out array (synchronises)."""
        names = ["draft", "draft_len", "match_len", "match_pos", "match_cnt", "features", "score",
                 "select", "sel_draft", "sel_len", "accepted", "committed", "n_commit", "target_tok",
                 "status", "hist", "hist_len", "freq_score", "match_src", "features_ext"]
        out = {k: getattr(self, k).cpu().numpy() for k in names}
        out["target_tok"] = out["target_tok"][:self.total_rows]
        out["state"] = self.state.cpu().numpy().reshape(-1).view(STATE_DTYPE)
        return out
