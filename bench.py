#!/usr/bin/env python
"""Benchmark of the HVD per-step path (lookup -> score/select -> verify/commit) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C3] [--impl b200|reference]

One step = one pass of the whole path over one batch of seeded synthetic input.  Prints ONE JSON line:
the headline workload (C3, the largest of the five that is a single uniform batch) at the top level and,
at N = 1, every workload C1-C5 under `per_config` (same fields: step time, roofline of the verify kernel
and of the lookup kernel, oracle baseline, end-to-end figure, clocks).  With N > 1 (launched by
torch.distributed.run) every rank runs its own copy of the batch: requests are independent, so the path
shards with no collective on the data path ("weak" scaling); only the timing is reduced (max over ranks).

Timing protocol: the K steps are captured in one CUDA graph (3 kernel launches per step); after W eager
warm-up steps and 3 untimed replays the graph is replayed 20 times, each replay between two CUDA events on
the launching stream with a barrier + synchronize around the series; `value` is K / median replay time, the
best replay is reported beside it.  Cold inputs: consecutive steps use rotating copies of the histories and
logits whose total exceeds twice the L2, and every step gets pristine per-step lengths / state; the `warm`
figure (same buffers every step) is reported separately and labelled.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "HVD select+verify steps/s"
UNIT = "steps/s"
L2_BYTES = 126 * 2**20
FALLBACK_HBM_GBS = 6650.0
HEADLINE = "C3"
ALL_CONFIGS = ("C1", "C2", "C3", "C4", "C5")
REPLAYS = 20          # timed replays of the K-step graph (median and best reported)
UNTIMED_REPLAYS = 3
# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the kernel on the workload, from the ncu captures
# summarised under profiles/ (per launch, like the algorithmic bytes; absent = not captured)
NCU_VERIFY_TRAFFIC_BYTES = {
    "C2": (260997504, "profiles/verify_window_kernel_c2_ncu.txt"),
    "C3": (2130413885, "profiles/verify_stream_kernel_c3_batch64_ncu.txt: captured at batch 64 (1.0064 x the algorithmic "
                       "bytes), scaled to the full launch by the needed rows"),
    "C4": (431483136, "profiles/verify_window_kernel_c4_ncu.txt"),
}
NCU_LOOKUP_TRAFFIC_BYTES = {
    "C2": (4242688, "profiles/lookup_kernel_c2_ncu.txt"),
    "C3": (33657856, "profiles/lookup_kernel_c3_ncu.txt"),
    "C4": (16831104, "profiles/lookup_kernel_c4_ncu.txt"),
    "C5": (29786880, "profiles/lookup_kernel_c5_ncu.txt"),
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default=HEADLINE, help="headline workload of the line (default: C3)")
    ap.add_argument("--only", action="store_true", help="measure the headline workload only (no per_config map)")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--predictor", default="config", choices=["config", "2x256"],
                    help="2x256: the paper's predictor shape (two hidden layers of 256 units) instead of the config's")
    ap.add_argument("--batch", type=int, default=0,
                    help="scale the workload to this many requests (profiling a workload's shape at a smaller size)")
    ap.add_argument("--profile", default=None, choices=["step", "lookup", "cycle", "prefix"],
                    help="profiling run, meant for ncu: W warm-up steps and K steps as plain stream launches on the "
                         "rotating inputs and nothing else (no graphs, no oracle, no end-to-end leg); `lookup`: only the "
                         "fused lookup + scoring kernel, and no logits are allocated; `cycle`: hvd_verify_commit_next "
                         "(commit fused with the next lookup) in place of the step's three kernels; `prefix`: the step with "
                         "hvd_verify_commit_prefix (one streaming launch and one gate per row window)")
    ap.add_argument("--unfused", action="store_true",
                    help="call hvd_lookup and hvd_score_select separately instead of hvd_lookup_score_select")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------------------------
# clocks during the timed region
# ----------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting",
               0x100: "display_clock_setting", 0x10: "sync_boost"}

    def __init__(self, device_index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self.stop_flag = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # pragma: no cover
            self.err = repr(e)

    def sample(self):
        nv = self.nv
        mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
        try:
            bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
        except Exception:
            bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
        self.samples.append(mhz)
        for bit, name in self.REASONS.items():
            if bits & bit:
                self.reasons.add(name)

    def run(self):
        if not self.ok:
            return
        while not self.stop_flag.is_set():
            try:
                self.sample()
            except Exception:
                break
            time.sleep(self.period)

    def summary(self, window: str):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "window": window}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples), "window": window}


def workload_config(w, n_gpus, extra=None):
    cfg = {"workload": f"{w.name}: batch {w.B}, histories {w.n} tokens, vocab {w.V}, K {w.K}, {w.dtype} logits",
           "requests_per_gpu": w.B, "parallelism": f"requests sharded over {n_gpus} GPU(s), no collective"}
    if extra:
        cfg.update(extra)
    return cfg


# ----------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on the host cores
# ----------------------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import hvd_workloads as W
    from oracle import pipeline as P
    w = W.CONFIGS[args.config]
    cores = P.host_threads()
    inp = P.prepare(w, device="cpu", nthreads=cores)
    # one full step to size the per-step sample
    rq = inp.rq.copy()
    t0 = time.perf_counter()
    P.step(inp, rq, nthreads=cores)
    t_full = time.perf_counter() - t0
    budget = 150.0
    B_s = w.B
    if (args.steps + args.warmup) * t_full > budget:
        B_s = max(1, int(w.B * budget / ((args.steps + args.warmup) * t_full)))
    sub = inp
    if B_s < w.B:
        # a bounded sample: the first B_s requests of the batch (own history slabs, own logits rows)
        rows = int(inp.rq.row_off[B_s])
        keep = slice(0, B_s)
        sub = P.Inputs(w, W.subset_requests(inp.rq, 0, B_s), inp.W1, inp.b1, inp.W2, inp.b2, inp.tau,
                       Wh=inp.Wh, bh=inp.bh, A=inp.A[keep], strict=inp.strict[keep], logits=inp.logits[:rows],
                       logits_np=inp.logits_np[:rows])
    times, committed = [], 0
    for i in range(args.warmup + args.steps):
        rq = sub.rq.copy()
        t0 = time.perf_counter()
        out = P.step(sub, rq, nthreads=cores)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
            committed += int(out.vf.n_commit.sum())
    total = float(np.sum(times))
    frac = B_s / w.B
    value = args.steps * frac / total
    sample = (f"{B_s} of {w.B} requests of {w.name} per step (whole-batch-equivalent steps/s = sampled "
              f"steps/s x {frac:.4f})" if B_s < w.B else f"the whole {w.name} batch every step")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps / frac,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": w.dtype,
            "data": "synthetic", "config": workload_config(w, args.gpus),
            "tokens_per_s": committed / total,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------
# the benchmark's own read-only probe kernel (libbench_probe.so, built from bench_probe.cu)
# ----------------------------------------------------------------------------------------------
class ReadProbe:
    def __init__(self, torch, dev):
        from paper_2606_01019_b200 import build
        self.lib = ctypes.CDLL(build.build_bench_probe())
        self.lib.bench_read_probe.restype = ctypes.c_int
        self.lib.bench_read_probe.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
        self.sink = torch.zeros(1, dtype=torch.int64, device=dev)
        self.grid = 8 * torch.cuda.get_device_properties(dev).multi_processor_count
        self.torch = torch

    def __call__(self, t):
        st = self.torch.cuda.current_stream().cuda_stream
        rc = self.lib.bench_read_probe(t.data_ptr(), t.numel() * t.element_size(), self.sink.data_ptr(), self.grid, st)
        if rc != 0:
            raise RuntimeError(f"bench_read_probe failed ({rc})")


# ----------------------------------------------------------------------------------------------
# one workload through the CUDA path
# ----------------------------------------------------------------------------------------------
def run_config(name, args, env, cpu_seconds):
    """Everything measured on one workload; returns the dict that becomes the line (headline) or an entry of
    per_config.  `env`: torch, dist, dev, rank, world, local, peak (GB/s), peak_kind, barrier, max_over_ranks."""
    torch, dev, rank, world = env["torch"], env["dev"], env["rank"], env["world"]
    barrier, peak_gbs, peak_kind = env["barrier"], env["peak"], env["peak_kind"]
    import hvd_workloads as W
    import paper_2606_01019_b200 as H

    w = W.CONFIGS[name]
    if args.predictor == "2x256":
        w = w.scaled(hidden=256, hidden_layers=2)
    if args.batch:
        w = w.scaled(B=args.batch)
    K_steps, W_steps = args.steps, args.warmup
    n_slots = K_steps + W_steps

    # ---- inputs: the product path itself produces the drafts the logits are planted on ----------
    rq = W.make_requests(w)
    W1, b1, W2, b2, tau = W.make_predictor(w)
    B, kc = rq.B, w.k_cap
    total_rows = int(rq.row_off[-1])
    ctx_kw = dict(max_batch=B, k_cap=kc, max_hist_len=int(rq.hist_cap.max()), max_rows=total_rows,
                  max_vocab=w.V, l_max=w.l_max, min_match=w.min_match, hidden=w.hidden)
    ctx = H.Context(**ctx_kw)
    # the same library with plain launches (no programmatic dependent launch): a call measured with nothing of its
    # neighbours overlapping it
    old_mask = os.environ.get("HVD_PDL_MASK")
    os.environ["HVD_PDL_MASK"] = "0"
    ctx_plain = H.Context(**ctx_kw)
    if old_mask is None:
        del os.environ["HVD_PDL_MASK"]
    else:
        os.environ["HVD_PDL_MASK"] = old_mask
    Wh, bh = W.make_second_layer(w) if w.hidden_layers == 2 else (None, None)

    def set_predictor(t):
        for c in (ctx, ctx_plain):
            if Wh is not None:
                c.hvd_set_predictor2(W1, b1, Wh, bh, W2, b2, t)
            else:
                c.hvd_set_predictor(W1, b1, W2, b2, t)

    set_predictor(tau)
    up = lambda a, dt: torch.as_tensor(np.ascontiguousarray(a, dt), device=dev)
    hist0 = up(rq.hist, np.int32)
    hist_off, hist_cap, Kt = up(rq.hist_off, np.int64), up(rq.hist_cap, np.int32), up(rq.K, np.int32)
    hist_len0, prompt_len = up(rq.hist_len, np.int32), up(rq.prompt_len, np.int32)
    state0 = torch.as_tensor(rq.state.view(np.int64).reshape(B, 2), device=dev)
    model_draft, model_len = up(rq.model_draft, np.int32), up(rq.model_len, np.int32)
    row_off = up(rq.row_off, np.int64)
    n_max = int(rq.hist_len.max())   # every timed step starts from the pristine lengths
    i32 = lambda *s: torch.zeros(s, dtype=torch.int32, device=dev)
    draft, draft_len, match_len, match_pos, match_cnt = i32(B, kc), i32(B), i32(B), i32(B), i32(B)
    score = torch.zeros(B, dtype=torch.float32, device=dev)
    select, sel_draft, sel_len = i32(B), i32(B, kc), i32(B)
    accepted, committed, n_commit, status = i32(B), i32(B, kc + 1), i32(B), i32(B)
    dtype = H.F32 if w.dtype == "f32" else H.BF16

    def lookup(hist, hist_len, c=ctx):
        c.hvd_lookup(B, hist, hist_off, hist_cap, hist_len, Kt, n_max, draft, draft_len, match_len, match_pos, match_cnt)

    def score_select(hist_len, state):
        ctx.hvd_score_select(B, hist_len, prompt_len, state, Kt, draft, draft_len, match_len, match_pos,
                             match_cnt, model_draft, model_len, None, score, select, sel_draft, sel_len)

    def lookup_score_select(hist, hist_len, state):
        ctx.hvd_lookup_score_select(B, hist, hist_off, hist_cap, hist_len, Kt, n_max, prompt_len, state,
                                    model_draft, model_len, draft, draft_len, match_len, match_pos, match_cnt,
                                    None, score, select, sel_draft, sel_len)

    def verify(logits, hist, hist_len, state, c=ctx):
        c.hvd_verify_commit(B, logits, dtype, w.V, row_off, 0, total_rows, sel_draft, sel_len, select, hist,
                            hist_off, hist_cap, hist_len, state, accepted, committed, n_commit, None, status)

    rows_streamed = torch.zeros(1, dtype=torch.int64, device=dev)

    def verify_prefix(logits, hist, hist_len, state):
        ctx.hvd_verify_commit_prefix(B, logits, dtype, w.V, row_off, 0, total_rows, sel_draft, sel_len, select, hist,
                                     hist_off, hist_cap, hist_len, state, accepted, committed, n_commit, rows_streamed,
                                     status)

    # the commit and the next cycle's lookup + selection in one call; the next selection goes to arrays of its
    # own, so that every timed step verifies the same (pristine) selection
    select_n, sel_draft_n, sel_len_n = i32(B), i32(B, kc), i32(B)
    n_max_next = min(int(rq.hist_cap.max()), n_max + kc + 1)

    def cycle(logits, hist, hist_len, state):
        ctx.hvd_verify_commit_next(B, logits, dtype, w.V, row_off, 0, total_rows, sel_draft, sel_len, select, hist,
                                   hist_off, hist_cap, hist_len, state, accepted, committed, n_commit, None, status,
                                   K=Kt, n_max=n_max_next, prompt_len=prompt_len, model_draft=model_draft,
                                   model_len=model_len, draft=draft, draft_len=draft_len, match_len=match_len,
                                   match_pos=match_pos, match_cnt=match_cnt, features=None, score=score,
                                   next_select=select_n, next_sel_draft=sel_draft_n, next_sel_len=sel_len_n)

    lookup(hist0, hist_len0)
    score_select(hist_len0, state0)
    if w.calibrate_cache_frac is not None:
        torch.cuda.synchronize()
        tau = W.calibrate_tau(score.cpu().numpy(), draft_len.cpu().numpy() > 0, w.calibrate_cache_frac)
        set_predictor(tau)
        score_select(hist_len0, state0)
    torch.cuda.synchronize()
    if args.profile == "lookup":
        nb = rq.hist.nbytes
        RH = int(max(2, min(64, -(-4 * L2_BYTES // nb))))
        hists = [hist0] + [hist0.clone() for _ in range(RH - 1)]
        for s in range(W_steps + K_steps):
            lookup_score_select(hists[s % RH], hist_len0, state0)
        torch.cuda.synchronize()
        ctx.close(); ctx_plain.close()
        return {"profile_run": "lookup", "config": workload_config(w, world), "steps": K_steps, "warmup": W_steps,
                "history_copies": RH, "lookup_algorithmic_bytes_per_launch": int(rq.hist_len.astype(np.int64).sum()) * 4}
    sel_len_h = sel_len.cpu().numpy()
    sel_draft_h = sel_draft.cpu().numpy()
    A = W.make_agreement(w, sel_len_h)
    logits0 = W.make_logits(w, total_rows, device=dev)
    W.plant_agreement(w, logits0, rq.row_off, sel_draft_h, sel_len_h, A)

    # ---- rotating copies of the big inputs, pristine per-step small arrays ------------------------
    hist_bytes_alloc = hist0.numel() * 4
    logits_bytes_alloc = logits0.numel() * logits0.element_size()
    R = int(max(2, -(-4 * L2_BYTES // (hist_bytes_alloc + logits_bytes_alloc))))
    # the histories alone rotate over enough copies to leave the L2 between two uses (at most 64 copies)
    RH = int(max(R, min(64, -(-4 * L2_BYTES // hist_bytes_alloc))))
    hist_cold = RH * hist_bytes_alloc >= 2 * L2_BYTES
    hists = [hist0] + [hist0.clone() for _ in range(RH - 1)]
    logits = [logits0] + [logits0.clone() for _ in range(R - 1)]
    hist_len_steps = hist_len0.repeat(n_slots, 1).contiguous()
    state_steps = state0.repeat(n_slots, 1, 1).contiguous()
    hist_len_pristine, state_pristine = hist_len_steps.clone(), state_steps.clone()
    probe = ReadProbe(torch, dev)

    stream = torch.cuda.Stream(device=dev)   # everything after the eager warm-up runs on this stream

    def restore():
        with torch.cuda.stream(stream):
            hist_len_steps.copy_(hist_len_pristine)
            state_steps.copy_(state_pristine)

    def step(slot, what="step", warm=False):
        rl, rh = (0, 0) if warm else (slot % R, slot % RH)
        hl, st = hist_len_steps[slot], state_steps[slot]
        if what == "cycle":       # verify + commit + the next cycle's lookup and selection: two kernels per step
            cycle(logits[rl], hists[rh], hl, st)
        elif what == "probe":     # plain read loop over the same logits buffer: the part's read-only speed
            probe(logits[rl])
        elif what == "lookup":
            lookup(hists[rh], hl)
        elif what == "lookup_plain":
            lookup(hists[rh], hl, ctx_plain)
        elif what == "verify":    # the selection of the last lookup is still in place: every step starts from the same state
            verify(logits[rl], hists[rh], hl, st)
        elif what == "verify_plain":
            verify(logits[rl], hists[rh], hl, st, ctx_plain)
        elif what == "verify_prefix":
            verify_prefix(logits[rl], hists[rh], hl, st)
        elif what == "step_prefix":
            lookup_score_select(hists[rh], hl, st)
            verify_prefix(logits[rl], hists[rh], hl, st)
        else:
            if args.unfused:
                lookup(hists[rh], hl)
                score_select(hl, st)
            else:
                lookup_score_select(hists[rh], hl, st)
            if what == "step":
                verify(logits[rl], hists[rh], hl, st)

    # ---- warm-up (eager), then graphs of the K steps ------------------------------------------------
    for s in range(W_steps):
        step(s)
    torch.cuda.synchronize()
    if args.profile:
        for s in range(K_steps):
            step(W_steps + s, {"cycle": "cycle", "prefix": "step_prefix"}.get(args.profile, "step"))
        torch.cuda.synchronize()
        needed = int((sel_len.cpu().numpy().astype(np.int64) + 1).sum())
        ctx.close(); ctx_plain.close()
        return {"profile_run": True, "config": workload_config(w, world), "steps": K_steps, "warmup": W_steps,
                "launches_per_step": 4 if args.unfused else 3, "needed_rows": needed,
                "verify_algorithmic_bytes_per_launch": needed * w.V * w.elt,
                "lookup_algorithmic_bytes_per_launch": int(rq.hist_len.astype(np.int64).sum()) * 4}

    def capture(what="step", warm=False):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            g.capture_begin()
            for s in range(K_steps):
                step(W_steps + s, what, warm)
            g.capture_end()
        torch.cuda.synchronize()
        return g

    def timed_replays(g, replays=REPLAYS, untimed=UNTIMED_REPLAYS, sampler=None):
        """Device times (ms) of `replays` replays of g, after `untimed` ones; barrier + synchronize around the series,
        every replay between two events on the launching stream, pristine lengths and state before each."""
        for _ in range(untimed):
            restore()
            with torch.cuda.stream(stream):
                g.replay()
        torch.cuda.synchronize()
        evs = []
        barrier()
        if sampler is not None:
            sampler.start()
        with torch.cuda.stream(stream):
            for _ in range(replays):
                restore()                      # on the same stream, outside the two events
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); g.replay(); e1.record()
                evs.append((e0, e1))
        barrier()
        ms = np.array([a.elapsed_time(b) for a, b in evs])
        restore()
        return ms

    sampler = ClockSampler(env["local"])
    g_step = capture("step")
    ms_step = timed_replays(g_step, sampler=sampler)
    window = "the 20 timed replays"
    # results of the timed steps (every step does the same work on identical copies)
    n_commit_h = n_commit.cpu().numpy()
    accepted_h = accepted.cpu().numpy()
    select_h = select.cpu().numpy()
    status_h = status.cpu().numpy()
    sel_len_after = sel_len.cpu().numpy()
    if len(sampler.samples) < 5:
        # region too short for the sampler: keep the same graph running, untimed, while sampling
        window = "the 20 timed replays + untimed repeats of the same graph"
        t_end = time.time() + 0.3
        while time.time() < t_end:
            restore()
            with torch.cuda.stream(stream):
                g_step.replay()
            torch.cuda.synchronize()
    sampler.stop_flag.set()
    sampler.join(timeout=2)
    clocks = sampler.summary(window)
    ms_step = env["max_over_ranks_vec"](ms_step)
    med_ms, best_ms = float(np.median(ms_step)), float(ms_step.min())
    del g_step

    def us_per_step(what, warm=False, replays=REPLAYS):
        g = capture(what, warm)
        ms = timed_replays(g, replays=replays, untimed=2)
        del g
        return 1e3 * float(np.median(ms)) / K_steps, 1e3 * float(ms.min()) / K_steps

    kt = {}
    kt["step_us_warm"], kt["step_us_warm_best"] = us_per_step("step", warm=True)
    kt["step_us_without_verify"], _ = us_per_step("noverify")
    kt["lookup_us"], kt["lookup_us_best"] = us_per_step("lookup")
    kt["lookup_us_plain_launches"], _ = us_per_step("lookup_plain")
    kt["lookup_us_warm"], _ = us_per_step("lookup", warm=True)
    kt["verify_commit_us_back_to_back"], _ = us_per_step("verify")
    kt["verify_commit_us_isolated"], kt["verify_commit_us_isolated_best"] = us_per_step("verify_plain")
    kt["verify_commit_us_by_difference"] = 1e3 * med_ms / K_steps - kt["step_us_without_verify"]
    kt["read_probe_us"], _ = us_per_step("probe")
    kt["step_us_commit_fused_with_next_lookup"], _ = us_per_step("cycle")
    # the same step with the verification that stops behind the first rejected draft token (same outputs: the
    # timed steps ask for no target_tok).  Rows streamed: counted by the kernels over one eager call.
    kt["step_us_prefix_verification"], kt["step_us_prefix_verification_best"] = us_per_step("step_prefix")
    kt["verify_prefix_us_back_to_back"], _ = us_per_step("verify_prefix")
    restore()
    with torch.cuda.stream(stream):
        rows_streamed.zero_()
        step(W_steps, "verify_prefix")
    torch.cuda.synchronize()
    prefix_rows = int(rows_streamed.item())
    prefix_same = bool((accepted.cpu().numpy() == accepted_h).all() and (n_commit.cpu().numpy() == n_commit_h).all())
    restore()

    steps_per_s = world * K_steps / (med_ms * 1e-3)
    tokens_per_step = int(n_commit_h.sum())
    assert (status_h == 0).all(), "a request reported a capacity or length problem"
    step_us = 1e3 * med_ms / K_steps

    # ---- rooflines: algorithmic bytes = needed rows x V x elt (verify), 4 bytes per history token (lookup) ----
    verify_bytes = int((sel_len_after.astype(np.int64) + 1).sum()) * w.V * w.elt
    lookup_bytes = int(rq.hist_len.astype(np.int64).sum()) * 4
    gbs = lambda nbytes, us: nbytes / (us * 1e-6) / 1e9
    v_iso, v_b2b = gbs(verify_bytes, kt["verify_commit_us_isolated"]), gbs(verify_bytes, kt["verify_commit_us_back_to_back"])
    probe_bytes = logits0.numel() * logits0.element_size()
    probe_gbs = gbs(probe_bytes, kt["read_probe_us"])
    # which streaming kernel hvd_verify_commit takes for this call (the rule of launch_verify in csrc/hvd_verify_commit.cu)
    grid_bytes = B * (kc + 1) * w.V * w.elt
    if 160 * 2**20 < grid_bytes <= 640 * 2**20 and B * (kc + 1) * 4 <= total_rows * 5:
        stream_kernel = "verify_window_kernel"
    elif logits_bytes_alloc > 160 * 2**20:
        stream_kernel = "verify_stream_kernel"
    else:
        stream_kernel = "verify_small_kernel"
    roofline = {"bound": "hbm", "kernel": stream_kernel + " (+ verify_commit_kernel)",
                "achieved": v_iso, "peak": peak_gbs, "unit": "GB/s", "frac": v_iso / peak_gbs,
                "traffic": NCU_VERIFY_TRAFFIC_BYTES.get(w.name, (None, None))[0] if not args.batch else None,
                "traffic_source": NCU_VERIFY_TRAFFIC_BYTES.get(w.name, (None, "not captured"))[1], "peak_kind": peak_kind,
                "algorithmic_bytes_per_launch": verify_bytes,
                "frac_of_8000_nominal": v_iso / 8000.0,
                "achieved_back_to_back": v_b2b, "frac_back_to_back": v_b2b / peak_gbs,
                "achieved_by_difference": gbs(verify_bytes, kt["verify_commit_us_by_difference"]),
                "read_only_kernel": {"achieved": probe_gbs, "unit": "GB/s", "bytes_per_launch": probe_bytes,
                                     "what": "bench_probe.cu: a plain grid-stride read of the whole logits buffer, K launches "
                                             "back to back on the rotating copies"},
                "frac_of_read_only_kernel": v_iso / probe_gbs,
                "timing": "CUDA events around a graph of K hvd_verify_commit calls (both kernels of the call) on rotating "
                          "inputs larger than L2; `achieved` = isolated: plain launches, every kernel starts after its "
                          "predecessor has completed; `achieved_back_to_back` = with programmatic dependent launch, the "
                          "next call's start-up hidden under this call's tail (as inside a step)"}
    rows_full = int((sel_len_after.astype(np.int64) + 1).sum())
    rows_needed = int((accepted_h.astype(np.int64) + 1)[status_h != 2].sum())
    prefix = {"entry_point": "hvd_lookup_score_select + hvd_verify_commit_prefix",
              "us_per_step": kt["step_us_prefix_verification"], "us_per_step_best": kt["step_us_prefix_verification_best"],
              "steps_per_s": world * 1e6 / kt["step_us_prefix_verification"],
              "speedup_over_the_full_verification": step_us / kt["step_us_prefix_verification"],
              "verify_us_back_to_back": kt["verify_prefix_us_back_to_back"],
              "rows_streamed": prefix_rows, "rows_the_results_depend_on": rows_needed, "rows_of_the_full_verification": rows_full,
              "bytes_streamed": prefix_rows * w.V * w.elt,
              "achieved_on_streamed_bytes": gbs(prefix_rows * w.V * w.elt, kt["verify_prefix_us_back_to_back"]),
              "frac_on_streamed_bytes": gbs(prefix_rows * w.V * w.elt, kt["verify_prefix_us_back_to_back"]) / peak_gbs,
              "unit": "GB/s", "same_results_as_the_full_verification": prefix_same,
              "what": "rows [0,2), [2,4), [4,8), ... of every request still accepted so far, one streaming launch per "
                      "window; accepted, committed tokens, histories and state as from hvd_verify_commit"}
    l_b2b = gbs(lookup_bytes, kt["lookup_us"])
    roofline_lookup = {"bound": "hbm", "kernel": "lookup_kernel / lookup_cluster_kernel (hvd_lookup alone, K calls back to back in one graph)",
                       "achieved": l_b2b, "peak": peak_gbs, "unit": "GB/s", "frac": l_b2b / peak_gbs,
                       "traffic": NCU_LOOKUP_TRAFFIC_BYTES.get(w.name, (None, None))[0] if not args.batch else None,
                       "traffic_source": NCU_LOOKUP_TRAFFIC_BYTES.get(w.name, (None, "not captured"))[1], "peak_kind": peak_kind,
                       "algorithmic_bytes_per_launch": lookup_bytes,
                       "cold": bool(hist_cold), "history_copies": RH,
                       "achieved_plain_launches": gbs(lookup_bytes, kt["lookup_us_plain_launches"]),
                       "achieved_warm_l2_resident": gbs(lookup_bytes, kt["lookup_us_warm"]),
                       "traffic_floor_us_at_peak": lookup_bytes / peak_gbs / 1e3}
    roofline_step = {"bound": "hbm", "algorithmic_bytes_per_step": lookup_bytes + verify_bytes,
                     "achieved": gbs(lookup_bytes + verify_bytes, step_us), "peak": peak_gbs, "unit": "GB/s",
                     "peak_kind": peak_kind, "frac": gbs(lookup_bytes + verify_bytes, step_us) / peak_gbs}

    # ---- end to end through the host-buffer entry point --------------------------------------------
    e2e = None
    if not args.no_e2e:
        E = max(1, min(args.e2e_steps, K_steps))
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        h_hist, h_off, h_cap = pin(rq.hist), pin(rq.hist_off), pin(rq.hist_cap)
        h_len, h_K, h_pl = pin(rq.hist_len), pin(rq.K), pin(rq.prompt_len)
        h_state = pin(rq.state.view(np.int64).reshape(B, 2))
        h_md, h_ml, h_ro = pin(rq.model_draft), pin(rq.model_len), pin(rq.row_off)
        h_logits = torch.empty(logits0.shape, dtype=logits0.dtype, pin_memory=True)
        h_logits.copy_(logits0)
        hz = lambda *s: torch.zeros(s, dtype=torch.int32).pin_memory()
        o_score = torch.zeros(B, dtype=torch.float32).pin_memory()
        o_sel, o_sd, o_sl, o_acc, o_com, o_nc, o_st = hz(B), hz(B, kc), hz(B), hz(B), hz(B, kc + 1), hz(B), hz(B)
        len0, st0 = h_len.clone(), h_state.clone()

        def host_step():
            h_len.copy_(len0)
            h_state.copy_(st0)
            ctx.hvd_step_host(B=B, n_max=n_max, hist=h_hist, hist_off=h_off, hist_cap=h_cap, hist_len=h_len,
                              K=h_K, prompt_len=h_pl, state=h_state, model_draft=h_md, model_len=h_ml,
                              logits=h_logits, dtype=dtype, V=w.V, row_off=h_ro, k_uniform=0,
                              total_rows=total_rows, score=o_score, select=o_sel, sel_draft=o_sd,
                              sel_len=o_sl, accepted=o_acc, committed=o_com, n_commit=o_nc, status=o_st)

        for _ in range(3):
            host_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(E):
            host_step()
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt = env["max_over_ranks"](dt)
        assert (o_acc.numpy() == accepted_h).all() and (o_nc.numpy() == n_commit_h).all()
        small = B * (8 + 4 * 5 + 16) + (B + 1) * 8 + B * kc * 4
        # of the logits the call copies the rows its verification reads: window by window, as hvd_verify_commit_prefix
        # does (the same rule on the same selection: the rows counted by the kernels above)
        logits_h2d = prefix_rows * w.V * w.elt
        h2d = int(h_hist.numel() * 4 + logits_h2d + small)
        d2h = int(B * 4 * 7 + B * kc * 4 + B * (kc + 1) * 4 + B * 16)
        e2e = {"value": world * E / dt, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "steps": E, "ms_per_step": 1e3 * dt / E, "tokens_per_s": world * E * tokens_per_step / dt,
               "api": "hvd_step_host (pinned host buffers)",
               "logits_bytes_on_host": int(h_logits.numel() * h_logits.element_size()),
               "note": "histories, per-request arrays and the logits rows that verification reads cross the bus "
                       "every step: rows window by window up to the window of a request's first rejected draft token "
                       "(hvd_verify_commit_prefix's rule), read in place from the pinned host buffer by the streaming "
                       "kernels; h2d_bytes_per_step counts those rows"}
        del h_logits, h_hist

    # ---- CPU baseline: the oracle, as it stands, on this machine's host cores (rank 0, N = 1) ----------
    cpu_baseline = None
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        from oracle import pipeline as P
        cores = P.host_threads()
        logits_np = W.logits_to_numpy(logits0)
        inp = P.Inputs(w, rq, W1, b1, W2, b2, tau, Wh=Wh, bh=bh, A=A, strict=np.ones(B, bool), logits_np=logits_np)
        times, out = [], None
        t_begin = time.perf_counter()
        while len(times) < 3 or (time.perf_counter() - t_begin < cpu_seconds and len(times) < 200):
            rq_c = rq.copy()
            t0 = time.perf_counter()
            out = P.step(inp, rq_c, nthreads=cores)
            times.append(time.perf_counter() - t0)
        med = float(np.median(times))
        same = bool((out.vf.accepted == accepted_h).all() and (out.vf.n_commit == n_commit_h).all()
                    and (out.sc.select == select_h).all())
        cpu_baseline = {"value": 1.0 / med, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"the whole {w.name} batch ({B} requests, {total_rows} logits rows), "
                                  f"median of {len(times)} repetitions",
                        "ms_per_step": 1e3 * med, "tokens_per_s": tokens_per_step / med,
                        "agrees_with_gpu_step": same}
        del logits_np, inp

    launches = 4 if args.unfused else 3
    res = {"metric": METRIC, "value": steps_per_s, "unit": UNIT, "n_gpus": world, "steps": K_steps,
           "warmup": W_steps, "ms_per_step": med_ms / K_steps, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
           "config": workload_config(w, world, {
               "cold_cache": f"{R} rotating copies of the logits ({logits_bytes_alloc / 2**20:.0f} MiB each) and {RH} of the "
                             f"histories ({hist_bytes_alloc / 2**20:.1f} MiB each); L2 is 126 MiB; "
                             + ("inputs per step exceed L2 and no copy is reused within 2x L2 of traffic"
                                if hist_cold else "the histories of the whole batch are too small to leave the L2"),
               "launch": f"graph: {K_steps} steps x {launches} kernels in one CUDA graph, replayed {REPLAYS} times "
                         f"after {UNTIMED_REPLAYS} untimed replays; value = K / median replay time",
               "entry_points": "hvd_lookup + hvd_score_select + hvd_verify_commit" if args.unfused
                               else "hvd_lookup_score_select + hvd_verify_commit",
               "tau": tau,
               "predictor": f"8->{w.hidden}" + (f"->{w.hidden}" if w.hidden_layers == 2 else "") + "->1 fp32"}),
           "replays": REPLAYS, "us_per_step": step_us, "us_per_step_best": 1e3 * best_ms / K_steps,
           "steps_per_s_best": world * K_steps / (best_ms * 1e-3),
           "tokens_per_s": world * K_steps * tokens_per_step / (med_ms * 1e-3),
           "tokens_per_step": tokens_per_step,
           "mean_accepted": float(accepted_h.mean()), "cache_selected_frac": float(select_h.mean()),
           "warm": {"us_per_step": kt["step_us_warm"], "us_per_step_best": kt["step_us_warm_best"],
                    "steps_per_s": 1.0 / (kt["step_us_warm"] * 1e-6),
                    "what": "the same K steps on ONE copy of the histories and logits (every step re-reads the buffers the "
                            "previous step read: L2-resident as far as they fit 126 MiB); per rank"},
           "kernel_us": kt, "prefix_verification": prefix, "roofline": roofline, "roofline_lookup": roofline_lookup, "roofline_step": roofline_step,
           "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": launches * K_steps * REPLAYS,
           "clocks": clocks,
           "us_per_step_x_sm_ghz": step_us * (clocks["sm_mhz"] or 0) / 1e3,
           # the same K steps with hvd_verify_commit_next (commit + next cycle's lookup and selection in one kernel:
           # two launches per step), single rank's figure; the headline keeps the separate entry points
           "variant_commit_fused_with_next_lookup": {
               "value": 1.0 / (kt["step_us_commit_fused_with_next_lookup"] * 1e-6), "unit": UNIT,
               "us_per_step": kt["step_us_commit_fused_with_next_lookup"],
               "entry_points": "hvd_verify_commit_next (after one hvd_lookup_score_select)"}}
    ctx.close()
    ctx_plain.close()
    del hists, logits, logits0, hist0
    torch.cuda.synchronize()
    torch.cuda.empty_cache()
    return res


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2606_01019_b200.sharding import max_over_ranks

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the HVD path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_vec(ms):
        if world == 1:
            return ms
        t = torch.as_tensor(ms, dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return t.cpu().numpy()

    peak_gbs, peak_kind = measured_peak()
    env = {"torch": torch, "dev": dev, "rank": rank, "world": world, "local": local, "peak": peak_gbs,
           "peak_kind": peak_kind, "barrier": barrier, "max_over_ranks": lambda x: max_over_ranks(x, dev),
           "max_over_ranks_vec": max_vec}
    line = run_config(args.config, args, env, cpu_seconds=10.0)
    if world == 1 and not args.only and not args.profile:
        # every workload in the same line; the oracle leg is capped at a few seconds per workload
        keep = ("us_per_step", "us_per_step_best", "value", "steps_per_s_best", "tokens_per_s", "tokens_per_step",
                "mean_accepted", "cache_selected_frac", "warm", "kernel_us", "prefix_verification", "roofline", "roofline_lookup",
                "roofline_step", "cpu_baseline", "e2e", "clocks", "us_per_step_x_sm_ghz", "dtype", "config")
        per = {}
        for name in ALL_CONFIGS:
            r = line if name == args.config else run_config(name, args, env, cpu_seconds=4.0)
            per[name] = {k: r[k] for k in keep}
            per[name]["steps_per_s"] = per[name].pop("value")
        line["per_config"] = per
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
