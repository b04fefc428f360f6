#!/usr/bin/env python
"""Benchmark of the TCA-Attention hot path on B200 (one process per GPU).

A step is one pass of the whole path over one batch of synthetic input: tca_score ->
tca_select -> tca_compact_kv -> tca_attn_prefill at L tokens, then `decode_steps` x
(tca_cache_append + tca_attn_decode).  Default workload: the 128K end-to-end
configuration (one Llama-3-8B-shaped layer, 32/8 heads, d = 128, bf16, batch 1,
L = 131072, 256 decode steps).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config4] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is prefill tokens/s over all GPUs with inputs
resident in HBM; `decode_us_per_step` is the mean of the decode steps; `e2e` repeats the
measurement through the same C-ABI calls with pinned HOST buffers copied in and the
outputs copied back inside the timed region.  N > 1 runs N independent replicas (the
path has no exchange step): no collective touches the data, only the timing is reduced.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
for _p in (ROOT, os.path.join(ROOT, "tests")):
    if _p not in sys.path:
        sys.path.insert(0, _p)

PREFILL_DRAM_BYTES_CONFIG4 = 1.99e9 + 1.04e9   # measured with ncu in one pass over the full-size launch (summary under profiles/)
DECODE_DRAM_READ_BYTES_CONFIG4 = 173.3e6        # one attention launch deep in the decode loop, same kind of capture: the rest of the 228.5 MB comes from L2
METRIC = "128K prefill tok/s"
UNIT = "tok/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------- multi-rank plumbing
def replica_workload(wl, rank: int):
    """Every rank runs its own replica of the workload on its own batch (seed shifted by rank).
    The path has no exchange step, so nothing but the timing crosses ranks."""
    return wl.scaled(seed=wl.seed + 1000 * rank)


def reduce_max(values, world: int, device="cpu"):
    """Element-wise maximum over ranks of a list of floats (a job is as slow as its slowest rank)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def job_throughput(world: int, batch: int, tokens: int, ms: float) -> float:
    """Tokens per second of the whole job: every rank processed batch * tokens in `ms`."""
    return world * batch * tokens / (ms * 1e-3)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.03)
        self.proc.terminate()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            try:
                pw.append(float(parts[2]))
            except ValueError:
                pass
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        busy = [x for x in sm if x > 0]
        return {"sm_mhz": float(np.median(busy)) if busy else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons), "samples": len(sm),
                "power_w": float(np.median(pw)) if pw else None}


# ----------------------------------------------------------------------------- workload on the device
class Pipeline:
    def __init__(self, wl, data, p, torch, B, host_io: bool = False, flags: int = 0):
        self.wl, self.torch, self.B = wl, torch, B
        self.L, self.steps_decode = wl.L, wl.decode_steps
        T = wl.L + wl.decode_steps
        self.prm = B.make_params(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.block, wl.window,
                                 alpha=wl.alpha, dtype=B.TCA_BF16 if wl.dtype == "bf16" else B.TCA_F32, flags=flags)
        tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32

        def host(a):
            t = torch.from_numpy(a.view(np.int16) if wl.dtype == "bf16" else a)
            return t.view(tdt) if wl.dtype == "bf16" else t

        self.dev = {k: host(v).cuda() for k, v in data.items()}
        U = wl.batch * wl.n_kv_heads
        self.U = U
        self.m = wl.n_blocks
        self.n_k, self.n_sel, self.tbar = B.tca_budget_resolve(p, self.m)
        per_unit = np.tile(self.n_sel, wl.batch)
        self.offsets = np.zeros(U + 1, dtype=np.int64)
        self.offsets[1:] = np.cumsum(per_unit)
        self.offsets_dev = torch.from_numpy(self.offsets).cuda()
        tk = np.tile(self.tbar, wl.batch).astype(np.int64)
        n_compress = (wl.L + wl.decode_steps - wl.window) // wl.block - self.m
        self.cache = B.Cache(self.prm, per_unit + (n_compress + 1) * tk, wl.window + wl.block, tk)
        self.logscore = torch.empty(U, wl.L, dtype=torch.float64, device="cuda")
        self.idx = torch.empty(max(1, int(self.offsets[-1])), dtype=torch.int32, device="cuda")
        self.ws_score = B.alloc_workspace(self.prm, wl.L, B.TCA_OP_SCORE)
        self.ws_select = B.alloc_workspace(self.prm, wl.L, B.TCA_OP_SELECT)
        self.ws_score_select = B.alloc_workspace(self.prm, wl.L, B.TCA_OP_SCORE_SELECT)
        self.ws_prefill = B.alloc_workspace(self.prm, wl.L, B.TCA_OP_PREFILL)
        self.ws_decode = B.alloc_workspace(self.prm, self.cache.rows_total, B.TCA_OP_DECODE)
        # device views used by the step (Q/K/V of the prompt are the first L tokens)
        self.Qp = self.dev["q"][:, :, :wl.L].contiguous()
        self.Kp = self.dev["k"][:, :, :wl.L].contiguous()
        self.Vp = self.dev["v"][:, :, :wl.L].contiguous()
        self.q_last = self.Qp[:, :, wl.L - 1].contiguous()
        self.O = torch.empty_like(self.Qp)
        # decode-step tensors laid out [step, B, H, d] so that a step is one contiguous slice
        self.qd = self.dev["q"][:, :, wl.L:].permute(2, 0, 1, 3).contiguous()
        self.kd = self.dev["k"][:, :, wl.L:].permute(2, 0, 1, 3).contiguous()
        self.vd = self.dev["v"][:, :, wl.L:].permute(2, 0, 1, 3).contiguous()
        self.Od = torch.empty_like(self.qd)
        if host_io:
            hq, hk, hv = host(data["q"]), host(data["k"]), host(data["v"])
            self.h_Qp = hq[:, :, :wl.L].contiguous().pin_memory()
            self.h_Kp = hk[:, :, :wl.L].contiguous().pin_memory()
            self.h_Vp = hv[:, :, :wl.L].contiguous().pin_memory()
            self.h_qd = hq[:, :, wl.L:].permute(2, 0, 1, 3).contiguous().pin_memory()
            self.h_kd = hk[:, :, wl.L:].permute(2, 0, 1, 3).contiguous().pin_memory()
            self.h_vd = hv[:, :, wl.L:].permute(2, 0, 1, 3).contiguous().pin_memory()
            self.h_O = torch.empty_like(self.h_Qp).pin_memory()
            self.h_q_last = self.h_Qp[:, :, wl.L - 1].contiguous().pin_memory()
            self.s_in, self.s_out = torch.cuda.Stream(), torch.cuda.Stream()
            n_ranges = max(1, min(16, wl.L // 4096))
            step_rows = -(-wl.L // n_ranges)
            step_rows = -(-step_rows // 128) * 128               # TCA_PREFILL_ROW_ALIGN
            cuts = list(range(0, wl.L, step_rows)) + [wl.L]
            self.row_ranges = list(zip(cuts[:-1], cuts[1:]))          # ascending: range i needs K, V rows below its end only
            self.ws_rows = [B.alloc_workspace(self.prm, wl.L, B.TCA_OP_PREFILL) for _ in self.row_ranges]
            self.h_Od = torch.empty_like(self.h_qd).pin_memory()
        self.launches_per_step = 4 + 1 + 1 + wl.decode_steps * 3   # score + select fused: 4, compact, prefill; append + split + combine per step
        self.ev = {}

    def _ev(self, name):
        e = self.torch.cuda.Event(enable_timing=True)
        e.record()
        self.ev.setdefault(name, []).append(e)

    def step(self, host_io: bool = False, mark: bool = False):
        if host_io:
            return self.step_from_host(mark)
        B, prm, L = self.B, self.prm, self.L
        if mark: self._ev("t_begin")
        if mark: self._ev("t0")
        B.tca_score_select(prm, self.q_last, self.Kp, L, self.n_k, self.logscore, self.idx, self.offsets_dev, None, None,
                           self.ws_score_select)
        if mark: self._ev("t_score_select")
        B.tca_compact_kv(prm, self.Kp, self.Vp, L, self.idx, self.offsets_dev, self.offsets, self.cache)
        if mark: self._ev("t_compact")
        B.tca_attn_prefill(prm, self.Qp, self.Kp, self.Vp, L, self.cache, self.O, self.ws_prefill)
        if mark: self._ev("t_prefill")
        if mark: self._ev("t_prefill_io")
        for s in range(self.steps_decode):
            B.tca_cache_append(prm, self.cache, self.kd[s], self.vd[s], self.qd[s])
            B.tca_attn_decode(prm, self.qd[s], self.cache, self.Od[s], self.ws_decode)
        if mark: self._ev("t_decode")

    def time_gather_prefill(self, reps: int = 3):
        """score + select, then the prefill that gathers the selected rows itself (no compaction, no cache):
        the prefill-only form of the path, timed with CUDA events, median of `reps` after one warm-up."""
        B, prm, L, torch = self.B, self.prm, self.L, self.torch
        ms_sel, ms_pf = [], []
        for r in range(reps + 1):
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            e[0].record()
            B.tca_score_select(prm, self.q_last, self.Kp, L, self.n_k, self.logscore, self.idx, self.offsets_dev, None,
                               None, self.ws_score_select)
            e[1].record()
            B.tca_attn_prefill_gather(prm, self.Qp, self.Kp, self.Vp, L, 0, L, self.idx, self.offsets_dev, self.O,
                                      self.ws_prefill)
            e[2].record()
            torch.cuda.synchronize()
            if r > 0:
                ms_sel.append(e[0].elapsed_time(e[1]))
                ms_pf.append(e[1].elapsed_time(e[2]))
        assert B.tca_ws_status(self.ws_prefill) == B.TCA_OK
        sel, pf = float(np.median(ms_sel)), float(np.median(ms_pf))
        return {"score_select_ms": sel, "prefill_ms": pf, "total_ms": sel + pf, "reps": reps,
                "note": "tca_attn_prefill_gather: selected rows fetched from K, V by the kernel's two producer warps (16-byte asynchronous copies)"}

    def step_from_host(self, mark: bool = False):
        """The same step with every input in pinned host memory and every output read back.

        K and the newest query go first (score and select need nothing else).  V and Q then arrive
        in row ranges, in ascending order, on a copy stream: a range of query rows attends only to
        positions below its end, so tca_compact_kv_range gathers the retained rows of each piece of
        V as it lands and tca_attn_prefill_rows starts on range i while the later pieces are still
        on the bus; each finished range of O leaves on a third stream.
        """
        B, prm, L, torch = self.B, self.prm, self.L, self.torch
        cs = torch.cuda.current_stream()
        if mark: self._ev("t_begin")
        start = torch.cuda.Event()
        start.record(cs)
        self.s_in.wait_event(start)          # the previous step has finished with these buffers
        self.s_out.wait_event(start)
        heads = [(b, h) for b in range(self.wl.batch) for h in range(self.wl.n_q_heads)]
        kv_heads = [(b, h) for b in range(self.wl.batch) for h in range(self.wl.n_kv_heads)]
        ev_q, ev_v = [], []
        with torch.cuda.stream(self.s_in):
            self.Kp.copy_(self.h_Kp, non_blocking=True)
            self.q_last.copy_(self.h_q_last, non_blocking=True)
            ev_k = torch.cuda.Event(); ev_k.record(self.s_in)
            for (r0, r1) in self.row_ranges:
                for (b, h) in kv_heads:
                    self.Vp[b, h, r0:r1].copy_(self.h_Vp[b, h, r0:r1], non_blocking=True)
                e = torch.cuda.Event(); e.record(self.s_in)
                ev_v.append(e)
                for (b, h) in heads:
                    self.Qp[b, h, r0:r1].copy_(self.h_Qp[b, h, r0:r1], non_blocking=True)
                e = torch.cuda.Event(); e.record(self.s_in)
                ev_q.append(e)
            self.qd.copy_(self.h_qd, non_blocking=True)
            self.kd.copy_(self.h_kd, non_blocking=True)
            self.vd.copy_(self.h_vd, non_blocking=True)
            ev_dec = torch.cuda.Event(); ev_dec.record(self.s_in)
        cs.wait_event(ev_k)
        if mark: self._ev("t0")
        B.tca_score_select(prm, self.q_last, self.Kp, L, self.n_k, self.logscore, self.idx, self.offsets_dev, None, None,
                           self.ws_score_select)
        if mark: self._ev("t_score_select")
        if mark: self._ev("t_compact")          # the compaction is part of the ranges below
        for i, (r0, r1) in enumerate(self.row_ranges):
            cs.wait_event(ev_v[i])
            B.tca_compact_kv_range(prm, self.Kp, self.Vp, L, r0, r1, self.idx, self.offsets_dev, self.offsets,
                                   self.cache)
            cs.wait_event(ev_q[i])
            B.tca_attn_prefill_rows(prm, self.Qp, self.Kp, self.Vp, L, r0, r1, self.cache, self.O, self.ws_rows[i])
            done = torch.cuda.Event(); done.record(cs)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(done)
                for (b, h) in heads:
                    self.h_O[b, h, r0:r1].copy_(self.O[b, h, r0:r1], non_blocking=True)
        if mark: self._ev("t_prefill")
        cs.wait_stream(self.s_out)
        cs.wait_event(ev_dec)
        if mark: self._ev("t_prefill_io")
        for s in range(self.steps_decode):
            B.tca_cache_append(prm, self.cache, self.kd[s], self.vd[s], self.qd[s])
            B.tca_attn_decode(prm, self.qd[s], self.cache, self.Od[s], self.ws_decode)
        self.h_Od.copy_(self.Od, non_blocking=True)
        if mark: self._ev("t_decode")

    def step_ms(self):
        """Milliseconds of every marked step (begin of the step to the end of its decode loop)."""
        return [x.elapsed_time(y) for x, y in zip(self.ev["t_begin"], self.ev["t_decode"])]

    def stage_ms(self):
        """Mean milliseconds per stage over the marked steps."""
        names = ["t_begin", "t0", "t_score_select", "t_compact", "t_prefill", "t_prefill_io", "t_decode"]
        out = {}
        for a, b in zip(names[:-1], names[1:]):
            out["h2d" if b == "t0" else b[2:]] = float(np.mean([x.elapsed_time(y) for x, y in zip(self.ev[a], self.ev[b])]))
        return out

    # ---- algorithmic work, counted from the realised index sets
    def algorithmic_work(self):
        wl = self.wl
        idx = self.idx.cpu().numpy()
        elt = 2 if wl.dtype == "bf16" else 4
        d, L, w, G = wl.head_dim, wl.L, wl.window, wl.group
        mb = self.m * wl.block
        i = np.arange(L, dtype=np.int64)
        c = np.minimum(np.maximum(0, i - w + 1), mb)
        pairs = 0
        for u in range(self.U):
            S = idx[self.offsets[u]:self.offsets[u + 1]]
            pairs += G * int((np.searchsorted(S, c, side="left") + (i - c + 1)).sum())
        n_rows = (self.offsets[1:] - self.offsets[:-1]) + (L - mb)
        dense_pairs = self.U * G * L * (L + 1) // 2
        return {
            "prefill_flops": 4.0 * d * pairs,
            "dense_prefill_flops": 4.0 * d * dense_pairs,
            "score_bytes": float(self.U * L * (d * elt + 8)),
            "compact_bytes": float(2 * 2 * int(n_rows.sum()) * d * elt),
            "decode_bytes_per_step": float(2 * int(n_rows.sum()) * d * elt),
            "dense_decode_bytes_per_step": float(2 * self.U * L * d * elt),
            "retained_fraction": float(n_rows.sum() / (self.U * L)),
        }


# ----------------------------------------------------------------------------- offline calibration (Algorithm 1)
def calibration_leg(pipe, torch, B, sm_max_mhz, n_candidates: int = 14, tau: float = 0.9, reps: int = 2):
    """Algorithm 1 on the prompt of the workload: column means of the causal attention map (two
    dense passes on the tensor cores), then the 14 candidates of Eq. 3 through select + Eq. 4.
    Not part of the timed step: it runs once per model, offline.  Reported against the MUFU
    roof: one ex2 per (query, key) pair of each dense pass, 16 per clock and SM."""
    wl, prm, L, U = pipe.wl, pipe.prm, pipe.L, pipe.U
    col = torch.empty(U, L, dtype=torch.float64, device="cuda")
    ws = B.alloc_workspace(prm, L, B.TCA_OP_CALIB)
    B.tca_calib_colmean(prm, pipe.Qp, pipe.Kp, L, col, ws)          # warm-up
    torch.cuda.synchronize()
    e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    e0.record()
    for _ in range(reps):
        B.tca_calib_colmean(prm, pipe.Qp, pipe.Kp, L, col, ws)
    e1.record()
    cands = B.tca_calib_candidates(wl.block, n_candidates, 1.0)
    B.tca_score(prm, pipe.q_last, pipe.Kp, L, pipe.logscore, pipe.ws_score)
    a_dev = torch.empty(n_candidates, U, dtype=torch.float64, device="cuda")
    sizes = np.zeros((n_candidates, U), dtype=np.int64)
    idx = torch.empty(max(1, U * pipe.m * wl.block), dtype=torch.int32, device="cuda")
    for i in range(n_candidates):
        n_k, n_sel, _ = B.tca_budget_resolve(np.tile(cands[i], (wl.n_kv_heads, 1)), pipe.m)
        per_unit = np.tile(n_sel, wl.batch)
        offsets = np.zeros(U + 1, dtype=np.int64)
        offsets[1:] = np.cumsum(per_unit)
        off_dev = torch.from_numpy(offsets).cuda()
        B.tca_select(prm, pipe.logscore, L, n_k, idx, off_dev, None, None, pipe.ws_select)
        B.tca_calib_score(prm, col, L, idx, off_dev, a_dev[i])
        sizes[i] = per_unit
    e2.record()
    torch.cuda.synchronize()
    assert B.tca_ws_status(ws) == B.TCA_OK
    a = a_dev.cpu().numpy()
    choice = [B.tca_calib_choose(a[:, u], sizes[:, u], tau) for u in range(U)]
    colmean_ms = e0.elapsed_time(e1) / reps
    pairs = wl.batch * wl.n_q_heads * (L * (L + 1) // 2)            # causal (query, key) pairs, all heads
    ex2_per_s = 2 * pairs / (colmean_ms * 1e-3)                     # both passes exponentiate every pair
    peak = 16 * 148 * sm_max_mhz * 1e6
    rows_sum = float((col[0] * (L - torch.arange(L, device="cuda", dtype=torch.float64))).sum().item())
    # The same scores against lower thresholds: on these inputs the retained share of the score
    # follows the retained share of the tokens, so tau = 0.9 is out of reach of the sparsest-to-densest
    # sweep of Eq. 3 with sigma = 1 (its last candidate keeps 76 % of the candidates) and Algorithm 1 ends
    # at its fall-back; lower thresholds take the valid branch.
    sweep = {f"{t:.2f}": [B.tca_calib_choose(a[:, u], sizes[:, u], t) for u in range(U)] for t in (0.9, 0.8, 0.7, 0.5)}
    return {"colmean_ms": colmean_ms, "candidates_ms": e1.elapsed_time(e2), "n_candidates": n_candidates, "tau": tau,
            "choice_per_unit": choice, "choice_per_unit_by_tau": sweep,
            "a_by_candidate_mean_over_units": [float(x) for x in a.mean(axis=1)],
            "share_of_candidates_kept_by_candidate": [float(sizes[i, 0]) / (pipe.m * wl.block) for i in range(n_candidates)],
            "retained_share_of_candidates": [float(sizes[choice[u], u]) / (pipe.m * wl.block) for u in range(U)],
            "a_of_choice": [float(a[choice[u], u]) for u in range(U)],
            "row_sum_check_unit0": rows_sum / L,
            "roofline": {"bound": "alu", "achieved": ex2_per_s / 1e12, "peak": peak / 1e12, "unit": "Tex2/s",
                         "frac": ex2_per_s / peak,
                         "peak_kind": "16 MUFU ex2 per clock and SM x 148 SMs x clocks.max.sm"}}


# ----------------------------------------------------------------------------- oracle timing (CPU baseline)
def time_oracle(wl, data, p, budget_s: float = 20.0):
    """The oracle as it stands on the host cores, on a bounded sample of the workload:
    selection of ONE KV head at full length plus attention for a few query rows of one of
    its query heads; the full prefill time is extrapolated from those two costs."""
    from oracle import tca_oracle as O
    import tca_harness as H
    from paper_2512_09238_b200 import inputs as I
    L, G = wl.L, wl.group
    scale = H.scale_of(wl)
    t0 = time.perf_counter()
    K = I.widen(data["k"][0, 0, :L])
    V = I.widen(data["v"][0, 0, :L])
    res = O.select_head(I.widen(data["q"][0, :G, L - 1]), K, p[0], wl.block, wl.window, float(wl.alpha), scale)
    t_select = time.perf_counter() - t0
    Q = I.widen(data["q"][0, 0, :L])
    rows = list(np.linspace(0, L - 1, 9).astype(int))
    n_done, t1 = 0, time.perf_counter()
    while n_done < 64 and (time.perf_counter() - t1) < max(2.0, budget_s - t_select):
        O.attention_rows(Q, K, V, res["T"], wl.window, scale, rows=[rows[n_done % len(rows)]])
        n_done += 1
    t_row = (time.perf_counter() - t1) / max(1, n_done)
    full = t_select * wl.batch * wl.n_kv_heads + t_row * L * wl.batch * wl.n_q_heads
    # one decode step of the oracle: one query of one head over the retained rows, times the heads
    T = res["T"]
    Kt, Vt = K[T], V[T]
    t2 = time.perf_counter()
    for _ in range(3):
        O.attention_over_set(Q[L - 1], Kt, Vt, scale)
    t_dec = (time.perf_counter() - t2) / 3 * wl.batch * wl.n_q_heads
    return {"value": wl.batch * L / full, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
            "decode_us_per_step": t_dec * 1e6,
            "sample": f"select of 1 of {wl.batch * wl.n_kv_heads} KV heads at L={L} ({t_select:.2f} s) + "
                      f"{n_done} query rows of 1 head ({t_row * 1e3:.1f} ms/row); prefill time extrapolated "
                      f"to {wl.batch * wl.n_q_heads} heads x {L} rows"}


# ----------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="config4")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--length", type=int, default=0, help="override L (smaller runs for profiling)")
    ap.add_argument("--decode-steps", type=int, default=-1)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-dense", action="store_true", help="skip the 100 %-budget comparison run")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="config5: skip the five-budget sweep")
    ap.add_argument("--prefill-order", default="band", choices=["global", "band"],
                    help="key-tile order of the prefill in the timed run: selected keys first, or the window band first "
                         "(the band needs no selection, so the prefill then starts under score/select/compact)")
    ap.add_argument("--no-order-compare", action="store_true", help="skip timing the other prefill order")
    ap.add_argument("--no-calibration", action="store_true", help="skip the offline calibration (Algorithm 1) leg")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    from paper_2512_09238_b200 import inputs as I
    wl = I.WORKLOADS[args.workload]
    if args.length:
        wl = wl.scaled(L=args.length)
    if args.decode_steps >= 0:
        wl = wl.scaled(decode_steps=args.decode_steps)
    elt_bytes = 2 if wl.dtype == "bf16" else 4
    qo_mib = wl.batch * wl.n_q_heads * wl.L * wl.head_dim * elt_bytes / 2 ** 20
    if qo_mib > 126:
        l2_note = (f"inputs larger than L2 (Q and O are {qo_mib:.0f} MiB each; a decode step reads the whole "
                   "retained cache, which at this size is larger than L2 too: the decode kernel asks the tiles of "
                   "about 45 % of the L2's size to stay resident from step to step and reads those from L2, the "
                   "rest from HBM; decode bytes in `stages` are the algorithmic ones)")
    else:
        l2_note = f"inputs smaller than L2 (Q is {qo_mib:.1f} MiB): a parity-size workload, not a bench line"
    config = {"workload": f"{wl.name}: 1 attention layer, {wl.n_q_heads}/{wl.n_kv_heads} heads, d={wl.head_dim}, "
                          f"{wl.dtype}, batch {wl.batch}, causal prefill L={wl.L} with selection and compaction, "
                          f"then {wl.decode_steps} decode steps (append + attend)",
              "block": wl.block, "window": wl.window, "alpha": wl.alpha, "seed": wl.seed,
              "l2": l2_note,
              "parallelism": "replicas only" if world > 1 else "1 GPU"}

    if args.impl == "reference":
        if rank != 0:
            return
        data = I.generate(wl.scaled(seed=wl.seed))
        p = I.budget_table(wl)
        vals = []
        for _ in range(args.warmup + args.steps):
            vals.append(time_oracle(wl, data, p, budget_s=8.0))
        vals = vals[args.warmup:]
        v = float(np.mean([x["value"] for x in vals]))
        base = dict(vals[-1])
        base["value"] = v
        print(json.dumps({"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": wl.batch * wl.L / v * 1e3,
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                          "data": "synthetic", "config": config, "cpu_baseline": base,
                          "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    import torch
    import torch.distributed as dist
    from paper_2512_09238_b200 import _build, binding as B
    if rank == 0:
        _build.build()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    B.lib()

    wl_rank = replica_workload(wl, rank)
    data = I.generate(wl_rank)
    p = I.budget_table(wl)
    order_flag = B.TCA_FLAG_PREFILL_BAND_FIRST if args.prefill_order == "band" else 0
    pipe = Pipeline(wl_rank, data, p, torch, B, host_io=not args.no_e2e, flags=order_flag)
    peaks, peak_kind = load_peaks()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(host_io: bool):
        pipe.ev = {}
        for _ in range(args.warmup):
            pipe.step(host_io=host_io)
        barrier()
        sampler = ClockSampler(local_rank)
        sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            pipe.step(host_io=host_io, mark=True)
        e1.record()
        barrier()
        clocks = sampler.stop()
        ms = e0.elapsed_time(e1)
        stages = pipe.stage_ms()
        per_step = pipe.step_ms()
        stages["step_median"], stages["step_min"] = float(np.median(per_step)), float(np.min(per_step))
        red = reduce_max([ms] + [stages[k] for k in sorted(stages)], world, device="cuda")
        ms, stages = red[0], dict(zip(sorted(stages), red[1:]))
        return ms / args.steps, stages, clocks

    ms_step, stages, clocks = timed(host_io=False)
    assert B.tca_ws_status(pipe.ws_prefill) == B.TCA_OK
    assert B.tca_ws_status(pipe.ws_decode) == B.TCA_OK     # no decode step timed on stale partials
    work = pipe.algorithmic_work()
    prefill_ms = stages["score_select"] + stages["compact"] + stages["prefill"]
    value = job_throughput(world, wl.batch, wl.L, prefill_ms)
    decode_us = stages["decode"] * 1e3 / wl.decode_steps if wl.decode_steps > 0 else None   # no decode phase: no figure

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic", "config": config,
           "ms_per_step_median": stages["step_median"], "ms_per_step_min": stages["step_min"],
           "decode_us_per_step": decode_us, "prefill_ms": prefill_ms, "clocks": clocks,
           "gpu_launches": pipe.launches_per_step * args.steps,
           "prefill_order": args.prefill_order + " first"}
    if clocks.get("power_w") and clocks.get("sm_mhz"):
        # the prefill runs at the board's power cap: what limits it shows as energy per flop and as clocks per
        # step (time x clock), not as time alone
        out["energy"] = {"median_power_w": clocks["power_w"], "joule_per_step": clocks["power_w"] * ms_step * 1e-3,
                         "prefill_ms_x_sm_mhz": stages["prefill"] * clocks["sm_mhz"],
                         "note": "median board power and SM clock sampled during the timed steps"}

    tf_peak = peaks["bf16_tflops_sustained"]
    achieved_tf = work["prefill_flops"] / (stages["prefill"] * 1e-3) / 1e12
    # DRAM bytes of one launch of the prefill kernel (dram__bytes_read.sum + dram__bytes_write.sum), from the
    # one-pass ncu capture of this very workload summarised under profiles/; other sizes were not captured.
    traffic = PREFILL_DRAM_BYTES_CONFIG4 if (wl.name == "config4" and wl.L == 131072) else None
    out["roofline"] = {"kernel": "tca_attn_prefill", "bound": "tensor", "achieved": achieved_tf, "peak": tf_peak,
                       "unit": "TFLOP/s", "frac": achieved_tf / tf_peak, "traffic": traffic,
                       "peak_kind": f"bf16 sustained, {peak_kind}", "frac_of_burst": achieved_tf / peaks["bf16_tflops"]}
    hbm = peaks["hbm_gbs"]

    def hbm_stage(bytes_, ms):
        gbs = bytes_ / (ms * 1e-3) / 1e9
        return {"ms": ms, "bytes": bytes_, "achieved_gbs": gbs, "frac_of_measured": gbs / hbm, "frac_of_8tbs": gbs / 8000.0}

    out["stages"] = {
        "score_select": dict(hbm_stage(work["score_bytes"], stages["score_select"]), launches=4,
                             note="tca_score_select: logits, finalize + block metric, rank, top-t; bytes are the score's"),
        "compact": hbm_stage(work["compact_bytes"], stages["compact"]),
        "prefill": {"ms": stages["prefill"], "flops": work["prefill_flops"], "dense_flops": work["dense_prefill_flops"]},
        "decode_step": dict(hbm_stage(work["decode_bytes_per_step"], decode_us * 1e-3),
                            dram_read_bytes_ncu=DECODE_DRAM_READ_BYTES_CONFIG4 if (wl.name == "config4" and wl.L == 131072) else None,
                            note="bytes are algorithmic (every retained row of K and V once); part of them is served "
                                 "from L2, where the kernel keeps about 45 % of the L2's size in cache tiles from step to step")
                       if decode_us else None,
        "retained_fraction": work["retained_fraction"],
        "hbm_peak_gbs": hbm, "hbm_peak_kind": peak_kind,
    }

    if "energy" in out:
        out["energy"]["picojoule_per_prefill_flop"] = (clocks["power_w"] * stages["prefill"] * 1e-3 /
                                                       work["prefill_flops"] * 1e12)

    if not args.no_order_compare and wl.dtype == "bf16":
        # the same steps with the other key-tile order of the prefill (latency hiding: band first lets the prefill
        # start under score/select/compact); both orders are parity-tested, the timed run uses --prefill-order
        pipe.prm.flags ^= B.TCA_FLAG_PREFILL_BAND_FIRST
        _, st_o, _ = timed(host_io=False)
        pipe.prm.flags ^= B.TCA_FLAG_PREFILL_BAND_FIRST
        other_ms = st_o["score_select"] + st_o["compact"] + st_o["prefill"]
        names = ("band_first", "global_first") if args.prefill_order == "global" else ("global_first", "band_first")
        out["prefill_order_compare"] = {names[0] + "_prefill_ms": other_ms, names[1] + "_prefill_ms": prefill_ms,
                                        "stages_other_order": {k: st_o[k] for k in ("score_select", "compact", "prefill")}}

    if not args.no_order_compare and wl.dtype == "bf16":
        out["prefill_gather"] = pipe.time_gather_prefill(reps=max(3, min(5, args.steps)))
        out["prefill_gather"]["with_compaction_ms"] = prefill_ms

    if not args.no_dense:
        # this library's own dense path: the same calls with a 100 % budget (p_b = 1 for every head)
        dense_wl = wl_rank.scaled(budget=("fixed", 1.0))
        main_pipe = pipe
        pipe = Pipeline(dense_wl, data, I.budget_table(dense_wl), torch, B, host_io=False)
        _, st_dense, _ = timed(host_io=False)
        dense_prefill = st_dense["score_select"] + st_dense["compact"] + st_dense["prefill"]
        dense_decode_us = st_dense["decode"] * 1e3 / wl.decode_steps if wl.decode_steps > 0 else None
        out["dense_baseline"] = {"budget": 1.0, "prefill_ms": dense_prefill, "decode_us_per_step": dense_decode_us,
                                 "speedup_prefill": dense_prefill / prefill_ms,
                                 "speedup_decode": dense_decode_us / decode_us if decode_us else None,
                                 "kv_rows_retained_vs_dense": work["retained_fraction"]}
        del pipe
        torch.cuda.empty_cache()
        pipe = main_pipe

    if wl.name == "config5" and not args.no_sweep:
        # the budget sweep of this configuration in one invocation: 5, 10, 25, 50 and 100 % of the candidates,
        # each with its own prefill and its own decode steps, timed like the main run
        main_pipe, sweep = pipe, {}
        for frac in (0.05, 0.10, 0.25, 0.50, 1.0):
            wl_f = wl_rank.scaled(budget=("fixed", frac))
            pipe = Pipeline(wl_f, data, I.budget_table(wl_f), torch, B, host_io=False)
            _, st_f, _ = timed(host_io=False)
            assert B.tca_ws_status(pipe.ws_prefill) == B.TCA_OK and B.tca_ws_status(pipe.ws_decode) == B.TCA_OK
            wk = pipe.algorithmic_work()
            pf = st_f["score_select"] + st_f["compact"] + st_f["prefill"]
            dus = st_f["decode"] * 1e3 / wl.decode_steps if wl.decode_steps > 0 else None
            sweep[f"{frac:.2f}"] = {
                "prefill_ms": pf, "prefill_tok_s": job_throughput(world, wl.batch, wl.L, pf),
                "attention_tflops": wk["prefill_flops"] / (st_f["prefill"] * 1e-3) / 1e12,
                "decode_us_per_step": dus,
                "decode_frac_of_measured_hbm": (wk["decode_bytes_per_step"] / (dus * 1e-6) / 1e9 / hbm) if dus else None,
                "retained_fraction": wk["retained_fraction"]}
            del pipe
            torch.cuda.empty_cache()
        out["budget_sweep"] = sweep
        pipe = main_pipe

    if not args.no_e2e:
        ms_e2e, st_e2e, _ = timed(host_io=True)
        assert all(B.tca_ws_status(w) == B.TCA_OK for w in pipe.ws_rows)
        elt = 2 if wl.dtype == "bf16" else 4
        nQ = wl.batch * wl.n_q_heads * wl.head_dim * elt
        nKV = wl.batch * wl.n_kv_heads * wl.head_dim * elt
        h2d = wl.L * (nQ + 2 * nKV) + nQ + wl.decode_steps * (nQ + 2 * nKV)   # prompt, newest query again, decode tokens
        d2h = wl.L * nQ + wl.decode_steps * nQ
        e2e_prefill_ms = sum(st_e2e[k] for k in ("h2d", "score_select", "compact", "prefill", "prefill_io"))
        out["e2e"] = {"value": job_throughput(world, wl.batch, wl.L, e2e_prefill_ms), "unit": UNIT,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e,
                      "prefill_ms": e2e_prefill_ms,
                      "decode_us_per_step": st_e2e["decode"] * 1e3 / wl.decode_steps if wl.decode_steps > 0 else None,
                      "note": "pinned host buffers: K and the newest query copied in first (score + select); V and Q "
                              "copied in, and O copied back, in ascending row ranges on two copy streams while "
                              "tca_compact_kv_range gathers each piece of V as it lands and tca_attn_prefill_rows "
                              "computes the ranges already present; decode tokens copied in, decode outputs copied "
                              "back; the timed prefill ends when the last range of O has reached the host",
                      "row_ranges": len(pipe.row_ranges)}

    if rank == 0 and world == 1 and not args.no_calibration and wl.dtype == "bf16":
        out["calibration"] = calibration_leg(pipe, torch, B, clocks.get("sm_max_mhz") or 1965.0)

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = time_oracle(wl_rank, data, p)

    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
