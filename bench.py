#!/usr/bin/env python
"""Throughput of one SVIP speculative-decoding round (draft steps + ragged packing + verify).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload stress] [--impl ours|reference]

A step is one whole round over one batch of the workload: one svip_draft_step call per draft
position over the sequences still drafting, one svip_pack_ragged, one svip_verify.  The default
workload is `stress`, the largest of the five published configurations that fits one GPU (B = 256
sequences, V = 256000 fp32 logits, K = 8: 4.7 GB of logits per round); `--workload ragged` is the
long-form configuration with entropy-driven draft lengths.  The metric is logits GB/s: bytes of logits
the round has to read (every draft row once, every target row once, plus the draft row of each
rejected position) divided by the device time of the step.  Prints ONE JSON line on rank 0.  With
N > 1 (torchrun) every rank runs its own batch on its own GPU (weak scaling, no data-path
collective); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2411_18462_b200 import sharding, workloads  # noqa: E402

METRIC = "logits GB/s (% of B200 HBM peak) for draft-step+verify; us/step at B=1"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of row_stats_kernel<bf16> per algorithmic byte, from an
# ncu capture of a 1056-row launch (321.20 MB read and 10.73 MB written for 321.16 MB of logits); traffic
# grows in proportion to the rows, so a full launch is scaled by its bytes
ROW_STATS_TRAFFIC_PER_ALGORITHMIC_BYTE = 331.93 / 321.16
# the same for draft_step_kernel<f32, sampling> in the launch shape timed on `stress` (clusters of 2,
# three blocks per SM), from a capture of 160-row launches (166.44 MB read and 9.27 MB written for
# 163.84 MB of logits)
DRAFT_F32_TRAFFIC_PER_ALGORITHMIC_BYTE = 175.71 / 163.84


def describe(w, B=None):
    lens = "K_i~U{1..%d} set by the entropy stop rule" % w.K_max if w.name == "ragged" else "K=%d" % w.K_max
    return "%s: B=%d V=%d %s logits, %s, T=%g, h=%g" % (w.name, B or w.B, w.V, w.dtype, lens, w.T, w.h)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid = uuid
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out = self.proc.communicate(timeout=10)[0]
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.splitlines():
            p = [x.strip() for x in line.split(",")]
            if len(p) < 8:
                continue
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except ValueError:
                continue
            for n, v in zip(names, p[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------- the round on one GPU

class Round:
    """Device buffers and pre-marshalled calls of one speculative-decoding round of a workload.

    Draft logits live position-major, [K, B, V] with the sequences sorted by decreasing draft
    length: step j reads the first active[j] rows of slab j (the sequences still drafting), which is
    the layout a serving loop produces.  Target rows are packed sequence after sequence."""

    def __init__(self, ctx, w, torch, stream):
        self.ctx, self.w, self.torch, self.stream = ctx, w, torch, stream
        order, q_pm, active = workloads.position_major(w)
        B, V, K = w.B, w.V, q_pm.shape[0]
        self.B, self.V, self.K, self.active, self.order = B, V, K, active, order
        lens = w.draft_len[order].astype(np.int32)
        cu_sorted = np.concatenate([[0], np.cumsum(lens.astype(np.int64) + 1)])
        t_sorted = np.empty_like(w.target_logits)
        uv_sorted = np.empty_like(w.verify_uniforms)
        ud_pm = np.zeros((K, B), dtype=np.float32)
        for k, i in enumerate(order):
            n = int(lens[k]) + 1
            t_sorted[cu_sorted[k]:cu_sorted[k] + n] = w.target_logits[w.cu_rows[i]:w.cu_rows[i] + n]
            uv_sorted[cu_sorted[k]:cu_sorted[k] + n] = w.verify_uniforms[w.cu_rows[i]:w.cu_rows[i] + n]
            r0 = int(w.cu_rows[i]) - int(i)
            ud_pm[:n - 1, k] = w.draft_uniforms[r0:r0 + n - 1]
        self.Rp = int(cu_sorted[-1])
        self.lens = lens
        as_t = (lambda a: torch.from_numpy(a.view(np.int16))) if w.dtype == "bf16" else torch.from_numpy
        # pinned host copies (the end-to-end leg copies from these every step)
        self.h_q = as_t(q_pm.reshape(K * B, V)).pin_memory()
        self.h_t = as_t(t_sorted).pin_memory()
        self.h_ud = torch.from_numpy(ud_pm.reshape(-1)).pin_memory()
        self.h_uv = torch.from_numpy(uv_sorted).pin_memory()
        self.h_len = torch.from_numpy(lens).pin_memory()
        dev = torch.device("cuda", torch.cuda.current_device())
        self.d_q = torch.empty_like(self.h_q, device=dev)
        self.d_t = torch.empty_like(self.h_t, device=dev)
        self.d_ud = torch.empty_like(self.h_ud, device=dev)
        self.d_uv = torch.empty_like(self.h_uv, device=dev)
        self.d_len = torch.empty_like(self.h_len, device=dev)
        self.d_tok = torch.zeros(K * B, dtype=torch.int32, device=dev)
        self.d_ent = torch.zeros(K * B, dtype=torch.float32, device=dev)
        self.d_stop = torch.zeros(K * B, dtype=torch.uint8, device=dev)
        self.d_stats = torch.zeros(K * B, 2, dtype=torch.float32, device=dev)
        self.d_cu = torch.zeros(B + 1, dtype=torch.int32, device=dev)
        self.d_nacc = torch.zeros(B, dtype=torch.int32, device=dev)
        self.d_next = torch.zeros(B, dtype=torch.int32, device=dev)
        self.h_nacc = torch.zeros(B, dtype=torch.int32).pin_memory()
        self.h_next = torch.zeros(B, dtype=torch.int32).pin_memory()
        self.h_stop = torch.zeros(K * B, dtype=torch.uint8).pin_memory()
        self.h_tok = torch.zeros(K * B, dtype=torch.int32).pin_memory()
        self.esz = w.elem_bytes
        self.dt = 1 if w.dtype == "bf16" else 0
        self.upload()
        self.prepare()
        torch.cuda.synchronize()

    def upload(self):
        """Host -> device copy of one step's inputs (active rows only); returns the bytes copied."""
        n = 0
        B = self.B
        for j in range(self.K):
            a = int(self.active[j])
            self.d_q[j * B:j * B + a].copy_(self.h_q[j * B:j * B + a], non_blocking=True)
            n += a * self.V * self.esz
        for d, h in ((self.d_t, self.h_t), (self.d_ud, self.h_ud), (self.d_uv, self.h_uv), (self.d_len, self.h_len)):
            d.copy_(h, non_blocking=True)
            n += h.numel() * h.element_size()
        return n

    def download(self):
        """Device -> host read of the step's results; returns the bytes copied."""
        n = 0
        for h, d in ((self.h_nacc, self.d_nacc), (self.h_next, self.d_next), (self.h_stop, self.d_stop),
                     (self.h_tok, self.d_tok)):
            h.copy_(d, non_blocking=True)
            n += h.numel() * h.element_size()
        return n

    def prepare(self):
        """Pre-marshals the calls of one step (the pointers and shapes never change)."""
        ctx, w, B, V, sp = self.ctx, self.w, self.B, self.V, self.stream
        q, ud, tok, ent = self.d_q.data_ptr(), self.d_ud.data_ptr(), self.d_tok.data_ptr(), self.d_ent.data_ptr()
        stop, stats = self.d_stop.data_ptr(), self.d_stats.data_ptr()
        calls = []
        for j in range(self.K):
            o = j * B
            calls.append(ctx.bind("draft_step", q + o * V * self.esz, self.dt, int(self.active[j]), V, V, w.T, w.h,
                                  ud + 4 * o, tok + 4 * o, ent + 4 * o, stop + o, stats + 8 * o, sp))
        calls.append(ctx.bind("pack_ragged", self.d_len, B, w.K_max, self.d_cu, None, None, sp))
        calls.append(ctx.bind("verify", self.d_tok, self.d_q, V, self.d_stats, 1, B, self.d_t, V, self.dt,
                              self.d_cu, B, w.K_max, self.Rp, V, w.T, self.d_uv, self.d_nacc, self.d_next, sp))
        self.calls = calls

    def step(self, draft_events=None):
        """One round.  draft_events = (before, after): torch events recorded on the launching stream
        around the draft-step launches of this round."""
        if draft_events is None:
            for c in self.calls:
                c()
            return
        draft_events[0].record()
        for c in self.calls[:-2]:
            c()
        draft_events[1].record()
        self.calls[-2]()
        self.calls[-1]()

    def logits_bytes(self):
        """Algorithmic logits bytes of one step (needs the results of a finished step)."""
        self.torch.cuda.synchronize()
        nacc = self.d_nacc.cpu().numpy()
        rejected = int((nacc < self.lens).sum())
        rows = int(self.lens.sum()) + self.Rp + rejected
        return rows * self.V * self.esz, rejected

    def results_by_sequence(self):
        """The last step's outputs in the workload's own indexing: per packed draft row (token, entropy,
        stop flag) and per sequence (n_accepted, next_token)."""
        self.torch.cuda.synchronize()
        w, B = self.w, self.B
        tok = self.d_tok.cpu().numpy().reshape(self.K, B); ent = self.d_ent.cpu().numpy().reshape(self.K, B)
        stop = self.d_stop.cpu().numpy().reshape(self.K, B)
        nacc = self.d_nacc.cpu().numpy(); nxt = self.d_next.cpu().numpy()
        out = {"token": np.zeros(w.n_draft_rows, np.int64), "entropy": np.zeros(w.n_draft_rows),
               "stop": np.zeros(w.n_draft_rows, np.uint8), "n_accepted": np.zeros(B, np.int64),
               "next_token": np.zeros(B, np.int64)}
        for k, i in enumerate(self.order):
            n = int(self.lens[k]); r0 = int(w.cu_rows[i]) - int(i)
            out["token"][r0:r0 + n] = tok[:n, k]; out["entropy"][r0:r0 + n] = ent[:n, k]
            out["stop"][r0:r0 + n] = stop[:n, k]
            out["n_accepted"][i] = nacc[k]; out["next_token"][i] = nxt[k]
        return out

    def check_stop_flags(self):
        """The stop rule must reproduce the workload's draft lengths (generator contract)."""
        stop = self.d_stop.cpu().numpy().reshape(self.K, self.B)
        for k in range(self.B):
            n = int(self.lens[k])
            if stop[:n - 1, k].any() or not (stop[n - 1, k] == 1 or n == self.w.K_max):
                return False
        return True


def b1_latency(ctx, torch):
    """us per replay of a CUDA graph holding a whole B = 1 round of the `tiny` workload."""
    w = workloads.make_workload("tiny")
    st = torch.cuda.Stream()
    K, V = w.K_max, w.V
    dq = torch.from_numpy(w.q_logits).cuda(); dt = torch.from_numpy(w.target_logits).cuda()
    ud = torch.from_numpy(w.draft_uniforms).cuda(); uv = torch.from_numpy(w.verify_uniforms).cuda()
    tok = torch.zeros(K, dtype=torch.int32, device="cuda"); ent = torch.zeros(K, device="cuda")
    stop = torch.zeros(K, dtype=torch.uint8, device="cuda"); stats = torch.zeros(K, 2, device="cuda")
    lens = torch.tensor([K], dtype=torch.int32, device="cuda"); cu = torch.zeros(2, dtype=torch.int32, device="cuda")
    nacc = torch.zeros(1, dtype=torch.int32, device="cuda"); nxt = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()

    def enqueue(s, verify=None):
        for j in range(K):
            ctx.draft_step(dq.data_ptr() + j * V * 4, 0, 1, V, V, w.T, w.h, ud.data_ptr() + 4 * j,
                           tok.data_ptr() + 4 * j, ent.data_ptr() + 4 * j, stop.data_ptr() + j,
                           stats.data_ptr() + 8 * j, s)
        ctx.pack_ragged(lens, 1, K, cu, None, None, s)
        (verify or ctx.verify)(tok, dq, V, stats, -1, 0, dt, V, 0, cu, 1, K, K + 1, V, w.T, uv, nacc, nxt, s)

    out = {}
    with torch.cuda.stream(st):
        ctx.graph_begin(st); enqueue(st); g = ctx.graph_end(st)
        ctx.graph_begin(st); enqueue(st, ctx.verify_early_exit); ge = ctx.graph_end(st)
        one = None
        ctx.graph_begin(st)
        ctx.draft_step(dq, 0, 1, V, V, w.T, w.h, ud, tok, ent, stop, stats, st)
        one = ctx.graph_end(st)
        for name, graph, reps in (("round_us", g, 200), ("round_early_exit_us", ge, 200), ("draft_step_us", one, 500)):
            for _ in range(20):
                graph.launch(st)
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            st.synchronize()
            e0.record(st)
            for _ in range(reps):
                graph.launch(st)
            e1.record(st)
            st.synchronize()
            out[name] = 1000.0 * e0.elapsed_time(e1) / reps
            # launch to result visible on the host: one replay, then wait for it, timed on the host clock
            t0 = time.perf_counter()
            for _ in range(reps):
                graph.launch(st)
                st.synchronize()
            out[name.replace("_us", "_to_host_us")] = 1e6 * (time.perf_counter() - t0) / reps
        out["accepted_in_this_round"] = int(nacc.item())
        g.destroy(); ge.destroy(); one.destroy()

        # one truncated draft step (top-k 50, top-p 0.9) at B = 1, by graph replay
        thr1 = torch.zeros(1, device="cuda")
        st.synchronize()
        ctx.graph_begin(st)
        ctx.draft_step_truncated(dq, 0, 1, V, V, w.T, w.h, 50, 0.9, ud, None, thr1, tok, ent, stop, stats, st)
        tg = ctx.graph_end(st)
        for _ in range(20):
            tg.launch(st)
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        st.synchronize()
        e0.record(st)
        for _ in range(500):
            tg.launch(st)
        e1.record(st)
        st.synchronize()
        out["truncated_draft_step_us"] = 1000.0 * e0.elapsed_time(e1) / 500
        tg.destroy()

        # the drafting phase as a loop inside the graph (each token: draft step at the sequence's own
        # position + the policy kernel that also decides the loop), against the same two kernels
        # driven from the host, which must read the count of drafting sequences back after every token
        gamma = torch.tensor([K], dtype=torch.int32, device="cuda"); dlen = torch.zeros(1, dtype=torch.int32, device="cuda")
        act = torch.ones(1, dtype=torch.uint8, device="cuda"); nact = torch.zeros(1, dtype=torch.int32, device="cuda")
        stop1 = torch.zeros(1, dtype=torch.uint8, device="cuda")
        st.synchronize()
        CONSTANT = 1
        # `unroll` tokens per loop iteration: the loop node costs a few microseconds per iteration, which a
        # body of several (masked) steps spreads over as many tokens
        for unroll, key in ((1, "draft_loop_us_per_token"), (4, "draft_loop_unrolled4_us_per_token")):
            ctx.graph_begin(st)
            ctx.policy_update(CONSTANT, None, dlen, gamma, act, 1, K, st)
            body = ctx.graph_loop_begin(st, nact, K)
            for _ in range(unroll):
                ctx.draft_step_at(dq, 0, 1, V, V, V, dlen, 1, w.T, w.h, ud, act, tok, ent, stop1, stats, body)
                ctx.policy_advance(CONSTANT, stop1, gamma, dlen, act, 1, K, nact, body)
            ctx.graph_loop_end()
            loop = ctx.graph_end(st)
            for _ in range(20):
                loop.launch(st)
            st.synchronize()
            assert int(dlen.item()) == K
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(st)
            for _ in range(200):
                loop.launch(st)
            e1.record(st)
            st.synchronize()
            out[key] = 1000.0 * e0.elapsed_time(e1) / 200 / K
            loop.destroy()

        def host_loop():
            ctx.policy_update(CONSTANT, None, dlen, gamma, act, 1, K, st)
            n = 0
            while True:
                ctx.draft_step_at(dq, 0, 1, V, V, V, dlen, 1, w.T, w.h, ud, act, tok, ent, stop1, stats, st)
                ctx.policy_advance(CONSTANT, stop1, gamma, dlen, act, 1, K, nact, st)
                n += 1
                if int(nact.item()) == 0:      # device -> host read, once per token
                    return n
        for _ in range(5):
            host_loop()
        t0 = time.perf_counter()
        n = sum(host_loop() for _ in range(50))
        st.synchronize()
        out["host_loop_us_per_token"] = 1e6 * (time.perf_counter() - t0) / n
    out["kernels_per_round"] = K + 3
    return out


def truncated_round(ctx, torch, rnd, top_k=50, top_p=0.9, reps=10):
    """The same round with top-k / nucleus truncated distributions, on the resident buffers of `rnd`:
    thresholds of the draft rows of every step and of all target rows, truncated draft steps, truncated
    verify.  Returns us per part and the logits GB/s of the whole truncated round."""
    w, B, V, K = rnd.w, rnd.B, rnd.V, rnd.K
    if not w.T > 0:
        return None
    sp = rnd.stream
    dev = rnd.d_q.device
    q_thr = torch.zeros(K * B, device=dev); p_thr = torch.zeros(rnd.Rp, device=dev)
    p_stats = torch.zeros(rnd.Rp, 2, device=dev)
    q, ud, tok, ent = rnd.d_q.data_ptr(), rnd.d_ud.data_ptr(), rnd.d_tok.data_ptr(), rnd.d_ent.data_ptr()
    stop, stats = rnd.d_stop.data_ptr(), rnd.d_stats.data_ptr()
    thr_calls, draft_calls, one_calls = [], [], []
    for j in range(K):
        o = j * B
        a = int(rnd.active[j])
        thr_calls.append(ctx.bind("row_threshold", q + o * V * rnd.esz, rnd.dt, a, V, V, w.T, top_k, top_p,
                                  q_thr.data_ptr() + 4 * o, None, sp))
        draft_calls.append(ctx.bind("draft_step_filtered", q + o * V * rnd.esz, rnd.dt, a, V, V, w.T, w.h, ud + 4 * o,
                                    None, q_thr.data_ptr() + 4 * o, tok + 4 * o, ent + 4 * o, stop + o,
                                    stats + 8 * o, sp))
        one_calls.append(ctx.bind("draft_step_truncated", q + o * V * rnd.esz, rnd.dt, a, V, V, w.T, w.h, top_k, top_p,
                                  ud + 4 * o, None, q_thr.data_ptr() + 4 * o, tok + 4 * o, ent + 4 * o, stop + o,
                                  stats + 8 * o, sp))
    t_thr = ctx.bind("row_threshold", rnd.d_t, rnd.dt, rnd.Rp, V, V, w.T, top_k, top_p, p_thr, p_stats, sp)
    pack = ctx.bind("pack_ragged", rnd.d_len, B, w.K_max, rnd.d_cu, None, None, sp)
    ver = ctx.bind("verify_filtered", rnd.d_tok, rnd.d_q, V, rnd.d_stats, q_thr, 1, B, rnd.d_t, V, p_thr, p_stats, rnd.dt,
                   rnd.d_cu, B, w.K_max, rnd.Rp, V, w.T, rnd.d_uv, rnd.d_nacc, rnd.d_next, sp)

    def timed(calls):
        for c in calls:
            c()
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            for c in calls:
                c()
        e1.record()
        torch.cuda.synchronize()
        return 1000.0 * e0.elapsed_time(e1) / reps

    out = {"top_k": top_k, "top_p": top_p,
           "draft_thresholds_us": timed(thr_calls), "draft_steps_us": timed(draft_calls),
           "draft_steps_one_call_us": timed(one_calls),
           "target_thresholds_us": timed([t_thr]), "verify_us": timed([pack, ver])}
    whole = one_calls + [t_thr, pack, ver]
    out["round_us"] = timed(whole)
    nbytes, _ = rnd.logits_bytes()
    out["logits_GBps"] = nbytes / (out["round_us"] * 1e-6) / 1e9
    out["threshold_passes_per_row"] = "2 (top_k small against the threads of a cluster: candidate path)"
    return out


def pair_stats_leg(ctx, torch, rnd, peak, reps=10):
    """The analysis quantities (Eq. 1-6) of every (draft row, target row under it) pair of the round, on
    contiguous copies of the resident rows (gathered outside the timed region).  Algorithmic bytes: both rows of
    a pair once.  Two forms: svip_pair_stats (normalisers computed inside: the rows are streamed twice) and
    svip_pair_stats_given with the normalisers a round has anyway (the draft step's row_stats; for the target
    rows one svip_row_threshold pass with nothing cut, timed beside it)."""
    w, B, V = rnd.w, rnd.B, rnd.V
    if not w.T > 0:
        return None
    rnd.step()          # the draft rows' normalisers of the plain round (other legs reuse the buffer)
    torch.cuda.synchronize()
    dev = rnd.d_q.device
    cu = np.concatenate([[0], np.cumsum(rnd.lens.astype(np.int64) + 1)])
    q_idx = np.concatenate([np.arange(rnd.lens[k]) * B + k for k in range(B)])
    t_idx = np.concatenate([cu[k] + np.arange(rnd.lens[k]) for k in range(B)])
    n = int(q_idx.size)
    qi = torch.from_numpy(q_idx).to(dev)
    q = rnd.d_q.index_select(0, qi)
    t = rnd.d_t.index_select(0, torch.from_numpy(t_idx).to(dev))
    q_stats = rnd.d_stats.index_select(0, qi).contiguous()
    p_stats = torch.zeros(n, 2, device=dev); thr = torch.zeros(n, device=dev)
    out = torch.zeros(n, 8, device=dev)
    calls = {"pair_stats": ctx.bind("pair_stats", q, V, t, V, rnd.dt, n, V, w.T, 0.18, out, rnd.stream),
             "target_normalisers": ctx.bind("row_threshold", t, rnd.dt, n, V, V, w.T, 0, 1.0, thr, p_stats, rnd.stream),
             "pair_stats_given": ctx.bind("pair_stats_given", q, V, q_stats, t, V, p_stats, rnd.dt, n, V, w.T, 0.18,
                                          out, rnd.stream)}
    nbytes = 2 * n * V * rnd.esz
    res = {"pairs": n, "algorithmic_bytes": nbytes}
    for name, call in calls.items():
        call()
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            call()
        e1.record()
        torch.cuda.synchronize()
        us = 1000.0 * e0.elapsed_time(e1) / reps
        if name == "target_normalisers":
            res[name + "_us"] = us
            continue
        o = out.cpu().numpy()
        res[name] = {"us_per_call": us, "GBps": nbytes / (us * 1e-6) / 1e9,
                     "frac_of_measured_peak": nbytes / (us * 1e-6) / 1e9 / peak,
                     "mean_beta": float(o[:, 0].mean()), "mean_H_q": float(o[:, 1].mean()),
                     "nan_outputs": int(np.isnan(o).sum())}
    return res


def graph_loop_round(ctx, torch, rnd, reps=20):
    """The same round as one CUDA graph whose drafting phase is a loop on the device (Algorithm 1's do-while):
    every iteration is one svip_draft_step_at over all sequences at their own positions (finished ones masked)
    and the entropy policy, which also decides the loop; then packing from the device-side draft lengths and
    svip_verify.  No host round trip and no host launch per draft position."""
    w, B, V, K = rnd.w, rnd.B, rnd.V, rnd.K
    if not w.T > 0:
        return None
    dev = rnd.d_q.device
    st = torch.cuda.Stream()
    dlen = torch.zeros(B, dtype=torch.int32, device=dev); act = torch.ones(B, dtype=torch.uint8, device=dev)
    nact = torch.zeros(1, dtype=torch.int32, device=dev); stop1 = torch.zeros(B, dtype=torch.uint8, device=dev)
    ENTROPY = 0
    rnd.step()
    torch.cuda.synchronize()
    want_nacc = rnd.d_nacc.clone(); want_next = rnd.d_next.clone()
    with torch.cuda.stream(st):
        ctx.graph_begin(st)
        ctx.policy_update(ENTROPY, None, dlen, None, act, B, w.K_max, st)
        body = ctx.graph_loop_begin(st, nact, w.K_max)
        ctx.draft_step_at(rnd.d_q, rnd.dt, B, V, V, B * V, dlen, B, w.T, w.h, rnd.d_ud, act, rnd.d_tok, rnd.d_ent,
                          stop1, rnd.d_stats, body)
        ctx.policy_advance(ENTROPY, stop1, None, dlen, act, B, w.K_max, nact, body)
        ctx.graph_loop_end()
        ctx.pack_ragged(dlen, B, w.K_max, rnd.d_cu, None, None, st)
        ctx.verify(rnd.d_tok, rnd.d_q, V, rnd.d_stats, 1, B, rnd.d_t, V, rnd.dt, rnd.d_cu, B, w.K_max, rnd.Rp, V, w.T,
                   rnd.d_uv, rnd.d_nacc, rnd.d_next, st)
        g = ctx.graph_end(st)
        for _ in range(3):
            g.launch(st)
        st.synchronize()
        same = bool(torch.equal(dlen.cpu(), torch.from_numpy(rnd.lens)) and torch.equal(rnd.d_nacc, want_nacc)
                    and torch.equal(rnd.d_next, want_next))
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for _ in range(reps):
            g.launch(st)
        e1.record(st)
        st.synchronize()
        us = 1000.0 * e0.elapsed_time(e1) / reps
        g.destroy()
    nbytes, _ = rnd.logits_bytes()
    return {"us_per_round": us, "logits_GBps": nbytes / (us * 1e-6) / 1e9, "loop_iterations": int(rnd.lens.max()),
            "same_results_as_host_driven_round": same}


def early_exit_leg(ctx, torch, rnd, reps=10):
    """The round with svip_verify_early_exit in place of svip_verify: the target rows of a sequence are read in order
    up to its first rejection.  Times the verify call alone in both forms and the whole round in both forms; counts
    the target rows the early-exit form needs (n_accepted + 1 per sequence)."""
    w, B, V = rnd.w, rnd.B, rnd.V
    rnd.step()
    torch.cuda.synchronize()
    plain = (rnd.d_nacc.clone(), rnd.d_next.clone())
    early = ctx.bind("verify_early_exit", rnd.d_tok, rnd.d_q, V, rnd.d_stats, 1, B, rnd.d_t, V, rnd.dt, rnd.d_cu, B,
                     w.K_max, rnd.Rp, V, w.T, rnd.d_uv, rnd.d_nacc, rnd.d_next, rnd.stream)

    def timed(calls):
        for c in calls:
            c()
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            for c in calls:
                c()
        e1.record()
        torch.cuda.synchronize()
        return 1000.0 * e0.elapsed_time(e1) / reps

    res = {"verify_us": timed(rnd.calls[-1:]), "verify_early_exit_us": timed([early]),
           "round_us": timed(rnd.calls), "round_early_exit_us": timed(rnd.calls[:-1] + [early])}
    nacc = rnd.d_nacc.cpu().numpy()
    res["target_rows"] = rnd.Rp
    res["target_rows_needed"] = int((nacc + 1).sum())
    res["same_n_accepted"] = int((rnd.d_nacc == plain[0]).sum())
    res["same_next_token"] = int((rnd.d_next == plain[1]).sum())
    res["sequences"] = B
    res["note"] = ("one kernel, one cluster per sequence; the rows of a sequence are read one after another, so it "
                   "pays where rejections come early or the batch fills the GPU")
    rnd.step()      # leave the plain round's results in the buffers
    torch.cuda.synchronize()
    return res


def tree_leg(ctx, torch, reps=20):
    """svip_verify_tree on synthetic candidate trees: 64 sequences, binary trees of depth 3 (14 candidate
    nodes: the two most likely tokens of every node's draft row), V = 32000 bf16, target = draft + N(0, 0.5^2)."""
    B, V, T = 64, 32000, 1.0
    parent = [-1, -1] + [i // 2 - 1 for i in range(4, 16)]       # nodes 2k, 2k+1 are the children of node k-1
    N = len(parent)
    g = torch.Generator(device="cuda").manual_seed(20241118)
    q = torch.randn(B * (N + 1), V, device="cuda", generator=g) * 2.0
    t = q + torch.randn(B * (N + 1), V, device="cuda", generator=g) * 0.5
    top2 = q.view(B, N + 1, V).topk(2, dim=2).indices                 # [B, N+1, 2]
    par = torch.tensor(parent, device="cuda")
    tokens = torch.stack([top2[:, parent[i] + 1, i % 2] for i in range(N)], dim=1).to(torch.int32).contiguous()
    parent_t = par.to(torch.int32).repeat(B, 1).contiguous()
    qb = q.to(torch.bfloat16).view(torch.int16); tb = t.to(torch.bfloat16).view(torch.int16)
    u = torch.rand(B, N + 1, device="cuda", generator=g)
    n_acc = torch.zeros(B, dtype=torch.int32, device="cuda"); path = torch.zeros(B, N, dtype=torch.int32, device="cuda")
    nxt = torch.zeros(B, dtype=torch.int32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    call = ctx.bind("verify_tree", tokens, parent_t, qb, V, None, tb, V, 1, B, N, V, T, u, n_acc, path, nxt, st)
    before = ctx.launch_count()
    call()
    kernels = ctx.launch_count() - before
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        call()
    e1.record()
    torch.cuda.synchronize()
    us = 1000.0 * e0.elapsed_time(e1) / reps
    rows_bytes = 2 * B * (N + 1) * V * 2
    return {"sequences": B, "nodes": N, "V": V, "dtype": "bf16", "us_per_call": us, "kernels": kernels,
            "mean_accepted": float(n_acc.float().mean()), "normaliser_passes_GBps": rows_bytes / (us * 1e-6) / 1e9,
            "note": "two passes of row statistics over all 2 x B x (N+1) rows, then the walk (a chain of passes over "
                    "single row pairs: latency-bound)"}


def vocab_parallel_leg(ctx, torch, rnd, peak, G=8, reps=20):
    """One rank's share of a vocabulary-parallel draft step over the first draft launch of the round: the rows'
    columns cut into G shards, this rank holding shard 0 (svip_vp_partial on the shard, svip_vp_combine on the G
    partials, svip_vp_locate on the shard).  The two small collectives between them need G GPUs and are not timed."""
    from paper_2411_18462_b200 import vocab_parallel as VP
    w, V = rnd.w, rnd.V
    B = int(rnd.active[0])
    dev = rnd.d_q.device
    sp = rnd.stream
    partials = torch.zeros(G, B, 4, device=dev)
    for r in range(G):
        lo, hi = VP.shard_bounds(V, G, r)
        ctx.vp_partial(rnd.d_q.data_ptr() + lo * rnd.esz, rnd.dt, B, hi - lo, V, w.T, lo, partials[r], sp)
    lo, hi = VP.shard_bounds(V, G, 0)
    ent = torch.zeros(B, device=dev); stop = torch.zeros(B, dtype=torch.uint8, device=dev)
    tok = torch.zeros(B, dtype=torch.int32, device=dev); owner = torch.zeros(B, dtype=torch.int32, device=dev)
    tgt = torch.zeros(B, device=dev); act = torch.zeros(B, dtype=torch.uint8, device=dev)
    calls = [ctx.bind("vp_partial", rnd.d_q, rnd.dt, B, hi - lo, V, w.T, lo, partials[0], sp),
             ctx.bind("vp_combine", partials, G, 0, B, w.T, w.h, rnd.d_ud, ent, stop, tok, owner, tgt, act, sp)]
    if w.T > 0:
        calls.append(ctx.bind("vp_locate", rnd.d_q, rnd.dt, B, hi - lo, V, w.T, tgt, act, lo, tok, sp))
    for c in calls:
        c()
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        for c in calls:
            c()
    e1.record()
    torch.cuda.synchronize()
    us = 1000.0 * e0.elapsed_time(e1) / reps
    owned = int(act.sum().item())
    nbytes = (B + owned) * (hi - lo) * rnd.esz          # the shard once, the owned rows' shard once more
    return {"ranks_emulated": G, "rows": B, "shard_columns": hi - lo, "rows_owned_by_this_rank": owned,
            "us_per_step_on_one_rank": us, "shard_GBps": nbytes / (us * 1e-6) / 1e9,
            "frac_of_measured_peak": nbytes / (us * 1e-6) / 1e9 / peak, "kernels": len(calls)}


CDF_TOL = 1e-5        # a sampled token may differ from the oracle's only across a CDF boundary closer than this
ACCEPT_GUARD = 1e-4   # an accept decision may differ only if the draw is this close to the acceptance probability
STOP_GUARD = 1e-3     # a stop flag may differ only if sqrt(H) is this close to h
ENTROPY_ATOL = 1e-4


def _within_cdf_tolerance(weights, u, token):
    c = np.cumsum(np.asarray(weights, dtype=np.float64))
    total = c[-1]
    if not total > 0 or not (0 <= token < len(c)) or not weights[token] > 0:
        return False
    lo = (c[token - 1] if token > 0 else 0.0) / total
    return bool(lo - CDF_TOL <= float(u) <= c[token] / total + CDF_TOL)


def _oracle_sample(w, n_seq):
    """The first n_seq sequences of the workload as packed arrays of their own."""
    sel = list(range(n_seq))
    rows_q = np.concatenate([np.arange(w.cu_rows[i] - i, w.cu_rows[i] - i + w.draft_len[i]) for i in sel])
    rows_t = np.concatenate([np.arange(w.cu_rows[i], w.cu_rows[i + 1]) for i in sel])
    lens = w.draft_len[sel]
    cu = np.concatenate([[0], np.cumsum(lens.astype(np.int64) + 1)])
    return {"rows_q": rows_q, "rows_t": rows_t, "lens": lens, "cu": cu,
            "q": np.ascontiguousarray(w.q_logits[rows_q]), "t": np.ascontiguousarray(w.target_logits[rows_t]),
            "ud": w.draft_uniforms[rows_q], "uv": w.verify_uniforms[rows_t]}


def _oracle_pass(O, w, s, threads):
    """One pass of the oracle over a sample: every draft row, then the verification round.  Returns
    (seconds, algorithmic bytes, results)."""
    t0 = time.perf_counter()
    tok, H, stop = O.draft_step(s["q"], w.T, w.h, s["ud"], threads=threads)
    nacc, nxt, _ = O.verify(tok.astype(np.int32), s["q"], s["t"], s["cu"], w.T, s["uv"], threads=threads)
    dt = time.perf_counter() - t0
    rejected = int((nacc < s["lens"]).sum())
    nbytes = (len(s["rows_q"]) + len(s["rows_t"]) + rejected) * w.V * w.elem_bytes
    return dt, nbytes, (tok, H, stop, nacc, nxt)


def _boundary_checks(O, w, s, oracle_out, gpu, threads):
    """Untimed comparison of the GPU's last step with the oracle on the sample: how many results are identical
    and how many of the others fall inside the stated tolerances (and are therefore allowed to differ)."""
    tok, H, stop, nacc, nxt = oracle_out
    rq = s["rows_q"]
    g_tok, g_H, g_stop = gpu["token"][rq], gpu["entropy"][rq], gpu["stop"][rq]
    out = {"draft_rows": int(len(rq)), "sequences": int(len(s["lens"]))}
    out["entropy_max_abs_err"] = float(np.max(np.abs(g_H - H)))
    near = np.abs(np.sqrt(H) - w.h) <= STOP_GUARD
    out["stop_near_threshold"] = int(near.sum())
    out["stop_flags_wrong"] = int((g_stop[~near] != stop[~near]).sum())
    bad = np.nonzero(g_tok != tok)[0]
    out["draft_tokens_identical"] = int(len(rq) - bad.size)
    tb = beyond = 0
    for r in bad:
        if w.T > 0 and _within_cdf_tolerance(O.softmax(s["q"][r], w.T), s["ud"][r], int(g_tok[r])):
            tb += 1
        else:
            beyond += 1
    out["token_boundary"] = tb
    out["draft_tokens_beyond_tolerance"] = beyond
    # verification: only sequences whose draft tokens are the oracle's can be compared
    cu, lens = s["cu"], s["lens"]
    same_draft = np.array([np.array_equal(g_tok[cu[i] - i: cu[i] - i + lens[i]], tok[cu[i] - i: cu[i] - i + lens[i]])
                           for i in range(len(lens))])
    out["sequences_not_compared"] = int((~same_draft).sum())
    inside = wrong = n_same = nx_same = nx_boundary = nx_beyond = 0
    guard_draws = 0
    aprob = None
    if w.T > 0:
        _, _, aprob = O.verify(tok.astype(np.int32), s["q"], s["t"], cu, w.T, s["uv"], want_accept_prob=True,
                               threads=threads)
        for i, a in enumerate(aprob):
            r = s["uv"][cu[i]: cu[i] + lens[i]].astype(np.float64)
            guard_draws += int(((np.abs(r - a) < ACCEPT_GUARD) & (a < 1.0)).sum())
    for i in np.nonzero(same_draft)[0]:
        gn, gx = int(gpu["n_accepted"][i]), int(gpu["next_token"][i])
        if gn != nacc[i]:
            j = min(gn, int(nacc[i]))
            ok = aprob is not None and abs(float(s["uv"][cu[i] + j]) - aprob[i][j]) < ACCEPT_GUARD
            inside += int(ok); wrong += int(not ok)
            continue
        n_same += 1
        if gx == nxt[i]:
            nx_same += 1
            continue
        ok = False
        if w.T > 0:
            p = O.softmax(s["t"][cu[i] + nacc[i]], w.T)
            wts = p
            if nacc[i] < lens[i]:
                wts, S = O.residual(p, O.softmax(s["q"][cu[i] - i + nacc[i]], w.T))
                if not S > 0:
                    wts = p
            ok = _within_cdf_tolerance(wts, s["uv"][cu[i] + lens[i]], gx)
        nx_boundary += int(ok); nx_beyond += int(not ok)
    out.update({"accept_draws_inside_guard": guard_draws, "n_accepted_identical": n_same,
                "n_accepted_decided_inside_guard": inside, "n_accepted_wrong": wrong,
                "next_identical": nx_same, "next_boundary": nx_boundary, "next_beyond_tolerance": nx_beyond})
    out["tolerances"] = {"entropy_abs": ENTROPY_ATOL, "cdf": CDF_TOL, "accept_guard": ACCEPT_GUARD, "stop_guard": STOP_GUARD}
    out["ok"] = bool(out["entropy_max_abs_err"] <= ENTROPY_ATOL and out["stop_flags_wrong"] == 0 and beyond == 0
                     and wrong == 0 and nx_beyond == 0)
    return out


def cpu_baseline(w, gpu_results=None, passes=3):
    """The fp64 oracle, as it stands, on a bounded sample of the same workload, on all host cores: median of
    `passes` passes.  With the GPU's results of the same sequences, an untimed comparison follows (`checks`:
    identical results and boundary cases, counted)."""
    from oracle import svip_oracle as O
    cores = len(os.sched_getaffinity(0))
    # about 4500 rows: a few seconds of CPU work per pass
    rows_per_seq = 2.0 * float(w.draft_len.mean()) + 1.0
    n_seq = min(w.B, max(64, int(round(4500.0 / rows_per_seq))))
    s = _oracle_sample(w, n_seq)
    O.lib()
    runs = [_oracle_pass(O, w, s, cores) for _ in range(passes)]
    runs.sort(key=lambda r: r[0])
    dt, nbytes, res = runs[len(runs) // 2]
    n_rows = len(s["rows_q"]) + len(s["rows_t"])
    # the same on one thread, over a sixteenth of the sample (whole sequences)
    n1 = max(1, n_seq // 16)
    s1 = _oracle_sample(w, n1)
    dt1, bytes1, _ = _oracle_pass(O, w, s1, 1)
    out = {"value": nbytes / dt / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
           "sample": "%d of %d sequences (%d draft + %d target rows), median of %d passes, %.2f s per pass" % (
               n_seq, w.B, len(s["rows_q"]), len(s["rows_t"]), passes, dt),
           "rows_per_s": n_rows / dt, "us_per_step": 1e6 * dt * (w.B / n_seq),
           "us_per_step_note": "one pass scaled to the whole batch (%d sequences)" % w.B,
           "single_thread_value": bytes1 / dt1 / 1e9,
           "single_thread_sample": "%d sequences (%d rows), one pass, %.1f s" % (
               n1, len(s1["rows_q"]) + len(s1["rows_t"]), dt1)}
    checks = _boundary_checks(O, w, s, res, gpu_results, cores) if gpu_results is not None else None
    return out, checks


# --------------------------------------------------------------------------- timing one workload

def measure(ctx, torch, dist, world, rnd, steps, warmup):
    """`warmup` untimed rounds, then `steps` timed ones (CUDA events on the launching stream, barrier and
    synchronize on both sides).  The row-statistics kernel is timed by the library's event pair around its
    launch, the draft-step kernel as the mean over the draft launches of a round."""
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        rnd.step()
    step_bytes, rejected = rnd.logits_bytes()
    stops_ok = rnd.check_stop_flags()
    status = ctx.read_status(stream.cuda_stream)
    ctx.profile_enable(True)
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    n_timed = min(steps, 1024)
    draft_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_timed)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = ctx.launch_count()
    e0.record(stream)
    for k in range(steps):
        rnd.step(draft_ev[k] if k < n_timed else None)
    e1.record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    m = {"steps": steps, "step_bytes": step_bytes, "rejected": rejected, "stops_ok": stops_ok, "status": status,
         "launches": ctx.launch_count() - launches0, "local_ms": e0.elapsed_time(e1), "n_timed": n_timed,
         "draft_ms": sum(a.elapsed_time(b) for a, b in draft_ev)}
    m["stats_ms"], m["stats_n"] = ctx.profile_read()
    ctx.profile_enable(False)
    return m


def rooflines(w, rnd, m, total_ms, peak, peak_kind):
    """The two streaming kernels against the HBM roofline; the one with the larger share of the step first."""
    steps = m["steps"]
    stats_bytes = w.n_target_rows * w.V * w.elem_bytes
    stats_n, stats_ms = m["stats_n"], m["stats_ms"]
    stats_gbs = stats_bytes / (stats_ms / max(stats_n, 1) * 1e-3) / 1e9 if stats_n else None
    n_draft = rnd.K
    draft_bytes = w.n_draft_rows * w.V * w.elem_bytes / n_draft
    draft_us = m["draft_ms"] * 1e3 / max(m["n_timed"] * n_draft, 1)
    draft_gbs = draft_bytes / (draft_us * 1e-6) / 1e9
    dt_name = "bf16" if w.dtype == "bf16" else "f32"
    mode = "sampling" if w.T > 0 else "greedy"
    roof_stats = {"bound": "hbm", "kernel": "row_stats_kernel<%s> (target rows of svip_verify)" % dt_name,
                  "achieved": stats_gbs, "peak": peak, "peak_kind": "%s copy bandwidth" % peak_kind, "unit": "GB/s",
                  "frac": (stats_gbs / peak) if stats_gbs else None, "launches_timed": stats_n,
                  "bytes_per_launch": stats_bytes, "us_per_launch": stats_ms * 1e3 / max(stats_n, 1),
                  "share_of_step": stats_ms / max(stats_n, 1) / (total_ms / steps),
                  "traffic": ROW_STATS_TRAFFIC_PER_ALGORITHMIC_BYTE * stats_bytes
                  if (w.dtype == "bf16" and ROW_STATS_TRAFFIC_PER_ALGORITHMIC_BYTE) else None}
    roof_draft = {"bound": "hbm", "kernel": "draft_step_kernel<%s, %s> (mean over the %d launches of a round)"
                  % (dt_name, mode, n_draft), "achieved": draft_gbs, "peak": peak,
                  "peak_kind": "%s copy bandwidth" % peak_kind, "unit": "GB/s", "frac": draft_gbs / peak,
                  "launches_timed": m["n_timed"] * n_draft, "bytes_per_launch": draft_bytes, "us_per_launch": draft_us,
                  "share_of_step": m["draft_ms"] / m["n_timed"] / (total_ms / steps),
                  "traffic": DRAFT_F32_TRAFFIC_PER_ALGORITHMIC_BYTE * draft_bytes
                  if (w.dtype == "f32" and DRAFT_F32_TRAFFIC_PER_ALGORITHMIC_BYTE) else None}
    return (roof_draft, roof_stats) if roof_draft["share_of_step"] >= roof_stats["share_of_step"] \
        else (roof_stats, roof_draft)


def other_workload(ctx, torch, name, rank, peak, peak_kind, steps):
    """A short timed run of another published configuration on the same GPU (kept small: a few hundred ms)."""
    spec = workloads.SPECS[name]
    w = workloads.make_workload(name, seed=sharding.rank_seed(workloads.BASE_SEED + spec["index"], rank))
    rnd = Round(ctx, w, torch, torch.cuda.current_stream().cuda_stream)
    m = measure(ctx, torch, None, 1, rnd, steps, 3)
    ms = m["local_ms"]
    first, second = rooflines(w, rnd, m, ms, peak, peak_kind)
    keep = ("kernel", "achieved", "frac", "us_per_launch", "bytes_per_launch", "share_of_step", "launches_timed")
    out = {"workload": describe(w), "dtype": w.dtype, "steps": steps, "us_per_step": 1e3 * ms / steps,
           "logits_GBps": m["step_bytes"] * steps / (ms * 1e-3) / 1e9,
           "frac_of_measured_peak": m["step_bytes"] * steps / (ms * 1e-3) / 1e9 / peak,
           "kernels_per_step": m["launches"] // steps, "rejected_sequences": m["rejected"],
           "stop_flags_match_draft_lengths": bool(m["stops_ok"]) if name == "ragged" else None,
           "status_word": m["status"],
           "roofline": {k: first[k] for k in keep}, "roofline_other": {k: second[k] for k in keep}}
    try:
        out["early_exit"] = early_exit_leg(ctx, torch, rnd, reps=5)
    except Exception as exc:
        out["early_exit"] = {"error": repr(exc)}
    if name == "ragged":
        try:
            out["device_loop_graph"] = graph_loop_round(ctx, torch, rnd)
        except Exception as exc:
            out["device_loop_graph"] = {"error": repr(exc)}
    del rnd
    torch.cuda.empty_cache()
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2411_18462_b200 import Context, build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.cuda.current_device()
    if build.is_stale():
        build.build()
    spec = workloads.SPECS[args.workload]
    w = workloads.make_workload(args.workload, seed=sharding.rank_seed(workloads.BASE_SEED + spec["index"], rank),
                                B=args.batch)
    ctx = Context(dev, max(1 << 14, w.n_target_rows))
    stream = torch.cuda.current_stream()
    rnd = Round(ctx, w, torch, stream.cuda_stream)
    warmup = max(args.warmup, 3)

    # the clocks are sampled from before the warm-up until the end-to-end leg is over
    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
    sampler = ClockSampler(uuid)
    sampler.start()
    m = measure(ctx, torch, dist, world, rnd, args.steps, warmup)
    step_bytes = m["step_bytes"]
    total_ms, total_bytes = sharding.aggregate(m["local_ms"], step_bytes * args.steps, device=torch.device("cuda", dev))

    # end to end: host buffers in, results out, every step
    e2e_steps = 0 if (args.skip_extras or args.only_leg) else max(1, min(args.steps, 5))
    h2d = d2h = 0
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for _ in range(e2e_steps):
        h2d = rnd.upload()
        rnd.step()
        d2h = rnd.download()
        stream.synchronize()
    t1.record(stream)
    torch.cuda.synchronize()
    e2e_ms, e2e_bytes = sharding.aggregate(t0.elapsed_time(t1), step_bytes * e2e_steps, device=torch.device("cuda", dev))
    clocks = sampler.stop()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_kind = measured_peak()
    value = total_bytes / (total_ms * 1e-3) / 1e9
    dominant, other = rooflines(w, rnd, m, total_ms, peak, peak_kind)
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": describe(w), "sequences_per_gpu": w.B, "draft_rows": w.n_draft_rows,
                   "target_rows": w.n_target_rows, "rejected_sequences": m["rejected"],
                   "logits_bytes_per_step": step_bytes, "l2": "inputs (%.2f GB per step) larger than L2, no flush" % (step_bytes / 1e9),
                   "launch": "one stream, %d kernels per step" % (m["launches"] // max(args.steps, 1)),
                   "stop_flags_match_draft_lengths": bool(m["stops_ok"]) if w.name == "ragged" else None,
                   "status_word": m["status"]},
        "pct_of_hbm_peak_nominal": 100.0 * value / world / NOMINAL_HBM_GBS,
        "pct_of_hbm_peak_measured": 100.0 * value / world / peak,
        "us_per_step": 1e3 * total_ms / args.steps,
        "roofline": dominant, "roofline_other": other,
        "e2e": {"value": (e2e_bytes / (e2e_ms * 1e-3) / 1e9) if e2e_steps else None, "unit": "GB/s",
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": m["launches"], "clocks": clocks,
    }
    gpu_results = rnd.results_by_sequence()
    if args.only_leg:       # for profiling one of the extra legs without the others' launches
        legs = {"pair_stats": lambda: pair_stats_leg(ctx, torch, rnd, peak, reps=2),
                "vocab_parallel": lambda: vocab_parallel_leg(ctx, torch, rnd, peak, reps=2),
                "tree": lambda: tree_leg(ctx, torch, reps=2),
                "truncated": lambda: truncated_round(ctx, torch, rnd, reps=2),
                "early_exit": lambda: early_exit_leg(ctx, torch, rnd, reps=2)}
        line[args.only_leg] = legs[args.only_leg]()
        print(json.dumps(line))
        return
    if not args.skip_extras:
        try:
            line["b1"] = b1_latency(ctx, torch)
        except Exception as exc:   # the headline number does not depend on the latency probe
            line["b1"] = {"error": repr(exc)}
        try:
            line["truncated"] = truncated_round(ctx, torch, rnd)
        except Exception as exc:
            line["truncated"] = {"error": repr(exc)}
        for key, leg in (("pair_stats", lambda: pair_stats_leg(ctx, torch, rnd, peak)),
                         ("vocab_parallel", lambda: vocab_parallel_leg(ctx, torch, rnd, peak)),
                         ("early_exit", lambda: early_exit_leg(ctx, torch, rnd)),
                         ("tree", lambda: tree_leg(ctx, torch))):
            try:
                line[key] = leg()
            except Exception as exc:
                line[key] = {"error": repr(exc)}
    if not args.no_cpu_baseline and not args.skip_extras:
        line["cpu_baseline"], line["checks"] = cpu_baseline(w, gpu_results)
    if not args.skip_extras and world == 1 and args.batch is None:
        del rnd
        torch.cuda.empty_cache()
        line["other_workloads"] = {}
        for name in ("ragged", "reasoning"):
            if name == args.workload:
                continue
            try:
                line["other_workloads"][name] = other_workload(ctx, torch, name, rank, peak, peak_kind,
                                                               max(3, min(args.steps, 50)))
            except Exception as exc:
                line["other_workloads"][name] = {"error": repr(exc)}
    line["paper_context"] = ("end-to-end speedups over fixed draft length reported by the paper: up to 17% "
                             "(MT-Bench, 8K context) and 22% (QwQ long-form reasoning); hardware not stated")
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_reference(args):
    """The oracle as the reference arm, on the same workload.  A step is one pass of the oracle over a bounded
    sample of whole sequences: the whole batch when a pass takes about a second or less, else as many sequences
    (a multiple of the core count, never fewer than that) as keep the run within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import svip_oracle as O
    spec = workloads.SPECS[args.workload]
    cores = len(os.sched_getaffinity(0))
    w = workloads.make_workload(args.workload, seed=workloads.BASE_SEED + spec["index"], B=args.batch)
    O.lib()
    warmup = max(args.warmup, 1)
    # size the sample from one pass over `cores` sequences
    n0 = min(w.B, cores)
    dt0, _, _ = _oracle_pass(O, w, _oracle_sample(w, n0), cores)
    budget_s = 150.0
    per_seq = dt0 / n0
    n_seq = int(budget_s / max(args.steps + warmup, 1) / per_seq)
    n_seq = min(w.B, max(n0, (n_seq // cores) * cores))
    s = _oracle_sample(w, n_seq)
    for _ in range(warmup):
        _oracle_pass(O, w, s, cores)
    times, nbytes = [], 0
    t_all = time.perf_counter()
    for _ in range(args.steps):
        dt, nbytes, _ = _oracle_pass(O, w, s, cores)
        times.append(dt)
    total = time.perf_counter() - t_all
    value = nbytes * args.steps / total / 1e9
    med = float(np.median(times))
    n_rows = len(s["rows_q"]) + len(s["rows_t"])
    sample = "%d of %d sequences of the workload per step (%d draft + %d target rows)" % (
        n_seq, w.B, len(s["rows_q"]), len(s["rows_t"]))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": warmup, "ms_per_step": 1000.0 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": describe(w), "sample": sample, "whole_batch": bool(n_seq == w.B)},
        "median_step": {"GBps": nbytes / med / 1e9, "rows_per_s": n_rows / med, "us_per_step": 1e6 * med,
                        "us_per_whole_batch": 1e6 * med * w.B / n_seq},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="stress", choices=sorted(workloads.SPECS))
    ap.add_argument("--batch", type=int, default=None,
                    help="sequences per GPU instead of the published batch size (smaller cases for profiling)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only-leg", default=None, choices=["pair_stats", "vocab_parallel", "tree", "truncated", "early_exit"],
                    help="after the timed region run just this extra leg, briefly (for profiling it)")
    ap.add_argument("--skip-extras", action="store_true",
                    help="only the timed region: no end-to-end leg, no B=1 latency, no CPU baseline (for profiling)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
