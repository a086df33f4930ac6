#!/usr/bin/env python
"""Benchmark of the chunkwise hard-routing SMat prefill on B200.

One "step" is one pass of the whole hot path over one batch of seeded synthetic input:
smat_forward for the forward workloads, smat_forward + smat_backward for the fwd+bwd workload.
Prints ONE JSON line (rank 0).  `value` is prefill tokens/s with inputs resident in HBM; `e2e`
is the same metric through the C-ABI call with pinned HOST buffers (H2D of Q, K, V and D2H of O —
and of dQ, dK, dV — inside the timed region).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--no-sweep]
    python bench.py --impl reference ...      # the fp64 CPU oracle on a bounded sample of the same workload

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of the
workload: (batch, head) pairs share no data, so there is no collective on the data path
(weak scaling, `value` = N x tokens / max-over-ranks time).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2609_36062_b200 import replicas, roofline, synth  # noqa: E402

DEFAULT_WORKLOAD = "t16k_d4"
SWEEP = ["t4k_d3", "t64k_d1", "t64k_d2", "t64k_d3", "t64k_d4", "t8k_d3_fwdbwd", "t16k_d4_hashed", "t16k_d4_normalized",
         "t4k_d3_gated", "t4k_d3_gated_fwdbwd"]
METRIC = "SMat prefill tokens/s"
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant stage per step — the tabulation, one
# launch of radon_tc_kernel — from an ncu capture of the 8-head copy of the workload (351.3 MB read + 530.1 MB
# written), scaled by heads (every head owns its tables; the per-CTA exchange buffer, the only shared footprint,
# is the same 55 MB at 8 and at 32 heads).
NCU_TRAFFIC_BYTES = {("t16k_d4", "tabulate_tc"): 881.4e6 * 4}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(synth.WORKLOADS))
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-sweep", action="store_true", help="skip the short runs of the other workloads")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--flags", type=int, default=0, help="plan flags (see include/smat.h)")
    ap.add_argument("--decode-only", action="store_true",
                    help="only the cached-decoding measurement, on --workload (a decode_* workload); prints its JSON object")
    return ap.parse_args()


# ------------------------------------------------------------------------------------------------ oracle leg
def oracle_sample(w: synth.Workload, budget_s: float, backward: bool):
    """Times the fp64 dense-mask oracle, as it stands, on sampled rows of head 0 of the workload.

    Returns (tokens/s extrapolated to the whole workload, threads used, description, rows done, seconds)."""
    from oracle import smat_oracle as so
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    geo = so.geometry(w.T, w.chunk, w.d)
    names = ("q", "k", "v", "do") if backward else ("q", "k", "v")
    rng = np.random.default_rng(0)
    done, heads_touched, t0 = 0, 0, time.perf_counter()
    batch = 8
    for head in range(w.bh):            # head after head, rows in random order, until the time budget is used up
        host = {x: synth.as_float64(w, synth.stored(w, x, head)) for x in names}
        order = rng.permutation(w.T)
        heads_touched += 1
        pos = 0
        while pos < w.T and time.perf_counter() - t0 <= budget_s:
            rows = order[pos:pos + batch]
            so.forward_rows(host["q"], host["k"], host["v"], geo, rows)
            if backward:
                so.dq_rows(host["q"], host["k"], host["v"], host["do"], geo, rows)
                so.dkdv_cols(host["q"], host["k"], host["v"], host["do"], geo, rows)
            pos += len(rows)
            done += len(rows)
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    # a token is done when its row is done in every head of its batch element
    tokens_per_s = done / dt / w.heads
    what = (f"{done} uniformly sampled rows of O" + (" and of dQ, dK, dV" if backward else "") +
            f" of the first {heads_touched} head(s) ({dt:.1f} s), scaled by 1/heads to whole tokens")
    return tokens_per_s, threads, what, done, dt


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = synth.WORKLOADS[args.workload]
    steps, warm = max(1, args.steps), max(0, args.warmup)
    budget = min(6.0, 120.0 / (steps + warm))
    for _ in range(warm):
        oracle_sample(w, min(budget, 1.0), w.backward)
    vals, secs, rows, threads, what = [], 0.0, 0, 1, ""
    for _ in range(steps):
        v, threads, what, r, dt = oracle_sample(w, budget, w.backward)
        vals.append(v); secs += dt; rows += r
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": 1e3 * secs / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, 1),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle",
                         "sample": f"each step: {what}"},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ helpers
def workload_config(w: synth.Workload, n_gpus: int):
    return {"workload": w.name, "d": w.d, "batch": w.batch, "heads": w.heads, "T": w.T, "d_k": w.d_k, "d_v": w.d_v,
            "chunk": w.chunk, "routing": w.routing, "variant": w.variant, "pass": "fwd+bwd (backward reuses the forward's profile/type tables left in the shared workspace)"
            if w.backward else "fwd", "input_dtype": w.dtype,
            "replicas": n_gpus, "l2": "inputs and tables exceed the 126 MB L2; no flush"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def wait_ready(self, timeout_s: float = 3.0):
        """Blocks until nvidia-smi has delivered its first sample, so that the timed region is covered."""
        t0 = time.perf_counter()
        while self.proc and not self.lines and time.perf_counter() - t0 < timeout_s:
            time.sleep(0.01)
        self.idle = len(self.lines)   # samples taken before any work was queued

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines[getattr(self, "idle", 0):]:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def make_inputs(w: synth.Workload, torch):
    """Pinned host tensors [batch, heads, T, dim] in the storage dtype."""
    names = ("q", "k", "v", "do") if w.backward else ("q", "k", "v")
    out = {}
    for x in names:
        arr = synth.full_tensor(w, x)
        if w.dtype == "f32":
            t = torch.from_numpy(arr)
        else:
            t = torch.from_numpy(arr.view(np.int16)).view(torch.bfloat16)
        out[x] = t.reshape(w.batch, w.heads, w.T, -1).pin_memory()
    return out


class Runner:
    def __init__(self, w: synth.Workload, torch, binding, flags=0):
        self.w, self.torch = w, torch
        if w.backward and w.variant in ("plain", "gated"):  # one workspace per step: the backward reuses the forward's F, U
            flags |= binding.FLAG_KEEP_FORWARD_TABLES
        flags |= {"gated": binding.FLAG_GATED, "normalized": binding.FLAG_NORMALIZED}.get(w.variant, 0)
        self.plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype, flags=flags)
        self.host = make_inputs(w, torch)
        self.dev = {k: v.cuda(non_blocking=True) for k, v in self.host.items()}
        self.O = torch.empty_like(self.dev["v"])
        self.ws = self.plan.workspace(for_backward=w.backward)
        if w.backward:
            self.dQ, self.dK, self.dV = (torch.empty_like(self.dev[x]) for x in ("q", "k", "v"))
        self.log_a = None
        if w.variant == "gated":
            self.log_a = torch.from_numpy(np.stack([synth.log_gates(w, h) for h in range(w.bh)])).cuda()
        self.routing = {}
        if w.routing == "hashed":   # user-supplied routing: int32 cell / type of every token, resident on the device
            g = self.plan.geometry()
            prof = np.stack([synth.hashed_cells(w, h, g.n, g.P) for h in range(w.bh)])
            typ = np.stack([synth.hashed_types(w, h, g.m, g.B) for h in range(w.bh)])
            self.routing = {"prof": torch.from_numpy(prof).cuda(), "type": torch.from_numpy(typ).cuda()}
        self.host_out = {"o": torch.empty_like(self.host["v"]).pin_memory()}
        if w.backward:
            for nm, src in (("dq", "q"), ("dk", "k"), ("dv", "v")):
                self.host_out[nm] = torch.empty_like(self.host[src]).pin_memory()
        torch.cuda.synchronize()

    def run_forward(self, d, O, stream=None):
        if self.w.variant == "gated":
            return self.plan.forward_gated(d["q"], d["k"], d["v"], self.log_a, O, self.ws, stream=stream)
        if self.w.variant == "normalized":
            return self.plan.forward_normalized(d["q"], d["k"], d["v"], O, self.ws, stream=stream)
        return self.plan.forward(d["q"], d["k"], d["v"], O, self.ws, stream=stream, **self.routing)

    def run_backward(self, d, outs, stream=None):
        if self.w.variant == "gated":
            if getattr(self, "dlog_a", None) is None:
                self.dlog_a = self.torch.empty_like(self.log_a)
            return self.plan.backward_gated(d["q"], d["k"], d["v"], self.log_a, d["do"], outs[0], outs[1], outs[2],
                                            self.dlog_a, self.ws, stream=stream)
        return self.plan.backward(d["q"], d["k"], d["v"], d["do"], outs[0], outs[1], outs[2], self.ws, stream=stream,
                                  **self.routing)

    def step(self):
        d = self.dev
        self.run_forward(d, self.O)
        n = self.plan.last_launch_count()
        if self.w.backward:
            self.run_backward(d, (self.dQ, self.dK, self.dV))
            n += self.plan.last_launch_count()
        return n

    def time_e2e(self, steps, warmup, barrier=None):
        """Seconds per step of the end-to-end loop: every step copies its inputs from pinned host memory, runs the
        path through the C call and copies the results back.  The three legs run on three streams with two sets of
        device buffers, so the copy-in of step i+1 and the copy-out of step i-1 overlap the kernels of step i
        (PCIe is full duplex); every step still moves all of its bytes inside the timed region."""
        torch = self.torch
        w = self.w
        s_in, s_cmp, s_out = (torch.cuda.Stream() for _ in range(3))
        dev = [self.dev, {k: torch.empty_like(v) for k, v in self.dev.items()}]
        outs = [{"o": self.O}, {"o": torch.empty_like(self.O)}]
        if w.backward:
            outs[0].update(dq=self.dQ, dk=self.dK, dv=self.dV)
            outs[1].update({k: torch.empty_like(v) for k, v in (("dq", self.dQ), ("dk", self.dK), ("dv", self.dV))})
        host_out = [self.host_out, {k: torch.empty_like(v).pin_memory() for k, v in self.host_out.items()}]
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_cmp = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]

        def one(i):
            b = i & 1
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_cmp[b])      # the kernels of step i-2 have read these inputs
                for k, v in self.host.items():
                    dev[b][k].copy_(v, non_blocking=True)
                ev_in[b].record(s_in)
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(ev_in[b])
                if i >= 2:
                    s_cmp.wait_event(ev_out[b])     # the results of step i-2 have left these buffers
                d, o = dev[b], outs[b]
                self.run_forward(d, o["o"], stream=s_cmp)
                if w.backward:
                    self.run_backward(d, (o["dq"], o["dk"], o["dv"]), stream=s_cmp)
                ev_cmp[b].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[b])
                for k, v in outs[b].items():
                    host_out[b][k].copy_(v, non_blocking=True)
                ev_out[b].record(s_out)

        for i in range(warmup):
            one(i)
        torch.cuda.synchronize()
        if barrier:
            barrier()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(s_in)
        for i in range(warmup, warmup + steps):
            one(i)
        end.record(s_out)                              # the last copy-out is the last operation of the loop
        torch.cuda.synchronize()
        if barrier:
            barrier()
        return start.elapsed_time(end) / 1e3 / steps

    def bytes_e2e(self):
        h2d = sum(v.numel() * v.element_size() for v in self.host.values())
        d2h = sum(v.numel() * v.element_size() for v in self.host_out.values())
        return h2d, d2h

    def time_steps(self, fn, steps, warmup, barrier=None):
        torch = self.torch
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        if barrier:
            barrier()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record()
        for _ in range(steps):
            fn()
        end.record()
        torch.cuda.synchronize()
        if barrier:
            barrier()
        return start.elapsed_time(end) / 1e3   # seconds for `steps` steps

    def time_each(self, fn, steps, warmup):
        """Per-step durations (seconds) from one CUDA event pair per step, after `warmup` untimed steps."""
        torch = self.torch
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        evs[0].record()
        for i in range(steps):
            fn()
            evs[i + 1].record()
        torch.cuda.synchronize()
        return [evs[i].elapsed_time(evs[i + 1]) / 1e3 for i in range(steps)]

    def time_sustained(self, fn, seconds_per_step, index, min_seconds=1.2):
        """The same step back to back for at least `min_seconds` (long enough for the board power limit to act),
        with the clocks sampled during the region."""
        torch = self.torch
        steps = max(20, int(min_seconds / max(seconds_per_step, 1e-6)) + 1)
        sampler = ClockSampler(index)
        sampler.start()
        sampler.wait_ready()
        total = self.time_steps(fn, steps, 3)
        clocks = sampler.stop()
        return {"steps": steps, "seconds": total, "ms_per_step": 1e3 * total / steps, "clocks": clocks}

    def stage_profile(self, steps):
        """Average per-kernel durations (ms) over `steps` steps, CUDA events on the launching stream."""
        self.plan.profile_enable(True)
        acc, order = {}, []
        for _ in range(steps):
            d = self.dev
            self.run_forward(d, self.O)
            recs = self.plan.profile_read()
            if self.w.backward:
                self.run_backward(d, (self.dQ, self.dK, self.dV))
                # stages the backward shares with the forward (the rebuilt forward tables) get their own prefix, so that
                # they cannot merge with an adjoint stage of the same base name
                recs += [(n if n.startswith("bwd_") else "bwd_fwd_" + n, t) for n, t in self.plan.profile_read()]
            for n, t in recs:
                if n not in acc:
                    acc[n] = 0.0; order.append(n)
                acc[n] += t
        self.plan.profile_enable(False)
        return [(n, acc[n] / steps) for n in order]


def table_bytes(plan):
    """Bytes per entry of the type and profile tables as the kernels that ran keep them (a gated plan whose passes run
    on the tensor cores keeps bf16 tables in its inner plan)."""
    if plan.gated_forward_uses_tensor_cores():
        return 2, 2
    return plan.type_table_element_bytes(), plan.profile_table_element_bytes()


def gated_tc_mode(plan) -> int:
    """0: not a gated plan on the tensor cores; 1: its forward only; 2: forward and backward."""
    if not plan.gated_forward_uses_tensor_cores():
        return 0
    return 2 if plan.gated_backward_uses_tensor_cores() else 1


def path_report(w, geo, seconds_per_step, peaks, u_bytes=4, f_bytes=4, gated_tc_forward=0):
    """Fractions against the path roofline.  The bytes are those of the design that ran: where a table is kept as
    bf16 its round trip is charged at 2 bytes per entry, and the fraction against the roofline with fp32 tables is
    given beside it.  gated_tc_forward: 0 = not a gated tensor-core pass; 1 = a gated plan whose forward runs on the
    tensor cores (bf16 tables) while its backward rebuilds fp32 tables on the ALU kernels; 2 = both passes on the
    tensor cores.  Each pass is charged with the tables it keeps."""
    e = 4 if w.dtype == "f32" else 2
    def total(ub, fb):
        if gated_tc_forward and (ub, fb) != (4, 4):
            wk = roofline.forward_work(w.T, w.chunk, w.d_k, w.d_v, e, geo, 2, 2)
            if w.backward:   # the gated backward rebuilds the forward tables; fp32 tables where it runs on the ALU kernels
                tb = 2 if gated_tc_forward == 2 else 4   # the tensor-core backward reuses the forward's tables
                wk = wk + roofline.backward_work(w.T, w.chunk, w.d_k, w.d_v, e, geo, tb, tb,
                                                 keep_forward_tables=gated_tc_forward == 2, f_bytes=tb, ubar_bytes=tb)
            return wk.scaled(w.bh)
        wk = roofline.forward_work(w.T, w.chunk, w.d_k, w.d_v, e, geo, ub, fb)
        if w.backward:  # bench.py's fwd+bwd step keeps the forward's tables; the adjoint tables follow the forward's
            fbar = 2 if (fb == 2 or (ub == 2 and geo.d <= 3)) else 4
            ubar = 2 if (fb == 2 and geo.d >= 3) or (ub == 2 and geo.d == 2) else 4
            wk = wk + roofline.backward_work(w.T, w.chunk, w.d_k, w.d_v, e, geo, ub, fbar, keep_forward_tables=True,
                                             f_bytes=fb, ubar_bytes=ubar)
        return wk.scaled(w.bh)
    work = total(2, 2) if gated_tc_forward else total(u_bytes, f_bytes)
    t = roofline.roofline_times(work, peaks)
    t32 = roofline.roofline_times(total(4, 4), peaks)
    return {
        "frac_2term": t["t_2term"] / seconds_per_step, "frac_3term": t["t_3term"] / seconds_per_step,
        "frac_2term_fp32_tables": t32["t_2term"] / seconds_per_step,
        "type_table_bytes_per_entry": 2 if gated_tc_forward else u_bytes,
        "profile_table_bytes_per_entry": 2 if gated_tc_forward else f_bytes,
        "roofline_ms_2term": 1e3 * t["t_2term"], "roofline_ms_3term": 1e3 * t["t_3term"],
        "t_tensor_ms": 1e3 * t["t_tensor"], "t_alu_ms": 1e3 * t["t_alu"], "t_hbm_ms": 1e3 * t["t_hbm"],
        "alu_peak_adds_per_s": t["alu_peak_adds"], "alu_peak_source": t["alu_peak_source"],
        "algorithmic": {"tensor_flop": work.flops, "alu_adds": work.adds, "hbm_bytes": work.bytes},
        "peaks": peaks["source"],
    }


def dominant_kernel_report(w, geo, stages, peaks, u_bytes=4, f_bytes=4):
    """Roofline of the stage that takes the longest.  Its bound is the slower of its bytes at the HBM peak and its
    operations (contraction flop plus Algorithm 2's additions, one flop each) at the tensor peak; a tabulation that
    adds on the fp32 ALUs is held against the measured fp32-add rate instead when that is the slower term."""
    e = 4 if w.dtype == "f32" else 2
    total = sum(t for _, t in stages)
    name, ms = max(stages, key=lambda s: s[1])
    base = name[len("bwd_fwd_"):] if name.startswith("bwd_fwd_") else name   # a forward stage re-run by the backward
    work = roofline.stage_work(base, w.T, w.chunk, w.d_k, w.d_v, e, geo, u_bytes, f_bytes).scaled(w.bh)
    t = roofline.roofline_times(work, peaks, sustained=True)
    ops = work.flops + work.adds
    t_ops = ops / (peaks["bf16_tflops_sustained"] * 1e12)
    sec = ms / 1e3
    if base in roofline.ALU_STAGES and t["t_alu"] > t["t_hbm"]:   # sums formed on the fp32 pipes: measured add rate
        bound, achieved, peak, unit = "alu", work.adds / sec / 1e9, t["alu_peak_adds"] / 1e9, "Gadd/s"
    elif t["t_hbm"] >= t_ops:
        bound, achieved, peak, unit = "hbm", work.bytes / sec / 1e9, peaks["hbm_gbs"], "GB/s"
    else:
        bound, achieved, peak, unit = "tensor", ops / sec / 1e12, peaks["bf16_tflops_sustained"], "TFLOP/s"
    return {"kernel": name, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit,
            "frac": achieved / peak if peak else None, "traffic": NCU_TRAFFIC_BYTES.get((w.name, base)),
            "algorithmic_bytes": work.bytes, "algorithmic_ops": ops,
            "ms": ms, "share": ms / total if total else None, "peak_source": peaks["source"],
            "kernels_ms": {n: round(t_, 4) for n, t_ in stages}}


def decode_report(torch, binding, peaks, steps=64, name="decode_t2k_d3"):
    """Cached decoding (one token per sequence and step): steps/s, tokens/s and the fraction of the HBM peak of the
    step kernel, whose algorithmic bytes per head are the running state read and written (fp32) and one type state."""
    w = synth.WORKLOADS[name]
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype)
    g = plan.geometry()
    host = make_inputs(w, torch)
    K, V = host["k"].cuda(), host["v"].cuda()
    cache = plan.decode_cache()
    plan.decode_begin(K, V, cache)
    rows = {x: [host[x][:, :, t].contiguous().cuda() for t in range(g.n, g.n + 8)] for x in ("q", "k", "v")}
    o = torch.empty_like(rows["v"][0])
    def run(count, t0):
        for i in range(count):
            plan.decode_step(rows["q"][i % 8], rows["k"][i % 8], rows["v"][i % 8], t0 + i, cache, o)
    run(8, g.n)
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    run(steps, g.n + 8)
    end.record()
    torch.cuda.synchronize()
    plan.check_status()
    sec = start.elapsed_time(end) / 1e3 / steps
    state = w.d_k * w.d_v
    by = w.bh * state * (4 + 4 + plan.type_table_element_bytes())
    return {"workload": w.name, "batch": w.batch, "heads": w.heads, "type_states_B": g.B, "us_per_step": 1e6 * sec,
            "value": w.batch / sec, "unit": "tokens/s", "cache_bytes": int(cache.numel()),
            "roofline": {"bound": "hbm", "achieved": by / sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": by / sec / 1e9 / peaks["hbm_gbs"], "algorithmic_bytes": by, "traffic": None}}


def run_native(args):
    import torch
    import torch.distributed as dist

    from paper_2609_36062_b200 import binding, build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback for the hot path")
    torch.cuda.set_device(local)
    build.build()
    binding.load_library()
    barrier = None
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        barrier = dist.barrier

    peaks = roofline.load_peaks(ROOT)
    if rank == 0:   # fp32 add rate of the plain ALUs, measured here (scalar and two-lane adds; the faster one counts)
        rates = {"scalar": binding.measure_fadd_rate(False), "packed": binding.measure_fadd_rate(True)}
        peaks["fadd_adds_per_s"] = max(rates.values())
        peaks["fadd_rates"] = rates
    if args.decode_only:
        if rank == 0:
            name = args.workload if args.workload.startswith("decode") else "decode_t2k_d3"
            print(json.dumps(decode_report(torch, binding, peaks, max(8, args.steps), name)))
        return
    w = synth.WORKLOADS[args.workload]
    steps, warm = max(1, args.steps), max(3, args.warmup)
    runner = Runner(w, torch, binding, args.flags)
    g = runner.plan.geometry()

    sampler = ClockSampler(local)
    sampler.start()
    sampler.wait_ready()
    launches = runner.step()
    secs = runner.time_steps(runner.step, steps, warm, barrier)
    clocks = sampler.stop()
    each = runner.time_each(runner.step, max(15, steps), 5)
    secs_e2e = runner.time_e2e(max(4, steps // 2), 2, barrier)
    secs, secs_e2e = replicas.max_over_ranks([secs, secs_e2e], device="cuda")
    per_step = secs / steps
    value = world * w.tokens / per_step
    h2d, d2h = runner.bytes_e2e()

    line = None
    if rank == 0:
        ub, fb = table_bytes(runner.plan)
        stages = runner.stage_profile(min(steps, 10))
        line = {
            "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": steps, "warmup": warm,
            "ms_per_step": 1e3 * per_step, "ms_per_step_median": 1e3 * float(np.median(each)),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if w.dtype == "f32" else "bf16 in, f32 accumulate", "data": "synthetic",
            "config": workload_config(w, world),
            "e2e": {"value": world * w.tokens / secs_e2e, "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h},
            "gpu_launches": launches * steps,
            "clocks": clocks,
            "roofline": dominant_kernel_report(w, g, stages, peaks, ub, fb),
            "path_roofline": path_report(w, g, per_step, peaks, ub, fb, gated_tc_mode(runner.plan)),
            "tables": {"profile_states_P": g.P, "cached_subset_states_B": g.B, "nnzC": g.nnzC, "q": g.q},
            "fadd_rates_adds_per_s": peaks.get("fadd_rates"),
        }
    del runner
    torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.no_sweep:
        sweep = []
        for name in SWEEP:
            if name == args.workload:
                continue
            ws_ = synth.WORKLOADS[name]
            r = Runner(ws_, torch, binding, args.flags)
            gg = r.plan.geometry()
            each_ = r.time_each(r.step, 15, 5)
            s = float(np.median(each_))
            rep = path_report(ws_, gg, s, peaks, r.plan.type_table_element_bytes(), r.plan.profile_table_element_bytes(),
                              gated_tc_mode(r.plan))
            st_ = r.stage_profile(3)
            dom = dominant_kernel_report(ws_, gg, st_, peaks, *table_bytes(r.plan))
            sweep.append({"workload": name, "dominant": {k: dom[k] for k in ("kernel", "bound", "achieved", "peak", "unit",
                                                                              "frac", "ms", "share")}, "value": ws_.tokens / s, "unit": "tokens/s", "ms_per_step": 1e3 * s,
                          "timing": "median of 15 steps after 5 warm-ups, one CUDA event pair per step",
                          "ms_min": 1e3 * min(each_), "ms_max": 1e3 * max(each_),
                          "frac_2term": rep["frac_2term"], "frac_3term": rep["frac_3term"],
                          "frac_2term_fp32_tables": rep["frac_2term_fp32_tables"],
                          "roofline_ms_2term": rep["roofline_ms_2term"],
                          "cached_subset_states_B": gg.B, "profile_states_P": gg.P,
                          "kernels_ms": {n: round(t_, 4) for n, t_ in st_}})
            del r
            torch.cuda.empty_cache()
        line["sweep"] = sweep
        line["decode"] = decode_report(torch, binding, peaks)
        # last, because it heats the board: the headline workload back to back for more than a second
        r = Runner(w, torch, binding, args.flags)
        sus = r.time_sustained(r.step, per_step, local)
        line["sustained"] = dict(sus, value=w.tokens * sus["steps"] / sus["seconds"], unit="tokens/s")
        del r
        torch.cuda.empty_cache()

    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            v, threads, what, _, _ = oracle_sample(w, 12.0, w.backward)
            line["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": what}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_native(args)


if __name__ == "__main__":
    main()
