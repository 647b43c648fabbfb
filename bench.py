#!/usr/bin/env python
"""Benchmark of the FP8 delayed-scaling linear-layer hot path (F + dI + dW, split-backward schedule).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C2] [--mode graph|eager] [--impl ours|reference]

One "step" is one optimizer step of the configuration: every microbatch's F, dI and dW for every linear
of the block in zero-bubble order (dW deferred), all weight gradients accumulated in place in one flat
FP32 buffer, then the optimizer boundary of every layer (which makes the next step re-quantise the
weights).  Prints ONE JSON line.  N > 1 runs N independent replicas (the path does not shard).
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
sys.path.insert(0, ROOT)

from paper_2609_23536_b200 import inputs  # noqa: E402
from paper_2609_23536_b200.schedules import peak_live, sched  # noqa: E402

METRIC = "fp8_linear_layer_F_dI_dW_tflops"
IDLE_BEFORE_BURST_S = 3.0  # idle time before a leg whose figures are compared with the burst (idle-part) peak
UNIT = "TFLOP/s"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"], "bf16_sustained": d["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


def step_flops(cfg) -> float:
    per_mb = 6.0 * cfg["T"] * sum(K * N for _, K, N in cfg["linears"])
    return per_mb * cfg["M"] * cfg["layers"]


# ------------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
            t0 = time.time()
            while not self.rows and time.time() - t0 < 5.0:  # nvidia-smi takes a moment to deliver its first sample
                time.sleep(0.01)
            self.first = len(self.rows)
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([time.time()] + [c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, t0=None, t1=None):
        """Median SM clock and the throttle reasons seen, over all samples or over those taken between the host times
        t0 and t1 (one timed block)."""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows[getattr(self, "first", 0):]:
            if t0 is not None and not (t0 <= r[0] <= t1):
                continue
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------ our arm
class Stage:
    """All linears of the configuration on one device, with resident per-microbatch inputs and outputs."""

    def __init__(self, qe, cfg_name, cfg, mode, device, host_io=False, same_stream=True, overlap_dw=False, staged=False,
                 group_dw=True, arena=False, chain=False, pair_f_di=True, together=True, plan_window=0):
        import torch

        self.qe, self.cfg, self.dev = qe, cfg, device
        self.boundary_per_layer = False
        self.group_dw = group_dw and not staged and not arena
        self.chain = chain
        self.pair_f_di = pair_f_di and not chain and not host_io
        self.together = together and self.pair_f_di and not staged and not arena
        self.plan_window = plan_window
        # the context executes on the stream the benchmark issues from: no cross-stream event hops between actions
        self.ctx = qe.Context(qe.GRAPH if mode == "graph" else qe.EAGER, device.index or 0,
                              exec_stream=(torch.cuda.current_stream().cuda_stream or None) if same_stream else None,
                              overlap_dw=overlap_dw, step_window=max(2, cfg["sched"][0] + cfg["sched"][1]))
        self.schedule = sched(cfg["M"], *cfg["sched"])
        P = peak_live(self.schedule)
        if plan_window:
            from paper_2609_23536_b200.schedules import plan_rounds
            self.rounds = plan_rounds(self.schedule, len(cfg["linears"]) * cfg["layers"], P, 8, plan_window)
        T, M = cfg["T"], cfg["M"]
        self.layers, self.offsets = [], []
        lin = cfg["linears"]
        offs, per_layer = inputs.grad_offsets(lin)
        self.grad = torch.zeros(per_layer * cfg["layers"], dtype=torch.float32, device=device)
        self.temp = torch.empty(max(K * N for _, K, N in lin), dtype=torch.float32, device=device) if staged else None
        # per-microbatch arena variant: M bf16 views per linear (capacity M * sum of sizeof(W)), summed at the boundary
        self.arena = torch.empty(M * per_layer * cfg["layers"], dtype=torch.bfloat16, device=device) if arena else None
        for l in range(cfg["layers"]):
            for j, (_, K, N) in enumerate(lin):
                w = inputs.weights(cfg_name, l, j, N, K, device=device)
                self.layers.append(qe.Layer(self.ctx, T, K, N, cfg["H"], cfg["margin"], P, w, stage=0, unit=l * len(lin) + j, host_io=host_io))
                self.offsets.append(l * per_layer + offs[j])
        # groups of directly chainable linears (next K == this N, T and N multiples of 256), at most 16 long
        self.groups = []
        for i, L in enumerate(self.layers):
            fits = (self.groups and len(self.groups[-1]) < 16 and self.layers[self.groups[-1][-1]].N == L.K
                    and L.N % 256 == 0 and L.T % 256 == 0 and self.layers[self.groups[-1][-1]].N % 256 == 0)
            if chain and fits:
                self.groups[-1].append(i)
            else:
                self.groups.append([i])
        # distinct synthetic tensors per (microbatch, linear), drawn once, outside any timed region, by the device's
        # generator (config 3 holds 73 GB of them; the CPU generator would take minutes)
        g = torch.Generator(device=device)
        g.manual_seed(inputs.seed_for(cfg_name, "bench"))
        draw = lambda shape, std: (torch.randn(shape, generator=g, dtype=torch.float32, device=device) * std).to(torch.bfloat16)
        # the end-to-end leg keeps inputs and outputs in pinned host memory only: one set of buffers per microbatch
        # while that stays under 12 GB, else as many sets as fit (at least two), taken in turn -- every step still
        # copies every microbatch's bytes in and out
        set_bytes = sum(4 * T * (L.K + L.N) for L in self.layers)
        self.host_sets = M if M * set_bytes <= 12e9 else max(2, int(12e9 // set_bytes))
        self.X, self.dY, self.Y, self.dX, self.Xh, self.dYh, self.Yh, self.dXh = [], [], [], [], [], [], [], []
        for m in range(M):
            xs, gs, ys, dxs, xh, gh, yh, dxh = [], [], [], [], [], [], [], []
            if host_io and m >= self.host_sets:
                k = m % self.host_sets
                self.X.append(xs); self.dY.append(gs); self.Y.append(ys); self.dX.append(dxs)
                self.Xh.append(self.Xh[k]); self.dYh.append(self.dYh[k]); self.Yh.append(self.Yh[k]); self.dXh.append(self.dXh[k])
                continue
            for L in self.layers:
                x = draw((T, L.K), 1.0)
                dy = draw((T, L.N), 1e-3)
                if host_io:
                    xh.append(torch.empty((T, L.K), dtype=torch.bfloat16).pin_memory().copy_(x))
                    gh.append(torch.empty((T, L.N), dtype=torch.bfloat16).pin_memory().copy_(dy))
                    yh.append(torch.empty((T, L.N), dtype=torch.bfloat16).pin_memory())
                    dxh.append(torch.empty((T, L.K), dtype=torch.bfloat16).pin_memory())
                else:
                    xs.append(x)
                    gs.append(dy)
                    ys.append(torch.empty((T, L.N), dtype=torch.bfloat16, device=device))
                    dxs.append(torch.empty((T, L.K), dtype=torch.bfloat16, device=device))
            self.X.append(xs); self.dY.append(gs); self.Y.append(ys); self.dX.append(dxs)
            self.Xh.append(xh); self.dYh.append(gh); self.Yh.append(yh); self.dXh.append(dxh)
        self.grad_host = torch.empty(self.grad.shape, dtype=torch.float32).pin_memory() if host_io else None
        self.epoch = 0
        self.h2d = self.d2h = 0
        self.issue_s = 0.0

    def boundary(self):
        """The optimizer boundary of the whole stage: one drain and one gathered status read (default), or layer by layer."""
        if self.boundary_per_layer:
            for L in self.layers:
                L.optimizer_boundary(self.cfg["M"])
        else:
            self.qe.optimizer_boundary_all(self.layers, self.cfg["M"])

    def make_plan(self):
        """The whole step as one qe_step_run call (native host loop; one graph for the step in graph mode)."""
        n = len(self.layers)
        acts = [(a, i, m) for a, m in self.schedule for i in (range(n) if a == "F" else range(n - 1, -1, -1))]
        self.plan = self.qe.StepPlan(self.ctx, self.layers, acts, self.cfg["M"], self.X, self.Y, self.dY, self.dX,
                                     self.grad, self.offsets, self.temp)

    def step(self, host_io=False):
        if getattr(self, "plan", None) is not None and not host_io:
            t_issue = time.perf_counter()
            self.plan.run()
            self.issue_s += time.perf_counter() - t_issue
            self.boundary()
            self.epoch += 1
            return
        tapes = {}
        n = len(self.layers)
        t_issue = time.perf_counter()
        if self.plan_window:
            # the schedule cut into rounds of independent per-linear actions (schedules.plan_rounds), one call each;
            # host_io: host pointers straight into the C-ABI (qe_run_together_host stages, runs and reads back)
            X, Y, dY, dX = (self.Xh, self.Yh, self.dYh, self.dXh) if host_io else (self.X, self.Y, self.dY, self.dX)
            for group in self.rounds:
                acts, keys = [], []
                for a, i, m in group:
                    if a == "F":
                        acts.append(("F", self.layers[i], m, self.epoch, X[m][i], Y[m][i]))
                        keys.append((m, i))
                        if host_io:
                            self.h2d += X[m][i].numel() * 2
                            self.d2h += Y[m][i].numel() * 2
                    elif a == "dI":
                        acts.append(("dI", self.layers[i], tapes[(m, i)], dY[m][i], dX[m][i]))
                        if host_io:
                            self.h2d += dY[m][i].numel() * 2
                            self.d2h += dX[m][i].numel() * 2
                    else:
                        acts.append(("dW", self.layers[i], tapes[(m, i)], self.offsets[i]))
                for key, t in zip(keys, self.qe.run_together(self.ctx, acts, self.grad, host=host_io)):
                    tapes[key] = t
            self.issue_s += time.perf_counter() - t_issue
            self.boundary()
            if host_io:  # the step's result: the accumulated gradients, complete after the boundary
                self.grad_host.copy_(self.grad, non_blocking=True)
                self.d2h += self.grad.numel() * 4
            self.epoch += 1
            return
        skip = 0
        for k, (a, m) in enumerate(self.schedule):
            if skip:  # this dI (and dW) went out together with the forward before it
                skip -= 1
                continue
            order = range(n) if a == "F" else range(n - 1, -1, -1)
            if (self.pair_f_di and not host_io and a == "F" and k + 1 < len(self.schedule) and self.schedule[k + 1][0] == "dI"):
                # steady state: a forward unit and an input-gradient unit are both at hand; F of linear i goes out
                # with dI of linear n-1-i (the two chains are independent), one shared GEMM launch per pair
                mb_b = self.schedule[k + 1][1]
                # ... and a deferred weight-gradient unit too, when the schedule has one next: its GEMM for linear i
                # joins the same launch (qe_run_together), no second stream needed
                mb_w = self.schedule[k + 2][1] if (self.together and k + 2 < len(self.schedule) and self.schedule[k + 2][0] == "dW") else None
                for i in range(n):
                    j = n - 1 - i
                    if mb_w is not None and i != j:
                        acts = [("F", self.layers[i], m, self.epoch, self.X[m][i], self.Y[m][i]),
                                ("dI", self.layers[j], tapes[(mb_b, j)], self.dY[mb_b][j], self.dX[mb_b][j]),
                                ("dW", self.layers[i], tapes[(mb_w, i)], self.offsets[i])]
                        tapes[(m, i)] = self.qe.run_together(self.ctx, acts, self.grad)[0]
                        continue
                    if i == j:
                        tapes[(m, i)] = self.layers[i].forward(m, self.epoch, self.X[m][i], self.Y[m][i])
                        self.layers[j].backward_dI(tapes[(mb_b, j)], self.dY[mb_b][j], self.dX[mb_b][j])
                    else:
                        tapes[(m, i)] = self.qe.forward_dI_pair(self.layers[i], m, self.epoch, self.X[m][i], self.Y[m][i],
                                                                 self.layers[j], tapes[(mb_b, j)], self.dY[mb_b][j], self.dX[mb_b][j])
                skip = 1
                if mb_w is not None:
                    skip = 2
                    if n % 2:  # the middle linear went out alone above: its weight gradient too
                        self.layers[n // 2].backward_dW(tapes[(mb_w, n // 2)], self.grad, self.offsets[n // 2])
                continue
            if self.together and not host_io and a == "F" and k + 1 < len(self.schedule) and self.schedule[k + 1][0] == "F":
                # warm-up: several forward units in a row (the last of them goes out with what follows it).  Their chains
                # through the linears are independent, so they advance as a wavefront: round r holds F of linear r-j of
                # the j-th unit; each linear still sees the microbatches in order
                ms, kk = [], k
                while kk + 1 < len(self.schedule) and self.schedule[kk][0] == "F" and self.schedule[kk + 1][0] == "F" and len(ms) < 4:
                    ms.append(self.schedule[kk][1])
                    kk += 1
                for r in range(n + len(ms) - 1):
                    acts, keys = [], []
                    for j, mm in enumerate(ms):
                        i = r - j
                        if 0 <= i < n:
                            acts.append(("F", self.layers[i], mm, self.epoch, self.X[mm][i], self.Y[mm][i]))
                            keys.append((mm, i))
                    for key, t in zip(keys, self.qe.run_together(self.ctx, acts)):
                        tapes[key] = t
                skip = len(ms) - 1
                continue
            if (self.together and not host_io and a == "dI" and k + 1 < len(self.schedule) and self.schedule[k + 1][0] == "dW"
                    and self.schedule[k + 1][1] != m):
                # cool-down: an input-gradient unit and a deferred weight-gradient unit of an earlier microbatch: dI of
                # linear n-1-i goes out with dW of linear i
                mb_w = self.schedule[k + 1][1]
                for i in range(n):
                    j = n - 1 - i
                    self.qe.run_together(self.ctx, [("dI", self.layers[j], tapes[(m, j)], self.dY[m][j], self.dX[m][j]),
                                                    ("dW", self.layers[i], tapes[(mb_w, i)], self.offsets[i])], self.grad)
                skip = 1
                continue
            if self.chain and a != "dW" and not host_io:
                # the linears as directly chained groups of up to 16 (FP8 hand-off: one cast per group and direction)
                for g in (self.groups if a == "F" else reversed(self.groups)):
                    ls = [self.layers[i] for i in g]
                    if a == "F":
                        for i, t in zip(g, self.qe.forward_chain(ls, m, self.epoch, self.X[m][g[0]], self.Y[m][g[-1]])):
                            tapes[(m, i)] = t
                    else:
                        self.qe.backward_dI_chain(ls, [tapes[(m, i)] for i in g], self.dY[m][g[-1]], self.dX[m][g[0]])
                continue
            if a == "dW" and self.group_dw:  # one call for the microbatch's weight gradients of all linears
                ordl = list(order)
                for lo in range(0, n, 16):
                    idx = ordl[lo:lo + 16]
                    self.qe.backward_dW_multi([self.layers[i] for i in idx], [tapes[(m, i)] for i in idx], self.grad,
                                              [self.offsets[i] for i in idx])
                continue
            for i in order:
                L = self.layers[i]
                if a == "F":
                    if host_io:  # host pointers straight into the C-ABI: it stages, runs and reads back
                        tapes[(m, i)] = L.forward_host(m, self.epoch, self.Xh[m][i], self.Yh[m][i])
                        self.h2d += self.Xh[m][i].numel() * 2
                        self.d2h += self.Yh[m][i].numel() * 2
                    else:
                        tapes[(m, i)] = L.forward(m, self.epoch, self.X[m][i], self.Y[m][i])
                elif a == "dI":
                    if host_io:
                        L.backward_dI_host(tapes[(m, i)], self.dYh[m][i], self.dXh[m][i])
                        self.h2d += self.dYh[m][i].numel() * 2
                        self.d2h += self.dXh[m][i].numel() * 2
                    else:
                        L.backward_dI(tapes[(m, i)], self.dY[m][i], self.dX[m][i])
                elif self.arena is not None:
                    L.backward_dW_arena(tapes[(m, i)], self.arena, self.cfg["M"] * self.offsets[i], self.cfg["M"])
                elif self.temp is not None:
                    L.backward_dW_staged(tapes[(m, i)], self.grad, self.offsets[i], self.temp)
                else:
                    L.backward_dW(tapes[(m, i)], self.grad, self.offsets[i])
        if self.arena is not None:
            for i, L in enumerate(self.layers):
                L.arena_finalize(self.arena, self.cfg["M"] * self.offsets[i], self.cfg["M"], self.grad, self.offsets[i])
        self.issue_s += time.perf_counter() - t_issue  # host time to enqueue the step (before the boundary's sync)
        self.boundary()
        if host_io:  # the step's result: the accumulated gradients, complete after the boundary
            self.grad_host.copy_(self.grad, non_blocking=True)
            self.d2h += self.grad.numel() * 4
        self.epoch += 1


def max_over_ranks(ms: float, dist, device="cuda") -> float:
    """Slowest rank's time (every rank returns it); dist is torch.distributed or None for a single process."""
    if dist is None:
        return ms
    import torch

    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(flop_per_step: float, steps: int, world: int, ms_max: float) -> float:
    """Aggregate TFLOP/s of all replicas: every rank did `steps` steps within the slowest rank's time."""
    return flop_per_step * steps * world / (ms_max * 1e-3) / 1e12


def time_steps(stage, steps, warmup, host_io, dist, min_s=0.0, clk=None, max_blocks=400):
    """Warm-up, then timed blocks of EXACTLY `steps` steps each (barrier + synchronize on both sides, CUDA events on the
    issuing stream, max over ranks), repeated until `min_s` seconds of device time have been timed: what a caller reads
    must not depend on how short it made the block.  Returns (ms of the median block, kernels launched per block, list
    of per-block records)."""
    import torch

    for _ in range(warmup):
        stage.step(host_io)
    torch.cuda.synchronize()
    blocks, total_ms, launches = [], 0.0, 0
    while True:
        if dist is not None:
            dist.barrier()
        stage.h2d = stage.d2h = 0
        stage.issue_s = 0.0
        k0 = stage.ctx.stats()["kernels_launched"]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0 = time.time()
        e0.record()
        for _ in range(steps):
            stage.step(host_io)
        e1.record()
        torch.cuda.synchronize()
        t1 = time.time()
        ms = max_over_ranks(e0.elapsed_time(e1), dist)  # the same number on every rank, so all ranks stop together
        launches = stage.ctx.stats()["kernels_launched"] - k0
        rec = {"ms": ms, "issue_s": stage.issue_s}
        if clk is not None:
            c = clk.summary(t0, t1)
            rec["sm_mhz"], rec["reasons"] = c["sm_mhz"], c["reasons"]
        blocks.append(rec)
        total_ms += ms
        if total_ms >= min_s * 1e3 or len(blocks) >= max_blocks:
            break
    if dist is not None:
        dist.barrier()
    order = sorted(range(len(blocks)), key=lambda i: blocks[i]["ms"])
    med = blocks[order[len(order) // 2]]
    stage.issue_s = med["issue_s"]
    return med["ms"], launches, blocks


def block_summary(blocks, steps, flop_per_step, world):
    """What the timed blocks say beyond the median: fastest and slowest block, total timed time, and the clock."""
    ms = sorted(b["ms"] for b in blocks)
    mhz = [b["sm_mhz"] for b in blocks if b.get("sm_mhz")]
    tf = lambda t: round(flop_per_step * steps * world / (t * 1e-3) / 1e12, 2)
    out = {"blocks": len(blocks), "timed_region_s": round(sum(ms) * 1e-3, 3),
           "ms_per_step_median": round(ms[len(ms) // 2] / steps, 4), "ms_per_step_min": round(ms[0] / steps, 4),
           "ms_per_step_max": round(ms[-1] / steps, 4), "value_median": tf(ms[len(ms) // 2]), "value_best_block": tf(ms[0]),
           "value_first_block": tf(blocks[0]["ms"]), "value_last_block": tf(blocks[-1]["ms"])}
    if mhz:
        out["sm_mhz_first_block"], out["sm_mhz_last_block"], out["sm_mhz_median_of_blocks"] = mhz[0], mhz[-1], float(np.median(mhz))
    return out


# dram__bytes_read + dram__bytes_write per GEMM launch of one step (mean over the step's launches), from ncu captures of
# `python profile_case.py gemm_step` (config-2 shapes with --small); each entry names the capture's summary and the
# commit of the kernel it was taken with, so that a stale figure shows
QE_TRAFFIC = {
    # config: (bytes per launch, launches per step, summary under profiles/, commit of the kernel source captured)
    "C2": (287.3e6, 19, "gemm_fp8_pair_dram_traffic_config2_microbatch.md", "3398557"),
    # config 3 holds 59 GB of GEMM operands and outputs per step, too much to capture: the five launches of ONE
    # layer-microbatch (12 GEMMs, 3770.3 MB read + written, 1.9 GB on the device) were captured and scaled by the 64
    # layer-microbatches of a step over its 135 launches; every operand and output of a step is distinct data that is
    # streamed once, so the traffic grows in proportion to the layer-microbatches processed
    "C3": (3770.3e6 * 64 / 135, 135, "gemm_fp8_pair_dram_traffic_config3_layer_microbatch.md", "3398557"),
}


def gemm_roofline(qe, cfg_name, cfg, peaks, device):
    """Times the dominant kernel (the tcgen05 FP8 GEMM) alone, live, through the C-ABI on the current stream with CUDA
    events around the loop: first every GEMM shape of one microbatch in a launch of its own over rotating operand sets
    larger than L2 (per-action rates), then the GEMM launches of one whole step as the issue plan groups them (the
    roofline figure: achieved = algorithmic flops of the step / time of its GEMM launches)."""
    import torch

    T = cfg["T"]
    shapes = []
    for _, K, N in cfg["linears"]:
        # (name, M, N, Kc, A format, A MN-major, B MN-major, epilogue): operand majors as the layer uses them
        shapes += [("F", T, N, K, 0, 0, 0, 0), ("dI", T, K, N, 1, 0, 1, 0), ("dW", N, K, T, 1, 1, 1, 2)]
    one = torch.ones(1, dtype=torch.float32, device=device)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    tot_flops = tot_ms = 0.0
    per, per_shape_ms = {}, {}
    for name, M_, N_, Kc, af, amn, bmn, kind in shapes:
        nset = max(2, int(160e6 // (M_ * Kc + N_ * Kc + M_ * N_ * (2 if kind == 0 else 8))) + 1)
        nset = min(nset, 24)
        A = [torch.randint(0, 120, (Kc, M_) if amn else (M_, Kc), dtype=torch.uint8, device=device) for _ in range(nset)]
        B = [torch.randint(0, 120, (Kc, N_) if bmn else (N_, Kc), dtype=torch.uint8, device=device) for _ in range(nset)]
        D = [torch.zeros((M_, N_), dtype=torch.bfloat16 if kind == 0 else torch.float32, device=device) for _ in range(nset)]
        reps = 3 * nset
        for i in range(nset):
            qe.qe_gemm_fp8_ex(A[i], af, bool(amn), B[i], 0, bool(bmn), one, one, D[i], kind, None, status)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for r in range(reps):
            i = r % nset
            qe.qe_gemm_fp8_ex(A[i], af, bool(amn), B[i], 0, bool(bmn), one, one, D[i], kind, None, status)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        fl = 2.0 * M_ * N_ * Kc
        tot_flops += fl
        tot_ms += ms
        per_shape_ms[(name, M_, N_, Kc)] = ms
        per.setdefault(name, [0.0, 0.0])
        per[name][0] += fl
        per[name][1] += ms
        del A, B, D
    assert status.item() == 0
    # ... and the GEMM launches of one whole step as the default issue plan makes them (schedules.plan_rounds: up to
    # eight independent per-linear GEMMs per launch), every (linear, microbatch) with operands and outputs of its own
    from paper_2609_23536_b200 import step_gemms

    launches, g_flops, g_bytes = step_gemms.build(cfg, device)
    step_gemms.run(qe, launches, status)
    torch.cuda.synchronize()
    reps = 3
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(device.index or 0) as gclk:  # which regime the launches were timed in (burst or power-capped)
        e0.record()
        for _ in range(reps):
            step_gemms.run(qe, launches, status)
        e1.record()
        torch.cuda.synchronize()
    g_clocks = gclk.summary()
    g_ms = e0.elapsed_time(e1) / reps
    g_launches = len(launches)
    del launches
    assert status.item() == 0
    lib = None
    try:  # context only: the vendor library's FP8 GEMM (cuBLASLt through torch._scaled_mm) on the forward shapes
        lf = lm = 0.0
        for _, K, N in cfg["linears"]:
            a = torch.randn((T, K), device=device).to(torch.float8_e4m3fn)
            b = torch.randn((N, K), device=device).to(torch.float8_e4m3fn)
            f = lambda: torch._scaled_mm(a, b.t(), scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
            for _ in range(3):
                f()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(20):
                f()
            e1.record()
            torch.cuda.synchronize()
            lf += 2.0 * T * K * N
            lm += e0.elapsed_time(e1) / 20
        lib = round(lf / (lm * 1e-3) / 1e12, 1)
    except Exception as e:  # noqa: BLE001
        lib = "unavailable: " + str(e)[:80]
    single = tot_flops / (tot_ms * 1e-3) / 1e12
    achieved = g_flops / (g_ms * 1e-3) / 1e12
    tr = QE_TRAFFIC.get(cfg_name)
    if tr is not None and tr[1] != g_launches:
        tr = None  # the issue plan changed since the capture
    # FP8 dense = 2 x the bf16 peak (nominal ratio).  Which measured bf16 figure: the burst one for launches timed in a
    # short loop; the sustained one when the loop is long enough for the power cap to engage and the sampled clocks
    # say it did (config 3: 0.5 s at ~1.2 GHz) -- the regime the sustained figure was itself measured in
    sustained = g_ms * reps >= 250.0 and "sw_power_cap" in g_clocks.get("reasons", [])
    peak = 2.0 * (peaks["bf16_sustained"] if sustained else peaks["bf16_burst"])
    burst_peak = 2.0 * peaks["bf16_burst"]
    # the weight-gradient launches are bound by the tensor pipe AND by the FP32 read-modify-write of the gradient slice:
    # both fractions, one problem per launch over rotating operand sets
    dw_fl, dw_ms = per["dW"]
    dw_bytes = sum(T * N + T * K + 8.0 * N * K for _, K, N in cfg["linears"])
    dw_tf, dw_gbs = dw_fl / (dw_ms * 1e-3) / 1e12, dw_bytes / (dw_ms * 1e-3) / 1e9
    return {
        "bound": "tensor", "kernel": "gemm_fp8_pair_group_kernel (the GEMM launches of one step as the issue plan groups them)",
        "achieved": round(achieved, 1), "peak": round(peak, 1),
        "unit": "TFLOP/s", "frac": round(achieved / peak, 4), "traffic": tr[0] if tr else None,
        "traffic_source": ("ncu capture summarised in profiles/%s, kernel as of commit %s" % (tr[2], tr[3])) if tr else None,
        "algorithmic_bytes_per_launch": round(g_bytes / g_launches),
        "flop_per_launch": round(g_flops / g_launches), "launches_timed": g_launches,
        "peak_source": peaks["source"] + (" bf16 sustained x2 (launches timed in a %.2f s loop under sw_power_cap)" % (g_ms * reps * 1e-3) if sustained else " bf16 burst x2"),
        "frac_of_bf16_burst_x2": round(achieved / burst_peak, 4),
        "frac_of_nominal_4500": round(achieved / 4500.0, 4),
        # the same launches against the figure for a kernel timed inside a long step, with the clock they ran at: the
        # loop above lasts 0.4 s at config 3 (the power cap engages within it), 6 ms at config 2 (it does not)
        "frac_of_bf16_sustained_x2": round(achieved / (2.0 * peaks["bf16_sustained"]), 4),
        "clocks_while_timed": g_clocks,
        "one_problem_per_launch_tflops": round(single, 1),
        "per_action_tflops": {k: round(v[0] / (v[1] * 1e-3) / 1e12, 1) for k, v in per.items()},
        "dw": {"tflops": round(dw_tf, 1), "frac_tensor": round(dw_tf / burst_peak, 4), "frac_tensor_of_nominal_4500": round(dw_tf / 4500.0, 4),
               "GB/s": round(dw_gbs, 1), "frac_hbm": round(dw_gbs / peaks["hbm_gbs"], 4),
               "what": "weight-gradient GEMMs of one microbatch, one problem per launch in a short loop (tensor fraction of bf16 burst x2): 2TNK flop and T(N+K) + 8NK bytes each"},
        "gemm_ms_per_step": round(g_ms, 4),
        "vendor_library_fp8_forward_tflops_same_shapes": lib,
    }


def hbm_kernels(qe, cfg, peaks, device):
    """Quantise(+transpose+amax) and standalone amax on tensors larger than L2: achieved algorithmic GB/s."""
    import torch

    rows, cols = 8192, 16384  # 268 MB bf16 in: larger than L2
    x = (torch.randn((rows, cols), device=device) * 1.0).to(torch.bfloat16)
    s = torch.ones(1, device=device)
    q = torch.empty((rows, cols), dtype=torch.uint8, device=device)
    qT = torch.empty((cols, rows), dtype=torch.uint8, device=device)
    amax = torch.zeros(1, device=device)
    part = torch.empty(qe.qe_amax_partials(), device=device)
    out = {}

    def timeit(fn, nbytes, reps=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        gbs = nbytes / (e0.elapsed_time(e1) / reps * 1e-3) / 1e9
        return {"GB/s": round(gbs, 1), "frac": round(gbs / peaks["hbm_gbs"], 4)}

    n = rows * cols
    out["quantize_transpose_amax_4B_per_elt"] = timeit(lambda: qe.qe_quantize(x, s, 0, q, qT, amax), 4 * n)
    out["quantize_amax_3B_per_elt"] = timeit(lambda: qe.qe_quantize(x, s, 0, q, None, amax), 3 * n)
    out["amax_2B_per_elt"] = timeit(lambda: qe.qe_amax(x, part, amax), 2 * n)
    g = torch.zeros(n // 2, device=device)
    t = torch.ones(n // 2, device=device)
    out["accumulate_12B_per_elt"] = timeit(lambda: qe.qe_accumulate(g, t, True), 12 * (n // 2))
    views = x.view(8, -1)  # 8 bf16 views of 16.8 M elements -> one FP32 gradient
    dst = torch.empty(views.shape[1], device=device)
    out["arena_reduce_8_views_20B_per_elt"] = timeit(lambda: qe.qe_arena_reduce(views, 8, dst), 20 * views.shape[1])
    out["peak_GB/s"] = peaks["hbm_gbs"]
    out["peak_source"] = peaks["source"]
    return out


# ------------------------------------------------------------------------------------------------ oracle legs
def oracle_sample(cfg_name, cfg, only=None):
    """One microbatch of every linear of the block (F + dI + dW) through the CPU oracle, as it stands
    (`only` = index of a single linear, for a smaller sample)."""
    from oracle.layer import OracleLinear

    T = cfg["T"]
    t_total, flops = 0.0, 0.0
    for j, (_, K, N) in enumerate(cfg["linears"]):
        if only is not None and j != only:
            continue
        L = OracleLinear(T, K, N, cfg["H"], cfg["margin"], 1)
        L.set_weight(inputs.bits(inputs.weights(cfg_name, 0, j, N, K)))
        X = inputs.bits(inputs.activations(cfg_name, 0, 0, j, 0, T, K))
        dY = inputs.bits(inputs.upstream_grads(cfg_name, 0, 0, j, 0, T, N))
        buf = np.zeros(N * K, np.float32)
        t0 = time.perf_counter()
        tape, _ = L.forward(0, 0, X)
        L.backward_dI(tape, dY)
        L.backward_dW(tape, buf, 0)
        t_total += time.perf_counter() - t0
        flops += 6.0 * T * K * N
    return t_total, flops


def oracle_sample_choice(cfg_name, cfg, many=False):
    """Which bounded sample of the workload the oracle is timed on: one microbatch of the whole block while that is
    about 10-30 s of CPU work (config 2: 120 M elements to cast, 0.63 TFLOP in float64), else (or when many samples
    are asked for) one microbatch of the block's smallest linear."""
    T = cfg["T"]
    casts = sum(T * K + T * N + N * K for _, K, N in cfg["linears"])
    if casts <= 150e6 and not many:
        return None, "one microbatch of all %d linears of %s (F+dI+dW), 1/%d of a step" % (len(cfg["linears"]), cfg_name, cfg["M"] * cfg["layers"])
    only = min(range(len(cfg["linears"])), key=lambda j: cfg["linears"][j][1] * cfg["linears"][j][2])
    _, K, N = cfg["linears"][only]
    share = K * N / (sum(k * n for _, k, n in cfg["linears"]) * cfg["M"] * cfg["layers"])
    return only, "one microbatch of the smallest linear of %s (%s %dx%d, T=%d: F+dI+dW), 1/%.0f of a step" % (cfg_name, cfg["linears"][only][0], K, N, T, 1 / share)


def _threads():
    try:
        from threadpoolctl import threadpool_info

        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def run_reference(args, cfg_name, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    only, sample = oracle_sample_choice(cfg_name, cfg, many=args.steps + min(args.warmup, 1) > 10)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(cfg_name, cfg, only)
    t0 = time.perf_counter()
    tot_s = tot_f = 0.0
    for _ in range(args.steps):
        s, f = oracle_sample(cfg_name, cfg, only)
        tot_s += s
        tot_f += f
    val = tot_f / tot_s / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": tot_s / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg_name, "note": "CPU oracle on the host cores; each step is a bounded sample: " + sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": _threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "wall_s": time.perf_counter() - t0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20, help="steps per timed block")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="repeat the timed block of --steps steps until this much device time has been timed; the median block is reported")
    ap.add_argument("--config", default="C3", help="C3 (default): the largest single-GPU configuration; config 2 rides along as a second object")
    ap.add_argument("--mode", default="graph", choices=["graph", "eager"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the e2e, roofline, HBM-kernel and CPU-baseline legs")
    ap.add_argument("--no-overlap-dw", dest="overlap_dw", action="store_false",
                    help="run dW on the execution stream too (default: QE_CTX_OVERLAP_DW, dW on a second stream joined at the optimizer boundary)")
    ap.add_argument("--step-api", action="store_true",
                    help="qe_step_run: the whole step in one C call (native host loop; ONE graph per step in graph mode; dW not overlapped). "
                         "Default: one C-ABI call per action with dW overlapped on the context's second stream")
    ap.add_argument("--no-group-dw", dest="group_dw", action="store_false",
                    help="one qe_backward_dW call per linear instead of qe_backward_dW_multi per microbatch")
    ap.add_argument("--no-pair-f-di", dest="pair_f_di", action="store_false",
                    help="never issue a forward and the input gradient that follows it in the schedule as qe_forward_dI_pair calls")
    ap.add_argument("--plan", type=int, default=-1, metavar="WINDOW",
                    help="issue the step as rounds of independent per-linear actions planned by schedules.plan_rounds, looking WINDOW "
                         "schedule units ahead (default: warm-up depth + deferral of the schedule, the units a stage holds at once; 0: "
                         "issue unit by unit, pairing only direct neighbours)")
    ap.add_argument("--no-together", dest="together", action="store_false",
                    help="keep the deferred dW out of the shared F + dI launches (it then goes to the second stream)")
    ap.add_argument("--chain", action="store_true",
                    help="treat consecutive linears whose shapes fit (K of the next = N of this) as directly chained: "
                         "qe_forward_chain / qe_backward_dI_chain with FP8 hand-off (config C5)")
    ap.add_argument("--arena", action="store_true",
                    help="per-microbatch arena variant: dW writes one bf16 view per linear and microbatch, summed into the FP32 buffer before the boundary")
    ap.add_argument("--staged", action="store_true", help="copied-gradient comparison path: dW into a temporary, then a copy-add kernel")
    ap.add_argument("--boundary-per-layer", action="store_true",
                    help="one qe_optimizer_boundary call per layer (a drain and a blocking status read each) instead of qe_optimizer_boundary_all")
    ap.add_argument("--own-stream", action="store_true", help="let the context create its own execution stream (event handoff on every action)")
    args = ap.parse_args()
    cfg_name, cfg = args.config, inputs.CONFIGS[args.config]
    if args.impl == "reference":
        return run_reference(args, cfg_name, cfg)

    import torch

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle arm")
    from paper_2609_23536_b200 import build

    build.build()
    from paper_2609_23536_b200 import binding as qe

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    device = torch.device("cuda", local)
    torch.cuda.set_stream(torch.cuda.Stream(device))  # everything below is issued on this (non-default) stream
    peaks = _peaks()
    args.warmup = max(args.warmup, 3)

    def measure(name, c, own_stream, min_s):
        """One configuration through the default issue path: warm-up, timed blocks, clocks; returns the result dict."""
        use_step = args.step_api
        window = 0 if (use_step or args.staged or args.arena or args.chain or not args.together or not args.pair_f_di) else (
            max(2, c["sched"][0] + c["sched"][1]) if args.plan < 0 else args.plan)
        stage = Stage(qe, name, c, args.mode, device, same_stream=not own_stream,
                      overlap_dw=args.overlap_dw and not use_step, staged=args.staged, group_dw=args.group_dw, arena=args.arena,
                      chain=args.chain, pair_f_di=args.pair_f_di, together=args.together, plan_window=window)
        stage.boundary_per_layer = args.boundary_per_layer
        if use_step:
            stage.make_plan()
        with ClockSampler(local) as clk:
            ms, launches, blocks = time_steps(stage, args.steps, args.warmup, False, dist, min_s, clk)
        res = {"ms": ms, "launches": launches, "blocks": blocks, "clocks": clk.summary(), "window": stage.plan_window,
               "stats": stage.ctx.stats(), "status": max(L.state()["device_status"] for L in stage.layers),
               "issue_ms": stage.issue_s / args.steps * 1e3, "flop": step_flops(c)}
        res["value"] = whole_job_value(res["flop"], args.steps, world, ms)
        del stage
        torch.cuda.empty_cache()
        return res

    def fractions(value, mhz, mhz_max):
        """The whole-step rate against the dense FP8 peak: nominal first, then the measured bf16 GEMM rates x 2 (the
        nominal FP8 : bf16 ratio).  The sustained figure was taken at the clock the power cap leaves a long GEMM loop;
        the last entry scales the nominal peak to the clock sampled during THIS timed region instead."""
        out = {"of_nominal_4500": round(value / world / 4500.0, 4),
               "of_measured_bf16_burst_x2": round(value / world / (2 * peaks["bf16_burst"]), 4),
               "of_measured_bf16_sustained_x2": round(value / world / (2 * peaks["bf16_sustained"]), 4)}
        if mhz and mhz_max:
            out["of_nominal_4500_at_sampled_clock"] = round(value / world / (4500.0 * mhz / mhz_max), 4)
            out["tflops_per_sm_ghz"] = round(value / world / (mhz / 1e3), 1)
        return out

    r = measure(cfg_name, cfg, args.own_stream, args.min_seconds)
    ms, value, clocks, stats = r["ms"], r["value"], r["clocks"], r["stats"]
    line = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms / args.steps, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "fp8_e4m3_e5m2_fp32acc", "data": "synthetic",
        "config": {
            "workload": cfg_name, "tokens": cfg["T"], "linears": [[n, K, N] for n, K, N in cfg["linears"]],
            "layers": cfg["layers"], "microbatches": cfg["M"], "schedule": "sched(M,%d,%d) zero-bubble style, dW deferred" % cfg["sched"],
            "history_len": cfg["H"], "exec": args.mode, "overlap_dw": bool(args.overlap_dw and not args.step_api), "issue": "qe_step_run (one call per step)" if args.step_api else ("rounds of independent per-linear actions (schedules.plan_rounds, window %d), one qe_run_together call each" % r["window"]) if r["window"] else "one C-ABI call per action; a forward and the input gradient (and deferred dW) that follow it in the schedule go out linear by linear through qe_forward_dI_pair / qe_run_together" if args.pair_f_di else "one C-ABI call per action", "chained_fp8_handoff": bool(args.chain), "f_with_next_dI": "one shared GEMM launch per (F of linear i, dI of linear n-1-i)" if (args.pair_f_di and not args.chain and not args.step_api) else "separate", "gradient_path": "per-microbatch bf16 arena + reduction" if args.arena else "staged copy-add" if args.staged else "direct placement", "dw_launches": "shared by up to 4 linears" if (args.group_dw and not args.staged and not args.arena) else "one per linear", "exec_stream": "context-owned (event handoffs)" if args.own_stream else "caller's stream", "parallelism": "replicas x%d (path does not shard)" % world,
            "l2": "per-step inputs (%.0f MB) exceed L2; distinct tensors per microbatch" % (
                sum(cfg["T"] * (K + N) * 2 for _, K, N in cfg["linears"]) * cfg["M"] * cfg["layers"] / 1e6),
            "flop_per_step": step_flops(cfg),
            "timing": "median of the timed blocks of --steps steps each, repeated until %.1f s of device time" % args.min_seconds,
        },
        "gpu_launches": int(r["launches"]),
        "host_issue_ms_per_step": round(r["issue_ms"], 3),
        "clocks": clocks,
        "timed": block_summary(r["blocks"], args.steps, r["flop"], world),
        "frac_of_fp8_peak": fractions(value, clocks.get("sm_mhz"), clocks.get("sm_max_mhz")),
        "stats": {k: (round(v, 3) if isinstance(v, float) else v) for k, v in stats.items()},
        "device_status": int(r["status"]),
    }

    if not args.no_extras:
        if not args.own_stream:
            # the same step with a context-owned execution stream: the caller->exec wait and the exec->caller event of
            # Sec. 4.4 on every call (the default run executes on the caller's own stream, where stream order gives
            # the same guarantee and no event is needed)
            o = measure(cfg_name, cfg, True, min(args.min_seconds, 1.0))
            line["own_stream"] = {"value": round(o["value"], 2), "ms_per_step": round(o["ms"] / args.steps, 4),
                                  "handoffs_per_step": o["stats"]["handoffs"] // max(1, (args.steps * len(o["blocks"]) + args.warmup)),
                                  "sm_mhz": o["clocks"].get("sm_mhz"), "blocks": len(o["blocks"])}
        # (one host call per action: finer-grained than qe_run_together_host per round, so more of the transfers overlap)
        stage = Stage(qe, cfg_name, cfg, args.mode, device, host_io=True, same_stream=not args.own_stream, overlap_dw=args.overlap_dw)
        big = step_flops(cfg) > 50e12
        n2 = 3 if big else min(20, max(2, args.steps // 2))
        ms2, _, _ = time_steps(stage, n2, 3, True, dist)
        line["e2e"] = {"value": round(step_flops(cfg) * n2 * world / (ms2 * 1e-3) / 1e12, 2), "unit": UNIT,
                       "h2d_bytes_per_step": stage.h2d // n2, "d2h_bytes_per_step": stage.d2h // n2,
                       "ms_per_step": round(ms2 / n2, 3), "steps": n2, "warmup": 3, "host_buffer_sets": stage.host_sets,
                       "what": "qe_forward_host / qe_backward_dI_host with pinned host X, dY, Y, dX for every microbatch; gradient buffer read back after each step"}
        del stage
        torch.cuda.empty_cache()
        if rank == 0:
            line["roofline"] = gemm_roofline(qe, cfg_name, cfg, peaks, device)
            line["roofline"]["gemm_share_of_step"] = round(line["roofline"]["gemm_ms_per_step"] / (ms / args.steps), 3)
            torch.cuda.empty_cache()
            line["hbm_kernels"] = hbm_kernels(qe, cfg, peaks, device)
        if cfg_name != "C2" and not (args.staged or args.arena or args.chain):
            # the Llama-block configuration with hidden size 2048 rides along: its weight-gradient GEMMs are as much
            # HBM- as tensor-bound and every launch's fixed cost weighs more, so it is the harder shape set
            c2 = inputs.CONFIGS["C2"]
            r2 = measure("C2", c2, args.own_stream, min(args.min_seconds, 1.0))
            line["c2"] = {"workload": "C2", "value": round(r2["value"], 2), "ms_per_step": round(r2["ms"] / args.steps, 4),
                          "timed": block_summary(r2["blocks"], args.steps, r2["flop"], world), "clocks": r2["clocks"],
                          "frac_of_fp8_peak": fractions(r2["value"], r2["clocks"].get("sm_mhz"), r2["clocks"].get("sm_max_mhz")),
                          "gpu_launches": int(r2["launches"]), "device_status": int(r2["status"])}
            if rank == 0:
                # its per-action rates and its 6 ms launch loop are set against the burst figure, which was measured on an
                # idle part: let the part idle first too (the config-2 blocks above just ran under the power cap)
                torch.cuda.synchronize()
                time.sleep(IDLE_BEFORE_BURST_S)
                line["c2"]["idle_before_roofline_s"] = IDLE_BEFORE_BURST_S
                line["c2"]["roofline"] = gemm_roofline(qe, "C2", c2, peaks, device)
                line["c2"]["roofline"]["gemm_share_of_step"] = round(line["c2"]["roofline"]["gemm_ms_per_step"] / (r2["ms"] / args.steps), 3)
                torch.cuda.empty_cache()
        if rank == 0 and world == 1:
            only, sample = oracle_sample_choice(cfg_name, cfg)
            s_, f_ = oracle_sample(cfg_name, cfg, only)
            line["cpu_baseline"] = {"value": round(f_ / s_ / 1e12, 5), "unit": UNIT, "cores": _threads(), "kind": "oracle",
                                    "sample": "%s, %.1f s" % (sample, s_)}
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
