#!/usr/bin/env python
"""Benchmark of the routed-MoE expert hot path on B200.

A "step" is one pass of the whole path -- moe_plan (counts, offsets, permutation, tile list)
and moe_run (the persistent kernel: gate/up GEMM + SwiGLU, down GEMM, combine) -- over one
synthetic batch of the chosen workload (for c4: all 8 layers, with moe_set_budget between
them).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4] [--impl reference]

N > 1 runs N independent replicas (one process per GPU, no data-path collective); the
reported value is all ranks' work over the slowest rank's device time.
`--impl reference` times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import synth  # noqa: E402

METRIC = "moe_expert_tflops"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
def plan_kernels(n_tokens: int, top_k: int, n_experts: int) -> int:
    """Kernels one moe_plan call launches: histogram, scan + tile list, scatter -- or one block
    that runs all three passes when the op has at most 8192 routed rows and 256 experts."""
    return 1 if (n_tokens * top_k <= 8192 and n_experts <= 256) else 3


DEFAULT_STEPS = {"c2": (200, 10), "c3": (30, 5), "c4": (4, 3), "c5": (30, 5), "c2s": (20, 3), "c3s": (10, 3), "c4s": (5, 3), "c5s": (10, 3)}



# DRAM bytes per launch of the persistent kernel (dram__bytes_read.sum + dram__bytes_write.sum) from one ncu
# capture each.  The captures are of the small variants (c3s, c2s, c5s: a full-size launch under the profiler's
# save/restore is too large); the full-size figures scale them by the number of active experts, because the
# traffic is the weights of the active experts, read about once (c3: 256/64, c2: 251/63, c5: 256/32).
NCU_DRAM_BYTES = {
    ("c3s", "moe_apk_pair_kernel"): 2.050e9 + 0.163e9,
    ("c3", "moe_apk_pair_kernel"): (2.050e9 + 0.163e9) * 256 / 64,
    ("c2s", "moe_apk_pair_kernel"): 1.816e9 + 0.016e9,
    ("c2", "moe_apk_pair_kernel"): (1.816e9 + 0.016e9) * 251 / 63,
    ("c4s", "moe_apk_pair_kernel"): 3.116e9 + 0.337e9,           # decode + prefill op paired (carrier tiles)
    ("c4", "moe_apk_pair_kernel"): (3.116e9 + 0.337e9) * 256 / 64,
    ("c5s", "moe_apk_kernel"): 1.570e9 + 0.062e9,                # paired, decode budget 96
    ("c5", "moe_apk_kernel"): (1.570e9 + 0.062e9) * 256 / 32,
}

def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap"}

    def __init__(self, index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
            self._period = period_s
        except Exception:
            self._nv = None

    def _loop(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self._period)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)

    def summary(self):
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------------ workloads

def visible_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


class Workload:
    """Device-resident inputs of one workload plus the calls of one step."""

    def __init__(self, name: str, rank: int, device: torch.device, tile_log: int = 0, pair: bool = True):
        """Generates the workload's seeded inputs on the host, uploads them and plans nothing yet.
        pair: a co-scheduled decode + prefill op of a layer run in their paired form (moe_plan_pair: decode rows
        travel in carrier tiles with prefill rows of the same expert, each weight tile is streamed once)."""
        self.pair = pair
        import paper_2607_18002_b200 as moe
        self.moe = moe
        self.name = name
        base = synth.SPECS[name]
        self.spec = synth.scaled(base, seed=base.seed + 100 * rank)
        sh = self.spec.shape
        self.sh = sh
        self.device = device
        n_sets = 2 if self.spec.layers > 1 else 1          # c4 alternates two weight sets
        threads = os.cpu_count() or 8
        self.W_host = [synth.make_weights(self.spec, layer=i, threads=threads) for i in range(n_sets)]
        dev = lambda t: None if t is None else t.to(device)
        self.W = [synth.Weights(dev(w.w_gate_up), dev(w.w_down), dev(w.s_gate_up), dev(w.s_down))
                  for w in self.W_host]
        self.fp8 = sh.dtype == "fp8"
        el = 1 if self.fp8 else 2
        self.layers = []
        # the paired form keeps the rows of both ops in one slot's scratch
        self.max_tokens = sum(T for _, T in self.spec.ops) if len(self.spec.ops) > 1 else self.spec.ops[0][1]
        self.ctx = moe.Context(sh.E, sh.k, sh.H, sh.I, self.max_tokens,
                               max_ops=len(self.spec.ops), tile_log_entries=tile_log,
                               dtype=moe.MOE_DTYPE_FP8_E4M3 if self.fp8 else moe.MOE_DTYPE_BF16,
                               device=device)
        self.flops = 0.0
        self.bytes_alg = 0.0
        self.h2d = self.d2h = 0
        for layer in range(self.spec.layers):
            ops = synth.make_ops(self.spec, layer)
            W = self.W[layer % n_sets]
            bound, host = [], []
            active = np.zeros(sh.E, dtype=bool)
            for op in ops:
                hx = op.x.pin_memory()
                hi = torch.from_numpy(op.ids).pin_memory()
                hw = torch.from_numpy(op.w).pin_memory()
                dx, di, dw = hx.to(device), hi.to(device), hw.to(device)
                hs = None if op.x_scale is None else op.x_scale.pin_memory()
                b = self.ctx.bind(op.cls, dx, di, dw, W.w_gate_up, W.w_down, x_scale=dev(hs),
                                  s_gate_up=W.s_gate_up, s_down=W.s_down)
                hy = torch.empty(b.y.shape, dtype=b.y.dtype).pin_memory()
                bound.append(b)
                host.append((hx, hi, hw, hy, hs))
                active[np.unique(op.ids)] = True
                self.flops += 6.0 * op.ids.size * sh.H * sh.I
                self.bytes_alg += op.T * sh.H * (el + 2)         # X once, y (bf16) once
                if hs is not None:
                    self.bytes_alg += hs.numel() * 4
                self.h2d += hx.numel() * el + hi.numel() * 4 + hw.numel() * 4 + (0 if hs is None else hs.numel() * 4)
                self.d2h += hy.numel() * 2
            # weights of the union of active experts of the launch, once
            self.bytes_alg += float(active.sum()) * 3 * sh.H * sh.I * el
            if self.fp8:
                self.bytes_alg += float(active.sum()) * 3 * (sh.H // 128) * (sh.I // 128) * 4
            self.layers.append((ops, bound, host))
        self.launches_per_step = sum(sum(plan_kernels(o.T, sh.k, sh.E) for o in ops_) + 1 + (1 if self.budget_for(li_) is not None else 0)
                                     + (2 if self._pairs(ops_) else 0) for li_, (ops_, _, _) in enumerate(self.layers))

    def budget_for(self, li: int):
        """Decode SM budget written ahead of layer li's launch (None: the budget word is left alone)."""
        if self.spec.layers > 1:
            return synth.C4_BUDGETS[li % len(synth.C4_BUDGETS)]
        if len(self.spec.ops) > 1:
            return synth.C5_BUDGET
        return None

    def _pairs(self, ops):
        """(prefill slot, decode slot) of a layer that runs paired, else None."""
        if not self.pair or len(ops) != 2:
            return None
        cls = [o.cls for o in ops]
        if sorted(cls) != [synth.DECODE, synth.PREFILL]:
            return None
        return cls.index(synth.PREFILL), cls.index(synth.DECODE)

    def plan_layer(self, ctx, ops, bound):
        for s, b in enumerate(bound):
            ctx.plan(s, b)
        pr = self._pairs(ops)
        if pr:
            ctx.plan_pair(pr[0], pr[1], 0)

    def step(self, ev=None):
        """Whole hot path for one batch; ev (optional) collects (before_run, after_run) events."""
        ctx = self.ctx
        for li, (ops, bound, _) in enumerate(self.layers):
            if self.budget_for(li) is not None:
                ctx.set_budget(self.budget_for(li))
            self.plan_layer(ctx, ops, bound)
            if ev is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            ctx.run(list(range(len(bound))), fuse_combine=True)
            if ev is not None:
                e1.record()
                ev.append((e0, e1))

    def _second_set(self):
        """A second context and a second set of device buffers for every op: the end-to-end loop
        alternates between the two sets, so that the copies of one step overlap the kernels of the
        neighbouring steps (what a serving loop does with its input and output staging)."""
        if getattr(self, "ctx2", None) is not None:
            return
        moe, sh, device = self.moe, self.sh, self.device
        dev = lambda t: None if t is None else t.to(device)
        self.ctx2 = moe.Context(sh.E, sh.k, sh.H, sh.I, self.max_tokens,
                                max_ops=len(self.spec.ops),
                                dtype=moe.MOE_DTYPE_FP8_E4M3 if self.fp8 else moe.MOE_DTYPE_BF16, device=device)
        n_sets = len(self.W)
        self.layers2 = []
        for layer, (ops, bound, host) in enumerate(self.layers):
            W = self.W[layer % n_sets]
            b2 = []
            for op, (hx, hi, hw, hy, hs) in zip(ops, host):
                b2.append(self.ctx2.bind(op.cls, hx.to(device), hi.to(device), hw.to(device), W.w_gate_up, W.w_down,
                                         x_scale=dev(hs), s_gate_up=W.s_gate_up, s_down=W.s_down))
            self.layers2.append((ops, b2, host))
        self.s_h2d, self.s_comp, self.s_d2h = (torch.cuda.Stream(device=device) for _ in range(3))

    def run_e2e_serial(self, steps: int):
        """The same end-to-end step on ONE stream, nothing overlapped: copy in, plan, run, copy out, and the
        host waits for the result before it starts the next step.  The difference to run_e2e is what the
        copies cost when they are not hidden behind the neighbouring steps' kernels."""
        ctx = self.ctx
        for _ in range(steps):
            for li, (ops, bound, host) in enumerate(self.layers):
                for b, (hx, hi, hw, hy, hs) in zip(bound, host):
                    b.x.copy_(hx, non_blocking=True)
                    if hs is not None:
                        b.x_scale.copy_(hs, non_blocking=True)
                    b.topk_ids.copy_(hi, non_blocking=True)
                    b.topk_w.copy_(hw, non_blocking=True)
                if self.budget_for(li) is not None:
                    ctx.set_budget(self.budget_for(li))
                self.plan_layer(ctx, ops, bound)
                ctx.run(list(range(len(bound))), fuse_combine=True)
                for b, (_, _, _, hy, _) in zip(bound, host):
                    hy.copy_(b.y, non_blocking=True)
            torch.cuda.synchronize(self.device)

    def run_e2e(self, steps: int):
        """`steps` steps with host buffers: every step copies its inputs from pinned host memory,
        plans, runs and copies its result back to pinned host memory.  Copies and kernels run on
        three streams over two sets of device buffers; a set is reused only after its results have
        left the device.  Returns when everything has finished."""
        self._second_set()
        sets = [(self.ctx, self.layers), (self.ctx2, self.layers2)]
        free = {}
        for step in range(steps):
            ctx, layers = sets[step % 2]
            for li, (ops_l, bound, host) in enumerate(layers):
                key = (step % 2, li)
                with torch.cuda.stream(self.s_h2d):
                    if key in free:
                        self.s_h2d.wait_event(free[key])
                    for b, (hx, hi, hw, hy, hs) in zip(bound, host):
                        b.x.copy_(hx, non_blocking=True)
                        if hs is not None:
                            b.x_scale.copy_(hs, non_blocking=True)
                        b.topk_ids.copy_(hi, non_blocking=True)
                        b.topk_w.copy_(hw, non_blocking=True)
                    e_in = torch.cuda.Event()
                    e_in.record(self.s_h2d)
                with torch.cuda.stream(self.s_comp):
                    self.s_comp.wait_event(e_in)
                    if self.budget_for(li) is not None:
                        ctx.set_budget(self.budget_for(li))
                    self.plan_layer(ctx, ops_l, bound)
                    ctx.run(list(range(len(bound))), fuse_combine=True)
                    e_run = torch.cuda.Event()
                    e_run.record(self.s_comp)
                with torch.cuda.stream(self.s_d2h):
                    self.s_d2h.wait_event(e_run)
                    for b, (_, _, _, hy, _) in zip(bound, host):
                        hy.copy_(b.y, non_blocking=True)
                    e_out = torch.cuda.Event()
                    e_out.record(self.s_d2h)
                free[key] = e_out
        torch.cuda.synchronize(self.device)


def oracle_sample(w: Workload, seconds_target: float = 12.0):
    """Times the CPU oracle, as it stands, on a bounded token sample of the workload's first
    op.  Returns (TFLOP/s, cores, description)."""
    import oracle
    sh = w.sh
    ops, _, _ = w.layers[0]
    op = max(ops, key=lambda o: o.T)
    Wh = w.W_host[0]
    OW = oracle.Weights(sh.E, sh.k, sh.H, sh.I, Wh.w_gate_up, Wh.w_down, Wh.s_gate_up, Wh.s_down)
    rA = oracle.ROUND_E4M3_1X128 if sh.dtype == "fp8" else oracle.ROUND_NONE
    cores = oracle.threads()
    n, spent, done_tokens = max(2, cores // sh.k), 0.0, 0
    rng = np.random.default_rng(0)
    while True:                       # grow the sample until the time budget is used
        toks = rng.choice(op.T, size=min(n, op.T), replace=False).astype(np.int32)
        t0 = time.perf_counter()
        oracle.plan(op.ids, sh.E)
        oracle.forward_tokens(OW, op.x, op.x_scale, op.ids, op.w, toks, round_A=rA)
        dt = time.perf_counter() - t0
        spent += dt
        done_tokens, last_dt = len(toks), dt
        if spent + 3 * dt > seconds_target or len(toks) == op.T:
            break
        n *= 2
    tflops = 6.0 * done_tokens * sh.k * sh.H * sh.I / last_dt / 1e12
    return tflops, cores, (f"oracle plan on all {op.T} tokens + FFN/combine on {done_tokens} "
                           f"seeded tokens of {w.name} ({last_dt:.2f} s)")


def _pcts(v):
    return {"n": int(len(v)), "p50_us": float(np.percentile(v, 50)), "p99_us": float(np.percentile(v, 99)),
            "mean_us": float(v.mean()), "max_us": float(v.max())}


def _log_summary(log):
    """Per class and tile kind, two readings of a tile's time from the kernel's tile log: its SERVICE time
    (claim -> commit) and its LATENCY (the moment it could first have run -> commit; every op of these
    launches is ready at launch, so that moment is the launch's first claim).  Plus op spans, CTA occupancy."""
    out = {"records": int(len(log))}
    if len(log) == 0:
        return out
    t0 = int(log["t_claim"].min())
    span = (int(log["t_commit"].max()) - t0) / 1e3
    out["kernel_span_us"] = span
    service = (log["t_commit"].astype(np.int64) - log["t_claim"].astype(np.int64)) / 1e3
    latency = (log["t_commit"].astype(np.int64) - t0) / 1e3
    names = {0: "gate_up", 1: "down", 2: "combine"}
    for cls, cname in ((0, "decode"), (1, "prefill")):
        mc = log["cls"] == cls
        if not mc.any():
            continue
        gemm = mc & (log["kind"] < 2)
        if gemm.any():
            out[f"{cname}_tile"] = _pcts(service[gemm])
            out[f"{cname}_tile_latency"] = _pcts(latency[gemm])
        out[f"{cname}_op_us"] = float((int(log["t_commit"][mc].max()) - t0) / 1e3)
        out[f"{cname}_first_claim_us"] = float((int(log["t_claim"][mc].min()) - t0) / 1e3)
        for kind, kname in names.items():
            m = mc & (log["kind"] == kind)
            if m.any():
                out[f"{cname}_{kname}"] = _pcts(service[m])
    ctas = np.unique(log["cta"])
    out["ctas_with_tiles"] = int(len(ctas))
    # busy time per CTA = union of its (overlapping) tile intervals
    busy = 0.0
    for c in ctas:
        r = log[log["cta"] == c]
        order = np.argsort(r["t_claim"])
        a, b = r["t_claim"][order].astype(np.int64), r["t_commit"][order].astype(np.int64)
        end = np.maximum.accumulate(b)
        start_new = np.concatenate([[True], a[1:] > end[:-1]])
        seg_start = a[start_new]
        seg_end = np.concatenate([end[:-1][start_new[1:]], end[-1:]])
        busy += float((seg_end - seg_start).sum()) / 1e3
    out["queue_occupancy"] = busy / (len(ctas) * span) if span > 0 else None
    return out


def _ratios(co, iso):
    """Co-run over isolated, for both readings of a decode tile's time and for the whole decode op."""
    r = {}
    if "decode_tile" in co and "decode_tile" in iso:
        for key, name in (("decode_tile", "service"), ("decode_tile_latency", "latency")):
            r[f"decode_tile_{name}_p50_ratio"] = co[key]["p50_us"] / iso[key]["p50_us"]
            r[f"decode_tile_{name}_p99_ratio"] = co[key]["p99_us"] / iso[key]["p99_us"]
        r["decode_op_ratio"] = co["decode_op_us"] / iso["decode_op_us"]
        r["decode_op_us"] = {"corun": co["decode_op_us"], "isolated": iso["decode_op_us"]}
        if "prefill_op_us" in co:
            r["prefill_op_us_corun"] = co["prefill_op_us"]
    return r


def tile_stats(w: Workload):
    """Per-tile timing from the kernel's tile log (extra, untimed launches): the analogue of the paper's
    preemption-interval measurement (Section 7.6).  For a co-scheduled workload, one layer per decode budget
    of the workload is launched twice -- both ops together, then the decode op alone at the same budget
    ("isolated") -- and the decode tiles' times are compared under both readings (service: claim -> commit;
    latency: launch -> commit), next to the decode op's completion time."""
    ctx = w.ctx
    mixed = any(len(bound) > 1 for _, bound, _ in w.layers)
    if not mixed:
        w.step()
        ctx.check()
        return {"corun": _log_summary(ctx.tile_log())}
    out = {"per_budget": {}, "paired": bool(w.pair)}
    # the workload's own budgets, then larger ones: the latency of a decode op that streams most experts'
    # weights follows its share of the SMs (and with it of the HBM bandwidth)
    own = tuple(synth.C4_BUDGETS) if w.spec.layers > 1 else (w.budget_for(0),)
    budgets = own + ((96, 112, 128) if w.spec.layers > 1 else ())
    pooled = {"co": [], "iso": []}
    for bi, q in enumerate(budgets):
        li = bi % len(w.layers)
        ops, bound, _ = w.layers[li]
        dec = [s for s, b in enumerate(bound) if b.c.cls == 0]
        if q is not None:
            ctx.set_budget(q)
        w.plan_layer(ctx, ops, bound)
        ctx.run(list(range(len(bound))), fuse_combine=True)
        ctx.check()
        log_co = ctx.tile_log()
        co = _log_summary(log_co)
        ctx.run(dec, fuse_combine=True)           # one op of a pair alone: the plain form runs
        ctx.check()
        log_iso = ctx.tile_log()
        iso = _log_summary(log_iso)
        entry = {"layer": li, "corun": co, "decode_isolated": iso}
        entry.update(_ratios(co, iso))
        if w.pair:                                 # the same launch without pairing, for comparison
            for s, b in enumerate(bound):
                ctx.plan(s, b)
            ctx.run(list(range(len(bound))), fuse_combine=True)
            ctx.check()
            un = _log_summary(ctx.tile_log())
            entry["unpaired"] = {"kernel_span_us": un["kernel_span_us"], "decode_op_us": un["decode_op_us"],
                                 "decode_op_ratio": un["decode_op_us"] / iso["decode_op_us"]}
        out["per_budget"][str(q)] = entry
        if q not in own:
            continue                               # the pooled percentiles are over the workload's own budgets
        for key, lg in (("co", log_co), ("iso", log_iso)):
            m = (lg["cls"] == 0) & (lg["kind"] < 2)
            t0 = int(lg["t_claim"].min())
            pooled[key].append(np.stack([(lg["t_commit"][m].astype(np.int64) - lg["t_claim"][m].astype(np.int64)) / 1e3,
                                         (lg["t_commit"][m].astype(np.int64) - t0) / 1e3]))
    co, iso = np.concatenate(pooled["co"], axis=1), np.concatenate(pooled["iso"], axis=1)
    for i, name in enumerate(("service", "latency")):
        out[f"decode_tile_{name}_p50_ratio"] = float(np.percentile(co[i], 50) / np.percentile(iso[i], 50))
        out[f"decode_tile_{name}_p99_ratio"] = float(np.percentile(co[i], 99) / np.percentile(iso[i], 99))
        out[f"decode_tile_{name}_us"] = {"corun_p50": float(np.percentile(co[i], 50)), "corun_p99": float(np.percentile(co[i], 99)),
                                         "isolated_p50": float(np.percentile(iso[i], 50)),
                                         "isolated_p99": float(np.percentile(iso[i], 99))}
    out["decode_op_ratio"] = {q: e["decode_op_ratio"] for q, e in out["per_budget"].items() if "decode_op_ratio" in e}
    out["decode_tile_latency_p99_ratio_by_budget"] = {q: e["decode_tile_latency_p99_ratio"] for q, e in out["per_budget"].items()
                                                      if "decode_tile_latency_p99_ratio" in e}
    within = [int(q) for q, r in out["decode_tile_latency_p99_ratio_by_budget"].items() if q != "None" and r <= 1.3]
    out["smallest_budget_with_latency_p99_within_1.3x"] = min(within) if within else None
    out["readings"] = ("service = commit - claim of a decode tile; latency = commit - launch start (all ops ready at "
                       "launch); isolated = the same decode op alone in the launch at the same budget")
    _, bound, _ = w.layers[min(1, len(w.layers) - 1)]
    dec = [s for s, b in enumerate(bound) if b.c.cls == 0]
    if w.spec.layers > 1:
        ctx.set_budget(synth.C4_BUDGETS[1])
    out["decode_arrives_mid_prefill"] = _mid_run_arrival(w, bound, dec)
    return out


def _mid_run_arrival(w: Workload, bound, dec):
    """The decode op becomes ready while the prefill op of the same launch is being served: its
    ready word is the prefill op's notify word, which the kernel sets once a third of the prefill
    tiles have committed.  Reports the time from that commit to the first decode claim (the
    preemption delay, bounded by the tile a unit runs plus the one it claimed ahead) next to the
    prefill tile times."""
    pre = [s for s in range(len(bound)) if s not in dec]
    ps, ds = pre[0], dec[0]
    word = torch.zeros(1, dtype=torch.int32, device=w.device)
    w.ctx.plan(ps, bound[ps])
    n_pre = w.ctx.footprint(ps)[1]
    after = max(1, n_pre // 3)
    bp, bd = bound[ps], bound[ds]
    bp.c.notify, bp.c.notify_after, bd.c.ready = word.data_ptr(), after, word.data_ptr()
    try:
        w.ctx.plan(ps, bp)
        w.ctx.plan(ds, bd)
        w.ctx.run([ps, ds], fuse_combine=True)
        w.ctx.check()
        log = w.ctx.tile_log()
    finally:
        bp.c.notify, bp.c.notify_after, bd.c.ready = None, 0, None
        w.ctx.plan(ps, bp)
        w.ctx.plan(ds, bd)
    p, d = log[log["slot"] == ps], log[log["slot"] == ds]
    t_ready = int(np.sort(p["t_commit"])[after - 1])
    first = int(d["t_claim"].min())
    gemm = p[p["kind"] < 2]
    service = (gemm["t_commit"].astype(np.int64) - gemm["t_claim"].astype(np.int64)) / 1e3
    dsvc = (d["t_commit"].astype(np.int64) - d["t_claim"].astype(np.int64))[d["kind"] < 2] / 1e3
    return {"ready_after_prefill_tiles": int(after), "prefill_tiles": int(n_pre),
            "ready_to_first_decode_claim_us": (first - t_ready) / 1e3,
            "prefill_tile_p50_us": float(np.percentile(service, 50)), "prefill_tile_p99_us": float(np.percentile(service, 99)),
            "decode_tile_p50_us": float(np.percentile(dsvc, 50)), "decode_tile_p99_us": float(np.percentile(dsvc, 99)),
            "decode_op_us": float((int(d["t_commit"].max()) - t_ready) / 1e3)}


def persistent_layers(w: Workload, steps: int, warmup: int):
    """The multi-layer workload as ONE persistent launch per step: all ops of all layers in one
    moe_run, prefill l after prefill l-1 and decode l after prefill l-1 (after_op), every decode op
    carrying the SM budget of its layer (moe_op_t.decode_sms) -- no launch, no host call and no
    separate budget write between layers.  Same inputs, same plan calls as the per-layer step."""
    moe, sh = w.moe, w.sh
    n_layers = len(w.layers)
    ctx = moe.Context(sh.E, sh.k, sh.H, sh.I, w.max_tokens, max_ops=2 * n_layers,
                      dtype=moe.MOE_DTYPE_FP8_E4M3 if w.fp8 else moe.MOE_DTYPE_BF16, device=w.device)
    bound = []
    for l, (ops, b_old, _) in enumerate(w.layers):
        W = w.W[l % len(w.W)]
        prev_prefill = next((2 * (l - 1) + j for j, o in enumerate(w.layers[l - 1][0]) if o.cls == synth.PREFILL), -1) if l else -1
        for op, b in zip(ops, b_old):
            bound.append(ctx.bind(op.cls, b.x, b.topk_ids, b.topk_w, W.w_gate_up, W.w_down, x_scale=b.x_scale,
                                  s_gate_up=W.s_gate_up, s_down=W.s_down, after_op=prev_prefill,
                                  decode_sms=synth.C4_BUDGETS[l % len(synth.C4_BUDGETS)] if op.cls == synth.DECODE else 0))
    slots = list(range(len(bound)))

    def step():
        for s_, b in enumerate(bound):
            ctx.plan(s_, b)
        for l, (ops, _, _) in enumerate(w.layers):         # the two ops of a layer paired, as in the per-layer step
            pr = w._pairs(ops)
            if pr:
                ctx.plan_pair(2 * l + pr[0], 2 * l + pr[1], 0)
        ctx.run(slots, fuse_combine=True)

    for _ in range(warmup):
        step()
    ctx.check()
    torch.cuda.synchronize()
    # The two forms alternate step by step, so that both see the same clocks (the power limit moves
    # them over a run of this length).
    t_one, t_per = [], []
    for _ in range(steps):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        ev[0].record()
        step()
        ev[1].record()
        w.step()
        ev[2].record()
        torch.cuda.synchronize()
        t_one.append(ev[0].elapsed_time(ev[1]))
        t_per.append(ev[1].elapsed_time(ev[2]))
    ctx.check()
    w.ctx.check()
    ms = float(np.mean(t_one))
    same = all(torch.equal(b.y, bo.y) for b, (_, b_old, _) in zip([bound[i:i + 2] for i in range(0, len(bound), 2)], w.layers)
               for b, bo in zip(b, b_old)) if all(len(x[1]) == 2 for x in w.layers) else None
    return {"ms_per_step": ms, "value": w.flops / (ms / 1e3) / 1e12, "unit": UNIT, "ops_in_launch": len(bound),
            "launches_per_step": sum(plan_kernels(o.T, sh.k, sh.E) for ops_, _, _ in w.layers for o in ops_) + 1
                                 + sum(2 for ops_, _, _ in w.layers if w._pairs(ops_)),
            "outputs_equal_per_layer_launches": same,
            "per_layer_launches_ms_per_step_alternating": float(np.mean(t_per))}


# ------------------------------------------------------------------ arms

def run_reference(args):
    """The reference arm: the CPU oracle on the host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    spec = synth.SPECS[args.workload]
    sh = spec.shape
    Wh = synth.make_weights(spec, threads=os.cpu_count() or 8)
    op = max(synth.make_ops(spec), key=lambda o: o.T)
    OW = oracle.Weights(sh.E, sh.k, sh.H, sh.I, Wh.w_gate_up, Wh.w_down, Wh.s_gate_up, Wh.s_down)
    rA = oracle.ROUND_E4M3_1X128 if sh.dtype == "fp8" else oracle.ROUND_NONE
    cores = oracle.threads()
    n_tok = max(4, (2 * cores) // sh.k)
    rng = np.random.default_rng(0)
    times = []
    for i in range(args.warmup + args.steps):
        toks = rng.choice(op.T, size=min(n_tok, op.T), replace=False).astype(np.int32)
        t0 = time.perf_counter()
        oracle.plan(op.ids, sh.E)
        oracle.forward_tokens(OW, op.x, op.x_scale, op.ids, op.w, toks, round_A=rA)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * float(np.mean(times))
    value = 6.0 * min(n_tok, op.T) * sh.k * sh.H * sh.I / (ms / 1e3) / 1e12
    sample = f"per step: oracle plan on all {op.T} tokens + FFN/combine on {min(n_tok, op.T)} seeded tokens"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# steps / warm-up of the workloads that ride along with the default run (one JSON line for all targets)
SUB_STEPS = {"c2": (100, 5), "c4": (2, 3), "c5": (15, 4)}


def measure(name: str, args, K: int, Wm: int, rank: int, world: int, local: int, device, peaks, peak_src,
            tile_log: bool, e2e: bool, one_launch: bool):
    """Times one workload: device-resident steps (CUDA events, barrier on both sides), the live duration of
    every persistent launch for the roofline, optionally the end-to-end loops with host buffers and the
    tile-log statistics.  Returns the fields of a bench line."""
    from paper_2607_18002_b200 import dist
    w = Workload(name, rank, device, tile_log=(1 << 17) if tile_log else 0, pair=not args.no_pair)
    for _ in range(Wm):
        w.step()
    w.ctx.check()

    # ---- device-resident timing
    ev = []
    dist.barrier()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(visible_index(local)) as clk:
        start.record()
        for _ in range(K):
            w.step(ev)
        stop.record()
        torch.cuda.synchronize()
    dist.barrier()
    w.ctx.check()
    secs = start.elapsed_time(stop) / 1e3
    run_ms = [a.elapsed_time(b) for a, b in ev]
    value = dist.job_throughput(w.flops * K, secs) / 1e12
    ms_per_step = 1e3 * dist.reduce_scalar(secs, "max") / K

    # ---- end to end with host buffers (host clock around K steps, everything synchronised on both sides)
    e2e_out = e2e_serial = None
    if e2e:
        w.run_e2e(min(Wm, 3))
        dist.barrier()
        torch.cuda.synchronize()
        t_e2e = time.perf_counter()
        w.run_e2e(K)
        t_e2e = time.perf_counter() - t_e2e
        dist.barrier()
        w.ctx.check()
        w.ctx2.check()
        e2e_out = {"value": dist.job_throughput(w.flops * K, t_e2e) / 1e12, "unit": UNIT,
                   "h2d_bytes_per_step": w.h2d, "d2h_bytes_per_step": w.d2h,
                   "how": "two buffer sets over three streams: a step's copies overlap the neighbouring steps' kernels"}
        Ks = max(3, K // 3)
        w.run_e2e_serial(2)
        dist.barrier()
        t_ser = time.perf_counter()
        w.run_e2e_serial(Ks)
        t_ser = time.perf_counter() - t_ser
        dist.barrier()
        w.ctx.check()
        e2e_serial = {"value": dist.job_throughput(w.flops * Ks, t_ser) / 1e12, "unit": UNIT, "steps": Ks,
                      "ms_per_step": 1e3 * t_ser / Ks,
                      "how": "one stream, nothing overlapped, the host waits for every step's result"}

    # ---- roofline of the dominant kernel (the persistent kernel), from live CUDA events
    t_run = float(np.mean(run_ms)) / 1e3
    kernel_name = "moe_apk_pair_kernel" if w.ctx.ctas_per_tile == 2 else "moe_apk_kernel"
    flops_launch = w.flops / len(w.layers)
    bytes_launch = w.bytes_alg / len(w.layers)
    # the fp8 tensor peak is the measured bf16 peak x the nominal 2x ratio.  A kernel timed alone (one
    # launch per step) is held against the burst figure; the launches of a long multi-layer step run
    # under the power cap like the seconds-long cuBLAS loop, so they are held against the sustained one.
    long_step = len(w.layers) > 1
    tpeak = peaks["bf16_tflops_sustained" if long_step else "bf16_tflops"] * (2.0 if w.fp8 else 1.0)
    tensor_frac = flops_launch / t_run / 1e12 / tpeak
    hbm_frac = bytes_launch / t_run / 1e9 / peaks["hbm_gbs"]
    if name in ("c2", "c2s", "c5", "c5s"):
        roof = {"bound": "hbm", "achieved": bytes_launch / t_run / 1e9, "peak": peaks["hbm_gbs"],
                "unit": "GB/s", "frac": hbm_frac}
    else:
        roof = {"bound": "tensor", "achieved": flops_launch / t_run / 1e12,
                "peak": tpeak, "unit": "TFLOP/s", "frac": tensor_frac}
    # the captures of the co-scheduled workloads are of the paired form
    tkey = (name, kernel_name) if (w.pair or len(w.spec.ops) == 1) else None
    roof.update({"traffic": NCU_DRAM_BYTES.get(tkey), "kernel": kernel_name,
                 "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum of one launch of the small variant, "
                                   "scaled by active experts (see profiles/)"
                                   if tkey in NCU_DRAM_BYTES else None,
                 "peak_source": peak_src, "peak_kind": "sustained" if long_step else "burst",
                 "launch_ms_mean": 1e3 * t_run, "launch_ms_min": float(np.min(run_ms)),
                 "algorithmic_flops_per_launch": flops_launch,
                 "algorithmic_bytes_per_launch": bytes_launch,
                 "tensor_frac_of_burst": flops_launch / t_run / 1e12 / (peaks["bf16_tflops"] * (2.0 if w.fp8 else 1.0)),
                 "tensor_frac_of_sustained": flops_launch / t_run / 1e12 / (peaks["bf16_tflops_sustained"] * (2.0 if w.fp8 else 1.0)),
                 "hbm_frac": hbm_frac})

    tiles = tile_stats(w) if tile_log else None
    one = persistent_layers(w, K, Wm) if (one_launch and len(w.layers) > 1 and world == 1) else None

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and e2e:
        v, cores, sample = oracle_sample(w)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}

    sh = w.sh
    res = {"value": value, "unit": UNIT, "steps": K, "warmup": Wm, "ms_per_step": ms_per_step,
           "dtype": "fp8_e4m3" if w.fp8 else "bf16",
           "config": {"workload": name, "ops": [[c, t] for c, t in w.spec.ops],
                      "layers": w.spec.layers, "experts": sh.E, "top_k": sh.k, "hidden": sh.H,
                      "inter": sh.I, "l2": "inputs_exceed_l2 (weights >> 126 MB, no flush)",
                      "buffers": "the same X / y buffers every step: the step's 7-10 GB of weights pass through "
                                 "the 126 MB L2 between two uses of a buffer",
                      "replicas": world, "fused_combine": True,
                      "paired_ops": bool(w.pair and any(w._pairs(o) for o, _, _ in w.layers)),
                      "decode_budgets": sorted({w.budget_for(li) for li in range(len(w.layers))} - {None})},
           "clocks": clk.summary(), "gpu_launches": w.launches_per_step * K, "roofline": roof}
    if e2e_out:
        res["e2e"], res["e2e_serial"] = e2e_out, e2e_serial
    if cpu:
        res["cpu_baseline"] = cpu
    if tiles:
        res["tiles"] = tiles
    if one:
        res["one_launch_for_all_layers"] = one
    del w
    torch.cuda.empty_cache()
    return res


def run_ours(args):
    from paper_2607_18002_b200 import dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the library has no CPU path)")
    rank, world, local = dist.init_from_env()
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    peaks, peak_src = load_peaks()
    main_res = measure(args.workload, args, args.steps, args.warmup, rank, world, local, device, peaks, peak_src,
                       tile_log=args.tile_log, e2e=True, one_launch=args.one_launch)
    # The default run also measures the other targets of the metric on their own workloads: the decode-only
    # layer (HBM), the mixed 8-layer stream (decode-tile latency under prefill, from the tile log) and the
    # FP8 layer.  Each gets its own warm-up, timed region, clock record and status check.
    sub = {}
    if args.sub_results and world == 1:
        for name in ("c2", "c4", "c5"):
            if name == args.workload:
                continue
            k_, w_ = SUB_STEPS[name]
            sub[name] = measure(name, args, k_, w_, rank, world, local, device, peaks, peak_src,
                                tile_log=(name == "c4"), e2e=False, one_launch=False)
    if rank == 0:
        line = {"metric": METRIC, "value": main_res.pop("value"), "unit": UNIT, "n_gpus": world,
                "steps": main_res.pop("steps"), "warmup": main_res.pop("warmup"),
                "ms_per_step": main_res.pop("ms_per_step"), "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": main_res.pop("dtype"), "data": "synthetic"}
        line.update(main_res)
        line.setdefault("cpu_baseline", None)
        if sub:
            line["sub_results"] = sub
        print(json.dumps(line))
    dist.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="c3", choices=["c2", "c3", "c4", "c5", "c2s", "c3s", "c4s", "c5s"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tile-log", action="store_true", help="add per-tile timing statistics of one extra untimed step")
    ap.add_argument("--one-launch", action="store_true",
                    help="multi-layer workloads: also time all layers as one persistent launch per step")
    ap.add_argument("--no-pair", action="store_true",
                    help="co-scheduled workloads: run the decode and the prefill op unpaired (no carrier tiles)")
    ap.add_argument("--no-sub", action="store_true",
                    help="default workload only: skip the c2 / c4 / c5 sub-results")
    args = ap.parse_args()
    args.sub_results = args.workload == "c3" and not args.no_sub
    ds, dw = DEFAULT_STEPS[args.workload]
    if args.impl == "reference":
        ds, dw = 3, 1
    args.steps = ds if args.steps is None else args.steps
    args.warmup = max(3 if args.impl == "ours" else 0, dw if args.warmup is None else args.warmup)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
