#!/usr/bin/env python
"""Benchmark of the mixed-adapter LoRA apply on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config2|config5|config4|config3|config1|backward|moe_backward]
    python bench.py --impl reference ...        # the fp64 CPU oracle, timed on the host cores

A step is a fixed number of passes of the whole hot path over one batch: each
pass is one segment plan (token -> adapter grouping through the slot table)
followed by the fused apply of every LoRA target projection of every layer.
The default workload is the 4B-dense decode layer: T=256 requests, 64 resident
adapters with ranks from {1, 8, 16, 32}, Zipf(1.1) request->adapter, seven
projections per layer, 36 layers; every layer has its own pool, x and y so that
a pass streams about 4.2 GB (far beyond the 126 MB L2).  The step is captured
in a CUDA graph and replayed; times are CUDA-event times on the launching
stream.  The passes per step are chosen once, before timing, so that a step
lasts about 50 ms and the timed region (K steps) is long enough for the clock
sampler to see it.

Prints ONE JSON line (rank 0).  metric = tokens/s per layer: T * layers * passes
/ step time, summed over ranks (ranks are independent replicas: the path has no
exchange step, scaling is weak).  Besides the headline the line carries the
same measurement for the dependency-respecting call grouping, for the other
workloads, for the unfused pair of calls, for an L2-warm single layer and for
the admission path.
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "mixed-adapter LoRA apply tokens/s per layer"
UNIT = "tokens/s"
STAGES = [[0, 1, 2], [3], [4, 5], [6]]      # q,k,v | o | gate,up | down: what a decoder layer's dependencies allow


# --------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------
def build_workload(name: str, layers: int):
    """Host-side description: the cases of one layer plus the batch.  The device
    copies of the other layers are clones (values do not matter for timing,
    addresses do)."""
    from paper_2605_13779_b200 import synth
    if name == "config2":
        batch = synth.config2_batch()
        projs = list(synth.QWEN3_4B_PROJECTIONS)
        cases = [synth.config2_projection(batch, p, layer=0) for p in projs]
        return {"kind": "dense", "name": "config2: Qwen3-4B-shaped decode layer, T=256, 64 adapters r in {1,8,16,32}, Zipf(1.1), 7 projections",
                "T": batch.T, "cases": cases, "layers": layers or synth.QWEN3_4B_LAYERS}
    if name == "config5":
        case = synth.config5()
        return {"kind": "dense", "name": "config5: 7168->7168, T=2048, 4096 rank-1 slots of a 10^6 catalog, Zipf(0.9)",
                "T": case.T, "cases": [case], "layers": layers or 61}   # a 7168-wide model is about 61 layers deep
    if name == "config1":
        case = synth.config1()
        return {"kind": "dense", "name": "config1: 2560->2560, T=64, 4 rank-8 adapters", "T": case.T,
                "cases": [case], "layers": layers or 64}
    if name == "config3":
        batch = synth.config3_batch()
        cases = [synth.config3_projection(batch, d, n) for d, n in synth.DENSE_32B_PROJECTIONS.values()]
        return {"kind": "dense", "name": "config3: 32B-dense segmented prefill, 32 requests of 128..1024 tokens, 32 adapters r=64",
                "T": batch.T, "cases": cases, "layers": layers or 2}
    if name == "config4":
        batch = synth.config4_batch()
        cases = [synth.config4_projection(batch, p) for p in ("gate", "up", "down")]
        return {"kind": "moe", "name": "config4: 30B-A3B MoE expert LoRA, T=4096, top-8 of 128 experts, 16 adapters r=16",
                "T": batch.T, "cases": cases, "layers": layers or 16}
    raise SystemExit(f"unknown workload {name}")


def algorithmic_bytes(wl) -> list:
    from paper_2605_13779_b200 import accounting
    fn = accounting.algorithmic_bytes_moe if wl["kind"] == "moe" else accounting.algorithmic_bytes_dense
    return [fn(c) for c in wl["cases"]]


def hbm_peak():
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        return json.load(open(peaks_path))["hbm_gbs"], "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback"


# --------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi SM clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
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
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------
# CPU oracle legs
# --------------------------------------------------------------------------
def oracle_layer_seconds(wl, max_seconds: float = 12.0):
    """Times the fp64 oracle (as it stands) on whole layers of the workload until
    about max_seconds of CPU work have been spent; returns (tokens/s per layer,
    threads, description of the sample)."""
    from oracle import oracle
    threads = oracle.max_threads()
    t_total, n_layers = 0.0, 0
    while True:
        t0 = time.perf_counter()
        oracle.plan(wl["cases"][0].ids, wl["cases"][0].table.id_to_slot, wl["cases"][0].table.num_slots,
                    expert_ids=getattr(wl["cases"][0], "expert_ids", None),
                    num_experts=getattr(wl["cases"][0], "E", 0))
        for c in wl["cases"]:
            t = c.table
            if wl["kind"] == "moe":
                oracle.moe_lora_apply(c.ids, c.expert_ids, t.id_to_slot, t.slot_rank, t.slot_scale, c.A, c.B,
                                      c.x, c.y0, x_row=c.x_row)
            else:
                oracle.lora_apply(c.ids, t.id_to_slot, t.slot_rank, t.slot_scale, c.A, c.B, c.x, c.y0)
        t_total += time.perf_counter() - t0
        n_layers += 1
        if t_total >= max_seconds or n_layers >= 2000:
            break
    per_layer = t_total / n_layers
    return wl["T"] / per_layer, threads, f"{n_layers} layer(s) of the workload ({len(wl['cases'])} projections each, all {wl['T']} tokens), {t_total:.1f} s"


def run_reference(args):
    """The reference arm: the CPU oracle on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = build_workload(args.workload, args.layers)
    vals = []
    budget = max(2.0, 60.0 / max(1, args.steps + args.warmup))
    sample = ""
    for i in range(args.warmup + args.steps):
        v, threads, sample = oracle_layer_seconds(wl, max_seconds=budget)
        if i >= args.warmup:
            vals.append(v)
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wl["T"] / value,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic (seeded)", "config": {"workload": wl["name"]},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------
class DeviceWorkload:
    """A workload resident on the device: every layer has its own pool, x and y."""

    def __init__(self, wl, copies: int):
        import torch
        from paper_2605_13779_b200 import binding as mb, harness
        self.mb, self.torch = mb, torch
        self.wl = wl
        self.moe = wl["kind"] == "moe"
        self.T = wl["T"]
        self.L = copies
        self.base = [harness.upload_moe(c) if self.moe else harness.upload_dense(c) for c in wl["cases"]]
        self.table = self.base[0].table
        self.layers = []
        for li in range(copies):
            row = []
            for dv in self.base:
                if li == 0:
                    row.append((dv.pool, dv.x, dv.y))
                else:
                    A, B = dv.pool.A.clone(), dv.pool.B.clone()
                    pool = mb.Pool(A, B, dv.pool.d, dv.pool.n, dv.pool.r_max, dv.pool.num_slots,
                                   num_experts=dv.pool.num_experts)
                    row.append((pool, dv.x.clone(), dv.y.clone()))
            for i in range(1, len(row)):   # projections with the same input (q, k, v; gate, up) read one tensor
                ca, cb = wl["cases"][i - 1], wl["cases"][i]
                if ca.x.shape == cb.x.shape and np.array_equal(ca.x, cb.x):
                    row[i] = (row[i][0], row[i - 1][1], row[i][2])
            self.layers.append(row)
        self.ids = self.base[0].ids
        self.status = mb.new_status()
        self.expert_ids = self.base[0].expert_ids if self.moe else None
        self.E = wl["cases"][0].E if self.moe else 0
        self.K = wl["cases"][0].K if self.moe else 1
        self.plan = mb.Plan(self.T, self.K, self.table.num_slots, self.E)
        self.workspaces = ([mb.new_moe_workspace(dv.pool, self.T, self.K) for dv in self.base] if self.moe
                           else [mb.new_workspace(dv.pool, self.T) for dv in self.base])
        self.bytes_per_case = algorithmic_bytes(wl)
        self.layer_bytes = sum(b["total"] for b in self.bytes_per_case)
        self._groups = {}

    def groups_idx(self, grouping):
        ncase = len(self.wl["cases"])
        if grouping == "none" or ncase == 1:
            return [[i] for i in range(ncase)]
        if self.moe:   # gate and up share the routed pairs and the hidden rows; down reads their product
            return [[0, 1], [2]] if ncase == 3 else [[i] for i in range(ncase)]
        if grouping == "layer":
            return [list(range(ncase))]
        return STAGES if ncase == 7 else [[i] for i in range(ncase)]

    def enqueue_plan(self):
        self.mb.mint_lora_plan(self.table, self.ids, self.status, expert_ids=self.expert_ids, num_experts=self.E,
                               plan=self.plan)

    def enqueue_layer(self, li, grouping):
        mb = self.mb
        if self.moe:
            row = self.layers[li]
            for g in self.groups_idx(grouping):
                if len(g) == 1:
                    ci = g[0]
                    mb.mint_moe_lora_apply(row[ci][0], self.table, self.plan, row[ci][1], row[ci][2], self.status,
                                           x_row=self.base[ci].x_row, workspace=self.workspaces[ci])
                else:
                    mb.mint_moe_lora_apply_grouped([(row[ci][0], row[ci][1], row[ci][2], self.workspaces[ci]) for ci in g],
                                                   self.table, self.plan, self.status, x_row=self.base[g[0]].x_row)
            return
        key = (li, grouping)
        if key not in self._groups:
            row = self.layers[li]
            self._groups[key] = [mb.ApplyGroup([(row[i][0], row[i][1], row[i][2], self.workspaces[i]) for i in g])
                                 for g in self.groups_idx(grouping)]
        for grp in self._groups[key]:
            mb.mint_lora_apply_fused_grouped(grp, self.table, self.plan, self.status)

    def enqueue_layer_unfused(self, li, v_bufs):
        """shrink then expand through a v tensor of its own (dense workloads)."""
        mb = self.mb
        for ci, (pool, x, y) in enumerate(self.layers[li]):
            mb.mint_lora_shrink(pool, self.table, self.plan, x, self.status, v=v_bufs[ci])
            mb.mint_lora_expand(pool, self.table, self.plan, v_bufs[ci], y, self.status)

    def launches_per_pass(self, grouping):
        kernels_per_call = 4 if (not self.moe and self.T >= 4096) else 2
        return 1 + self.L * len(self.groups_idx(grouping)) * kernels_per_call

    def capture(self, stream, fn):
        torch = self.torch
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(g, stream=stream):
                fn()
        return g

    def check_status(self, what):
        st = self.status.cpu().numpy()
        if st[0] != 0:
            raise SystemExit(f"device status {self.mb.status_name(int(st[0]))} after {what}: the timed run is invalid")


def time_graph(torch, dist, world, stream, graph, steps, warmup, name="timed region"):
    """K replays bracketed by a barrier and a synchronize on both sides; max over ranks (ms).
    The timed replays sit in an NVTX range of the given name (visible to profilers)."""
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            graph.replay()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.nvtx.range_push(name)
        e0.record(stream)
        for _ in range(steps):
            graph.replay()
        e1.record(stream)
        torch.cuda.nvtx.range_pop()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return ms


def parity_of_first_layer(dw: DeviceWorkload, grouping):
    """One layer of the call the bench times, on fresh copies of y, against the fp64 oracle."""
    import torch
    from oracle import oracle
    from paper_2605_13779_b200 import harness, synth
    saved = [y.clone() for (_, _, y) in dw.layers[0]]
    for (_, _, y), c in zip(dw.layers[0], dw.wl["cases"]):      # (earlier replays have updated y: start from y0 again)
        y.copy_(dw.mb.bf16_from_bits(c.y0))
    dw.enqueue_plan()
    dw.enqueue_layer(0, grouping)
    torch.cuda.synchronize()
    out = {"max_abs": 0.0, "rel_fro": 0.0, "max_abs_y_ref": 0.0}
    for ci, c in enumerate(dw.wl["cases"]):
        t = c.table
        y = dw.layers[0][ci][2]
        if dw.moe:
            y_ref, _ = oracle.moe_lora_apply(c.ids, c.expert_ids, t.id_to_slot, t.slot_rank, t.slot_scale, c.A, c.B,
                                             c.x, c.y0, x_row=c.x_row)
            y_gpu = harness.y_to_f64(y)
        else:
            rows = None
            if c.T * c.n > 64_000_000:      # sampled rows where the full comparison would take minutes
                rows = np.sort(synth.stream("bench/parity", ci).choice(c.T, size=128, replace=False))
            sel = slice(None) if rows is None else rows
            y_ref, _, _ = oracle.lora_apply(c.ids[sel], t.id_to_slot, t.slot_rank, t.slot_scale, c.A, c.B, c.x[sel], c.y0[sel])
            y_gpu = harness.y_to_f64(y if rows is None else y[torch.from_numpy(rows).cuda()])
        out["max_abs"] = max(out["max_abs"], float(np.abs(y_gpu - y_ref).max()))
        out["rel_fro"] = max(out["rel_fro"], float(np.linalg.norm(y_gpu - y_ref) / np.linalg.norm(y_ref)))
        out["max_abs_y_ref"] = max(out["max_abs_y_ref"], float(np.abs(y_ref).max()))
    out["within_tolerance"] = bool(out["max_abs"] <= 3e-2 and out["rel_fro"] <= 5e-3)
    for (_, _, y), s in zip(dw.layers[0], saved):
        y.copy_(s)
    return out


def measure_side_workload(torch, dist, world, stream, name, peak):
    """A short device-timed loop of another workload: us per layer, tokens/s per layer, roofline fraction."""
    wl = build_workload(name, 0)
    dw = DeviceWorkload(wl, wl["layers"])
    dw.enqueue_plan()
    for li in range(dw.L):
        dw.enqueue_layer(li, "layer")
    torch.cuda.synchronize()

    def one_pass():
        dw.enqueue_plan()
        for li in range(dw.L):
            dw.enqueue_layer(li, "layer")

    def applies():
        for li in range(dw.L):
            dw.enqueue_layer(li, "layer")

    g = dw.capture(stream, one_pass)
    ga = dw.capture(stream, applies)
    est = time_graph(torch, dist, world, stream, g, 2, 2) / 2
    steps = int(min(200, max(5, 150.0 / max(est, 1e-3))))
    ms = time_graph(torch, dist, world, stream, g, steps, 3) / steps
    ms_a = time_graph(torch, dist, world, stream, ga, steps, 1) / steps
    dw.check_status(name)
    res = {"workload": wl["name"], "layers": dw.L, "us_per_layer": ms * 1e3 / dw.L,
           "us_per_layer_apply_only": ms_a * 1e3 / dw.L,
           "tokens_per_s": world * dw.T * dw.L / (ms * 1e-3), "bytes_per_layer": dw.layer_bytes,
           "GBps": dw.layer_bytes / (ms * 1e-3 / dw.L) / 1e9,
           "roofline_frac": dw.layer_bytes / (ms_a * 1e-3 / dw.L) / 1e9 / peak,
           "roofline_frac_with_plan": dw.layer_bytes / (ms * 1e-3 / dw.L) / 1e9 / peak,
           "replay_footprint_MB": dw.layer_bytes * dw.L / 1e6}
    if dw.moe:
        # Routing differs from layer to layer of a MoE model, so a served layer needs a plan of its own:
        # the same pass with one plan before every layer.
        def plan_every_layer():
            for li in range(dw.L):
                dw.enqueue_plan()
                dw.enqueue_layer(li, "layer")

        gp = dw.capture(stream, plan_every_layer)
        ms_p = time_graph(torch, dist, world, stream, gp, steps, 2) / steps
        dw.check_status(name)
        res["us_per_layer_plan_every_layer"] = ms_p * 1e3 / dw.L
        res["roofline_frac_plan_every_layer"] = dw.layer_bytes / (ms_p * 1e-3 / dw.L) / 1e9 / peak
        del gp
    if name != "config3":
        res["parity"] = parity_of_first_layer(dw, "layer")
    del g, ga, dw
    gc.collect()
    torch.cuda.empty_cache()
    return res


def measure_backward(torch, dist, world, stream, peak, layers=6, short=False):
    """The LoRA backward (dx, dA, dB) of every projection of config 2's layer, device-timed: one plan,
    then mint_lora_backward per projection and layer; every layer has its own tensors (about 0.4 GB each)."""
    from oracle import backward as oracle_backward
    from paper_2605_13779_b200 import accounting, binding as mb, harness, synth
    wl = build_workload("config2", 0)
    cases = wl["cases"]
    base = [harness.upload_dense(c) for c in cases]
    table, ids, status = base[0].table, base[0].ids, mb.new_status()
    dys = [synth.normal_bf16(synth.stream("bench/backward", c.name), (c.T, c.n), 1.0) for c in cases]
    rows = []
    for li in range(layers):
        row = []
        for dv, c, dy in zip(base, cases, dys):
            pool = dv.pool if li == 0 else mb.Pool(dv.pool.A.clone(), dv.pool.B.clone(), c.d, c.n, c.r_max,
                                                   dv.pool.num_slots)
            row.append((pool, dv.x if li == 0 else dv.x.clone(), mb.bf16_from_bits(dy),
                        torch.zeros(c.T, c.d, dtype=torch.bfloat16, device="cuda"),
                        torch.zeros(c.A.shape, dtype=torch.float32, device="cuda"),
                        torch.zeros(c.B.shape, dtype=torch.float32, device="cuda")))
        rows.append(row)
    ws = [mb.new_backward_workspace(dv.pool, wl["T"]) for dv in base]
    plan = mb.Plan(wl["T"], 1, table.num_slots, 0)

    groups = [mb.BackwardGroup([(pool, x, dy, dx, dA, dB, w) for (pool, x, dy, dx, dA, dB), w in zip(row, ws)])
              for row in rows]

    def one_pass():
        mb.mint_lora_plan(table, ids, status, plan=plan)
        for grp in groups:
            mb.mint_lora_backward_grouped(grp, table, plan, status)

    one_pass()
    torch.cuda.synchronize()
    # parity of the first layer's first call (all outputs started at zero) against the fp64 oracle
    par = {"max_abs_dx": 0.0, "rel_fro_dx": 0.0, "rel_fro_dA": 0.0, "rel_fro_dB": 0.0}
    for ci in (0, 6):
        c, (_, _, _, dx, dA, dB) = cases[ci], rows[0][ci]
        t = c.table
        dx_ref, dA_ref, dB_ref, _ = oracle_backward.lora_backward(c.ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                                                  c.A, c.B, c.x, dys[ci])
        dxg = harness.y_to_f64(dx)
        par["max_abs_dx"] = max(par["max_abs_dx"], float(np.abs(dxg - dx_ref).max()))
        par["rel_fro_dx"] = max(par["rel_fro_dx"], float(np.linalg.norm(dxg - dx_ref) / np.linalg.norm(dx_ref)))
        par["rel_fro_dA"] = max(par["rel_fro_dA"], float(np.linalg.norm(dA.cpu().numpy() - dA_ref) / np.linalg.norm(dA_ref)))
        par["rel_fro_dB"] = max(par["rel_fro_dB"], float(np.linalg.norm(dB.cpu().numpy() - dB_ref) / np.linalg.norm(dB_ref)))
    par["within_tolerance"] = bool(par["max_abs_dx"] <= 3e-2 and par["rel_fro_dx"] <= 5e-3 and
                                   par["rel_fro_dA"] <= 1e-4 and par["rel_fro_dB"] <= 1e-4)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(g, stream=stream):
            one_pass()
    est = time_graph(torch, dist, world, stream, g, 2, 2) / 2
    steps = 2 if short else int(min(100, max(5, 150.0 / max(est, 1e-3))))
    ms = time_graph(torch, dist, world, stream, g, steps, 3, name="backward") / steps
    st = status.cpu().numpy()
    if st[0] != 0:
        raise SystemExit(f"device status {mb.status_name(int(st[0]))} after the backward loop")
    layer_bytes = sum(accounting.algorithmic_bytes_backward(c)["total"] for c in cases)
    res = {"workload": "config2 layer: dx, dA, dB of the seven projections (one grouped call per layer)",
           "layers": layers, "us_per_layer": ms * 1e3 / layers, "bytes_per_layer": layer_bytes,
           "GBps": layer_bytes / (ms * 1e-3 / layers) / 1e9,
           "roofline_frac": layer_bytes / (ms * 1e-3 / layers) / 1e9 / peak,
           "tokens_per_s": world * wl["T"] * layers / (ms * 1e-3), "parity": par}
    del g, groups, rows, base, ws
    gc.collect()
    torch.cuda.empty_cache()
    return res


def measure_moe_backward(torch, dist, world, stream, peak, short=False):
    """The backward of config 4's three expert projections (per-pair dx, dA, dB of the packed tensors) at
    full size, device-timed: one MoE plan, then mint_moe_lora_backward per projection; two sets of
    tensors (about 2.5 GB each) are walked in turn."""
    from oracle import backward as oracle_backward
    from paper_2605_13779_b200 import accounting, binding as mb, harness, synth
    wl = build_workload("config4", 0)
    cases = wl["cases"][:1] if short else wl["cases"]   # (short: the gate projection alone, under a profiler)
    P = cases[0].T * cases[0].K
    base = [harness.upload_moe(c) for c in cases]
    table, ids, ex, status = base[0].table, base[0].ids, base[0].expert_ids, mb.new_status()
    dys = [synth.normal_bf16(synth.stream("bench/moe-backward", c.name), (P, c.n), 1.0) for c in cases]
    sets = []
    for si in range(1 if short else 2):
        row = []
        for dv, c, dy in zip(base, cases, dys):
            pool = dv.pool if si == 0 else mb.Pool(dv.pool.A.clone(), dv.pool.B.clone(), c.d, c.n, c.r_max,
                                                   dv.pool.num_slots, num_experts=c.E)
            row.append((pool, dv.x if si == 0 else dv.x.clone(), mb.bf16_from_bits(dy),
                        torch.zeros(P, c.d, dtype=torch.bfloat16, device="cuda"),
                        torch.zeros(c.A.shape, dtype=torch.float32, device="cuda"),
                        torch.zeros(c.B.shape, dtype=torch.float32, device="cuda"), dv.x_row))
        sets.append(row)
    nbytes = max(int(mb.load_library().mint_moe_lora_backward_workspace_bytes(dv.pool.handle, cases[0].T, cases[0].K))
                 for dv in base)
    ws = torch.empty(max(256, nbytes), dtype=torch.uint8, device="cuda")
    plan = mb.Plan(cases[0].T, cases[0].K, table.num_slots, cases[0].E)
    w = base[0].pair_weight

    def one_pass():
        for row in sets:
            mb.mint_lora_plan(table, ids, status, expert_ids=ex, num_experts=cases[0].E, plan=plan)
            for (pool, x, dy, dx, dA, dB, x_row) in row:
                mb.mint_moe_lora_backward(pool, table, plan, x, dy, status, dx=dx, dA=dA, dB=dB, x_row=x_row,
                                          pair_weight=w, workspace=ws)

    one_pass()
    torch.cuda.synchronize()
    # parity of the first set's gate projection (all outputs started at zero) against the fp64 oracle
    c, (_, _, _, dx, dA, dB, _) = cases[0], sets[0][0]
    t = c.table
    dx_ref, dA_ref, dB_ref, _ = oracle_backward.moe_lora_backward(c.ids, c.expert_ids, t.id_to_slot, t.slot_rank,
                                                                  t.slot_scale, c.A, c.B, c.x, dys[0], x_row=c.x_row,
                                                                  pair_weight=c.pair_weight)
    dxg = harness.y_to_f64(dx)
    par = {"max_abs_dx": float(np.abs(dxg - dx_ref).max()),
           "rel_fro_dx": float(np.linalg.norm(dxg - dx_ref) / np.linalg.norm(dx_ref)),
           "rel_fro_dA": float(np.linalg.norm(dA.cpu().numpy() - dA_ref) / np.linalg.norm(dA_ref)),
           "rel_fro_dB": float(np.linalg.norm(dB.cpu().numpy() - dB_ref) / np.linalg.norm(dB_ref))}
    par["within_tolerance"] = bool(par["max_abs_dx"] <= 3e-2 and par["rel_fro_dx"] <= 5e-3 and
                                   par["rel_fro_dA"] <= 1e-4 and par["rel_fro_dB"] <= 1e-4)
    del dx_ref, dA_ref, dB_ref, dxg
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(g, stream=stream):
            one_pass()
    est = time_graph(torch, dist, world, stream, g, 2, 2) / 2
    steps = 2 if short else int(min(100, max(5, 150.0 / max(est, 1e-3))))
    ms = time_graph(torch, dist, world, stream, g, steps, 3, name="moe_backward") / steps
    st = status.cpu().numpy()
    if st[0] != 0:
        raise SystemExit(f"device status {mb.status_name(int(st[0]))} after the MoE backward loop")
    layer_bytes = sum(accounting.algorithmic_bytes_moe_backward(c)["total"] for c in cases)
    res = {"workload": "config4 layer: per-pair dx, dA, dB of gate, up and down (one call per projection, a plan per layer)",
           "layers": len(sets), "us_per_layer": ms * 1e3 / len(sets), "bytes_per_layer": layer_bytes,
           "GBps": layer_bytes / (ms * 1e-3 / len(sets)) / 1e9,
           "roofline_frac": layer_bytes / (ms * 1e-3 / len(sets)) / 1e9 / peak,
           "tokens_per_s": world * cases[0].T * len(sets) / (ms * 1e-3), "parity": par}
    del g, sets, base, ws
    gc.collect()
    torch.cuda.empty_cache()
    return res


def measure_admission(torch, stream):
    """Admitting one adapter into the three expert projections of a 30B-A3B-shaped layer (128 experts):
    the packed representation (one call per projection) against one copy per tensor."""
    from paper_2605_13779_b200 import binding as mb, synth
    E, slots = 128, 4
    out = {}
    for rank in (1, 16):
        pools, packed = [], []
        for d, n in synth.MOE_30B_PROJECTIONS.values():
            A = torch.zeros(slots, E, d, 16, dtype=torch.bfloat16, device="cuda")
            B = torch.zeros(slots, E, 16, n, dtype=torch.bfloat16, device="cuda")
            pools.append(mb.Pool(A, B, d, n, 16, slots, num_experts=E))
            packed.append((torch.randn(E, d, rank, device="cuda").to(torch.bfloat16),
                           torch.randn(E, rank, n, device="cuda").to(torch.bfloat16)))
        nbytes = sum(a.numel() * 2 + b.numel() * 2 for a, b in packed)

        def admit_packed():
            for pool, (a, b) in zip(pools, packed):
                pool.admit_packed(1, a, b, rank)

        def admit_per_tensor():
            for pool, (a, b) in zip(pools, packed):
                for e in range(E):
                    pool.write_slot(1, a[e], b[e], rank, expert=e)

        res = {}
        with torch.cuda.stream(stream):
            for nm, fn, reps in (("packed", admit_packed, 20), ("per_tensor", admit_per_tensor, 3)):
                fn()
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                for _ in range(reps):
                    fn()
                torch.cuda.synchronize()
                res[nm] = (time.perf_counter() - t0) / reps
        out[f"rank{rank}"] = {"bytes": nbytes, "tensors_per_layer": {"packed": 6, "per_tensor": 6 * E},
                              "packed_us": res["packed"] * 1e6, "per_tensor_us": res["per_tensor"] * 1e6,
                              "packed_GBps": nbytes / res["packed"] / 1e9,
                              "admissions_per_s_packed_48_layers": 1.0 / (48 * res["packed"]),
                              "speedup": res["per_tensor"] / res["packed"]}
    out["what"] = ("one adapter into gate/up/down of one 128-expert layer, device-resident sources, "
                   "host-timed including launch; per_tensor = one copy call per (expert, tensor)")
    return out


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2605_13779_b200 import binding as mb

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    mb.load_library()
    peak, peak_src = hbm_peak()
    if args.workload in ("backward", "moe_backward"):   # a backward alone (the command profilers wrap): its own JSON line
        if args.workload == "backward":
            res = measure_backward(torch, dist, 1, torch.cuda.Stream(), peak, layers=args.layers or 6,
                                   short=args.profile)
        else:
            res = measure_moe_backward(torch, dist, 1, torch.cuda.Stream(), peak, short=args.profile)
        if rank == 0:
            print(json.dumps(res))
        return

    wl = build_workload(args.workload, args.layers)
    dw = DeviceWorkload(wl, wl["layers"])
    L, T = dw.L, dw.T
    grouping = args.grouping
    stream = torch.cuda.Stream()

    # warm-up outside any graph (first launches load the module)
    dw.enqueue_plan()
    for li in range(L):
        dw.enqueue_layer(li, grouping)
    torch.cuda.synchronize()
    parity = parity_of_first_layer(dw, grouping) if (rank == 0 and not args.profile) else None

    def one_pass(g=grouping):
        dw.enqueue_plan()
        for li in range(L):
            dw.enqueue_layer(li, g)

    def applies(g=grouping):
        for li in range(L):
            dw.enqueue_layer(li, g)

    # passes per step: a step of about 50 ms
    probe = dw.capture(stream, one_pass)
    est_ms = time_graph(torch, dist, world, stream, probe, 3, 2) / 3
    passes = 1 if args.profile else int(min(64, max(1, round(50.0 / max(est_ms, 1e-3)))))
    if world > 1:
        t = torch.tensor([passes], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        passes = int(t.item())

    def step_fn():
        for _ in range(passes):
            one_pass()

    def apply_fn():
        for _ in range(passes):
            applies()

    step_graph = dw.capture(stream, step_fn)
    apply_graph = dw.capture(stream, apply_fn)
    torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms_total = time_graph(torch, dist, world, stream, step_graph, args.steps, args.warmup, "steps: plan + applies")
    ms_apply = time_graph(torch, dist, world, stream, apply_graph, args.steps, 1, "applies only")
    clocks = sampler.stop() if rank == 0 else None
    ms_step = ms_total / args.steps
    value = world * T * L * passes / (ms_step * 1e-3)
    calls_per_layer = len(dw.groups_idx(grouping))
    dw.check_status("the timed region")

    if args.profile:
        if rank == 0:
            print(json.dumps({"profile_run": True, "workload": wl["name"], "layers": L, "ms_per_step": ms_step,
                              "us_per_layer": ms_step * 1e3 / (L * passes), "grouping": grouping,
                              "layer_GBps": dw.layer_bytes / (ms_step * 1e-3 / (L * passes)) / 1e9,
                              "avg_apply_call_us": ms_apply * 1e3 / args.steps / (L * passes * calls_per_layer)}))
        return

    # ---- the other schedules of the same workload (short loops) ---------------------
    other = {}
    if rank == 0 and not dw.moe and len(wl["cases"]) == 7:
        alt = "stage" if grouping == "layer" else "layer"
        ga = dw.capture(stream, lambda: applies(alt))
        n = 30
        ms = time_graph(torch, dist, 1, stream, ga, n, 3) / n
        other[alt] = {"us_per_layer": ms * 1e3 / L, "calls_per_layer": len(dw.groups_idx(alt)),
                      "roofline_frac": dw.layer_bytes / (ms * 1e-3 / L) / 1e9 / peak}
        del ga
    if rank == 0 and not dw.moe:
        # the unfused pair of calls: v goes through a tensor of its own
        v_bufs = [torch.empty(T, dv.pool.r_max, dtype=torch.float32, device="cuda") for dv in dw.base]
        for li in range(min(L, 2)):
            dw.enqueue_layer_unfused(li, v_bufs)
        torch.cuda.synchronize()

        def unfused():
            for li in range(L):
                dw.enqueue_layer_unfused(li, v_bufs)

        gu = dw.capture(stream, unfused)
        n = 10
        ms = time_graph(torch, dist, 1, stream, gu, n, 2) / n
        other["unfused_shrink_then_expand"] = {"us_per_layer": ms * 1e3 / L,
                                               "roofline_frac": dw.layer_bytes / (ms * 1e-3 / L) / 1e9 / peak}
        del gu, v_bufs
    if rank == 0:
        # L2-warm: the same single layer over and over (its working set stays in the 126 MB L2 where it fits)
        def warm():
            for _ in range(32):
                dw.enqueue_layer(0, grouping)

        gw = dw.capture(stream, warm)
        n = 10
        ms = time_graph(torch, dist, 1, stream, gw, n, 3) / n
        other["l2_warm_single_layer"] = {"us_per_layer": ms * 1e3 / 32, "layer_MB": dw.layer_bytes / 1e6}
        del gw

    # ---- end to end through the C ABI with host buffers --------------------------
    # Per step: ids, every x and every y0 come from pinned host memory, the plan and
    # all applies run, and every updated y goes back to pinned host memory.
    e2e_layers = min(L, 4)
    host_ids = dw.ids.cpu().pin_memory()
    host_x = [[x.cpu().pin_memory() for (_, x, _) in row] for row in dw.layers[:e2e_layers]]
    host_y = [[y.cpu().pin_memory() for (_, _, y) in row] for row in dw.layers[:e2e_layers]]
    h2d = host_ids.numel() * 8 + sum(t.numel() * 2 for row in host_x for t in row) + \
        sum(t.numel() * 2 for row in host_y for t in row)
    d2h = sum(t.numel() * 2 for row in host_y for t in row)

    # Three streams, as a caller that feeds layers from the host would use the API: inputs of layer i+1
    # come in while layer i is applied and the result of layer i-1 goes out (PCIe carries both directions
    # at once).  Events order a layer's apply after its inputs and its read-back after the apply; a layer's
    # next inputs wait for its previous read-back.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(e2e_layers)]
    ev_done = [torch.cuda.Event() for _ in range(e2e_layers)]
    ev_out = [torch.cuda.Event() for _ in range(e2e_layers)]
    ev_ids = torch.cuda.Event()

    def e2e_step(first):
        with torch.cuda.stream(s_in):
            if not first:
                s_in.wait_event(ev_done[e2e_layers - 1])   # the previous step's plan and applies have read ids
            dw.ids.copy_(host_ids, non_blocking=True)
            ev_ids.record(s_in)
            for li in range(e2e_layers):
                if not first:
                    s_in.wait_event(ev_out[li])
                for ci, (pool, x, y) in enumerate(dw.layers[li]):
                    x.copy_(host_x[li][ci], non_blocking=True)
                    y.copy_(host_y0[li][ci], non_blocking=True)
                ev_in[li].record(s_in)
        stream.wait_event(ev_ids)
        dw.enqueue_plan()
        for li in range(e2e_layers):
            stream.wait_event(ev_in[li])
            dw.enqueue_layer(li, grouping)
            ev_done[li].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[li])
                for ci, (pool, x, y) in enumerate(dw.layers[li]):
                    host_y[li][ci].copy_(y, non_blocking=True)
                ev_out[li].record(s_out)

    host_y0 = [[t.clone().pin_memory() for t in row] for row in host_y]
    with torch.cuda.stream(stream):
        for i in range(3):
            e2e_step(i == 0)
        torch.cuda.synchronize()
        e2e_steps = max(3, min(args.steps, 10))
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step(False)
        torch.cuda.synchronize()
        e2e_s = (time.perf_counter() - t0) / e2e_steps
    if world > 1:
        t = torch.tensor([e2e_s], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e_value = world * T * e2e_layers / e2e_s
    dw.check_status("the end-to-end leg")
    layer_bytes, launches = dw.layer_bytes, dw.launches_per_pass(grouping) * passes
    del step_graph, apply_graph, probe, host_x, host_y, host_y0
    if rank != 0:
        return

    # ---- roofline of the dominant kernel pair (the fused apply) ------------------------
    # the apply is a shrink launch and an expand launch that overlap (programmatic dependent launch),
    # so the roofline unit is the pair: bytes of one call / time of one call
    n_apply = L * calls_per_layer * passes
    avg_launch_s = ms_apply * 1e-3 / args.steps / n_apply
    avg_launch_bytes = layer_bytes / calls_per_layer
    achieved = avg_launch_bytes / avg_launch_s / 1e9
    roofline = {"bound": "hbm", "kernel": "shrink_stream_kernel+expand_stream_kernel",
                "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "frac_of_8TBps": achieved / 8000.0, "peak_source": peak_src,
                "bytes_per_launch": avg_launch_bytes, "avg_launch_us": avg_launch_s * 1e6,
                "launches_timed": n_apply * args.steps, "traffic": None}
    # dram__bytes_read.sum + dram__bytes_write.sum of one launch pair, as the ncu summary under profiles/ records it
    # for this workload and grouping (a line "traffic_bytes_per_launch = N"); null when there is no such record
    summary = os.path.join(ROOT, "profiles", f"stream_kernels_{args.workload}_{grouping}.md")
    if os.path.exists(summary):
        import re
        m = re.search(r"traffic_bytes_per_launch\s*=\s*(\d+)", open(summary).read())
        if m:
            roofline["traffic"] = int(m.group(1))
    us_layer = ms_step * 1e3 / (L * passes)
    us_layer_apply = ms_apply * 1e3 / args.steps / (L * passes)

    # ---- the other workloads, the admission path, the CPU oracle --------------------------
    del dw
    gc.collect()
    torch.cuda.empty_cache()
    workloads = {}
    if args.workload == "config2" and not args.no_side_workloads:
        for name in ("config5", "config4", "config3"):
            workloads[name] = measure_side_workload(torch, dist, 1, stream, name, peak)
    admission = None if args.no_side_workloads else measure_admission(torch, stream)
    backward = (measure_backward(torch, dist, 1, stream, peak)
                if (args.workload == "config2" and not args.no_side_workloads and rank == 0) else None)
    moe_backward = (measure_moe_backward(torch, dist, 1, stream, peak)
                    if (args.workload == "config2" and not args.no_side_workloads and rank == 0) else None)
    cpu_val, cores, sample = oracle_layer_seconds(wl)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 in, f32 accumulate", "data": "synthetic (seeded)",
        "config": {"workload": wl["name"], "layers_per_pass": L, "passes_per_step": passes, "tokens": T,
                   "l2": f"inputs larger than L2: every layer has its own pool/x/y, {layer_bytes * L / 1e6:.0f} MB algorithmic bytes per pass",
                   "grouping": grouping, "calls_per_layer": calls_per_layer,
                   "timing": "CUDA graph of (plan + all applies) x passes, CUDA events on the launching stream"},
        "us_per_layer": us_layer,
        "us_per_layer_apply_only": us_layer_apply,
        "plan_share_us_per_layer": us_layer - us_layer_apply,
        "layer_bytes": layer_bytes,
        "layer_GBps": layer_bytes / (us_layer * 1e-6) / 1e9,
        "clocks": clocks,
        "parity": parity,
        "roofline": roofline,
        "schedules": other,
        "workloads": workloads,
        "admission": admission,
        "backward": backward,
        "moe_backward": moe_backward,
        "cpu_baseline": {"value": cpu_val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "layers_per_step": e2e_layers},
        "gpu_launches": launches * args.steps,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def spawn_replicas(args):
    """--gpus N without a launcher: start N replica processes of this script (one per GPU)."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(args.gpus):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(args.gpus),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable] + sys.argv, env=env))
    rc = 0
    for p in procs:
        rc = p.wait() or rc
    sys.exit(rc)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config2")
    ap.add_argument("--layers", type=int, default=0, help="layers per pass (0 = the workload's own)")
    ap.add_argument("--grouping", default="layer", choices=["none", "stage", "layer"],
                    help="how the projections of a layer are grouped into fused calls")
    ap.add_argument("--profile", action="store_true",
                    help="device-timed part only, one pass per step (no end-to-end leg, no CPU oracle): the command profilers wrap")
    ap.add_argument("--no-side-workloads", action="store_true", help="skip the other workloads and the admission path")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_replicas(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
