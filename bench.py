#!/usr/bin/env python
"""Benchmark of the mixed-adapter LoRA apply on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config2|config5|config4|config3]
    python bench.py --impl reference ...        # the fp64 CPU oracle, timed on the host cores

A step is one pass of the whole hot path over one batch: one segment plan
(token -> adapter grouping through the slot table) followed by the fused apply
of every LoRA target projection of every layer.  The default workload is the
4B-dense decode layer: T=256 requests, 64 resident adapters with ranks from
{1, 8, 16, 32}, Zipf(1.1) request->adapter, seven projections per layer, 36
layers; every layer has its own pool, x and y so that a step streams about
4.5 GB (far beyond the 126 MB L2).  The step is captured in a CUDA graph and
replayed; times are CUDA-event times on the launching stream.

Prints ONE JSON line (rank 0).  metric = tokens/s per layer: T * layers / step
time, summed over ranks (ranks are independent replicas: the path has no
exchange step, scaling is weak).
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "mixed-adapter LoRA apply tokens/s per layer"
UNIT = "tokens/s"


# --------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------
def build_workload(name: str, layers: int):
    """Host-side description: a list of per-layer lists of cases, plus the
    batch.  Only `distinct_layers` layers are drawn on the host; the device
    copies cycle through them (values do not matter for timing, addresses do)."""
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
                "T": case.T, "cases": [case], "layers": layers or 16}
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
                "T": batch.T, "cases": cases, "layers": layers or 4}
    raise SystemExit(f"unknown workload {name}")


def algorithmic_bytes(wl) -> list:
    from paper_2605_13779_b200 import accounting
    fn = accounting.algorithmic_bytes_moe if wl["kind"] == "moe" else accounting.algorithmic_bytes_dense
    return [fn(c) for c in wl["cases"]]


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
def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2605_13779_b200 import binding as mb, harness

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    mb.load_library()

    wl = build_workload(args.workload, args.layers)
    L = wl["layers"]
    T = wl["T"]
    moe = wl["kind"] == "moe"
    bytes_per_case = algorithmic_bytes(wl)
    layer_bytes = sum(b["total"] for b in bytes_per_case)

    # ---- device-resident inputs: every layer has its own pool, x and y -------
    base = [harness.upload_moe(c) if moe else harness.upload_dense(c) for c in wl["cases"]]
    table = base[0].table
    layers = []
    for li in range(L):
        row = []
        for dv in base:
            if li == 0:
                row.append((dv.pool, dv.x, dv.y))
            else:
                A, B = dv.pool.A.clone(), dv.pool.B.clone()
                pool = mb.Pool(A, B, dv.pool.d, dv.pool.n, dv.pool.r_max, dv.pool.num_slots,
                               num_experts=dv.pool.num_experts)
                row.append((pool, dv.x.clone(), dv.y.clone()))
        layers.append(row)
    ids = base[0].ids
    status = mb.new_status()
    expert_ids = base[0].expert_ids if moe else None
    E = wl["cases"][0].E if moe else 0
    plan = mb.Plan(T, wl["cases"][0].K if moe else 1, table.num_slots, E)

    def enqueue_plan():
        mb.mint_lora_plan(table, ids, status, expert_ids=expert_ids, num_experts=E, plan=plan)

    # call grouping: "none" = one fused call per projection; "stage" = projections that can run at the
    # same point of a transformer layer share a call (q,k,v | o | gate,up | down); "layer" = one call per layer
    ncase = len(wl["cases"])
    if moe or args.grouping == "none" or ncase == 1:
        groups_idx = [[i] for i in range(ncase)]
    elif args.grouping == "layer":
        groups_idx = [list(range(ncase))]
    else:
        groups_idx = [[0, 1, 2], [3], [4, 5], [6]] if ncase == 7 else [[i] for i in range(ncase)]
    workspaces = ([mb.new_moe_workspace(dv.pool, T, wl["cases"][0].K) for dv in base] if moe
                  else [mb.new_workspace(dv.pool, T) for dv in base])
    groups = []
    if not moe:
        for row in layers:
            groups.append([mb.ApplyGroup([(row[i][0], row[i][1], row[i][2], workspaces[i]) for i in g])
                           for g in groups_idx])

    def enqueue_layer(li):
        if moe:
            for ci, (pool, x, y) in enumerate(layers[li]):
                mb.mint_moe_lora_apply(pool, table, plan, x, y, status, x_row=base[ci].x_row,
                                       workspace=workspaces[ci])
        else:
            for grp in groups[li]:
                mb.mint_lora_apply_fused_grouped(grp, table, plan, status)

    def enqueue_applies():
        for li in range(L):
            enqueue_layer(li)

    # a fused call is a shrink and an expand launch; batches that may hold dense segments add the two tensor-core kernels
    kernels_per_call = 4 if (not moe and T >= 4096) else 2
    calls_per_layer = len(groups_idx)
    launches_per_step = 1 + L * calls_per_layer * kernels_per_call

    # warm-up outside any graph (first launches load the module), then capture
    enqueue_plan()
    enqueue_applies()
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    step_graph = torch.cuda.CUDAGraph()
    apply_graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(step_graph, stream=stream):
            enqueue_plan()
            enqueue_applies()
        with torch.cuda.graph(apply_graph, stream=stream):
            enqueue_applies()
    torch.cuda.synchronize()

    def timed(graph, steps, warmup):
        with torch.cuda.stream(stream):
            for _ in range(warmup):
                graph.replay()
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(steps):
                graph.replay()
            e1.record(stream)
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            ms = e0.elapsed_time(e1)
        if world > 1:
            t = torch.tensor([ms], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms_total = timed(step_graph, args.steps, args.warmup)
    ms_apply = timed(apply_graph, args.steps, 1)
    clocks = sampler.stop() if rank == 0 else None
    ms_step = ms_total / args.steps
    value = world * T * L / (ms_step * 1e-3)

    if args.profile:
        if rank == 0:
            print(json.dumps({"profile_run": True, "workload": wl["name"], "layers": L, "ms_per_step": ms_step,
                              "us_per_layer": ms_step * 1e3 / L, "grouping": args.grouping,
                              "layer_GBps": layer_bytes / (ms_step * 1e-3 / L) / 1e9,
                              "avg_apply_call_us": ms_apply * 1e3 / args.steps / (L * calls_per_layer)}))
        return

    # ---- end to end through the C ABI with host buffers --------------------------
    # Per step: ids, every x and every y0 come from pinned host memory, the plan and
    # all applies run, and every updated y goes back to pinned host memory.
    e2e_layers = min(L, 4)
    host_ids = ids.cpu().pin_memory()
    host_x = [[x.cpu().pin_memory() for (_, x, _) in row] for row in layers[:e2e_layers]]
    host_y = [[y.cpu().pin_memory() for (_, _, y) in row] for row in layers[:e2e_layers]]
    h2d = host_ids.numel() * 8 + sum(t.numel() * 2 for row in host_x for t in row) + \
        sum(t.numel() * 2 for row in host_y for t in row)
    d2h = sum(t.numel() * 2 for row in host_y for t in row)

    def e2e_step():
        ids.copy_(host_ids, non_blocking=True)
        for li in range(e2e_layers):
            for ci, (pool, x, y) in enumerate(layers[li]):
                x.copy_(host_x[li][ci], non_blocking=True)
                y.copy_(host_y[li][ci], non_blocking=True)
        enqueue_plan()
        for li in range(e2e_layers):
            enqueue_layer(li)
            for ci, (pool, x, y) in enumerate(layers[li]):
                host_y[li][ci].copy_(y, non_blocking=True)

    with torch.cuda.stream(stream):
        for _ in range(3):
            e2e_step()
        torch.cuda.synchronize()
        e2e_steps = max(3, min(args.steps, 10))
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        torch.cuda.synchronize()
        e2e_s = (time.perf_counter() - t0) / e2e_steps
    if world > 1:
        t = torch.tensor([e2e_s], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e_value = world * T * e2e_layers / e2e_s

    st = status.cpu().numpy()
    if st[0] != 0:
        raise SystemExit(f"device status {mb.status_name(int(st[0]))}: the timed run is invalid")

    if rank != 0:
        return
    # ---- roofline of the dominant kernel (the fused apply) ------------------------
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = json.load(open(peaks_path))["hbm_gbs"], "measured (MEASURED_PEAKS.json hbm_gbs)"
    else:
        peak, peak_src = 6650.0, "fallback"
    # the apply is a shrink launch and an expand launch that overlap (programmatic dependent launch),
    # so the roofline unit is the pair: bytes of one call / time of one call
    n_apply = L * calls_per_layer
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
    summary = os.path.join(ROOT, "profiles", f"stream_kernels_{args.workload}_{args.grouping}.md")
    if os.path.exists(summary):
        import re
        m = re.search(r"traffic_bytes_per_launch\s*=\s*(\d+)", open(summary).read())
        if m:
            roofline["traffic"] = int(m.group(1))

    cpu_val, cores, sample = oracle_layer_seconds(wl)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 in, f32 accumulate", "data": "synthetic (seeded)",
        "config": {"workload": wl["name"], "layers_per_step": L, "tokens": T,
                   "l2": f"inputs larger than L2: every layer has its own pool/x/y, {layer_bytes * L / 1e6:.0f} MB algorithmic bytes per step",
                   "grouping": args.grouping, "calls_per_layer": calls_per_layer,
                   "timing": "CUDA graph of plan + all applies, CUDA events on the launching stream"},
        "us_per_layer": ms_step * 1e3 / L,
        "layer_bytes": layer_bytes,
        "layer_GBps": layer_bytes / (ms_step * 1e-3 / L) / 1e9,
        "clocks": clocks,
        "roofline": roofline,
        "cpu_baseline": {"value": cpu_val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "layers_per_step": e2e_layers},
        "gpu_launches": launches_per_step * args.steps,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config2")
    ap.add_argument("--layers", type=int, default=0, help="layers per step (0 = the workload's own)")
    ap.add_argument("--grouping", default="layer", choices=["none", "stage", "layer"],
                    help="how the projections of a layer are grouped into fused calls")
    ap.add_argument("--profile", action="store_true",
                    help="device-timed part only (no end-to-end leg, no CPU oracle): the command profilers wrap")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
