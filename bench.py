#!/usr/bin/env python
"""Benchmark of the full-graph GNN layer pass (InferTurbo's GAS hot path) on B200.

One step = it_infer over all layers of the workload for every vertex (gather, combine, apply,
write; all layers).  Default workload: "medium" (2M vertices, 40M edges, power-law in-degree,
fp32 dim 128, 2-layer GraphSAGE-sum with edge weights, hub threshold 1024).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `value` = vertices/s end to end with inputs resident in HBM; `e2e` = the
same through the C ABI from pinned host buffers (host->device copies of the graph and features
and the device->host read of the result inside the timed region).  With N > 1 every rank runs an
independent replica of the workload (the layer pass does not shard without an exchange step).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "vertices/sec end-to-end (all layers, full graph)"
UNIT = "vertices/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="medium")
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--threshold", type=int, default=None, help="hub-split threshold instead of the workload's (0 = no split)")
    ap.add_argument("--edge-dim", type=int, default=0, help="give every message an edge-feature vector of this length (GraphSAGE workloads)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="target CPU time of the oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    return ap.parse_args()


def workload_config(w, args):
    return {"workload": f"{w.name}" + ("" if args.scale == 1.0 else f" x{args.scale}"),
            "n_vertices": w.n, "n_edges": w.e, "feat_dim": int(w.layers[0].in_dim), "storage": w.dtype,
            "layers": [f"{l.op}:{l.in_dim}->{l.out_dim}:{l.act}" for l in w.layers],
            "edge_weights": w.edge_weights is not None, "edge_feature_dim": int(w.layers[0].edge_dim), "hub_threshold": w.threshold,
            "l2_policy": "inputs larger than L2 (features + CSR >> 126 MB); no explicit flush"}


# ----------------------------------------------------------------------------- CPU oracle timing

COMPACT_ABOVE_BYTES = 16e9   # fp64 bytes of one whole layer input above which the oracle sample is compacted


def affinity_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def time_oracle_sample(w, target_seconds: float):
    """The oracle as it stands, on destinations [0, m) of the workload's graph: every layer's
    pass over those vertices (layer inputs beyond the first are a seeded stand-in of the right
    shape: the time does not depend on the values).  Returns (vertices/s, m, seconds).
    Where fp64 copies of whole layer inputs would not fit comfortably in host memory (the 100M-vertex
    workload), the sampled destinations and the vertices they read are first relabelled to a compact
    graph, outside the timed region; the timed arithmetic is the same."""
    from oracle import oracle as O
    from workloads import rng as wrng
    O.lib()
    rng = np.random.default_rng(0)
    ef = w.edge_feat_as_f32()
    dims = [w.layers[0].in_dim] + [l.out_dim for l in w.layers[:-1]]
    compact = w.n * max(dims) * 8 > COMPACT_ABOVE_BYTES

    if not compact:
        X = w.x_as_f32().astype(np.float64)
        inputs = [X] + [rng.standard_normal((w.n, l.out_dim)) for l in w.layers[:-1]]

    def run(m):
        rows = np.arange(m, dtype=np.int64)
        if compact:
            ids, cip, cix, cw, ct = O.compact_neighbourhood(w.indptr, w.indices, w.edge_weights, rows, 1)[:5]
            x0 = w.x[ids] if w.dtype == "f32" else wrng.bf16_bits_to_f32(w.x[ids])
            ins = [x0.astype(np.float64)] + [rng.standard_normal((len(ids), l.out_dim)) for l in w.layers[:-1]]
            t0 = time.perf_counter()
            for H, layer in zip(ins, w.layers):
                O.layer_forward(cip, cix, cw, H, layer, storage=None, threshold=w.threshold, reorder=False, rows=ct)
            return time.perf_counter() - t0
        t0 = time.perf_counter()
        for H, layer in zip(inputs, w.layers):
            O.layer_forward(w.indptr, w.indices, w.edge_weights, H, layer, storage=None, threshold=w.threshold,
                            reorder=False, rows=rows, edge_feat=ef)
        return time.perf_counter() - t0

    m = min(w.n, 20_000)
    t = run(m)
    if m < w.n and t < target_seconds / 2:
        m = int(min(w.n, max(m, m * target_seconds / max(t, 1e-3))))
        if compact:
            m = min(m, 500_000)   # keeps the fp64 inputs of the compact graph to a few GB
        t = run(m)
    return m / t, m, t


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host cores, K steps of a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from workloads import make, with_edge_features
    w = with_edge_features(make(args.workload, args.scale), args.edge_dim)
    cores = affinity_cores()
    per_step = max(2.0, min(args.cpu_seconds, 120.0 / max(1, args.steps + args.warmup)))
    vals, m, secs = [], 0, 0.0
    for i in range(args.warmup + args.steps):
        v, m, t = time_oracle_sample(w, per_step)
        if i >= args.warmup:
            vals.append(v)
            secs += t
    value = float(np.mean(vals)) if vals else 0.0
    sample = f"all layers on destinations [0,{m}) of {w.name} per step, fp64, OpenMP"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * secs / max(1, args.steps), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload_config(w, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str | None):
        self.path = tempfile.mktemp(prefix="clocks_", suffix=".csv")
        cmd = ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"]
        if uuid:
            cmd.insert(1, f"--id={uuid}")
        try:
            self.proc = subprocess.Popen(cmd, stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "power_w_max": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                p = [t.strip() for t in line.split(",")]
                if len(p) < 7:
                    continue
                try:
                    sm.append(float(p[0])); mx.append(float(p[1])); pw.append(float(p[2]))
                except ValueError:
                    continue
                for nm, val in zip(names, p[3:7]):
                    if val == "Active":
                        reasons.add(nm)
            os.unlink(self.path)
        except OSError:
            pass
        if sm:
            # under load = samples in the upper half of the power range seen
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), power_w_max=float(max(pw)),
                       reasons=sorted(reasons), samples=len(sm))
        return out


# ----------------------------------------------------------------------------- ranks

def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's time: the replicas run side by side, so the whole job takes as long as that rank."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: int, world: int, ms_per_step: float) -> float:
    """Units all ranks processed per second (every rank runs the same workload: weak scaling)."""
    return world * units_per_rank / (ms_per_step * 1e-3)


# ----------------------------------------------------------------------------- the GPU arm

def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2307_00228_b200 import binding as B
    from paper_2307_00228_b200 import host
    from workloads import make, with_edge_features

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.lib()

    def barrier():
        if world > 1:
            dist.barrier()

    w = with_edge_features(make(args.workload, args.scale), args.edge_dim)
    if args.threshold is not None:
        w.threshold = args.threshold
    int32_csr = w.name == "large"   # that workload is defined with an int32 CSR
    d = host.upload(w, int32_indptr=int32_csr)
    dev = torch.device("cuda", local)

    for _ in range(max(3, args.warmup)):
        d.infer()
    torch.cuda.synchronize()

    # ---- preprocessing, reported apart from the layer pass: validate the CSR, split the hubs + bucket the rows
    def timed_ms(fn, reps=3):
        best = None
        for _ in range(reps):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            r = fn()
            torch.cuda.synchronize()
            dt = (time.perf_counter() - t0) * 1e3
            best = dt if best is None else min(best, dt)
        return best, r

    keep = d.graph._keep
    create_ms, g2 = timed_ms(lambda: B.it_graph_create(keep[0], keep[1], keep[2]))
    split_ms, _ = timed_ms(lambda: B.it_split_hubs(g2, w.threshold))
    del g2

    # ---- timed region: K steps, inputs resident in HBM
    uuid = None
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        pass
    sampler = ClockSampler(uuid)
    time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    launches0 = B.it_kernel_launch_count()
    B.it_profile_begin()
    ev0.record()
    for _ in range(args.steps):
        d.infer()
    ev1.record()
    torch.cuda.synchronize()
    barrier()
    stats = B.it_profile_end()
    launches = B.it_kernel_launch_count() - launches0
    ms_total = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    ms_total = max_over_ranks(ms_total, world, dev)
    ms_per_step = ms_total / args.steps
    value = whole_job_value(w.n, world, ms_per_step)

    # ---- per-layer edges/s (each layer alone, same buffers as a real pass)
    layer_stats = []
    h = d.x
    for lay, src in zip(d.layers, w.layers):
        ws = d.workspace   # sized for it_infer, so large enough for any single layer
        o = torch.empty((w.n, src.out_dim), dtype=d.x.dtype, device=dev)
        for _ in range(3):
            B.it_layer_forward(d.graph, lay, h, o, ws)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.steps):
            B.it_layer_forward(d.graph, lay, h, o, ws)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / args.steps
        layer_stats.append({"layer": f"{src.op}:{src.in_dim}->{src.out_dim}", "ms": ms, "edges_per_s": w.e / (ms * 1e-3)})
        h = o

    # ---- end to end from pinned host buffers through the C ABI
    e2e = None
    if not args.no_e2e:
        graph_t = d.graph._keep
        host_in = [torch.from_numpy(w.x if w.dtype == "f32" else w.x.view(np.int16)).pin_memory(),
                   torch.from_numpy(w.indptr.astype(np.int32) if int32_csr else w.indptr).pin_memory(),
                   torch.from_numpy(w.indices).pin_memory()]
        dev_in = [d.x.view(torch.int16) if w.dtype == "bf16" else d.x, graph_t[0], graph_t[1]]
        if w.edge_weights is not None:
            host_in.append(torch.from_numpy(w.edge_weights).pin_memory())
            dev_in.append(graph_t[2])
        if w.edge_feat is not None:
            host_in.append(torch.from_numpy(w.edge_feat if w.dtype == "f32" else w.edge_feat.view(np.int16)).pin_memory())
            dev_in.append(d.graph._edge_feat.view(torch.int16) if w.dtype == "bf16" else d.graph._edge_feat)
        host_out = torch.empty(d.out.shape, dtype=d.out.dtype).pin_memory()
        h2d = sum(t_.numel() * t_.element_size() for t_ in host_in)
        d2h = host_out.numel() * host_out.element_size()

        def e2e_step():
            for src_t, dst_t in zip(host_in, dev_in):
                dst_t.copy_(src_t, non_blocking=True)
            d.infer()
            host_out.copy_(d.out, non_blocking=True)

        e2e_step()
        torch.cuda.synchronize()
        k = max(3, min(args.steps, 10))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        a.record()
        for _ in range(k):
            e2e_step()
        b.record()
        torch.cuda.synchronize()
        e2e_ms = max_over_ranks(a.elapsed_time(b) / k, world, dev)
        e2e = {"value": whole_job_value(w.n, world, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": k}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (live CUDA-event time from the timed region)
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peaks = json.load(open(peaks_path))
        hbm_peak, peak_src = float(peaks["hbm_gbs"]), "measured"
    else:
        hbm_peak, peak_src = 6650.0, "fallback"
    tot_ms = sum(s["total_ms"] for s in stats) or 1.0
    kernels = sorted(({"name": s["name"], "launches": s["launches"], "ms_per_step": s["total_ms"] / args.steps,
                       "share": s["total_ms"] / tot_ms,
                       "algo_GBps": (s["algo_bytes"] / 1e9) / (s["total_ms"] * 1e-3) if s["total_ms"] > 0 else 0.0}
                      for s in stats), key=lambda r: -r["share"])
    top = max(stats, key=lambda s: s["total_ms"])
    achieved = (top["algo_bytes"] / 1e9) / (top["total_ms"] * 1e-3)
    # DRAM bytes per launch of that kernel from the committed ncu capture (lines "traffic <workload>:<kernel> <bytes>")
    traffic = None
    traffic_path = os.path.join(ROOT, "profiles", "traffic.md")
    if os.path.exists(traffic_path) and args.scale == 1.0:
        for line in open(traffic_path):
            parts = line.split()
            if len(parts) == 3 and parts[0] == "traffic" and parts[1] == f"{w.name}:{top['name']}":
                traffic = float(parts[2])
    roofline = {"bound": "hbm", "kernel": top["name"], "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                "frac": achieved / hbm_peak, "peak_source": peak_src, "traffic": traffic,
                "dram_GBps": None if traffic is None else traffic / 1e9 / (top["total_ms"] / max(1, top["launches"]) * 1e-3),
                "algo_bytes_per_launch": top["algo_bytes"] / max(1, top["launches"]),
                "ms_per_launch": top["total_ms"] / max(1, top["launches"])}

    cpu = None
    if not args.no_cpu_baseline:
        v, m, secs = time_oracle_sample(w, args.cpu_seconds)
        cpu = {"value": v, "unit": UNIT, "cores": affinity_cores(), "kind": "oracle",
               "sample": f"all layers on destinations [0,{m}) of {w.name} ({secs:.1f} s), fp64, OpenMP"}

    print(json.dumps({
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w.dtype, "data": "synthetic", "config": workload_config(w, args),
        "edges_per_sec_per_layer": layer_stats, "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline, "kernels": kernels, "cpu_baseline": cpu,
        "split": {"rows": d.n_rows, "split_owners": d.n_split_owners},
        "preprocess": {"graph_create_ms": create_ms, "split_and_bucket_ms": split_ms, "timing": "host clock around the call, best of 3"}}))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
