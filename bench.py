#!/usr/bin/env python
"""Benchmark of the aggregation hot path: one step = CSR build + chunked GCN aggregation on the
Reddit-shaped synthetic workload (config 4: 232,965 vertices, ~115M edges + self-loops, F = 602 fp32).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--chunk-width C]

Prints ONE JSON line.  With --gpus N > 1 (under torchrun) every rank processes its own graph of the
same shape (different seed): weak scaling, no data-path collective.  --impl reference times the CPU
oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import graphgen as gg  # noqa: E402

METRIC = "aggregated edge-features/sec"
UNIT = "edge-features/s"
WORKLOADS = {
    "config4": dict(kind="config4", desc="GCN, 232,965 vertices, ~115M power-law edges + self-loops, F=602 fp32 (ld 608)"),
    "config4_small": dict(kind="config4", factor=0.25, desc="config 4 recipe at 1/4 of the vertices and 1/16 of the edges"),
}


def make_workload(name: str, seed: int):
    spec = WORKLOADS[name]
    if "factor" in spec:
        return gg.scaled("config4", spec["factor"], seed)
    return gg.config4(seed)


def roofline_bytes(n: int, nnz: int, f: int, elem: int, weighted: bool = True) -> int:
    """CSR indices and weights once, each row pointer once, every gathered feature."""
    return 4 * (n + 1) + 4 * nnz + (4 * nnz if weighted else 0) + nnz * f * elem


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        self.proc.wait()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val == "Active":
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------ CPU oracle arm

def oracle_sample(w, rows_in_sample: int, seed: int = 0):
    """The in-edges of a random sample of destination rows: a bounded piece of the same workload."""
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(w.n, size=min(rows_in_sample, w.n), replace=False)).astype(np.int64)
    mask = np.zeros(w.n, bool)
    mask[rows] = True
    keep = mask[w.dst]
    return rows, w.src[keep], w.dst[keep]


def oracle_step(w, rows, src, dst, threads: int):
    """CSR build + GCN aggregation of the sampled rows with the CPU oracle; returns edge-features done."""
    import oracle as orc
    row_ptr, col, _ = orc.build_csr(w.n, src, dst, w.flags)
    orc.aggregate("gcn", row_ptr, col, w.x, w.f, chunk_width=w.f, rows=rows, threads=threads)
    deg = np.diff(row_ptr)
    return int(deg[rows].sum()) * w.f


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle as orc
    w = make_workload(args.workload, args.seed)
    threads = orc.max_threads()
    rows, src, dst = oracle_sample(w, args.cpu_rows)
    for _ in range(args.warmup):
        oracle_step(w, rows, src, dst, threads)
    t0 = time.perf_counter()
    units = 0
    for _ in range(args.steps):
        units += oracle_step(w, rows, src, dst, threads)
    dt = time.perf_counter() - t0
    value = units / dt
    sample = "CSR build + GCN aggregation (F=%d, fp64) of the in-edges of %d sampled destination rows per step" % (
        w.f, len(rows))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "description": WORKLOADS[args.workload]["desc"], "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------ CUDA arm

def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2104_03058_b200 as g

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    g.lib()

    w = make_workload(args.workload, args.seed + rank)
    e = len(w.src)
    h_src = torch.from_numpy(w.src).pin_memory()
    h_dst = torch.from_numpy(w.dst).pin_memory()
    h_x = torch.from_numpy(w.x).pin_memory()
    d_src, d_dst, d_x = h_src.to(device), h_dst.to(device), h_x.to(device)
    out = torch.empty((w.n, w.ld), dtype=torch.float32, device=device)
    h_out = torch.empty((w.n, w.ld), dtype=torch.float32).pin_memory()
    pb, sb = g.csr_workspace_bytes(w.n, e, w.flags)
    persistent = torch.empty(pb, dtype=torch.uint8, device=device)
    scratch = torch.empty(sb, dtype=torch.uint8, device=device)
    out_view = out[:, :w.f]
    cw = args.chunk_width

    state = {"agg_scratch": None, "csr": None}

    def step():
        if state["csr"] is not None:
            state["csr"].destroy()
        csr = g.build_csr(w.n, d_src, d_dst, w.flags, persistent=persistent, scratch=scratch)
        if state["agg_scratch"] is None:
            state["agg_scratch"] = torch.empty(max(g.aggregate_workspace_bytes(csr, w.f), 256), dtype=torch.uint8,
                                               device=device)
        g.aggregate_gcn(csr, d_x, f=w.f, chunk_width=cw, out=out_view, scratch=state["agg_scratch"])
        state["csr"] = csr
        return csr

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        csr = step()
    nnz = csr.nnz
    units_per_step = nnz * w.f

    # ---- timed region: device-resident inputs
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    g.kernel_timing_enable(True)
    g.kernel_timing_read()
    launches0 = g.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1)
    launches = g.launch_count() - launches0
    kernels = g.kernel_timing_read()
    g.kernel_timing_enable(False)
    clocks = sampler.stop()

    # ---- end to end: pinned host inputs in, result out, every step (the package's host-buffer front end:
    # double-buffered device copies, the next step's inputs and the previous result travel while the kernels run)
    from paper_2104_03058_b200.host import HostGcnPipeline
    pipe = HostGcnPipeline(w.n, e, w.f, w.ld, w.flags, cw, device=device)
    job = (h_src, h_dst, h_x)
    pipe.submit(*job, h_out)                         # warm-up job (allocates the aggregation workspace)
    pipe.finish()
    barrier()
    ev2, ev3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev2.record()
    for i in range(args.steps):
        pipe.submit(*job, h_out, next_job=job if i + 1 < args.steps else None)
    pipe.finish()
    ev3.record()
    barrier()
    ms_e2e = ev2.elapsed_time(ev3)
    h2d = h_src.numel() * 4 + h_dst.numel() * 4 + h_x.numel() * 4
    d2h = h_out.numel() * 4
    del pipe

    # ---- aggregation alone (context for the step time), a few calls
    agg_ms = {}
    for width in sorted(set(args.sweep + [cw])):
        g.aggregate_gcn(state["csr"], d_x, f=w.f, chunk_width=width, out=out_view, scratch=state["agg_scratch"])
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(3):
            g.aggregate_gcn(state["csr"], d_x, f=w.f, chunk_width=width, out=out_view, scratch=state["agg_scratch"])
        a1.record()
        torch.cuda.synchronize()
        agg_ms[width] = a0.elapsed_time(a1) / 3

    t = torch.tensor([ms, ms_e2e, float(units_per_step)], dtype=torch.float64, device=device)
    if world > 1:
        tmax = t.clone()
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        tsum = t.clone()
        dist.all_reduce(tsum, op=dist.ReduceOp.SUM)
        ms, ms_e2e, total_units = tmax[0].item(), tmax[1].item(), tsum[2].item()
    else:
        total_units = float(units_per_step)

    if rank == 0:
        peak, peak_src = measured_peaks()
        name = "gather_aggregate_gcn"
        k_ms, k_n = kernels.get(name, (0.0, 0))
        bytes_launch = roofline_bytes(w.n, nnz, w.f, 4)
        achieved = bytes_launch / (k_ms / k_n * 1e-3) / 1e9 if k_n else None
        total_kernel_ms = sum(v[0] for v in kernels.values())
        result = {
            "metric": METRIC, "value": total_units * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "description": WORKLOADS[args.workload]["desc"],
                       "step": "gnnfd_build_csr + gnnfd_aggregate_gcn", "n": w.n, "input_edges": e, "nnz": nnz,
                       "f": w.f, "chunk_width": cw, "parallelism": "independent graphs per GPU" if world > 1 else "1 GPU",
                       "l2": "inputs larger than L2 (x %d MB, col_idx+weights %d MB per sweep; L2 126 MB)"
                             % (w.n * w.ld * 4 // 2**20, nnz * 8 // 2**20)},
            "roofline": {"bound": "hbm", "kernel": name, "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak if achieved else None, "peak_source": peak_src,
                         "bytes_per_launch": bytes_launch, "kernel_ms": k_ms / k_n if k_n else None,
                         "frac_of_8TBs_nominal": achieved / 8000.0 if achieved else None, "traffic": None},
            "e2e": {"value": total_units * args.steps / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": launches,
            "clocks": clocks,
            "kernels": {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps,
                            "share": v[0] / total_kernel_ms if total_kernel_ms else None}
                        for k, v in sorted(kernels.items(), key=lambda kv: -kv[1][0])},
            "aggregate_only": {str(k): {"ms": v, "edge_features_per_s": units_per_step / (v * 1e-3),
                                        "roofline_GBs": roofline_bytes(w.n, nnz, w.f, 4) / (v * 1e-3) / 1e9}
                               for k, v in agg_ms.items()},
        }
        if world == 1 and not args.no_cpu_baseline:
            import oracle as orc
            threads = orc.max_threads()
            rows, s_src, s_dst = oracle_sample(w, args.cpu_rows)
            t0 = time.perf_counter()
            units = oracle_step(w, rows, s_src, s_dst, threads)
            dt = time.perf_counter() - t0
            result["cpu_baseline"] = {
                "value": units / dt, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": dt,
                "sample": "CSR build + GCN aggregation (F=%d, fp64) of the in-edges of %d sampled destination rows"
                          % (w.f, len(rows))}
        print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=sorted(WORKLOADS), default="config4")
    ap.add_argument("--chunk-width", type=int, default=64)
    ap.add_argument("--sweep", type=int, nargs="*", default=[], help="extra chunk widths to time (aggregation only)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--cpu-rows", type=int, default=16384, help="destination rows in the CPU-oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
