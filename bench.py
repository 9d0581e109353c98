#!/usr/bin/env python
"""Benchmark of the aggregation hot path.

One step = gnnfd_build_csr + one chunked aggregation (GCN, GraphSAGE mean or GAT, as the workload
says) over one synthetic graph.  The default workload is the Reddit-shaped config 4 (232,965
vertices, ~115M edges + self-loops, F = 602 fp32, GCN); the other configs are available with
--workload for the results tables and the profiles.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload W] [--chunk-width C]

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

# name -> (factory, default chunk width, description)
WORKLOADS = {
    "config1": (lambda s: gg.config1(s), 16, "GCN, 4,096 vertices, ~40k power-law edges + self-loops, F=16 fp32"),
    "config2": (lambda s: gg.config2(s), 64, "GraphSAGE mean, 100,000 vertices, avg degree 20 power law, F=128 fp32"),
    "config3": (lambda s: gg.config3(s), 64,
                "GAT, 200,000 vertices, avg degree 15 power law + self-loops, 8 heads x 8 dims fp32"),
    "config4": (lambda s: gg.config4(s), 64,
                "GCN, 232,965 vertices, ~115M power-law edges + self-loops, F=602 fp32 (ld 608)"),
    "config4_small": (lambda s: gg.scaled("config4", 0.25, s), 64,
                      "config 4 recipe at 1/4 of the vertices and 1/16 of the edges"),
    "config5_f256": (lambda s: gg.config5(s, f=256), 256,
                     "GCN, RMAT scale 21, 60M edges symmetrised + dedup + self-loops, F=256 bf16"),
    "config5_f64": (lambda s: gg.config5(s, f=64), 64, "GCN, RMAT scale 21 (as config5_f256), F=64 bf16"),
    "config5_f32": (lambda s: gg.config5(s, f=32), 32, "GCN, RMAT scale 21 (as config5_f256), F=32 bf16"),
    "config5_f16": (lambda s: gg.config5(s, f=16), 16, "GCN, RMAT scale 21 (as config5_f256), F=16 bf16"),
    "config5_f8": (lambda s: gg.config5(s, f=8), 8, "GCN, RMAT scale 21 (as config5_f256), F=8 bf16"),
}
# hidden-layer aggregation on the config-4 graph (the paper's Hid = 8 / 16 / 32 / 64 settings, Section III)
for _model in ("gcn", "sage", "gat"):
    for _hid in (8, 16, 32, 64):
        WORKLOADS["reddit_%s_hid%d" % (_model, _hid)] = (
            (lambda s, m=_model, h=_hid: gg.reddit_hidden(m, h, s)), _hid,
            "%s on the config-4 graph (232,965 vertices, ~115M edges + self-loops), hidden width %d fp32"
            % (_model.upper(), _hid))
WORKLOADS["reddit_small_gat_hid64"] = (
    (lambda s: gg.reddit_hidden("gat", 64, s, factor=0.25)), 64,
    "GAT on the config-4 recipe at 1/4 of the vertices and 1/16 of the edges, 8 heads x 8 dims fp32")
# DRAM bytes per launch of the dominant kernel from a one-pass ncu capture of the same launch
# (dram__bytes_read.sum + dram__bytes_write.sum), valid only for the kernel sources they were taken with.
NCU_TRAFFIC = {"config4": {"bytes": 16.823e9, "sources_sha1": "20fda6161c29e4d7927491bed812043bb79b7a77"},
               "config5_f256": {"bytes": 14.644e9, "sources_sha1": "20fda6161c29e4d7927491bed812043bb79b7a77"}}
KERNEL_SOURCES = ("paper_2104_03058_b200/csrc/aggregate.cu", "paper_2104_03058_b200/csrc/schedule.cuh",
                  "paper_2104_03058_b200/csrc/vec.cuh")
# L2-to-crossbar peak that ncu derives on this part (derived__lts__lts2xbar_bytes.sum.peak_sustained), bytes per clock
L2_PEAK_BYTES_PER_CLK = 11776


PROBE_SRC = os.path.join(ROOT, "bench_l2_probe.cu")
PROBE_LIB = os.path.join(ROOT, "libbench_l2_probe.so")


def build_l2_probe(force: bool = False) -> str:
    """Compiles the bench-only helper that measures random row reads out of a resident working set."""
    if force or not os.path.exists(PROBE_LIB) or os.path.getmtime(PROBE_LIB) < os.path.getmtime(PROBE_SRC):
        tmp = PROBE_LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call([os.environ.get("NVCC", "nvcc"), "-std=c++17", "-O3", "-gencode",
                               "arch=compute_100a,code=sm_100a", "-lineinfo", "-Xcompiler", "-fPIC", "-shared",
                               "-o", tmp, PROBE_SRC])
        os.replace(tmp, PROBE_LIB)
    return PROBE_LIB


def measure_random_row_reads(buf, rows: int, pitch_bytes: int = 256):
    """GB/s at which random 256-byte rows of a resident set reach the SMs (None if the helper cannot be built)."""
    import ctypes

    import torch
    try:
        lib = ctypes.CDLL(build_l2_probe())
    except (OSError, subprocess.CalledProcessError):
        return None
    lib.bench_random_row_reads.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int64, ctypes.c_int64,
                                           ctypes.c_void_p, ctypes.POINTER(ctypes.c_double)]
    out = ctypes.c_double()
    rc = lib.bench_random_row_reads(ctypes.c_void_p(buf.data_ptr()), buf.numel() * buf.element_size(), rows, pitch_bytes,
                                    ctypes.c_void_p(torch.cuda.current_stream().cuda_stream), ctypes.byref(out))
    return out.value if rc == 0 else None


def kernel_sources_sha1() -> str:
    import hashlib
    h = hashlib.sha1()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def ncu_traffic(workload: str):
    rec = NCU_TRAFFIC.get(workload)
    if rec is None or rec["sources_sha1"] != kernel_sources_sha1():
        return None
    return rec["bytes"]


KERNEL_OF_MODEL = {"gcn": "gather_aggregate_gcn", "sage": "gather_aggregate_sage", "gat": "gat_aggregate"}


def make_workload(name: str, seed: int):
    return WORKLOADS[name][0](seed)


def roofline_bytes(w, nnz: int, f: int | None = None) -> int:
    """Algorithmic bytes of one aggregation launch: every row pointer once, the CSR column indices once,
    the GCN weights once, every gathered feature (and, for GAT, every gathered score)."""
    elem = 2 if w.dtype == "bf16" else 4
    b = 4 * (w.n + 1) + 4 * nnz + nnz * (w.f if f is None else f) * elem
    if w.model == "gcn":
        b += 4 * nnz
    if w.model == "gat":
        b += 4 * nnz * w.heads
    return b


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, an earlier copy-bandwidth measurement on the same GPU model)"


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
            time.sleep(0.3)        # let the sampler come up before the timed region starts
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
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


def oracle_step(w, rows, src, dst, threads: int, chunk_width: int | None = None):
    """CSR build + aggregation of the sampled rows with the CPU oracle; returns edge-features done."""
    import oracle as orc
    row_ptr, col, _ = orc.build_csr(w.n, src, dst, w.flags)
    cw = w.f if chunk_width is None else chunk_width
    if w.model == "gat":
        orc.aggregate_gat(row_ptr, col, w.x, w.a_src, w.a_dst, w.heads, w.dim, w.negative_slope, chunk_width=cw,
                          rows=rows, threads=threads)
    else:
        orc.aggregate(w.model, row_ptr, col, w.x, w.f, chunk_width=cw, rows=rows, threads=threads)
    deg = np.diff(row_ptr)
    return int(deg[rows].sum()) * w.f


def oracle_single_core(w, n_rows: int, widths):
    """The oracle as it stands on ONE core, on a smaller row sample: undecomposed and at the given chunk
    widths (the paper's CPU effect, Section II-B: a narrower chunk keeps the gathered slice in the cache)."""
    rows, src, dst = oracle_sample(w, n_rows, seed=1)
    res = {"cores": 1, "kind": "oracle", "unit": UNIT, "sample": sample_text(w, len(rows)), "by_chunk_width": {}}
    for cw in [w.f] + [c for c in widths if c < w.f]:
        t0 = time.perf_counter()
        units = oracle_step(w, rows, src, dst, 1, chunk_width=cw)
        dt = time.perf_counter() - t0
        res["by_chunk_width"]["undecomposed" if cw >= w.f else str(cw)] = {"value": units / dt, "seconds": dt}
    res["value"] = res["by_chunk_width"]["undecomposed"]["value"]
    return res


def sample_text(w, n_rows: int) -> str:
    return "CSR build + %s aggregation (F=%d, fp64) of the in-edges of %d sampled destination rows" % (
        w.model.upper(), w.f, n_rows)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle as orc
    w = make_workload(args.workload, args.seed)
    threads = orc.max_threads()
    rows, src, dst = oracle_sample(w, args.cpu_rows or 16384)
    for _ in range(args.warmup):
        oracle_step(w, rows, src, dst, threads)
    t0 = time.perf_counter()
    units = 0
    for _ in range(args.steps):
        units += oracle_step(w, rows, src, dst, threads)
    dt = time.perf_counter() - t0
    value = units / dt
    sample = sample_text(w, len(rows)) + " per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "description": WORKLOADS[args.workload][2], "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------ CUDA arm

def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2104_03058_b200 as g
    from paper_2104_03058_b200 import sharding
    from paper_2104_03058_b200.host import HostPipeline

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    if not os.path.exists(g.build.LIB_PATH):      # a checkout without the built library: compile it (atomic replace)
        g.build.build_library()
    g.lib()

    # --shard columns: ONE graph for all ranks (same seed); each rank builds the CSR and aggregates only the
    # decomposition layers of its column slab (strong scaling).  Default: an independent graph per rank (weak).
    by_columns = args.shard == "columns"
    w = make_workload(args.workload, args.seed + (0 if by_columns else rank))
    cw = args.chunk_width or WORKLOADS[args.workload][1]
    j0, j1 = sharding.column_slab(w.f, cw, world, rank) if by_columns else (0, w.f)
    e = len(w.src)
    bf16 = w.dtype == "bf16"
    h_src = torch.from_numpy(w.src).pin_memory()
    h_dst = torch.from_numpy(w.dst).pin_memory()
    h_x = (torch.from_numpy(w.x.view(np.int16)).view(torch.bfloat16) if bf16 else torch.from_numpy(w.x)).pin_memory()
    d_src, d_dst, d_x = h_src.to(device), h_dst.to(device), h_x.to(device)
    out = torch.empty((w.n, w.ld), dtype=torch.float32, device=device)
    h_out = torch.empty((w.n, w.ld), dtype=torch.float32).pin_memory()
    pb, sb = g.csr_workspace_bytes(w.n, e, w.flags)
    persistent = torch.empty(pb, dtype=torch.uint8, device=device)
    scratch = torch.empty(sb, dtype=torch.uint8, device=device)
    out_view = out[:, :w.f]
    gat = w.model == "gat"
    a_src = torch.from_numpy(w.a_src).to(device) if gat else None
    a_dst = torch.from_numpy(w.a_dst).to(device) if gat else None

    state = {"agg_scratch": None, "csr": None}

    def aggregate(csr, width):
        if by_columns:
            sharding.aggregate_slab(csr, d_x, w.model, w.f, width, world, rank, out_view, a_src=a_src, a_dst=a_dst,
                                    heads=w.heads, dim=w.dim, negative_slope=w.negative_slope,
                                    scratch=state["agg_scratch"])
            if args.gather and world > 1:
                sharding.gather_slabs_(out_view, w.f, width)
        elif gat:
            g.aggregate_gat(csr, d_x, a_src, a_dst, w.heads, w.dim, w.negative_slope, chunk_width=width, out=out_view,
                            scratch=state["agg_scratch"])
        elif w.model == "sage":
            g.aggregate_sage(csr, d_x, f=w.f, chunk_width=width, out=out_view, scratch=state["agg_scratch"])
        else:
            g.aggregate_gcn(csr, d_x, f=w.f, chunk_width=width, out=out_view, scratch=state["agg_scratch"])

    def step():
        if state["csr"] is not None:
            state["csr"].destroy()
        csr = g.build_csr(w.n, d_src, d_dst, w.flags, persistent=persistent, scratch=scratch)
        if state["agg_scratch"] is None:
            need = g.gat_workspace_bytes(csr, w.heads, w.dim) if gat else g.aggregate_workspace_bytes(csr, w.f)
            state["agg_scratch"] = torch.empty(max(need, 256), dtype=torch.uint8, device=device)
        aggregate(csr, cw)
        state["csr"] = csr
        return csr

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        csr = step()
    nnz = csr.nnz
    units_per_step = nnz * (j1 - j0)

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
    job = (h_src, h_dst, h_x)
    if by_columns:
        # a rank moves the edge list, its own columns of x in and its own columns of the result out
        def e2e_step():
            d_src.copy_(h_src, non_blocking=True)
            d_dst.copy_(h_dst, non_blocking=True)
            d_x[:, j0:j1].copy_(h_x[:, j0:j1], non_blocking=True)
            step()
            h_out[:, j0:j1].copy_(out[:, j0:j1], non_blocking=True)
        e2e_step()
        barrier()
        ev2, ev3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev2.record()
        for i in range(args.steps):
            e2e_step()
        ev3.record()
        barrier()
        ms_e2e = ev2.elapsed_time(ev3)
        esize = h_x.element_size()
        h2d = h_src.numel() * h_src.element_size() * 2 + w.n * (j1 - j0) * esize
        d2h = w.n * (j1 - j0) * 4
    else:
        pipe = HostPipeline(w.n, e, w.f, w.ld, w.flags, cw, device=device, feature_dtype=h_x.dtype, model=w.model,
                            heads=w.heads, dim=w.dim, a_src=a_src, a_dst=a_dst, negative_slope=w.negative_slope)
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
        h2d = sum(t.numel() * t.element_size() for t in job)
        d2h = h_out.numel() * 4
        del pipe

    # ---- aggregation alone (context for the step time), a few calls per chunk width
    agg_ms, agg_cold_ms = {}, {}
    reps = 3 if units_per_step > 1e9 else 50
    l2_bytes = torch.cuda.get_device_properties(device).L2_cache_size
    flush = torch.empty(2 * l2_bytes, dtype=torch.uint8, device=device)
    for width in sorted(set(args.sweep + [cw])):
        aggregate(state["csr"], width)
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(reps):
            aggregate(state["csr"], width)
        a1.record()
        torch.cuda.synchronize()
        agg_ms[width] = a0.elapsed_time(a1) / reps
        # cold L2: a buffer of twice the L2 size is overwritten before every timed call (outside the timing)
        cold = []
        for _ in range(3):
            flush.zero_()
            a0.record()
            aggregate(state["csr"], width)
            a1.record()
            torch.cuda.synchronize()
            cold.append(a0.elapsed_time(a1))
        agg_cold_ms[width] = statistics.median(cold)

    softmax_ms = None
    if gat:        # the materialised edge softmax (alpha per CSR slot) on the same graph, timed alone
        s_src, s_dst = g.gat_scores(d_x, a_src, a_dst, w.heads, w.dim)
        alpha = torch.empty((nnz, w.heads), dtype=torch.float32, device=device)
        sm_scratch = torch.empty(max(g.edge_softmax_workspace_bytes(state["csr"], w.heads), 256), dtype=torch.uint8,
                                 device=device)
        g.edge_softmax(state["csr"], s_src, s_dst, w.negative_slope, out=alpha, scratch=sm_scratch)
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(reps):
            g.edge_softmax(state["csr"], s_src, s_dst, w.negative_slope, out=alpha, scratch=sm_scratch)
        a1.record()
        torch.cuda.synchronize()
        softmax_ms = a0.elapsed_time(a1) / reps

    def timed(fn, reps_):
        fn()
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(reps_):
            fn()
        t1.record()
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / reps_

    combine_ms = combine_fp32_ms = None
    layer_ms = {}
    if not bf16 and args.combine_out > 0 and not by_columns and not args.core_only:
        # the dense transform a layer runs ahead of its aggregation (Section III), timed alone: x [n, f] -> [n, combine_out];
        # then whole layers (transform + aggregation of the transformed columns) on the built CSR
        co = args.combine_out
        w_t = (torch.randn((co, w.ld), device=device) * 0.05)
        z = torch.empty((w.n, co), device=device)
        status = torch.zeros(1, dtype=torch.int32, device=device)
        combine_ms = timed(lambda: g.combine(d_x[:, :w.f], w_t[:, :w.f], out=z, status=status), 20)
        combine_fp32_ms = timed(lambda: g.combine(d_x[:, :w.f], w_t[:, :w.f], out=z, status=status, mode="fp32"), 20)
        lay_out = torch.empty((w.n, co), device=device)
        heads_l = max(co // 8, 1)
        att = torch.randn((heads_l, co // heads_l), device=device) * 0.1
        for lm in ("gcn", "sage", "gat"):
            if lm == "gat" and co % heads_l:
                continue
            kw = dict(a_src=att, a_dst=att, heads=heads_l, dim=co // heads_l) if lm == "gat" else {}
            scr = torch.empty(g.layer_workspace_bytes(state["csr"], lm, co, kw.get("heads", 0), kw.get("dim", 0)),
                              dtype=torch.uint8, device=device)
            for md in ("tf32", "fp32"):
                layer_ms[lm + "_" + md] = timed(lambda: g.layer(state["csr"], lm, d_x[:, :w.f], w_t[:, :w.f], mode=md, out=lay_out,
                                                               scratch=scr, status=status, **kw), 10)
            del scr
        if int(status.item()) != 0:
            raise SystemExit("gnnfd_combine reported a timed-out wait")
        del z, w_t, lay_out

    # the light set-up for graphs that are aggregated once: destination-only sort (rows in edge-id order), then
    # the same aggregation; and both in one call from one buffer
    light = None
    if not gat and not by_columns and not (w.flags & g.CSR_DEDUP) and not args.core_only:
        def light_step():
            c2 = g.build_csr(w.n, d_src, d_dst, w.flags | g.CSR_INPUT_ORDER, persistent=persistent, scratch=scratch)
            (g.aggregate_sage if w.model == "sage" else g.aggregate_gcn)(c2, d_x, f=w.f, chunk_width=cw, out=out_view,
                                                                        scratch=state["agg_scratch"])
            c2.destroy()
        one_scratch = torch.empty(g.oneshot_workspace_bytes(w.n, e, w.flags, w.f), dtype=torch.uint8, device=device)
        light = {"light_build_plus_aggregate_ms": timed(light_step, 5),
                 "oneshot_call_ms": timed(lambda: g.oneshot(w.model, w.n, d_src, d_dst, d_x, flags=w.flags, f=w.f,
                                                            chunk_width=cw, out=out_view, scratch=one_scratch), 5),
                 "full_build_plus_aggregate_ms": timed(step, 5)}
        del one_scratch
        step()          # leaves the fully ordered CSR in place for what follows

    # what L2 delivers for random row reads of one chunk's slice with nothing else going on: the measured
    # ceiling beside the L2 peak that ncu derives
    l2_measured = None
    slice_rows = min(w.n, out.numel() * 4 // 256)
    if slice_rows * 256 <= 0.6 * l2_bytes:
        l2_measured = measure_random_row_reads(out, slice_rows, 256)

    rank_ms = ms
    ms, total_units = sharding.reduce_job_timing(ms, float(units_per_step), device=device)
    ms_e2e, _ = sharding.reduce_job_timing(ms_e2e, 0.0, device=device)
    per_rank = [{"rank": rank, "columns": [j0, j1], "ms_per_step": rank_ms / args.steps}]
    if world > 1:
        gathered = [None] * world
        dist.all_gather_object(gathered, per_rank[0])
        per_rank = gathered

    if rank == 0:
        peak, peak_src = measured_peaks()
        name = KERNEL_OF_MODEL[w.model]
        k_ms, k_n = kernels.get(name, (0.0, 0))
        bytes_launch = roofline_bytes(w, nnz, j1 - j0)
        achieved = bytes_launch / (k_ms / k_n * 1e-3) / 1e9 if k_n else None
        total_kernel_ms = sum(v[0] for v in kernels.values())
        x_mb = w.n * w.ld * (2 if bf16 else 4) // 2 ** 20
        # The gathered bytes are served by L2 whenever one chunk's slice of x fits it (ncu: L1 hit rate ~0 at full
        # size), so the roof that binds the gather is then the L2-to-crossbar rate at the clock the run held; the
        # contract's count against the HBM copy peak stays beside it.
        l2_clock_mhz = clocks["sm_mhz"] or clocks["sm_max_mhz"] or 1965.0
        l2_peak = L2_PEAK_BYTES_PER_CLK * l2_clock_mhz / 1e3
        slice_bytes = w.n * min(cw, w.f) * (2 if bf16 else 4)
        hbm_counted = {"achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak if achieved else None,
                       "peak_source": peak_src, "frac_of_8TBs_nominal": achieved / 8000.0 if achieved else None,
                       "note": "algorithmic bytes charge every gathered feature, most of which L2 serves: a fraction "
                               "above 1 means the kernel runs above the HBM roof on cache hits"}
        l2_roofline = {"what": "algorithmic bytes / kernel time against the L2-to-crossbar peak ncu derives "
                               "(11,776 B/clk) at the median SM clock sampled during the timed region",
                       "achieved": achieved, "peak": l2_peak, "clock_mhz": l2_clock_mhz, "unit": "GB/s",
                       "frac": achieved / l2_peak if achieved else None,
                       "measured_random_row_read_GBs": l2_measured,
                       "frac_of_measured": achieved / l2_measured if achieved and l2_measured else None}
        l2_bound = slice_bytes <= l2_bytes
        roofline = {"bound": "l2" if l2_bound else "hbm", "kernel": name, "achieved": achieved,
                    "peak": l2_peak if l2_bound else peak, "unit": "GB/s",
                    "frac": (achieved / (l2_peak if l2_bound else peak)) if achieved else None,
                    "peak_source": ("ncu-derived L2-to-crossbar peak x sampled SM clock; one chunk's slice of x "
                                    "(%d MB) is L2-resident, HBM moves only the traffic below" % (slice_bytes >> 20))
                    if l2_bound else peak_src,
                    "bytes_per_launch": bytes_launch, "kernel_ms": k_ms / k_n if k_n else None,
                    "traffic": ncu_traffic(args.workload), "hbm_counted": hbm_counted}
        result = {
            "metric": METRIC, "value": total_units * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": warmup, "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "strong" if by_columns else "weak", "vs_baseline": None,
            "dtype": "bf16" if bf16 else "f32", "data": "synthetic",
            "config": {"workload": args.workload, "description": WORKLOADS[args.workload][2],
                       "arithmetic": "fp32 multiply-add (bf16 features are widened exactly)" if bf16 else "fp32",
                       "step": "gnnfd_build_csr + gnnfd_aggregate_" + w.model, "n": w.n, "input_edges": e, "nnz": nnz,
                       "f": w.f, "feature_dtype": w.dtype, "chunk_width": cw,
                       "parallelism": ("feature-chunk slabs: one graph, CSR built on every GPU, each GPU aggregates "
                                       "its chunk-aligned columns%s" % (", slabs all-gathered over NCCL" if args.gather
                                                                        else ", no exchange")) if by_columns
                       else ("independent graphs per GPU" if world > 1 else "1 GPU"),
                       "ranks": per_rank,
                       "l2": "inputs vs the 126 MB L2: x %d MB, col_idx+weights %d MB per sweep (no flush between steps)"
                             % (x_mb, nnz * 8 // 2 ** 20)},
            "roofline": roofline,
            "l2_roofline": l2_roofline,
            "e2e": {"value": total_units * args.steps / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": launches,
            "clocks": clocks,
            # device memory of one step (the paper's second axis, Fig. 6): the build scratch may be freed after the build
            "device_memory_bytes": {
                "edge_list": d_src.numel() * d_src.element_size() * 2,
                "features": d_x.numel() * d_x.element_size(), "output": out.numel() * 4,
                "csr_persistent": pb, "build_scratch": sb,
                "aggregation_scratch": state["agg_scratch"].numel() if state["agg_scratch"] is not None else 0,
                "total_during_build": d_src.numel() * d_src.element_size() * 2 + d_x.numel() * d_x.element_size()
                                      + out.numel() * 4 + pb + sb,
                "total_after_build": d_x.numel() * d_x.element_size() + out.numel() * 4 + pb
                                     + (state["agg_scratch"].numel() if state["agg_scratch"] is not None else 0)},
            "kernels": {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps,
                            "share": v[0] / total_kernel_ms if total_kernel_ms else None}
                        for k, v in sorted(kernels.items(), key=lambda kv: -kv[1][0])},
            "aggregate_only": {str(k): {"ms": v, "cold_l2_ms": agg_cold_ms[k],
                                        "edge_features_per_s": units_per_step / (v * 1e-3),
                                        "roofline_GBs": bytes_launch / (v * 1e-3) / 1e9}
                               for k, v in agg_ms.items()},
        }
        if softmax_ms is not None:
            # HBM bytes the softmax has to move: the column indices once and alpha once (the score gathers are cache hits)
            sm_bytes = 4 * (w.n + 1) + 4 * nnz + 4 * nnz * w.heads
            result["edge_softmax_only"] = {"ms": softmax_ms, "alpha_GBs_written": nnz * w.heads * 4 / (softmax_ms * 1e-3) / 1e9,
                                           "hbm_bytes": sm_bytes, "hbm_GBs": sm_bytes / (softmax_ms * 1e-3) / 1e9,
                                           "frac_of_hbm_peak": sm_bytes / (softmax_ms * 1e-3) / 1e9 / peak}
        if light is not None:
            result["one_shot"] = light
        if layer_ms:
            result["layer_ms"] = dict(layer_ms, f_out=args.combine_out,
                                      what="gnnfd_layer_*: transform to f_out columns + aggregation of them, built CSR")
        if combine_ms is not None:
            cb_bytes = 4 * (w.n * w.f + args.combine_out * w.f + w.n * args.combine_out)
            result["combine_fp32_faithful"] = {
                "kernel": "combine_fp32_3xtf32", "ms": combine_fp32_ms, "achieved_GBs": cb_bytes / (combine_fp32_ms * 1e-3) / 1e9,
                "frac_of_hbm_peak": cb_bytes / (combine_fp32_ms * 1e-3) / 1e9 / peak,
                "slowdown_vs_tf32": combine_fp32_ms / combine_ms}
            result["combine_only"] = {
                "kernel": "combine_tf32", "shape": "[%d, %d] x [%d, %d]" % (w.n, w.f, w.f, args.combine_out),
                "ms": combine_ms, "bound": "hbm", "hbm_bytes": cb_bytes,
                "achieved_GBs": cb_bytes / (combine_ms * 1e-3) / 1e9,
                "frac_of_hbm_peak": cb_bytes / (combine_ms * 1e-3) / 1e9 / peak,
                "tf32_TFLOPs": 2.0 * w.n * w.f * args.combine_out / (combine_ms * 1e-3) / 1e12}
        if world == 1 and not args.no_cpu_baseline:
            import oracle as orc
            threads = orc.max_threads()
            rows, s_src, s_dst = oracle_sample(w, args.cpu_rows or 98304)
            t0 = time.perf_counter()
            units = oracle_step(w, rows, s_src, s_dst, threads)
            dt = time.perf_counter() - t0
            result["cpu_baseline"] = {"value": units / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
                                      "seconds": dt, "sample": sample_text(w, len(rows)),
                                      "single_core": oracle_single_core(w, max(len(rows) // 8, 64), [cw])}
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
    ap.add_argument("--chunk-width", type=int, default=0, help="0 = the workload's default")
    ap.add_argument("--sweep", type=int, nargs="*", default=[], help="extra chunk widths to time (aggregation only)")
    ap.add_argument("--combine-out", type=int, default=64,
                    help="output width of the dense transform timed beside the step (0: skip; fp32 workloads only)")
    ap.add_argument("--shard", choices=["graphs", "columns"], default="graphs",
                    help="graphs: every rank its own graph (weak scaling); columns: one graph, each rank aggregates the "
                         "decomposition layers of its column slab (strong scaling)")
    ap.add_argument("--gather", action="store_true",
                    help="with --shard columns: all-gather the slabs (NCCL) so that every rank ends with the full result")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--cpu-rows", type=int, default=0,
                    help="destination rows in the CPU-oracle sample (0: 16384 per step of --impl reference, "
                         "98304 for the one cpu_baseline step of the CUDA arm)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--core-only", action="store_true",
                    help="leave out the side measurements (dense transform, layers, one-shot path): for profiler captures")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
