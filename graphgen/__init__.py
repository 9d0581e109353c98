"""Seeded synthetic inputs: graphs in COO form, feature matrices, attention vectors.

This module serves both the CPU oracle's tests and the GPU tests with the same
data.  It holds no aggregation arithmetic: only random structure and values.
The C source (``graphgen.c``) is compiled with gcc on first use.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "graphgen.c")
_LIB = os.path.join(_HERE, "libgraphgen.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile libgraphgen.so beside the source (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, u64, dbl, i32 = ctypes.c_int64, ctypes.c_uint64, ctypes.c_double, ctypes.c_int
        vp = ctypes.c_void_p
        lib.gg_mix64.restype = u64
        lib.gg_mix64.argtypes = [u64, u64, u64]
        lib.gg_powerlaw_graph.restype = i64
        lib.gg_powerlaw_graph.argtypes = [i64, i64, dbl, i64, u64, i32, vp, vp, i64]
        lib.gg_rmat_graph.restype = i32
        lib.gg_rmat_graph.argtypes = [i32, i64, dbl, dbl, dbl, u64, i32, vp, vp]
        lib.gg_uniform_graph.restype = i32
        lib.gg_uniform_graph.argtypes = [i64, i64, u64, vp, vp]
        lib.gg_fill_f32.restype = i32
        lib.gg_fill_f32.argtypes = [vp, i64, i64, i64, i32, dbl, dbl, u64, u64, ctypes.c_float]
        lib.gg_f32_to_bf16.restype = None
        lib.gg_f32_to_bf16.argtypes = [vp, vp, i64]
        lib.gg_bf16_to_f32.restype = None
        lib.gg_bf16_to_f32.argtypes = [vp, vp, i64]
        lib.gg_num_threads.restype = i32
        _lib = lib
    return _lib


def _p(a: np.ndarray) -> int:
    return a.ctypes.data


def mix64(seed: int, stream: int, index: int) -> int:
    return int(_load().gg_mix64(seed, stream, index))


def powerlaw_graph(n: int, target_edges: int, alpha: float = 2.1, dmax: int | None = None,
                   seed: int = 0, relabel: bool = True):
    """Directed power-law graph; returns (src, dst) int32 arrays in shuffled COO order."""
    lib = _load()
    dmax = n - 1 if dmax is None else dmax
    cap = int(target_edges * 1.01) + 16
    src = np.empty(cap, np.int32)
    dst = np.empty(cap, np.int32)
    e = lib.gg_powerlaw_graph(n, target_edges, alpha, dmax, seed, int(relabel), _p(src), _p(dst), cap)
    if e < 0:
        raise RuntimeError("gg_powerlaw_graph failed: %d" % e)
    return src[:e].copy() if e < cap // 2 else src[:e], dst[:e].copy() if e < cap // 2 else dst[:e]


def rmat_graph(scale: int, e: int, a: float = 0.57, b: float = 0.19, c: float = 0.19,
               seed: int = 0, relabel: bool = True):
    lib = _load()
    src = np.empty(e, np.int32)
    dst = np.empty(e, np.int32)
    rc = lib.gg_rmat_graph(scale, e, a, b, c, seed, int(relabel), _p(src), _p(dst))
    if rc:
        raise RuntimeError("gg_rmat_graph failed: %d" % rc)
    return src, dst


def uniform_graph(n: int, e: int, seed: int = 0):
    """Uniformly random directed multigraph (duplicates and self-loops occur)."""
    lib = _load()
    src = np.empty(e, np.int32)
    dst = np.empty(e, np.int32)
    rc = lib.gg_uniform_graph(n, e, seed, _p(src), _p(dst))
    if rc:
        raise RuntimeError("gg_uniform_graph failed: %d" % rc)
    return src, dst


def features_f32(rows: int, cols: int, ld: int | None = None, dist: str = "uniform",
                 p0: float = -1.0, p1: float = 1.0, seed: int = 0, stream: int = 4,
                 pad: float = 0.0, out: np.ndarray | None = None) -> np.ndarray:
    """[rows, ld] fp32 array; columns >= cols hold ``pad``.  dist: 'uniform' [p0,p1) or
    'normal' (mean p0, std p1)."""
    lib = _load()
    ld = cols if ld is None else ld
    if out is None:
        out = np.empty((rows, ld), np.float32)
    assert out.dtype == np.float32 and out.shape == (rows, ld) and out.flags.c_contiguous
    rc = lib.gg_fill_f32(_p(out), rows, cols, ld, {"uniform": 0, "normal": 1}[dist], p0, p1,
                         seed, stream, pad)
    if rc:
        raise RuntimeError("gg_fill_f32 failed: %d" % rc)
    return out


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even."""
    x = np.ascontiguousarray(x, np.float32)
    out = np.empty(x.shape, np.uint16)
    _load().gg_f32_to_bf16(_p(x), _p(out), x.size)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, np.uint16)
    out = np.empty(b.shape, np.float32)
    _load().gg_bf16_to_f32(_p(b), _p(out), b.size)
    return out


def num_threads() -> int:
    return int(_load().gg_num_threads())


# ---------------------------------------------------------------- workloads

FLAG_SELF_LOOPS, FLAG_DEDUP, FLAG_SYMMETRIZE = 1, 2, 4


@dataclass
class Workload:
    """One seeded synthetic workload: what the library is given, nothing derived."""
    name: str
    model: str                      # 'gcn' | 'sage' | 'gat'
    n: int
    src: np.ndarray                 # int32 [E]
    dst: np.ndarray                 # int32 [E]
    flags: int                      # CSR build flags
    f: int                          # feature width (heads*dim for gat)
    ld: int                         # leading dimension of x
    x: np.ndarray                   # fp32 [n, ld] or uint16 bf16 bits [n, ld]
    dtype: str                      # 'f32' | 'bf16'
    chunk_widths: tuple = ()
    heads: int = 1
    dim: int = 0
    a_src: np.ndarray | None = None
    a_dst: np.ndarray | None = None
    negative_slope: float = 0.2
    extra: dict = field(default_factory=dict)


def config1(seed: int = 0) -> Workload:
    """GCN, 4,096 vertices, ~40k power-law edges + self-loops, F=16 fp32 U(-1,1)."""
    n, f = 4096, 16
    src, dst = powerlaw_graph(n, 40_000, 2.1, None, seed)
    x = features_f32(n, f, dist="uniform", p0=-1.0, p1=1.0, seed=seed)
    return Workload("config1", "gcn", n, src, dst, FLAG_SELF_LOOPS, f, f, x, "f32", (4, 8, 16))


def config2(seed: int = 0, n: int = 100_000, avg_deg: int = 20, f: int = 128) -> Workload:
    """GraphSAGE mean, 100,000 vertices, avg degree 20 power law, F=128 fp32 N(0,1)."""
    src, dst = powerlaw_graph(n, n * avg_deg, 2.1, None, seed)
    x = features_f32(n, f, dist="normal", p0=0.0, p1=1.0, seed=seed)
    return Workload("config2", "sage", n, src, dst, 0, f, f, x, "f32", (8, 16, 32, 64, 128))


def config3(seed: int = 0, n: int = 200_000, avg_deg: int = 15, heads: int = 8, dim: int = 8) -> Workload:
    """GAT, 200,000 vertices, avg degree 15 power law + self-loops, 8 heads x 8 dims fp32 N(0,1),
    a_src/a_dst N(0, std 0.1), LeakyReLU slope 0.2."""
    src, dst = powerlaw_graph(n, n * avg_deg, 2.1, None, seed)
    f = heads * dim
    x = features_f32(n, f, dist="normal", p0=0.0, p1=1.0, seed=seed)
    a_src = features_f32(heads, dim, dist="normal", p0=0.0, p1=0.1, seed=seed, stream=5)
    a_dst = features_f32(heads, dim, dist="normal", p0=0.0, p1=0.1, seed=seed, stream=6)
    return Workload("config3", "gat", n, src, dst, FLAG_SELF_LOOPS, f, f, x, "f32", (8, 64),
                    heads=heads, dim=dim, a_src=a_src, a_dst=a_dst, negative_slope=0.2)


def config4(seed: int = 0, n: int = 232_965, edges: int = 114_615_892, dmax: int = 20_000,
            f: int = 602, ld: int = 608) -> Workload:
    """GCN input layer: 232,965 vertices, ~114M power-law edges (max degree 20k) + self-loops,
    F=602 fp32 U(0,1) with rows padded to 608 columns."""
    src, dst = powerlaw_graph(n, edges, 2.1, dmax, seed)
    x = features_f32(n, f, ld=ld, dist="uniform", p0=0.0, p1=1.0, seed=seed)
    return Workload("config4", "gcn", n, src, dst, FLAG_SELF_LOOPS, f, ld, x, "f32",
                    (32, 64, 128, 602))


def config5(seed: int = 0, scale: int = 21, edges: int = 60_000_000, f: int = 256,
            relabel: bool = True) -> Workload:
    """GCN on RMAT (a,b,c,d)=(0.57,0.19,0.19,0.05), symmetrised + deduplicated + self-loops,
    bf16 features U(-1,1); f = 256 (input layer) or a hidden width 8/16/32/64."""
    n = 1 << scale
    src, dst = rmat_graph(scale, edges, 0.57, 0.19, 0.19, seed, relabel)
    x = to_bf16_bits(features_f32(n, f, dist="uniform", p0=-1.0, p1=1.0, seed=seed))
    widths = (32, 64, 128, 256) if f == 256 else tuple(sorted({8, f}))
    return Workload("config5_f%d" % f, "gcn", n, src, dst,
                    FLAG_SELF_LOOPS | FLAG_DEDUP | FLAG_SYMMETRIZE, f, f, x, "bf16", widths)


def scaled(config: str, factor: float, seed: int = 0) -> Workload:
    """A smaller instance of config 2/3/4/5 with the same recipe (vertex and edge counts scaled),
    for cases the CPU oracle finishes in seconds."""
    if config == "config2":
        return config2(seed, n=max(64, int(100_000 * factor)))
    if config == "config3":
        return config3(seed, n=max(64, int(200_000 * factor)))
    if config == "config4":
        n = max(256, int(232_965 * factor))
        e = max(n, int(114_615_892 * factor * factor))
        return config4(seed, n=n, edges=e, dmax=min(20_000, n - 1))
    if config.startswith("config5"):
        f = int(config.split("_f")[1]) if "_f" in config else 256
        scale = max(8, 21 + int(round(np.log2(factor))))
        return config5(seed, scale=scale, edges=max(1024, int(60_000_000 * factor)), f=f)
    raise ValueError(config)


def reddit_hidden(model: str = "gcn", hidden: int = 32, seed: int = 0, dim: int = 8, factor: float = 1.0) -> Workload:
    """Hidden-layer aggregation on the Reddit-shaped graph of config 4 (the paper's Hid = 8 / 16 / 32 / 64
    settings of Section III): same graph and self-loops, features [n, hidden] fp32 N(0,1).  For GAT the
    hidden width is split into heads of ``dim`` columns (one head when hidden <= dim).  ``factor`` < 1
    scales the vertex count by factor and the edge count by factor squared, as ``scaled`` does."""
    n = max(256, int(232_965 * factor))
    src, dst = powerlaw_graph(n, max(n, int(114_615_892 * factor * factor)), 2.1, min(20_000, n - 1), seed)
    x = features_f32(n, hidden, dist="normal", p0=0.0, p1=1.0, seed=seed)
    if model == "gat":
        d = min(dim, hidden)
        heads = hidden // d
        a_src = features_f32(heads, d, dist="normal", p0=0.0, p1=0.1, seed=seed, stream=5)
        a_dst = features_f32(heads, d, dist="normal", p0=0.0, p1=0.1, seed=seed, stream=6)
        return Workload("reddit_gat_hid%d" % hidden, "gat", n, src, dst, FLAG_SELF_LOOPS, hidden, hidden, x, "f32",
                        tuple(sorted({d, hidden})), heads=heads, dim=d, a_src=a_src, a_dst=a_dst, negative_slope=0.2)
    return Workload("reddit_%s_hid%d" % (model, hidden), model, n, src, dst, FLAG_SELF_LOOPS, hidden, hidden, x, "f32",
                    tuple(sorted({min(hidden, 8), hidden})))
