"""ctypes binding of the CPU oracle (``oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, the smoke check and the
benchmark's CPU-baseline leg.  The CUDA package never imports this module and
this module never imports the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# The two overrides exist for the mutation test, which builds deliberately wrong copies of the source
# elsewhere and checks that the pins reject them.
_SRC = os.environ.get("GNNFD_ORACLE_SOURCE", os.path.join(_HERE, "oracle.cpp"))
_LIB = os.environ.get("GNNFD_ORACLE_LIB", os.path.join(_HERE, "liboracle.so"))
_lib = None

ADD_SELF_LOOPS, DEDUP, SYMMETRIZE = 1, 2, 4
ERR_INVALID, ERR_BAD_INDEX, ERR_TOO_LARGE = -1, -2, -3


def build(force: bool = False) -> str:
    """Compile liboracle.so beside the source (g++, C++17, OpenMP for the optional row-parallel loop)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["g++", "-std=c++17", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, i32, u32, dbl, vp = ctypes.c_int64, ctypes.c_int32, ctypes.c_uint32, ctypes.c_double, ctypes.c_void_p
        lib.orc_csr_capacity.restype = i64
        lib.orc_csr_capacity.argtypes = [i64, i64, u32]
        lib.orc_build_csr.restype = i64
        lib.orc_build_csr.argtypes = [i64, i64, vp, vp, i32, u32, vp, vp, vp]
        lib.orc_degree_norm.restype = None
        lib.orc_degree_norm.argtypes = [i64, vp, vp, vp, vp]
        lib.orc_aggregate.restype = i32
        lib.orc_aggregate.argtypes = [i32, i64, vp, vp, vp, i64, i32, i32, i32, vp, i64, vp, vp, i32]
        lib.orc_gat_scores.restype = i32
        lib.orc_gat_scores.argtypes = [i64, vp, i64, i32, vp, vp, i32, i32, vp, vp]
        lib.orc_edge_softmax.restype = i32
        lib.orc_edge_softmax.argtypes = [i64, vp, vp, vp, vp, i32, dbl, vp]
        lib.orc_edge_softmax_f32.restype = i32
        lib.orc_edge_softmax_f32.argtypes = [i64, vp, vp, vp, vp, i32, dbl, vp]
        lib.orc_aggregate_gat.restype = i32
        lib.orc_aggregate_gat.argtypes = [i64, vp, vp, vp, i64, i32, vp, vp, i32, i32, dbl, i32, vp, i64,
                                          vp, vp, i32]
        lib.orc_max_threads.restype = i32
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data


def _xinfo(x: np.ndarray):
    assert x.ndim == 2 and x.flags.c_contiguous
    if x.dtype == np.float32:
        return 0
    if x.dtype == np.uint16:        # bf16 bit patterns
        return 1
    raise TypeError("features must be float32 or uint16 (bf16 bits)")


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__("oracle error %d" % code)
        self.code = code


def build_csr(n: int, src: np.ndarray, dst: np.ndarray, flags: int = 0):
    """-> (row_ptr int32[n+1], col_idx int32[nnz], perm int32[nnz])."""
    lib = _load()
    assert src.dtype == dst.dtype and src.dtype in (np.int32, np.int64)
    src = np.ascontiguousarray(src)
    dst = np.ascontiguousarray(dst)
    e = len(src)
    cap = lib.orc_csr_capacity(n, e, flags)
    row_ptr = np.zeros(n + 1, np.int32)
    col = np.empty(max(cap, 1), np.int32)
    perm = np.empty(max(cap, 1), np.int32)
    nnz = lib.orc_build_csr(n, e, _p(src), _p(dst), 0 if src.dtype == np.int32 else 1, flags,
                            _p(row_ptr), _p(col), _p(perm))
    if nnz < 0:
        raise OracleError(nnz)
    return row_ptr, col[:nnz].copy(), perm[:nnz].copy()


def degree_norm(row_ptr: np.ndarray):
    """-> (deg int32[n], dinv float64[n], rdeg float64[n])."""
    n = len(row_ptr) - 1
    deg = np.empty(n, np.int32)
    dinv = np.empty(n, np.float64)
    rdeg = np.empty(n, np.float64)
    _load().orc_degree_norm(n, _p(row_ptr), _p(deg), _p(dinv), _p(rdeg))
    return deg, dinv, rdeg


def aggregate(model: str, row_ptr, col_idx, x, f: int, chunk_width: int | None = None, rows=None,
              threads: int = 1):
    """GCN / SAGE aggregation -> (out float64[R, f], abs float64[R, f])."""
    n = len(row_ptr) - 1
    xdt = _xinfo(x)
    chunk_width = f if chunk_width is None else chunk_width
    if rows is not None:
        rows = np.ascontiguousarray(rows, np.int64)
    r = n if rows is None else len(rows)
    out = np.zeros((r, f), np.float64)
    ab = np.zeros((r, f), np.float64)
    rc = _load().orc_aggregate({"gcn": 0, "sage": 1}[model], n, _p(row_ptr), _p(col_idx), _p(x),
                               x.shape[1], xdt, f, chunk_width, _p(rows), r, _p(out), _p(ab), threads)
    if rc:
        raise OracleError(rc)
    return out, ab


def gat_scores(z, a_src, a_dst, heads: int, dim: int):
    n = z.shape[0]
    a_src = np.ascontiguousarray(a_src, np.float32)
    a_dst = np.ascontiguousarray(a_dst, np.float32)
    s_src = np.empty((n, heads), np.float64)
    s_dst = np.empty((n, heads), np.float64)
    rc = _load().orc_gat_scores(n, _p(z), z.shape[1], _xinfo(z), _p(a_src), _p(a_dst), heads, dim,
                                _p(s_src), _p(s_dst))
    if rc:
        raise OracleError(rc)
    return s_src, s_dst


def edge_softmax(row_ptr, col_idx, s_src, s_dst, slope: float = 0.2):
    """alpha float64[nnz, heads] in CSR order; scores float64 or float32 [n, heads]."""
    n = len(row_ptr) - 1
    heads = s_src.shape[1]
    alpha = np.empty((len(col_idx), heads), np.float64)
    lib = _load()
    if s_src.dtype == np.float32:
        fn = lib.orc_edge_softmax_f32
        s_src = np.ascontiguousarray(s_src, np.float32)
        s_dst = np.ascontiguousarray(s_dst, np.float32)
    else:
        fn = lib.orc_edge_softmax
        s_src = np.ascontiguousarray(s_src, np.float64)
        s_dst = np.ascontiguousarray(s_dst, np.float64)
    rc = fn(n, _p(row_ptr), _p(col_idx), _p(s_src), _p(s_dst), heads, slope, _p(alpha))
    if rc:
        raise OracleError(rc)
    return alpha


def aggregate_gat(row_ptr, col_idx, z, a_src, a_dst, heads: int, dim: int, slope: float = 0.2,
                  chunk_width: int | None = None, rows=None, threads: int = 1):
    """GAT aggregation -> (out float64[R, heads*dim], abs float64[R, heads*dim])."""
    n = len(row_ptr) - 1
    f = heads * dim
    chunk_width = f if chunk_width is None else chunk_width
    a_src = np.ascontiguousarray(a_src, np.float32)
    a_dst = np.ascontiguousarray(a_dst, np.float32)
    if rows is not None:
        rows = np.ascontiguousarray(rows, np.int64)
    r = n if rows is None else len(rows)
    out = np.zeros((r, f), np.float64)
    ab = np.zeros((r, f), np.float64)
    rc = _load().orc_aggregate_gat(n, _p(row_ptr), _p(col_idx), _p(z), z.shape[1], _xinfo(z), _p(a_src),
                                   _p(a_dst), heads, dim, slope, chunk_width, _p(rows), r, _p(out),
                                   _p(ab), threads)
    if rc:
        raise OracleError(rc)
    return out, ab


def combine(x: np.ndarray, w_t: np.ndarray, tf32: bool = False):
    """Combination ahead of aggregation (Section III): z = x @ w_t.T in float64, and sum_k |x w| beside it.
    With ``tf32`` both operands are first cut to the 10 explicit mantissa bits a tf32 operand keeps (the
    low 13 bits of the fp32 pattern are dropped), which is what a tf32 tensor-core product computes
    exactly apart from the order of its fp32 additions."""
    x = np.ascontiguousarray(x, np.float32)
    w_t = np.ascontiguousarray(w_t, np.float32)
    if tf32:
        x = (x.view(np.uint32) & np.uint32(0xFFFFE000)).view(np.float32)
        w_t = (w_t.view(np.uint32) & np.uint32(0xFFFFE000)).view(np.float32)
    x64, w64 = x.astype(np.float64), w_t.astype(np.float64)
    return x64 @ w64.T, np.abs(x64) @ np.abs(w64).T


def max_threads() -> int:
    return int(_load().orc_max_threads())
