"""Thin ctypes binding of libgnnfd.so: argument marshalling only.

PyTorch supplies device memory and streams; every step of the aggregation runs inside the library's
CUDA kernels.  There is no fallback: if the shared library is missing or fails to load, importing
the entry points raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

F32, BF16 = 0, 1
I32, I64 = 0, 1
CSR_ADD_SELF_LOOPS, CSR_DEDUP, CSR_SYMMETRIZE, CSR_INPUT_ORDER = 1, 2, 4, 8
OK, INVALID_ARG, BAD_INDEX, TOO_LARGE, WORKSPACE_TOO_SMALL, UNSUPPORTED, CUDA_ERROR = 0, -1, -2, -3, -4, -5, -6
STATIC_SCRATCH_EXCEEDED = -7
COMBINE_TF32, COMBINE_FP32 = 0, 1
STATIC_SCRATCH_BYTES = 32 << 20
HUB_DEGREE, HUB_SEGMENT, HUB_RANGE_ROWS = 2048, 1024, 524288

_lib = None


class GnnfdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().gnnfd_status_string(status).decode()
        if status == CUDA_ERROR:
            msg += " (cudaError %d)" % lib().gnnfd_last_cuda_error()
        super().__init__("%s: %s" % (where, msg))


def lib() -> ctypes.CDLL:
    """Loads libgnnfd.so from the package directory (never builds, never falls back)."""
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            raise ImportError("libgnnfd.so is not built: run paper_2104_03058_b200.build.build_library()")
        L = ctypes.CDLL(path)
        i64, i32, u32, vp, sz, fl = (ctypes.c_int64, ctypes.c_int32, ctypes.c_uint32, ctypes.c_void_p,
                                     ctypes.c_size_t, ctypes.c_float)
        pp = ctypes.POINTER
        L.gnnfd_csr_workspace_bytes.argtypes = [i64, i64, u32, pp(sz), pp(sz)]
        L.gnnfd_build_csr.argtypes = [i64, i64, vp, vp, i32, u32, vp, sz, vp, sz, vp, pp(vp)]
        L.gnnfd_csr_info.argtypes = [vp, pp(i64), pp(i64), pp(vp), pp(vp), pp(vp), pp(vp), pp(vp), pp(vp), pp(i32)]
        L.gnnfd_csr_schedule.argtypes = [vp, pp(i64 * 5), pp(vp), pp(i64), pp(vp), pp(vp), pp(vp), pp(vp), pp(vp)]
        L.gnnfd_csr_destroy.argtypes = [vp]
        L.gnnfd_csr_destroy.restype = None
        L.gnnfd_aggregate_workspace_bytes.argtypes = [vp, i32, pp(sz)]
        agg = [vp, vp, i64, i32, vp, i64, i32, i32, i32, vp, sz, vp]
        L.gnnfd_aggregate_gcn.argtypes = agg
        L.gnnfd_aggregate_sage.argtypes = agg
        L.gnnfd_aggregate_gcn_static.argtypes = [vp, vp, i64, i32, vp, i64, i32, i32, i32, vp]
        L.gnnfd_oneshot_workspace_bytes.argtypes = [i64, i64, u32, i32, pp(sz)]
        one = [i64, i64, vp, vp, i32, u32, vp, i64, i32, vp, i64, i32, i32, i32, vp, sz, vp]
        L.gnnfd_oneshot_gcn.argtypes = one
        L.gnnfd_oneshot_sage.argtypes = one
        L.gnnfd_oneshot_gat_workspace_bytes.argtypes = [i64, i64, u32, i32, i32, pp(sz)]
        L.gnnfd_oneshot_gat.argtypes = [i64, i64, vp, vp, i32, u32, vp, i64, i32, vp, vp, i32, i32, fl, vp, i64, i32, i32,
                                        vp, sz, vp]
        L.gnnfd_default_chunk_candidates.argtypes = [i32, i32, pp(i32), ctypes.c_int]
        L.gnnfd_tune_chunk_width.argtypes = [vp, ctypes.c_int, vp, i64, i32, vp, i64, i32, i32, pp(i32), ctypes.c_int,
                                             vp, sz, vp, pp(i32), pp(fl)]
        L.gnnfd_gat_scores.argtypes = [i64, vp, i64, i32, vp, vp, i32, i32, vp, vp, vp]
        L.gnnfd_gat_workspace_bytes.argtypes = [vp, i32, i32, pp(sz)]
        L.gnnfd_aggregate_gat.argtypes = [vp, vp, i64, i32, vp, vp, i32, i32, fl, vp, i64, i32, i32, vp, sz, vp]
        L.gnnfd_edge_softmax_workspace_bytes.argtypes = [vp, i32, pp(sz)]
        L.gnnfd_edge_softmax.argtypes = [vp, vp, vp, i32, fl, vp, vp, sz, vp]
        L.gnnfd_combine.argtypes = [i64, vp, i64, i32, i32, vp, i64, i32, vp, i64, i32, vp, vp]
        L.gnnfd_combine_ex.argtypes = [i64, vp, i64, i32, i32, vp, i64, i32, vp, i64, i32, ctypes.c_int, vp, vp, i32, i32,
                                       vp, vp, vp, vp]
        L.gnnfd_layer_workspace_bytes.argtypes = [vp, ctypes.c_int, i32, i32, i32, i32, pp(sz)]
        layer = [vp, vp, i64, i32, i32, vp, i64, i32, ctypes.c_int, vp, i64, i32, i32, vp, sz, vp, vp]
        L.gnnfd_layer_gcn.argtypes = layer
        L.gnnfd_layer_sage.argtypes = layer
        L.gnnfd_layer_gat.argtypes = [vp, vp, i64, i32, i32, vp, i64, i32, i32, vp, vp, fl, ctypes.c_int, vp, i64, i32, i32,
                                      vp, sz, vp, vp]
        L.gnnfd_debug_combine_fault.argtypes = [i64, i32]
        L.gnnfd_status_string.argtypes = [ctypes.c_int]
        L.gnnfd_status_string.restype = ctypes.c_char_p
        L.gnnfd_last_cuda_error.restype = ctypes.c_int
        L.gnnfd_launch_count.restype = i64
        L.gnnfd_kernel_timing_enable.argtypes = [ctypes.c_int]
        L.gnnfd_kernel_timing_read.argtypes = [pp(ctypes.c_char_p), pp(ctypes.c_double), pp(i64), ctypes.c_int]
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != OK:
        raise GnnfdError(status, where)


def _stream_ptr(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("features must be float32 or bfloat16, got %s" % t.dtype)


def _matrix(t: torch.Tensor, cols: int, name: str):
    """(pointer, leading dimension) of a row-major device matrix with at least `cols` columns."""
    if not t.is_cuda or t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1) or t.shape[1] < cols:
        raise ValueError("%s must be a 2-D CUDA tensor with unit column stride and >= %d columns" % (name, cols))
    return ctypes.c_void_p(t.data_ptr()), t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def _alloc_bytes(nbytes: int, device, stream=None) -> torch.Tensor:
    """Scratch of at least `nbytes` (torch's caching allocator returns 512-byte aligned blocks).  The
    block is taken under the stream the work will run on, so that the allocator does not hand it to
    another stream's tensor while the kernels that use it are still queued."""
    if stream is None:
        return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    with torch.cuda.stream(stream):
        return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def _same_device(csr_device, **tensors):
    """Every operand must live on the device the CSR was built on (the library never migrates data)."""
    for name, t in tensors.items():
        if t is not None and torch.device(t.device) != torch.device(csr_device):
            raise ValueError("%s is on %s but the CSR is on %s" % (name, t.device, csr_device))


def _need_rows(t, rows: int, name: str):
    if t.shape[0] < rows:
        raise ValueError("%s has %d rows, the graph needs %d" % (name, t.shape[0], rows))


def _extent(t):
    """[first byte, one past the last byte) of the storage a strided 2-D / 1-D tensor touches."""
    if t.numel() == 0:
        return (t.data_ptr(), t.data_ptr())
    last = sum((n - 1) * st for n, st in zip(t.shape, t.stride()))
    return (t.data_ptr(), t.data_ptr() + (last + 1) * t.element_size())


def _no_overlap(a, b, name_a: str, name_b: str):
    """The kernels read features through the read-only data path, so an output that overlaps an input
    is undefined behaviour the header forbids: refuse it here."""
    a0, a1 = _extent(a)
    b0, b1 = _extent(b)
    if not (a0 < b1 and b0 < a1):
        return
    # Two column ranges of one row-major buffer interleave row by row without sharing an element: same row
    # pitch, and the column intervals (taken modulo the pitch) apart.
    if a.dim() == 2 and b.dim() == 2 and a.shape[0] > 1 and b.shape[0] > 1:
        pitch_a, pitch_b = a.stride(0) * a.element_size(), b.stride(0) * b.element_size()
        if pitch_a == pitch_b and pitch_a > 0:
            first, second = (a, b) if a0 <= b0 else (b, a)
            off = (max(a0, b0) - min(a0, b0)) % pitch_a
            w_first = first.shape[1] * first.element_size()
            w_second = second.shape[1] * second.element_size()
            if w_first <= off and off + w_second <= pitch_a:
                return
    raise ValueError("%s and %s overlap in memory" % (name_a, name_b))


def _check_aggregate_operands(csr, x, out, f: int, name_x: str = "x"):
    """Shape, device and aliasing rules of the aggregation entry points, checked before any launch."""
    _same_device(csr.device, **{name_x: x, "out": out})
    _need_rows(x, csr.n, name_x)
    _need_rows(out, csr.n, "out")
    _no_overlap(x, out, name_x, "out")


class Csr:
    """Handle of a built CSR; keeps the persistent device buffer alive."""

    def __init__(self, handle, persistent: torch.Tensor, device):
        self._h = handle
        self._persistent = persistent
        self.device = device
        n, nnz, md = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int32()
        ptrs = [ctypes.c_void_p() for _ in range(6)]
        _check(lib().gnnfd_csr_info(self._h, ctypes.byref(n), ctypes.byref(nnz), *[ctypes.byref(p) for p in ptrs],
                                    ctypes.byref(md)), "gnnfd_csr_info")
        self.n, self.nnz, self.max_degree = n.value, nnz.value, md.value
        self._ptrs = dict(zip(("row_ptr", "col_idx", "perm", "dinv_sqrt", "rdeg", "edge_weight"),
                              [p.value for p in ptrs]))
        bins = (ctypes.c_int64 * 5)()
        nseg = ctypes.c_int64()
        sp = [ctypes.c_void_p() for _ in range(6)]
        _check(lib().gnnfd_csr_schedule(self._h, ctypes.byref(bins), ctypes.byref(sp[0]), ctypes.byref(nseg),
                                        ctypes.byref(sp[1]), ctypes.byref(sp[2]), ctypes.byref(sp[3]), ctypes.byref(sp[4]),
                                        ctypes.byref(sp[5])),
               "gnnfd_csr_schedule")
        self.bin_count = list(bins)
        self.n_segments = nseg.value
        self._ptrs.update(dict(zip(("row_order", "seg_row", "seg_begin", "seg_end", "seg_slot", "hub_seg_ptr"),
                                   [p.value for p in sp])))

    @property
    def handle(self):
        if self._h is None:
            raise RuntimeError("CSR handle was destroyed")
        return self._h

    def _view(self, name: str, count: int, dtype) -> torch.Tensor:
        """A tensor view (no copy) of one of the arrays inside the persistent buffer."""
        off = self._ptrs[name] - self._persistent.data_ptr()
        size = torch.empty(0, dtype=dtype).element_size()
        return self._persistent[off:off + count * size].view(dtype)

    row_ptr = property(lambda self: self._view("row_ptr", self.n + 1, torch.int32))
    col_idx = property(lambda self: self._view("col_idx", self.nnz, torch.int32))
    perm = property(lambda self: self._view("perm", self.nnz, torch.int32))
    dinv_sqrt = property(lambda self: self._view("dinv_sqrt", self.n, torch.float32))
    rdeg = property(lambda self: self._view("rdeg", self.n, torch.float32))
    edge_weight = property(lambda self: self._view("edge_weight", self.nnz, torch.float32))
    row_order = property(lambda self: self._view("row_order", self.n, torch.int32))
    seg_row = property(lambda self: self._view("seg_row", self.n_segments, torch.int32))
    seg_begin = property(lambda self: self._view("seg_begin", self.n_segments, torch.int32))
    seg_end = property(lambda self: self._view("seg_end", self.n_segments, torch.int32))
    seg_slot = property(lambda self: self._view("seg_slot", self.n_segments, torch.int32))
    hub_seg_ptr = property(lambda self: self._view("hub_seg_ptr", self.bin_count[4] + 1, torch.int32))

    def destroy(self):
        if self._h is not None:
            lib().gnnfd_csr_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def csr_workspace_bytes(n: int, e: int, flags: int):
    p, s = ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib().gnnfd_csr_workspace_bytes(n, e, flags, ctypes.byref(p), ctypes.byref(s)), "gnnfd_csr_workspace_bytes")
    return p.value, s.value


def build_csr(n: int, src: torch.Tensor, dst: torch.Tensor, flags: int = 0, stream=None,
              persistent: torch.Tensor | None = None, scratch: torch.Tensor | None = None) -> Csr:
    """gnnfd_build_csr on device tensors src/dst (int32 or int64, same dtype and length)."""
    if not (src.is_cuda and dst.is_cuda) or src.dtype != dst.dtype or src.shape != dst.shape or src.dim() != 1:
        raise ValueError("src and dst must be 1-D CUDA tensors of the same dtype and length")
    if src.dtype not in (torch.int32, torch.int64):
        raise TypeError("edge ids must be int32 or int64")
    src, dst = src.contiguous(), dst.contiguous()
    e = src.numel()
    pb, sb = csr_workspace_bytes(n, e, flags)
    if persistent is None:
        persistent = _alloc_bytes(pb, src.device)
    if scratch is None:
        scratch = _alloc_bytes(sb, src.device)
    handle = ctypes.c_void_p()
    st = lib().gnnfd_build_csr(n, e, ctypes.c_void_p(src.data_ptr()), ctypes.c_void_p(dst.data_ptr()),
                               I32 if src.dtype == torch.int32 else I64, flags,
                               ctypes.c_void_p(persistent.data_ptr()), persistent.numel(),
                               ctypes.c_void_p(scratch.data_ptr()), scratch.numel(), _stream_ptr(stream),
                               ctypes.byref(handle))
    _check(st, "gnnfd_build_csr")
    return Csr(handle, persistent, src.device)


def aggregate_workspace_bytes(csr: Csr, f: int) -> int:
    s = ctypes.c_size_t()
    _check(lib().gnnfd_aggregate_workspace_bytes(csr.handle, f, ctypes.byref(s)), "gnnfd_aggregate_workspace_bytes")
    return s.value


def _aggregate(fn, name, csr: Csr, x, f, chunk_width, out, out_dtype, scratch, stream):
    f = x.shape[1] if f is None else f
    chunk_width = f if chunk_width is None else chunk_width
    if out is None:
        out = torch.empty((csr.n, f), dtype=out_dtype or torch.float32, device=x.device)
    xp, ldx = _matrix(x, f, "x")
    op, ldo = _matrix(out, f, "out")
    _check_aggregate_operands(csr, x, out, f)
    need = aggregate_workspace_bytes(csr, f)
    if scratch is None and need:
        scratch = _alloc_bytes(need, x.device, stream)
    _same_device(csr.device, scratch=scratch)
    sp = ctypes.c_void_p(scratch.data_ptr()) if scratch is not None else None
    sn = scratch.numel() * scratch.element_size() if scratch is not None else 0
    _check(fn(csr.handle, xp, ldx, _dtype_code(x), op, ldo, _dtype_code(out), f, chunk_width, sp, sn,
              _stream_ptr(stream)), name)
    return out


def aggregate_gcn(csr: Csr, x: torch.Tensor, f: int | None = None, chunk_width: int | None = None,
                  out: torch.Tensor | None = None, out_dtype=None, scratch=None, stream=None) -> torch.Tensor:
    return _aggregate(lib().gnnfd_aggregate_gcn, "gnnfd_aggregate_gcn", csr, x, f, chunk_width, out, out_dtype,
                      scratch, stream)


def aggregate_sage(csr: Csr, x: torch.Tensor, f: int | None = None, chunk_width: int | None = None,
                   out: torch.Tensor | None = None, out_dtype=None, scratch=None, stream=None) -> torch.Tensor:
    return _aggregate(lib().gnnfd_aggregate_sage, "gnnfd_aggregate_sage", csr, x, f, chunk_width, out, out_dtype,
                      scratch, stream)


def oneshot_workspace_bytes(n: int, e: int, flags: int, f: int) -> int:
    s = ctypes.c_size_t()
    _check(lib().gnnfd_oneshot_workspace_bytes(n, e, flags, f, ctypes.byref(s)), "gnnfd_oneshot_workspace_bytes")
    return s.value


def oneshot(model: str, n: int, src: torch.Tensor, dst: torch.Tensor, x: torch.Tensor, flags: int = 0, f: int | None = None,
            chunk_width: int | None = None, out: torch.Tensor | None = None, out_dtype=None, scratch=None, stream=None):
    """gnnfd_oneshot_gcn / gnnfd_oneshot_sage: light build + aggregation of a COO edge list in one call."""
    if not (src.is_cuda and dst.is_cuda) or src.dtype != dst.dtype or src.shape != dst.shape or src.dim() != 1:
        raise ValueError("src and dst must be 1-D CUDA tensors of the same dtype and length")
    if src.dtype not in (torch.int32, torch.int64):
        raise TypeError("edge ids must be int32 or int64")
    src, dst = src.contiguous(), dst.contiguous()
    f = x.shape[1] if f is None else f
    chunk_width = f if chunk_width is None else chunk_width
    if out is None:
        out = torch.empty((n, f), dtype=out_dtype or torch.float32, device=x.device)
    xp, ldx = _matrix(x, f, "x")
    op, ldo = _matrix(out, f, "out")
    _same_device(src.device, dst=dst, x=x, out=out)
    _need_rows(x, n, "x")
    _need_rows(out, n, "out")
    _no_overlap(x, out, "x", "out")
    if scratch is None:
        scratch = _alloc_bytes(oneshot_workspace_bytes(n, src.numel(), flags, f), x.device, stream)
    _same_device(src.device, scratch=scratch)
    fn = {"gcn": lib().gnnfd_oneshot_gcn, "sage": lib().gnnfd_oneshot_sage}[model]
    _check(fn(n, src.numel(), ctypes.c_void_p(src.data_ptr()), ctypes.c_void_p(dst.data_ptr()),
              I32 if src.dtype == torch.int32 else I64, flags, xp, ldx, _dtype_code(x), op, ldo, _dtype_code(out), f,
              chunk_width, ctypes.c_void_p(scratch.data_ptr()), scratch.numel() * scratch.element_size(),
              _stream_ptr(stream)), "gnnfd_oneshot_" + model)
    return out


def oneshot_gat(n: int, src: torch.Tensor, dst: torch.Tensor, z: torch.Tensor, a_src: torch.Tensor, a_dst: torch.Tensor,
                heads: int, dim: int, negative_slope: float = 0.2, flags: int = 0, chunk_width: int | None = None,
                out: torch.Tensor | None = None, out_dtype=None, scratch=None, stream=None):
    """gnnfd_oneshot_gat: light build + GAT aggregation of a COO edge list in one call."""
    if not (src.is_cuda and dst.is_cuda) or src.dtype != dst.dtype or src.shape != dst.shape or src.dim() != 1:
        raise ValueError("src and dst must be 1-D CUDA tensors of the same dtype and length")
    if src.dtype not in (torch.int32, torch.int64):
        raise TypeError("edge ids must be int32 or int64")
    src, dst = src.contiguous(), dst.contiguous()
    f = heads * dim
    chunk_width = f if chunk_width is None else chunk_width
    if out is None:
        out = torch.empty((n, f), dtype=out_dtype or torch.float32, device=z.device)
    zp, ldz = _matrix(z, f, "z")
    op, ldo = _matrix(out, f, "out")
    _same_device(src.device, dst=dst, z=z, out=out)
    _need_rows(z, n, "z")
    _need_rows(out, n, "out")
    _no_overlap(z, out, "z", "out")
    a_src, a_dst = _attention_vectors(a_src, a_dst, heads, dim, z.device, stream)
    if scratch is None:
        need = ctypes.c_size_t()
        _check(lib().gnnfd_oneshot_gat_workspace_bytes(n, src.numel(), flags, heads, dim, ctypes.byref(need)),
               "gnnfd_oneshot_gat_workspace_bytes")
        scratch = _alloc_bytes(need.value, z.device, stream)
    _same_device(src.device, scratch=scratch)
    _check(lib().gnnfd_oneshot_gat(n, src.numel(), ctypes.c_void_p(src.data_ptr()), ctypes.c_void_p(dst.data_ptr()),
                                   I32 if src.dtype == torch.int32 else I64, flags, zp, ldz, _dtype_code(z),
                                   ctypes.c_void_p(a_src.data_ptr()), ctypes.c_void_p(a_dst.data_ptr()), heads, dim,
                                   negative_slope, op, ldo, _dtype_code(out), chunk_width,
                                   ctypes.c_void_p(scratch.data_ptr()), scratch.numel() * scratch.element_size(),
                                   _stream_ptr(stream)), "gnnfd_oneshot_gat")
    return out


def default_chunk_candidates(f: int, dtype=torch.float32) -> list:
    buf = (ctypes.c_int32 * 16)()
    k = lib().gnnfd_default_chunk_candidates(f, F32 if dtype == torch.float32 else BF16, buf, 16)
    if k < 0:
        raise GnnfdError(k, "gnnfd_default_chunk_candidates")
    return list(buf[:k])


def tune_chunk_width(csr: Csr, x: torch.Tensor, model: str = "gcn", f: int | None = None, candidates=None,
                     out: torch.Tensor | None = None, scratch=None, stream=None):
    """gnnfd_tune_chunk_width: times the candidates on this graph and these features; -> (width, ms)."""
    f = x.shape[1] if f is None else f
    candidates = default_chunk_candidates(f, x.dtype) if candidates is None else list(candidates)
    if out is None:
        out = torch.empty((csr.n, f), dtype=torch.float32, device=x.device)
    xp, ldx = _matrix(x, f, "x")
    op, ldo = _matrix(out, f, "out")
    _check_aggregate_operands(csr, x, out, f)
    need = aggregate_workspace_bytes(csr, f)
    if scratch is None and need:
        scratch = _alloc_bytes(need, x.device, stream)
    _same_device(csr.device, scratch=scratch)
    sp = ctypes.c_void_p(scratch.data_ptr()) if scratch is not None else None
    sn = scratch.numel() * scratch.element_size() if scratch is not None else 0
    arr = (ctypes.c_int32 * len(candidates))(*candidates)
    best, ms = ctypes.c_int32(), ctypes.c_float()
    _check(lib().gnnfd_tune_chunk_width(csr.handle, {"gcn": 0, "sage": 1}[model], xp, ldx, _dtype_code(x), op, ldo,
                                        _dtype_code(out), f, arr, len(candidates), sp, sn, _stream_ptr(stream),
                                        ctypes.byref(best), ctypes.byref(ms)), "gnnfd_tune_chunk_width")
    return best.value, ms.value


def aggregate_gcn_static(csr: Csr, x: torch.Tensor, f: int | None = None, chunk_width: int | None = None,
                         out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """gnnfd_aggregate_gcn_static: GCN aggregation whose hub-row workspace is the library's built-in
    array, for callers that can neither allocate device memory nor spare a buffer.  ``out`` should be
    passed by such callers (when it is None this wrapper allocates it with torch, which the C entry
    point itself never does).  Raises GnnfdError(STATIC_SCRATCH_EXCEEDED) beyond the built-in size."""
    f = x.shape[1] if f is None else f
    chunk_width = f if chunk_width is None else chunk_width
    if out is None:
        out = torch.empty((csr.n, f), dtype=torch.float32, device=x.device)
    xp, ldx = _matrix(x, f, "x")
    op, ldo = _matrix(out, f, "out")
    _check_aggregate_operands(csr, x, out, f)
    _check(lib().gnnfd_aggregate_gcn_static(csr.handle, xp, ldx, _dtype_code(x), op, ldo, _dtype_code(out), f,
                                            chunk_width, _stream_ptr(stream)), "gnnfd_aggregate_gcn_static")
    return out


def _attention_vectors(a_src, a_dst, heads: int, dim: int, device, stream):
    """The two [heads, dim] fp32 attention vectors, contiguous and on `device`.  A conversion makes a
    temporary; it is created under the launch stream for the same reason as the scratch buffers."""
    for name, a in (("a_src", a_src), ("a_dst", a_dst)):
        if a.numel() != heads * dim:
            raise ValueError("%s must hold heads*dim = %d values" % (name, heads * dim))
        if torch.device(a.device) != torch.device(device):
            raise ValueError("%s is on %s, the features are on %s" % (name, a.device, device))
    if stream is None:
        return a_src.contiguous().float(), a_dst.contiguous().float()
    with torch.cuda.stream(stream):
        return a_src.contiguous().float(), a_dst.contiguous().float()


def gat_scores(z: torch.Tensor, a_src: torch.Tensor, a_dst: torch.Tensor, heads: int, dim: int, stream=None):
    n = z.shape[0]
    zp, ldz = _matrix(z, heads * dim, "z")
    a_src, a_dst = _attention_vectors(a_src, a_dst, heads, dim, z.device, stream)
    s_src = torch.empty((n, heads), dtype=torch.float32, device=z.device)
    s_dst = torch.empty((n, heads), dtype=torch.float32, device=z.device)
    _check(lib().gnnfd_gat_scores(n, zp, ldz, _dtype_code(z), ctypes.c_void_p(a_src.data_ptr()),
                                  ctypes.c_void_p(a_dst.data_ptr()), heads, dim, ctypes.c_void_p(s_src.data_ptr()),
                                  ctypes.c_void_p(s_dst.data_ptr()), _stream_ptr(stream)), "gnnfd_gat_scores")
    return s_src, s_dst


def gat_workspace_bytes(csr: Csr, heads: int, dim: int) -> int:
    s = ctypes.c_size_t()
    _check(lib().gnnfd_gat_workspace_bytes(csr.handle, heads, dim, ctypes.byref(s)), "gnnfd_gat_workspace_bytes")
    return s.value


def aggregate_gat(csr: Csr, z: torch.Tensor, a_src: torch.Tensor, a_dst: torch.Tensor, heads: int, dim: int,
                  negative_slope: float = 0.2, chunk_width: int | None = None, out: torch.Tensor | None = None,
                  out_dtype=None, scratch=None, stream=None) -> torch.Tensor:
    f = heads * dim
    chunk_width = f if chunk_width is None else chunk_width
    if out is None:
        out = torch.empty((csr.n, f), dtype=out_dtype or torch.float32, device=z.device)
    zp, ldz = _matrix(z, f, "z")
    op, ldo = _matrix(out, f, "out")
    _check_aggregate_operands(csr, z, out, f, "z")
    a_src, a_dst = _attention_vectors(a_src, a_dst, heads, dim, z.device, stream)
    if scratch is None:
        scratch = _alloc_bytes(gat_workspace_bytes(csr, heads, dim), z.device, stream)
    _same_device(csr.device, scratch=scratch)
    _check(lib().gnnfd_aggregate_gat(csr.handle, zp, ldz, _dtype_code(z), ctypes.c_void_p(a_src.data_ptr()),
                                     ctypes.c_void_p(a_dst.data_ptr()), heads, dim, negative_slope, op, ldo,
                                     _dtype_code(out), chunk_width, ctypes.c_void_p(scratch.data_ptr()),
                                     scratch.numel() * scratch.element_size(), _stream_ptr(stream)),
           "gnnfd_aggregate_gat")
    return out


def edge_softmax_workspace_bytes(csr: Csr, heads: int) -> int:
    s = ctypes.c_size_t()
    _check(lib().gnnfd_edge_softmax_workspace_bytes(csr.handle, heads, ctypes.byref(s)),
           "gnnfd_edge_softmax_workspace_bytes")
    return s.value


def edge_softmax(csr: Csr, s_src: torch.Tensor, s_dst: torch.Tensor, negative_slope: float = 0.2,
                 out: torch.Tensor | None = None, scratch=None, stream=None) -> torch.Tensor:
    heads = s_src.shape[1]
    if not (s_src.is_contiguous() and s_dst.is_contiguous()):
        raise ValueError("scores must be contiguous")
    if s_src.dtype != torch.float32 or s_dst.dtype != torch.float32 or s_src.shape != s_dst.shape:
        raise TypeError("scores must be float32 [n, heads]")
    if s_src.dim() != 2 or s_src.shape[0] != csr.n:
        raise ValueError("scores must be [n, heads] with n = %d rows, got %s" % (csr.n, tuple(s_src.shape)))
    if out is None:
        out = torch.empty((csr.nnz, heads), dtype=torch.float32, device=s_src.device)
    if out.dtype != torch.float32 or out.dim() != 2 or not out.is_contiguous() or out.shape[1] != heads \
            or out.shape[0] < csr.nnz:
        raise ValueError("alpha must be a contiguous float32 [nnz >= %d, heads = %d] tensor" % (csr.nnz, heads))
    _same_device(csr.device, s_src=s_src, s_dst=s_dst, alpha=out)
    _no_overlap(s_src, out, "s_src", "alpha")
    _no_overlap(s_dst, out, "s_dst", "alpha")
    if scratch is None:
        scratch = _alloc_bytes(edge_softmax_workspace_bytes(csr, heads), s_src.device, stream)
    _same_device(csr.device, scratch=scratch)
    _check(lib().gnnfd_edge_softmax(csr.handle, ctypes.c_void_p(s_src.data_ptr()), ctypes.c_void_p(s_dst.data_ptr()),
                                    heads, negative_slope, ctypes.c_void_p(out.data_ptr()),
                                    ctypes.c_void_p(scratch.data_ptr()), scratch.numel() * scratch.element_size(),
                                    _stream_ptr(stream)),
           "gnnfd_edge_softmax")
    return out


def _combine_mode(mode) -> int:
    if mode in (COMBINE_TF32, "tf32"):
        return COMBINE_TF32
    if mode in (COMBINE_FP32, "fp32"):
        return COMBINE_FP32
    raise ValueError("mode must be 'tf32' or 'fp32'")


def combine(x: torch.Tensor, w_t: torch.Tensor, f_in: int | None = None, out: torch.Tensor | None = None,
            out_dtype=None, status: torch.Tensor | None = None, stream=None, mode="tf32", a_src=None, a_dst=None,
            heads: int = 0, dim: int = 0):
    """gnnfd_combine_ex: z = x[:, :f_in] @ w_t[:, :f_in].T on the tensor cores with fp32 sums.  float32 inputs
    are multiplied as tf32 (``mode="tf32"``) or fp32-faithfully as tf32 pairs (``mode="fp32"``); bfloat16 inputs
    as they are.  ``status`` is an int32 tensor of one element that the kernel sets to 1 if a block gave up
    waiting.  With ``a_src`` / ``a_dst`` ([heads, dim], heads * dim == f_out) the GAT scores of z are formed in
    the same pass and the call returns (z, s_src, s_dst) instead of z."""
    f_in = w_t.shape[1] if f_in is None else f_in
    f_out = w_t.shape[0]
    if x.dtype != w_t.dtype:
        raise TypeError("x and w_t must have the same dtype")
    if out is None:
        out = torch.empty((x.shape[0], f_out), dtype=out_dtype or torch.float32, device=x.device)
    xp, ldx = _matrix(x, f_in, "x")
    wp, ldw = _matrix(w_t, f_in, "w_t")
    op, ldo = _matrix(out, f_out, "out")
    _same_device(x.device, w_t=w_t, out=out, status=status)
    _need_rows(out, x.shape[0], "out")
    _no_overlap(x, out, "x", "out")
    _no_overlap(w_t, out, "w_t", "out")
    sp = ctypes.c_void_p(status.data_ptr()) if status is not None else None
    scores = a_src is not None or a_dst is not None
    s_src = s_dst = None
    asp = adp = ssp = sdp = None
    if scores:
        a_src, a_dst = _attention_vectors(a_src, a_dst, heads, dim, x.device, stream)
        s_src = torch.empty((x.shape[0], heads), dtype=torch.float32, device=x.device)
        s_dst = torch.empty((x.shape[0], heads), dtype=torch.float32, device=x.device)
        asp, adp = ctypes.c_void_p(a_src.data_ptr()), ctypes.c_void_p(a_dst.data_ptr())
        ssp, sdp = ctypes.c_void_p(s_src.data_ptr()), ctypes.c_void_p(s_dst.data_ptr())
    _check(lib().gnnfd_combine_ex(x.shape[0], xp, ldx, _dtype_code(x), f_in, wp, ldw, f_out, op, ldo, _dtype_code(out),
                                  _combine_mode(mode), asp, adp, heads, dim, ssp, sdp, sp, _stream_ptr(stream)),
           "gnnfd_combine_ex")
    return (out, s_src, s_dst) if scores else out


def layer_workspace_bytes(csr: Csr, model: str, f_out: int, heads: int = 0, dim: int = 0, dtype=torch.float32) -> int:
    s = ctypes.c_size_t()
    _check(lib().gnnfd_layer_workspace_bytes(csr.handle, {"gcn": 0, "sage": 1, "gat": 2}[model], f_out, heads, dim,
                                             F32 if dtype == torch.float32 else BF16, ctypes.byref(s)),
           "gnnfd_layer_workspace_bytes")
    return s.value


def layer(csr: Csr, model: str, x: torch.Tensor, w_t: torch.Tensor, f_in: int | None = None, mode="tf32",
          chunk_width: int | None = None, out: torch.Tensor | None = None, out_dtype=None, a_src=None, a_dst=None,
          heads: int = 0, dim: int = 0, negative_slope: float = 0.2, scratch=None, status=None, stream=None):
    """gnnfd_layer_gcn / _sage / _gat: out = Aggregate(x[:, :f_in] @ w_t[:, :f_in].T) on a built CSR; the
    transformed features stay in the scratch buffer."""
    f_in = w_t.shape[1] if f_in is None else f_in
    f_out = w_t.shape[0]
    if x.dtype != w_t.dtype:
        raise TypeError("x and w_t must have the same dtype")
    if model == "gat" and heads * dim != f_out:
        raise ValueError("heads * dim must equal the number of rows of w_t")
    chunk_width = f_out if chunk_width is None else chunk_width
    if out is None:
        out = torch.empty((csr.n, f_out), dtype=out_dtype or torch.float32, device=x.device)
    xp, ldx = _matrix(x, f_in, "x")
    wp, ldw = _matrix(w_t, f_in, "w_t")
    op, ldo = _matrix(out, f_out, "out")
    _same_device(csr.device, x=x, w_t=w_t, out=out, status=status)
    _need_rows(x, csr.n, "x")
    _need_rows(out, csr.n, "out")
    _no_overlap(x, out, "x", "out")
    _no_overlap(w_t, out, "w_t", "out")
    if scratch is None:
        scratch = _alloc_bytes(layer_workspace_bytes(csr, model, f_out, heads, dim, x.dtype), x.device, stream)
    _same_device(csr.device, scratch=scratch)
    sp = ctypes.c_void_p(status.data_ptr()) if status is not None else None
    scr, scr_n = ctypes.c_void_p(scratch.data_ptr()), scratch.numel() * scratch.element_size()
    if model == "gat":
        a_src, a_dst = _attention_vectors(a_src, a_dst, heads, dim, x.device, stream)
        _check(lib().gnnfd_layer_gat(csr.handle, xp, ldx, _dtype_code(x), f_in, wp, ldw, heads, dim,
                                     ctypes.c_void_p(a_src.data_ptr()), ctypes.c_void_p(a_dst.data_ptr()), negative_slope,
                                     _combine_mode(mode), op, ldo, _dtype_code(out), chunk_width, scr, scr_n, sp,
                                     _stream_ptr(stream)), "gnnfd_layer_gat")
    else:
        fn = lib().gnnfd_layer_gcn if model == "gcn" else lib().gnnfd_layer_sage
        _check(fn(csr.handle, xp, ldx, _dtype_code(x), f_in, wp, ldw, f_out, _combine_mode(mode), op, ldo,
                  _dtype_code(out), chunk_width, scr, scr_n, sp, _stream_ptr(stream)), "gnnfd_layer_" + model)
    return out


def debug_combine_fault(wait_ns: int, skip_k_block: int):
    """gnnfd_debug_combine_fault: arms the give-up drill for this thread's next transform launch."""
    _check(lib().gnnfd_debug_combine_fault(wait_ns, skip_k_block), "gnnfd_debug_combine_fault")


def launch_count() -> int:
    return int(lib().gnnfd_launch_count())


def kernel_timing_enable(on: bool = True):
    _check(lib().gnnfd_kernel_timing_enable(int(on)), "gnnfd_kernel_timing_enable")


def kernel_timing_read() -> dict:
    """{kernel name: (total ms, launches)} since the last read."""
    cap = 64
    names = (ctypes.c_char_p * cap)()
    ms = (ctypes.c_double * cap)()
    cnt = (ctypes.c_int64 * cap)()
    k = lib().gnnfd_kernel_timing_read(names, ms, cnt, cap)
    if k < 0:
        raise GnnfdError(k, "gnnfd_kernel_timing_read")
    return {names[i].decode(): (ms[i], cnt[i]) for i in range(min(k, cap))}
