"""Host-buffer front end: graph and features in pinned host memory in, aggregated features out.

``HostPipeline.submit`` runs one job (CSR build + chunked GCN / SAGE / GAT aggregation) whose inputs and output
live in pinned host memory.  Device buffers are double-buffered and the copies run on their own
streams, so the host-to-device copy of the next job and the device-to-host copy of the previous
result overlap the kernels of the current one.  Only torch plumbing (streams, events, copies) lives
here; the work itself is the library's.
"""
from __future__ import annotations

import torch

from . import binding as g


class HostPipeline:
    def __init__(self, n: int, max_edges: int, f: int, ld: int, flags: int, chunk_width: int, device=None,
                 feature_dtype=torch.float32, index_dtype=torch.int32, depth: int = 2, model: str = "gcn",
                 heads: int = 1, dim: int = 0, a_src=None, a_dst=None, negative_slope: float = 0.2):
        if model not in ("gcn", "sage", "gat"):
            raise ValueError(model)
        self.n, self.f, self.ld, self.flags, self.chunk_width = n, f, ld, flags, chunk_width
        self.model, self.heads, self.dim, self.negative_slope = model, heads, dim, negative_slope
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
        self.depth = depth
        dev = self.device
        self.d_src = [torch.empty(max_edges, dtype=index_dtype, device=dev) for _ in range(depth)]
        self.d_dst = [torch.empty(max_edges, dtype=index_dtype, device=dev) for _ in range(depth)]
        self.d_x = [torch.empty((n, ld), dtype=feature_dtype, device=dev) for _ in range(depth)]
        self.d_out = [torch.empty((n, ld), dtype=torch.float32, device=dev) for _ in range(depth)]
        pb, sb = g.csr_workspace_bytes(n, max_edges, flags)
        self.persistent = torch.empty(pb, dtype=torch.uint8, device=dev)
        self.scratch = torch.empty(sb, dtype=torch.uint8, device=dev)
        self.agg_scratch = None
        self.a_src = None if a_src is None else a_src.to(dev)
        self.a_dst = None if a_dst is None else a_dst.to(dev)
        self.s_in = torch.cuda.Stream(device=dev)
        self.s_out = torch.cuda.Stream(device=dev)
        self.ev_in = [torch.cuda.Event() for _ in range(depth)]        # inputs of slot arrived
        self.ev_done = [torch.cuda.Event() for _ in range(depth)]      # kernels of slot finished
        self.ev_out = [torch.cuda.Event() for _ in range(depth)]       # result of slot copied out
        self.jobs = 0
        self._staged = None
        self.csr = None

    def _stage(self, h_src, h_dst, h_x):
        """Enqueue the host-to-device copies of a job on the input stream."""
        slot = self.jobs % self.depth
        e = h_src.numel()
        with torch.cuda.stream(self.s_in):
            if self.jobs >= self.depth:
                self.s_in.wait_event(self.ev_done[slot])               # the slot's previous job no longer reads it
            self.d_src[slot][:e].copy_(h_src, non_blocking=True)
            self.d_dst[slot][:e].copy_(h_dst, non_blocking=True)
            self.d_x[slot].copy_(h_x, non_blocking=True)
            self.ev_in[slot].record(self.s_in)
        return slot, e

    def submit(self, h_src, h_dst, h_x, h_out, next_job=None):
        """Runs one job.  ``next_job`` = (h_src, h_dst, h_x) of the following job, if known: its copies
        are enqueued before this job's kernels so that they overlap them."""
        staged = self._staged if self._staged is not None else self._stage(h_src, h_dst, h_x)
        slot, e = staged
        self.jobs += 1
        self._staged = self._stage(*next_job) if next_job is not None else None
        cur = torch.cuda.current_stream(self.device)
        cur.wait_event(self.ev_in[slot])
        if self.jobs > self.depth:
            cur.wait_event(self.ev_out[slot])                          # the slot's previous result has left
        if self.csr is not None:
            self.csr.destroy()
        self.csr = g.build_csr(self.n, self.d_src[slot][:e], self.d_dst[slot][:e], self.flags,
                               persistent=self.persistent, scratch=self.scratch)
        # the workspace depends on this graph's hub rows, so it is asked for per job and grown when needed
        # (the old buffer may still be in use by the previous job's kernels on this stream: torch frees it
        # in stream order)
        need = (g.gat_workspace_bytes(self.csr, self.heads, self.dim) if self.model == "gat"
                else g.aggregate_workspace_bytes(self.csr, self.f))
        if self.agg_scratch is None or self.agg_scratch.numel() < need:
            self.agg_scratch = torch.empty(max(need, 256), dtype=torch.uint8, device=self.device)
        out = self.d_out[slot][:, :self.f]
        if self.model == "gat":
            g.aggregate_gat(self.csr, self.d_x[slot], self.a_src, self.a_dst, self.heads, self.dim,
                            self.negative_slope, chunk_width=self.chunk_width, out=out, scratch=self.agg_scratch)
        elif self.model == "sage":
            g.aggregate_sage(self.csr, self.d_x[slot], f=self.f, chunk_width=self.chunk_width, out=out,
                             scratch=self.agg_scratch)
        else:
            g.aggregate_gcn(self.csr, self.d_x[slot], f=self.f, chunk_width=self.chunk_width, out=out,
                            scratch=self.agg_scratch)
        self.ev_done[slot].record(cur)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.ev_done[slot])
            h_out.copy_(self.d_out[slot], non_blocking=True)
            self.ev_out[slot].record(self.s_out)
        return self.csr

    def finish(self):
        """Makes the current stream wait for every copy still in flight."""
        cur = torch.cuda.current_stream(self.device)
        cur.wait_stream(self.s_in)
        cur.wait_stream(self.s_out)

