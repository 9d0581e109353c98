"""Host-side planning for more than one GPU.

The decomposition layers of Algorithm 1 are independent of one another, so the aggregation shards by
feature chunk with no exchange step: every rank holds the graph (CSR) and a slab of whole chunks
x[:, j0:j1], aggregates it with the single-GPU entry points (a column view with the full leading
dimension is enough, nothing is copied), and owns out[:, j0:j1].  Independent graphs (one per rank)
need no plan at all.  Only torch.distributed plumbing lives here; no arithmetic of the method.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def column_slab(f: int, chunk_width: int, world: int, rank: int) -> tuple[int, int]:
    """Columns [j0, j1) of rank `rank`: contiguous whole chunks, as even as possible (the first
    `n_chunks % world` ranks get one more chunk; a rank may get none)."""
    if f <= 0 or chunk_width <= 0 or world <= 0 or not 0 <= rank < world:
        raise ValueError("bad slab request")
    cw = min(chunk_width, f)
    n_chunks = (f + cw - 1) // cw
    base, extra = divmod(n_chunks, world)
    first = rank * base + min(rank, extra)
    count = base + (1 if rank < extra else 0)
    return min(f, first * cw), min(f, (first + count) * cw)


def gather_columns(local: torch.Tensor, f: int, chunk_width: int, group=None) -> torch.Tensor:
    """All-gathers the per-rank column slabs [n, j1-j0] into the full [n, f] matrix on every rank."""
    world = dist.get_world_size(group)
    n = local.shape[0]
    widths = [column_slab(f, chunk_width, world, r) for r in range(world)]
    widest = max(j1 - j0 for j0, j1 in widths)
    padded = torch.zeros((n, widest), dtype=local.dtype, device=local.device)
    padded[:, :local.shape[1]] = local
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded, group=group)
    out = torch.empty((n, f), dtype=local.dtype, device=local.device)
    for (j0, j1), part in zip(widths, parts):
        out[:, j0:j1] = part[:, :j1 - j0]
    return out


def reduce_job_timing(ms: float, units: float, device=None, group=None) -> tuple[float, float]:
    """(max over ranks of the elapsed milliseconds, sum over ranks of the units processed)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return ms, units
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    dist.all_reduce(u, op=dist.ReduceOp.SUM, group=group)
    return t.item(), u.item()
