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


def aggregate_slab(csr, x: torch.Tensor, model: str, f: int, chunk_width: int, world: int, rank: int,
                   out: torch.Tensor, a_src=None, a_dst=None, heads: int = 1, dim: int = 0,
                   negative_slope: float = 0.2, scratch=None, stream=None) -> tuple[int, int]:
    """Rank `rank`'s share of one aggregation: the decomposition layers (chunks) that fall in its column slab,
    computed by the single-GPU entry points on column views x[:, j0:j1] -> out[:, j0:j1] (same leading
    dimensions, nothing copied).  `x` and `out` are the full-width matrices (a rank that only holds its slab
    passes matrices whose other columns are never touched).  For GAT the slab has to consist of whole heads
    (chunk_width a multiple of `dim`), because a head's attention scores need all of its columns.
    Returns the slab [j0, j1)."""
    from . import binding as g
    j0, j1 = column_slab(f, chunk_width, world, rank)
    if j1 == j0:
        return j0, j1
    xs, outs = x[:, j0:j1], out[:, j0:j1]
    cw = min(chunk_width, f)
    if model == "gcn":
        g.aggregate_gcn(csr, xs, f=j1 - j0, chunk_width=cw, out=outs, scratch=scratch, stream=stream)
    elif model == "sage":
        g.aggregate_sage(csr, xs, f=j1 - j0, chunk_width=cw, out=outs, scratch=scratch, stream=stream)
    elif model == "gat":
        if dim <= 0 or j0 % dim or (j1 % dim and j1 != f) or f != heads * dim:
            raise ValueError("a GAT column slab must consist of whole heads: slab [%d, %d), head width %d" % (j0, j1, dim))
        h0, h1 = j0 // dim, (j1 + dim - 1) // dim
        g.aggregate_gat(csr, xs, a_src[h0:h1], a_dst[h0:h1], h1 - h0, dim, negative_slope, chunk_width=cw, out=outs,
                        scratch=scratch, stream=stream)
    else:
        raise ValueError(model)
    return j0, j1


def gather_slabs_(out: torch.Tensor, f: int, chunk_width: int, group=None) -> torch.Tensor:
    """Completes `out` [n, >= f] on every rank: each rank contributes the slab it computed (its columns of
    `out`), the others' slabs arrive by one all-gather (NCCL on GPUs) into local buffers and are copied into
    place.  No kernel ever reads another GPU's memory."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    slabs = [column_slab(f, chunk_width, world, r) for r in range(world)]
    widest = max(j1 - j0 for j0, j1 in slabs)
    n = out.shape[0]
    j0, j1 = slabs[rank]
    mine = torch.zeros((n, widest), dtype=out.dtype, device=out.device)
    mine[:, :j1 - j0] = out[:, j0:j1]
    parts = torch.empty((world, n, widest), dtype=out.dtype, device=out.device)
    dist.all_gather([parts[r] for r in range(world)], mine, group=group)
    for r, (a0, a1) in enumerate(slabs):
        if r != rank and a1 > a0:
            out[:, a0:a1] = parts[r, :, :a1 - a0]
    return out


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
