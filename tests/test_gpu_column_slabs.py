"""Sharding by feature chunk (Algorithm 1: decomposition layers are independent): one GPU plays 2, 3 and 5
ranks in turn, each rank aggregating only its chunk-aligned column slab through the single-GPU entry points
on column views; the reassembled matrix is compared with the CPU oracle element by element.  (The ranks
exchange nothing while they compute, so playing them one after the other on one device is the same work.)"""
import numpy as np
import pytest

import graphgen as gg
import oracle as orc

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

SENTINEL = -12345.0


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def close(got, want, scale):
    return (np.abs(got.astype(np.float64) - want) <= 1e-5 * scale + 1e-6).all()


@pytest.mark.parametrize("world", [2, 3, 5])
@pytest.mark.parametrize("model", ["gcn", "sage"])
def test_virtual_ranks_reassemble_gcn_and_sage(world, model):
    import paper_2104_03058_b200 as g
    from paper_2104_03058_b200 import sharding
    w = gg.scaled("config4", 0.05)                     # power-law graph with hub rows, F = 602 in ld = 608
    row_ptr, col, _ = orc.build_csr(w.n, w.src, w.dst, w.flags)
    csr = g.build_csr(w.n, dev(w.src), dev(w.dst), w.flags)
    f, cw = 150, 32                                     # 5 chunks, the last one 22 columns wide
    x = dev(w.x)
    want, scale = orc.aggregate(model, row_ptr, col, w.x, f, threads=orc.max_threads())
    out = torch.full((w.n, w.ld), SENTINEL, device="cuda")
    covered = np.zeros(f, bool)
    for rank in range(world):
        j0, j1 = sharding.aggregate_slab(csr, x, model, f, cw, world, rank, out)
        assert j0 % cw == 0 and not covered[j0:j1].any()
        covered[j0:j1] = True
        if rank < world - 1:                            # columns of the ranks still to come are untouched
            assert bool((out[:, j1:] == SENTINEL).all())
    assert covered.all()
    got = out.cpu().numpy()
    assert close(got[:, :f], want, scale)
    assert (got[:, f:] == SENTINEL).all()               # padding columns never written
    # the slabs are the very chunks a single call computes: the whole chunks come out with the same bits as in
    # one full-width call (the ragged last chunk may be laid out over fewer lanes when it is a slab's only chunk)
    full = g.aggregate_gcn(csr, x, f=f, chunk_width=cw) if model == "gcn" else g.aggregate_sage(csr, x, f=f, chunk_width=cw)
    whole = f // cw * cw
    assert torch.equal(out[:, :whole], full[:, :whole])
    assert csr.bin_count[4] > 0                         # hub rows (segment partials) were part of it


@pytest.mark.parametrize("world", [2, 3])
def test_virtual_ranks_reassemble_gat_by_whole_heads(world):
    import paper_2104_03058_b200 as g
    from paper_2104_03058_b200 import sharding
    w = gg.scaled("config3", 0.05)
    row_ptr, col, _ = orc.build_csr(w.n, w.src, w.dst, w.flags)
    csr = g.build_csr(w.n, dev(w.src), dev(w.dst), w.flags)
    z, a_src, a_dst = dev(w.x), dev(w.a_src), dev(w.a_dst)
    f = w.heads * w.dim
    want, scale = orc.aggregate_gat(row_ptr, col, w.x, w.a_src, w.a_dst, w.heads, w.dim, w.negative_slope)
    for cw in (w.dim, 2 * w.dim):                       # one head per chunk (the paper's GAT granularity), two heads
        out = torch.full((w.n, f), SENTINEL, device="cuda")
        for rank in range(world):
            sharding.aggregate_slab(csr, z, "gat", f, cw, world, rank, out, a_src=a_src, a_dst=a_dst, heads=w.heads,
                                    dim=w.dim, negative_slope=w.negative_slope)
        assert close(out.cpu().numpy(), want, scale)
    with pytest.raises(ValueError, match="whole heads"):
        sharding.aggregate_slab(csr, z, "gat", f, w.dim + 4, 2, 1, torch.empty((w.n, f), device="cuda"), a_src=a_src,
                                a_dst=a_dst, heads=w.heads, dim=w.dim)


def test_more_ranks_than_chunks_leaves_idle_ranks_without_work():
    import paper_2104_03058_b200 as g
    from paper_2104_03058_b200 import sharding
    n, f = 2000, 16
    src, dst = gg.uniform_graph(n, 20_000, seed=4)
    csr = g.build_csr(n, dev(src), dev(dst), 1)
    x = torch.randn((n, f), device="cuda")
    out = torch.zeros((n, f), device="cuda")
    before = g.launch_count()
    assert sharding.aggregate_slab(csr, x, "gcn", f, 16, 4, 3, out) == (16, 16)      # one chunk, rank 3 of 4: nothing to do
    assert g.launch_count() == before


def test_slab_gather_over_nccl_with_device_tensors():
    """gather_slabs_ on CUDA tensors through the NCCL backend.  One GPU is what a test gets, so the group has one
    rank: the collective runs on the device and must leave the rank's own columns and the padding as they are."""
    import os
    import socket

    import torch.distributed as dist
    from paper_2104_03058_b200 import sharding
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        out = torch.arange(300 * 20, dtype=torch.float32, device="cuda").reshape(300, 20).contiguous()
        want = out.clone()
        sharding.gather_slabs_(out, 17, 4)
        torch.cuda.synchronize()
        assert torch.equal(out, want)
        ms, units = sharding.reduce_job_timing(3.5, 10.0, device=torch.device("cuda", 0))
        assert (ms, units) == (3.5, 10.0)
    finally:
        dist.destroy_process_group()
