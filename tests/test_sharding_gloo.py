"""World-size-2 gloo runs of the multi-GPU host logic: chunk-aligned column slabs reassemble to the
full aggregation, and job timing reduces as max(time) / sum(units)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import graphgen as gg
import oracle as orc
from paper_2104_03058_b200 import sharding


def test_column_slabs_partition_the_columns_on_chunk_boundaries():
    for f, cw, world in [(602, 64, 2), (602, 64, 8), (16, 4, 3), (5, 7, 4), (64, 1, 5)]:
        slabs = [sharding.column_slab(f, cw, world, r) for r in range(world)]
        assert slabs[0][0] == 0 and slabs[-1][1] == f
        for (a0, a1), (b0, b1) in zip(slabs, slabs[1:]):
            assert a1 == b0 and a0 <= a1
        for j0, j1 in slabs:
            assert j0 % min(cw, f) == 0 or j0 == f
        sizes = [(j1 - j0 + min(cw, f) - 1) // min(cw, f) for j0, j1 in slabs]
        assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.column_slab(10, 2, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, f, cw, result_path):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        n = 500
        src, dst = gg.powerlaw_graph(n, 6000, 2.1, None, 1)
        x = gg.features_f32(n, f, dist="normal", p0=0, p1=1, seed=1)
        row_ptr, col, _ = orc.build_csr(n, src, dst, orc.ADD_SELF_LOOPS)
        j0, j1 = sharding.column_slab(f, cw, world, rank)
        # the rank's slab as the single-GPU entry points would see it: a column view of x
        slab = np.ascontiguousarray(x[:, j0:j1])
        local = np.zeros((n, 0)) if j1 == j0 else orc.aggregate("gcn", row_ptr, col, slab, j1 - j0, cw)[0]
        full = sharding.gather_columns(torch.from_numpy(local), f, cw)
        want = orc.aggregate("gcn", row_ptr, col, x, f, cw)[0]
        ok = np.array_equal(full.numpy(), want)
        # the in-place form the GPU ranks use: every rank holds the full-width output, has filled only its own
        # columns (the others hold a sentinel), and one all-gather completes it
        mine = torch.full((n, f + 3), -777.0, dtype=torch.float64)          # three padding columns stay untouched
        mine[:, j0:j1] = torch.from_numpy(local)
        sharding.gather_slabs_(mine, f, cw)
        ok = ok and np.array_equal(mine[:, :f].numpy(), want) and bool((mine[:, f:] == -777.0).all())
        ms, units = sharding.reduce_job_timing(10.0 + rank, 100.0 * (rank + 1))
        ok = ok and ms == 10.0 + world - 1 and units == 100.0 * world * (world + 1) / 2
        flag = torch.tensor([1 if ok else 0])
        dist.all_reduce(flag, op=dist.ReduceOp.MIN)
        if rank == 0:
            with open(result_path, "w") as fh:
                fh.write(str(int(flag.item())))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("f,cw", [(13, 4), (8, 8)])
def test_two_ranks_reassemble_the_full_result(tmp_path, f, cw):
    result = tmp_path / "ok.txt"
    mp.spawn(_worker, args=(2, _free_port(), f, cw, str(result)), nprocs=2, join=True)
    assert result.read_text() == "1"
