"""gnnfd_aggregate_gcn_static: the GCN aggregation for hosts that cannot allocate device memory.

Some users of the library own no allocator at the point of the call: the whole device was handed to
a memory pool when their process started, or they sit in a loop where a cudaMalloc (which
synchronises the device) is not acceptable, and they have no spare buffer either.  For them the
hub-row workspace is an array built into the library.  These tests call that entry point through the
C ABI, twice in a row (the array keeps the first call's contents), and compare with the ordinary
entry point, which gets a caller-allocated workspace, and with the CPU oracle.  The file is named to be
collected last.
"""
import numpy as np
import pytest

import graphgen as gg
import oracle as orc

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _graph_with_hub_rows(n, e, hubs, seed):
    src, dst = gg.uniform_graph(n, e, seed=seed)
    per = e // (2 * len(hubs))
    for i, v in enumerate(hubs):
        dst[i * per:(i + 1) * per] = v
    return src, dst


def test_static_workspace_matches_caller_workspace_twice_in_a_row():
    import paper_2104_03058_b200 as g
    n, f = 4000, 70
    src, dst = _graph_with_hub_rows(n, 60_000, hubs=(5, 1999, 3998), seed=21)
    csr = g.build_csr(n, torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda(), g.CSR_ADD_SELF_LOOPS)
    assert csr.bin_count[4] == 3 and 0 < g.aggregate_workspace_bytes(csr, f) <= g.STATIC_SCRATCH_BYTES
    row_ptr, col, _ = orc.build_csr(n, src, dst, orc.ADD_SELF_LOOPS)
    out_static = torch.empty((n, f), device="cuda")
    # The first call on a device resolves the built-in array's address (and lets the driver load that part
    # of the library image), as the header says; memory is watched from the second call on.
    g.aggregate_gcn_static(csr, torch.zeros((n, f), device="cuda"), f=f, chunk_width=f, out=out_static)
    torch.cuda.synchronize()
    for call, seed in enumerate((1, 2)):
        # different features on the second call: stale partial sums of the first would show up
        x_host = gg.features_f32(n, f, dist="normal", p0=0.0, p1=1.0, seed=seed)
        x = torch.from_numpy(x_host).cuda()
        oracle_out, oracle_scale = orc.aggregate("gcn", row_ptr, col, x_host, f)
        for width in (f, 16):
            want = g.aggregate_gcn(csr, x, f=f, chunk_width=width)
            out_static.fill_(float("nan"))
            torch.cuda.synchronize()
            free_before, allocated_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
            got = g.aggregate_gcn_static(csr, x, f=f, chunk_width=width, out=out_static)
            torch.cuda.synchronize()
            # the call took no device memory, neither through torch nor behind its back
            assert torch.cuda.memory_allocated() == allocated_before
            assert torch.cuda.mem_get_info()[0] == free_before
            # the same kernels on the same data: bit for bit what the ordinary entry point returns ...
            assert torch.equal(got, want), "call %d width %d" % (call, width)
            # ... and within the library's fp32 bar of the CPU oracle (whose tolerance scale is its own)
            err = np.abs(got.cpu().numpy().astype(np.float64) - oracle_out)
            assert (err <= 1e-5 * oracle_scale + 1e-6).all(), "call %d width %d: max error %g" % (
                call, width, err.max())


def test_static_workspace_rejects_what_does_not_fit():
    import paper_2104_03058_b200 as g
    n, f = 64, 9000
    src, dst = _graph_with_hub_rows(n, 2_200_000, hubs=(3,), seed=5)      # every row is a hub row
    csr = g.build_csr(n, torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda(), 0)
    assert g.aggregate_workspace_bytes(csr, f) > g.STATIC_SCRATCH_BYTES
    x = torch.zeros((n, f), device="cuda")
    out = torch.full((n, f), 7.0, device="cuda")
    before = g.launch_count()
    with pytest.raises(g.GnnfdError) as err:
        g.aggregate_gcn_static(csr, x, f=f, chunk_width=f, out=out)
    assert err.value.status == g.STATIC_SCRATCH_EXCEEDED
    assert "workspace" in str(err.value)
    assert g.launch_count() == before and bool((out == 7.0).all())      # nothing ran
    # a narrower feature matrix on the same graph fits
    f2 = 512
    x2 = x[:, :f2].contiguous() + 1.0
    got = g.aggregate_gcn_static(csr, x2, f=f2, chunk_width=128)
    want = g.aggregate_gcn(csr, x2, f=f2, chunk_width=128)
    assert torch.equal(got, want)
