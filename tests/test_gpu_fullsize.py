"""Full-size parity: config 4 exactly as bench.py launches it (232,965 vertices, ~115M edges,
F = 602 in rows of 608, chunk width 64).  The CSR is compared bit for bit with the oracle's; the
aggregation on sampled rows (every degree class and the hub rows included) element by element, and on
all rows through closed forms that hold at any size."""
import numpy as np
import pytest

import graphgen as gg
import oracle as orc

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def big():
    import paper_2104_03058_b200 as g
    w = gg.config4()
    row_ptr, col, perm = orc.build_csr(w.n, w.src, w.dst, w.flags)
    csr = g.build_csr(w.n, torch.from_numpy(w.src).cuda(), torch.from_numpy(w.dst).cuda(), w.flags)
    return g, w, csr, (row_ptr, col, perm)


def test_config4_csr_bit_exact(big):
    g, w, csr, (row_ptr, col, perm) = big
    assert csr.nnz == len(col) and abs(csr.nnz - w.n - 114_615_892) < 0.02 * 114_615_892
    assert torch.equal(csr.row_ptr.cpu(), torch.from_numpy(row_ptr))
    assert torch.equal(csr.col_idx.cpu(), torch.from_numpy(col))
    assert torch.equal(csr.perm.cpu(), torch.from_numpy(perm))
    assert csr.max_degree == int(np.diff(row_ptr).max()) and csr.bin_count[4] > 1000


def test_config4_gcn_sampled_rows_in_the_bench_configuration(big):
    g, w, csr, (row_ptr, col, _) = big
    deg = np.diff(row_ptr)
    rng = np.random.default_rng(4)
    rows = np.concatenate([rng.choice(w.n, 192, replace=False), np.argsort(deg)[-16:], np.argsort(deg)[:16]])
    rows = np.unique(rows).astype(np.int64)
    want, scale = orc.aggregate("gcn", row_ptr, col, w.x, w.f, rows=rows, threads=orc.max_threads())
    xd = torch.from_numpy(w.x).cuda()
    out = torch.full((w.n, w.ld), float("nan"), device="cuda")
    for width in (64, 128, 602):
        out.fill_(float("nan"))
        g.aggregate_gcn(csr, xd, f=w.f, chunk_width=width, out=out[:, :w.f])
        torch.cuda.synchronize()
        got = out[torch.from_numpy(rows).cuda()][:, :w.f].cpu().numpy()
        err = np.abs(got - want)
        assert (err <= 1e-5 * scale + 1e-6).all(), "width %d: worst %.3e" % (width, (err - 1e-5 * scale).max())
        assert bool(torch.isnan(out[:, w.f:]).all()) and not bool(torch.isnan(out[:, :w.f]).any())


def test_config4_closed_forms_on_every_row(big):
    g, w, csr, (row_ptr, _, _) = big
    deg = np.diff(row_ptr).astype(np.float64)
    # x[u, :] = sqrt(deg u)  =>  GCN out[v, :] = sum_u deg_u^-1/2 deg_v^-1/2 sqrt(deg_u) = sqrt(deg v)
    f = 8
    x = torch.from_numpy(np.repeat(np.sqrt(deg)[:, None], f, axis=1).astype(np.float32)).cuda()
    got = g.aggregate_gcn(csr, x, f=f, chunk_width=4).cpu().numpy()
    np.testing.assert_allclose(got, np.sqrt(deg)[:, None] * np.ones((1, f)), rtol=2e-5)
    # the mean of a constant is the constant
    c = torch.full((w.n, f), 3.25, device="cuda")
    got = g.aggregate_sage(csr, c, f=f, chunk_width=8).cpu().numpy()
    np.testing.assert_allclose(got, 3.25, rtol=2e-5)


def test_config4_tuner_prefers_a_decomposed_sweep(big):
    g, w, csr, _ = big
    xd = torch.from_numpy(w.x).cuda()
    out = torch.empty((w.n, w.ld), device="cuda")
    width, ms = g.tune_chunk_width(csr, xd, "gcn", f=w.f, candidates=[602, 128, 64, 32], out=out[:, :w.f])
    # the slice gathered per sweep must fit L2: the undecomposed sweep (561 MB) and very narrow chunks lose
    assert width in (64, 128) and 5.0 < ms < 60.0


def test_config4_graph_gat_and_sage_hidden64_sampled_rows(big):
    """The paper's GAT / GraphSAGE setting on the Reddit-shaped graph (hidden width 64): sampled rows,
    the hub rows among them, against the oracle; chunk width 8 is the paper's GAT granularity."""
    g, w, csr, (row_ptr, col, _) = big
    deg = np.diff(row_ptr)
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([rng.choice(w.n, 96, replace=False), np.argsort(deg)[-8:]])).astype(np.int64)
    heads, dim = 8, 8
    z = gg.features_f32(w.n, heads * dim, dist="normal", p0=0.0, p1=1.0, seed=1)
    a_src = gg.features_f32(heads, dim, dist="normal", p0=0.0, p1=0.1, seed=1, stream=5)
    a_dst = gg.features_f32(heads, dim, dist="normal", p0=0.0, p1=0.1, seed=1, stream=6)
    zd = torch.from_numpy(z).cuda()
    sel = torch.from_numpy(rows).cuda()
    want, scale = orc.aggregate_gat(row_ptr, col, z, a_src, a_dst, heads, dim, 0.2, rows=rows, threads=orc.max_threads())
    for width in (8, 64):
        got = g.aggregate_gat(csr, zd, torch.from_numpy(a_src).cuda(), torch.from_numpy(a_dst).cuda(), heads, dim, 0.2,
                              chunk_width=width)[sel].cpu().numpy()
        assert (np.abs(got - want) <= 1e-5 * scale + 1e-6).all(), "gat width %d" % width
    want, scale = orc.aggregate("sage", row_ptr, col, z, heads * dim, rows=rows, threads=orc.max_threads())
    for width in (4, 64):
        got = g.aggregate_sage(csr, zd, f=heads * dim, chunk_width=width)[sel].cpu().numpy()
        assert (np.abs(got - want) <= 1e-5 * scale + 1e-6).all(), "sage width %d" % width


def test_config4_graph_edge_softmax_sampled_rows(big):
    """alpha of every slot of sampled rows of the Reddit-shaped graph (8 heads), hub rows and the
    shortest rows among them, against the oracle run on the sub-CSR of those rows; every row's alphas
    sum to one."""
    g, w, csr, (row_ptr, col, _) = big
    deg = np.diff(row_ptr)
    rng = np.random.default_rng(6)
    rows = np.unique(np.concatenate([rng.choice(w.n, 256, replace=False), np.argsort(deg)[-8:],
                                     np.argsort(deg)[:8]])).astype(np.int64)
    heads = 8
    s_src = gg.features_f32(w.n, heads, dist="normal", p0=0.0, p1=1.5, seed=2, stream=5)
    s_dst = gg.features_f32(w.n, heads, dist="normal", p0=0.0, p1=1.5, seed=2, stream=6)
    alpha = g.edge_softmax(csr, torch.from_numpy(s_src).cuda(), torch.from_numpy(s_dst).cuda(), 0.2)
    slots = np.concatenate([np.arange(row_ptr[v], row_ptr[v + 1]) for v in rows])
    sub_ptr = np.concatenate([[0], np.cumsum(deg[rows])]).astype(np.int32)
    want = orc.edge_softmax(sub_ptr, col[slots], s_src.astype(np.float64), s_dst[rows].astype(np.float64), 0.2)
    got = alpha[torch.from_numpy(slots).cuda()].cpu().numpy()
    assert (np.abs(got - want) <= 1e-5 * want + 1e-7).all()
    # row sums over the whole graph: segmented sum of alpha by row on the device, in fp64
    sums = torch.zeros((w.n, heads), dtype=torch.float64, device="cuda")
    row_of_slot = torch.repeat_interleave(torch.arange(w.n, device="cuda"), torch.from_numpy(deg).cuda().long())
    sums.index_add_(0, row_of_slot, alpha.double())
    assert float((sums - 1.0).abs().max()) <= 1e-5


def test_config4_features_combined_to_64_columns_sampled_rows(big):
    """The dense transform ahead of aggregation at the bench's size ([232,965, 602] in rows of 608 times a
    [602, 64] matrix): sampled rows, the last partial row tile among them, against the oracle's tf32
    reading (summation order only) and the exact product (the tf32 bound)."""
    g, w, _, _ = big
    f_out = 64
    w_t = gg.features_f32(f_out, w.ld, dist="normal", p0=0.0, p1=0.05, seed=3, stream=8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    z = g.combine(torch.from_numpy(w.x).cuda()[:, :w.f], torch.from_numpy(w_t).cuda()[:, :w.f], status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rng = np.random.default_rng(7)
    rows = np.unique(np.concatenate([rng.choice(w.n, 2000, replace=False), np.arange(w.n - 130, w.n), np.arange(130)]))
    got = z[torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.float64)
    exact, scale = orc.combine(w.x[rows][:, :w.f], w_t[:, :w.f])
    cut, _ = orc.combine(w.x[rows][:, :w.f], w_t[:, :w.f], tf32=True)
    assert (np.abs(got - cut) <= 1e-5 * scale + 1e-6).all()
    assert (np.abs(got - exact) <= 2.0 ** -9 * scale + 1e-6).all()


def test_config5_full_size_csr_and_bf16_aggregation():
    """Config 5 at its full size (RMAT scale 21, 60M edges, symmetrised + deduplicated + self-loops, bf16
    features of width 64): the CSR bit for bit, the kept-entry count against a direct count of distinct
    off-diagonal pairs, and the aggregation on sampled rows of every degree class."""
    import paper_2104_03058_b200 as g
    w = gg.config5(f=64)
    row_ptr, col, perm = orc.build_csr(w.n, w.src, w.dst, w.flags)
    csr = g.build_csr(w.n, torch.from_numpy(w.src).cuda(), torch.from_numpy(w.dst).cuda(), w.flags)
    assert csr.nnz == len(col)
    assert torch.equal(csr.row_ptr.cpu(), torch.from_numpy(row_ptr))
    assert torch.equal(csr.col_idx.cpu(), torch.from_numpy(col))
    assert torch.equal(csr.perm.cpu(), torch.from_numpy(perm))
    # distinct undirected pairs, both directions, plus one loop per vertex
    a, b = w.src.astype(np.int64), w.dst.astype(np.int64)
    off = a != b
    pairs = np.unique(np.minimum(a[off], b[off]) * w.n + np.maximum(a[off], b[off]))
    assert csr.nnz == 2 * len(pairs) + w.n
    deg = np.diff(row_ptr)
    rng = np.random.default_rng(8)
    rows = np.unique(np.concatenate([rng.choice(w.n, 256, replace=False), np.argsort(deg)[-8:], np.argsort(deg)[:8]]))
    rows = rows.astype(np.int64)
    want, scale = orc.aggregate("gcn", row_ptr, col, w.x, w.f, rows=rows, threads=orc.max_threads())
    xd = torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16)
    sel = torch.from_numpy(rows).cuda()
    for width in (64, 8):
        got = g.aggregate_gcn(csr, xd, f=w.f, chunk_width=width)[sel].cpu().numpy()
        assert (np.abs(got - want) <= 1e-2 * np.abs(want) + 1e-5 * scale + 1e-6).all(), "width %d" % width


def test_config5_full_size_input_width_256():
    """Config 5 at the input width (F = 256 bf16, 1.07 GB of features, the launch `bench.py --workload config5_f256`
    times): sampled rows of every degree class (hub rows are cut at four source ranges on this graph) against the
    oracle, undecomposed and at chunk width 64; a sentinel shows that every output element is written; two runs
    give the same bits."""
    import paper_2104_03058_b200 as g
    w = gg.config5(f=256)
    row_ptr, col, _ = orc.build_csr(w.n, w.src, w.dst, w.flags)
    csr = g.build_csr(w.n, torch.from_numpy(w.src).cuda(), torch.from_numpy(w.dst).cuda(), w.flags)
    assert csr.nnz == len(col) and csr.bin_count[4] > 0
    # the hub rows' segments span several source ranges
    seg_first = csr.col_idx[csr.seg_begin.long()].cpu().numpy() // g.HUB_RANGE_ROWS
    assert len(np.unique(seg_first)) == (w.n + g.HUB_RANGE_ROWS - 1) // g.HUB_RANGE_ROWS == 4
    deg = np.diff(row_ptr)
    rng = np.random.default_rng(9)
    by_class = [np.flatnonzero((deg > lo) & (deg <= hi)) for lo, hi in ((0, 8), (8, 32), (32, 128), (128, 2048), (2048, 1 << 30))]
    rows = np.unique(np.concatenate([rng.choice(c, min(len(c), 48), replace=False) for c in by_class] +
                                    [np.argsort(deg)[-4:]])).astype(np.int64)
    want, scale = orc.aggregate("gcn", row_ptr, col, w.x, w.f, rows=rows, threads=orc.max_threads())
    xd = torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16)
    sel = torch.from_numpy(rows).cuda()
    out = torch.full((w.n, w.f), float("nan"), device="cuda")
    first = None
    for width in (256, 64, 256):
        out.fill_(float("nan"))
        g.aggregate_gcn(csr, xd, f=w.f, chunk_width=width, out=out)
        assert not bool(torch.isnan(out).any()), "width %d left elements unwritten" % width
        got = out[sel].cpu().numpy()
        assert (np.abs(got - want) <= 1e-2 * np.abs(want) + 1e-5 * scale + 1e-6).all(), "width %d" % width
        # the fp32 bar alone holds too: bf16 inputs are widened exactly, only the summation order differs
        assert (np.abs(got - want) <= 1e-5 * scale + 1e-6).all(), "width %d (fp32 bar)" % width
        if width == 256:
            if first is None:
                first = out.clone()
            else:
                assert torch.equal(out, first)
