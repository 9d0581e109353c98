"""Parity of the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs.

Bars: CSR structure bit-exact; fp32 aggregation |gpu - oracle| <= 1e-5 * sum|w x| + 1e-6 per element;
bf16-feature / fp32-accumulate outputs within 1e-2 relative (plus the same absolute terms);
alpha within 1e-5 relative + 1e-7 and rows summing to 1 within 1e-5.
"""
import numpy as np
import pytest

import graphgen as gg
import oracle as orc

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

SL, DD, SY = 1, 2, 4


@pytest.fixture(scope="module")
def g():
    import paper_2104_03058_b200 as lib
    lib.lib()                     # raises if libgnnfd.so is missing: there is no fallback
    return lib


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def to_dev_features(w):
    if w.dtype == "bf16":
        return torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16)
    return dev(w.x)


def assert_close_f32(got, want, scale, what=""):
    err = np.abs(got.astype(np.float64) - want)
    bound = 1e-5 * scale + 1e-6
    bad = err > bound
    assert not bad.any(), "%s: %d elements out of tolerance, worst %.3e vs bound %.3e" % (
        what, bad.sum(), err[bad].max(), bound[bad][np.argmax(err[bad])])


def assert_close_bf16(got, want, scale, what=""):
    err = np.abs(got.astype(np.float64) - want)
    bound = 1e-2 * np.abs(want) + 1e-5 * scale + 1e-6
    assert (err <= bound).all(), "%s: worst excess %.3e" % (what, (err - bound).max())


def check_csr(g, n, src, dst, flags):
    csr = g.build_csr(n, dev(src), dev(dst), flags)
    row_ptr, col, perm = orc.build_csr(n, src, dst, flags)
    assert csr.nnz == len(col)
    np.testing.assert_array_equal(csr.row_ptr.cpu().numpy(), row_ptr)
    np.testing.assert_array_equal(csr.col_idx.cpu().numpy(), col)
    np.testing.assert_array_equal(csr.perm.cpu().numpy(), perm)
    deg, dinv, rdeg = orc.degree_norm(row_ptr)
    assert csr.max_degree == (deg.max() if n else 0)
    np.testing.assert_array_equal(csr.dinv_sqrt.cpu().numpy(), dinv.astype(np.float32))
    np.testing.assert_array_equal(csr.rdeg.cpu().numpy(), rdeg.astype(np.float32))
    rows = np.repeat(np.arange(n), deg)
    d32 = dinv.astype(np.float32)
    np.testing.assert_array_equal(csr.edge_weight.cpu().numpy(), d32[col] * d32[rows])
    check_schedule(g, csr, deg)
    return csr, (row_ptr, col, perm)


def degree_class(deg, hub_degree):
    """Fine degree classes of the launch schedule: exact degree up to 8, quarter octaves of deg - 1 up to
    the hub threshold, one class for hub rows (restated from the header's description)."""
    deg = np.asarray(deg, np.int64)
    t = np.maximum(deg - 1, 8)
    o = np.floor(np.log2(t)).astype(np.int64)
    mid = 9 + (o - 3) * 4 + ((t >> (o - 2)) & 3)
    return np.where(deg <= 8, deg, np.where(deg > hub_degree, 41, mid))


def check_schedule(g, csr, deg):
    order = csr.row_order.cpu().numpy()
    n = len(deg)
    assert sorted(order.tolist()) == list(range(n))
    bounds = [8, 32, 128, g.HUB_DEGREE]
    bins = np.searchsorted(bounds, deg, side="left")          # first bound >= deg; 4 = hub
    cls = degree_class(deg, g.HUB_DEGREE)
    start = 0
    for b in range(5):
        part = order[start:start + csr.bin_count[b]]
        assert (bins[part] == b).all()
        start += csr.bin_count[b]
    assert start == n
    # rows are ordered by (class, row id)
    key = cls[order] * (n + 1) + order
    assert (np.diff(key) > 0).all()
    hubs = order[n - csr.bin_count[4]:]
    seg_ptr = csr.hub_seg_ptr.cpu().numpy()
    seg_row = csr.seg_row.cpu().numpy()
    seg_begin = csr.seg_begin.cpu().numpy()
    seg_end = csr.seg_end.cpu().numpy()
    seg_slot = csr.seg_slot.cpu().numpy()
    row_ptr = csr.row_ptr.cpu().numpy()
    col = csr.col_idx.cpu().numpy()
    assert seg_ptr[0] == 0 and seg_ptr[-1] == csr.n_segments
    assert sorted(seg_slot.tolist()) == list(range(csr.n_segments))          # every slot is scheduled exactly once
    # source ranges: GNNFD_HUB_RANGE_ROWS ids, doubled until at most 64 cover the graph
    width = g.HUB_RANGE_ROWS
    while (n + width - 1) // width > 64:
        width *= 2
    by_slot = np.argsort(seg_slot)                                # schedule position of slot s
    for i, v in enumerate(hubs):
        pos = by_slot[seg_ptr[i]:seg_ptr[i + 1]]                  # the row's segments in slot order
        assert (seg_row[pos] == v).all()
        b, e = seg_begin[pos], seg_end[pos]
        # in slot order the segments tile the row: ascending, gap-free, none empty, none above the segment size
        assert b[0] == row_ptr[v] and e[-1] == row_ptr[v + 1] and (b[1:] == e[:-1]).all()
        assert ((e - b) > 0).all() and ((e - b) <= g.HUB_SEGMENT).all()
        # a segment stays inside one source range, and a range's piece of the row is cut into as few segments as fit
        r_first, r_last = col[b] // width, col[e - 1] // width
        assert (r_first == r_last).all()
        for r in np.unique(r_first):
            piece = (e - b)[r_first == r]
            assert len(piece) == (piece.sum() + g.HUB_SEGMENT - 1) // g.HUB_SEGMENT
    # launch order: range by range, inside a range hub row by hub row (in row_order), inside a row ascending
    if csr.n_segments:
        hub_index = {int(v): i for i, v in enumerate(hubs)}
        key = [(int(col[seg_begin[p]]) // width, hub_index[int(seg_row[p])], int(seg_begin[p])) for p in range(csr.n_segments)]
        assert key == sorted(key)


# ------------------------------------------------------------------ CSR build

@pytest.mark.parametrize("flags", [0, SL, DD, SY, SL | DD, SY | DD | SL])
@pytest.mark.parametrize("n,e", [(50, 400), (1000, 30_011), (70_000, 9_000)])
def test_csr_bit_exact_multigraph(g, flags, n, e):
    src, dst = gg.uniform_graph(n, e, seed=n + flags)
    check_csr(g, n, src, dst, flags)


def test_csr_int64_ids_and_hub_rows(g):
    n = 3000
    src, dst = gg.uniform_graph(n, 40_000, seed=3)
    dst[:9000] = 7                      # one row above the hub threshold, with duplicates
    dst[9000:12_500] = 11
    csr, _ = check_csr(g, n, src.astype(np.int64), dst.astype(np.int64), SL)
    assert csr.bin_count[4] == 2 and csr.n_segments >= 6


def test_csr_degenerate_inputs(g):
    empty = np.zeros(0, np.int32)
    check_csr(g, 1, empty, empty, 0)
    check_csr(g, 5, empty, empty, SL)
    check_csr(g, 1, np.zeros(3, np.int32), np.zeros(3, np.int32), DD)
    check_csr(g, 2, np.array([0, 1, 1], np.int32), np.array([1, 0, 0], np.int32), SY | DD)


def test_csr_rejects_bad_ids_without_fault(g):
    src = np.array([0, 9, 2], np.int32)
    dst = np.array([1, 2, -4], np.int32)
    with pytest.raises(g.GnnfdError) as err:
        g.build_csr(5, dev(src), dev(dst), 0)
    assert err.value.status == g.BAD_INDEX
    # the context is still usable
    check_csr(g, 5, np.array([0, 4], np.int32), np.array([1, 2], np.int32), 0)


def test_workspace_too_small_and_invalid_args(g):
    src, dst = gg.uniform_graph(100, 1000, seed=1)
    pb, sb = g.csr_workspace_bytes(100, 1000, 0)
    small = torch.empty(pb // 2, dtype=torch.uint8, device="cuda")
    with pytest.raises(g.GnnfdError) as err:
        g.build_csr(100, dev(src), dev(dst), 0, persistent=small)
    assert err.value.status == g.WORKSPACE_TOO_SMALL
    csr = g.build_csr(100, dev(src), dev(dst), 0)
    x = torch.zeros((100, 8), device="cuda")
    with pytest.raises(g.GnnfdError) as err:
        g.aggregate_gcn(csr, x, f=8, chunk_width=0)
    assert err.value.status == g.INVALID_ARG
    with pytest.raises(g.GnnfdError):
        g.csr_workspace_bytes(0, 10, 0)
    with pytest.raises(g.GnnfdError) as err:
        g.csr_workspace_bytes(10, 2 ** 31, 0)
    assert err.value.status == g.TOO_LARGE


# ------------------------------------------------------------------ GCN / SAGE

def run_model(g, w, csr, xd, width, out_dtype=None):
    fn = g.aggregate_gcn if w.model == "gcn" else g.aggregate_sage
    out = fn(csr, xd, f=w.f, chunk_width=width, out_dtype=out_dtype)
    torch.cuda.synchronize()
    return out


def check_workload(g, w, widths=None, rows=None):
    csr, (row_ptr, col, _) = check_csr(g, w.n, w.src, w.dst, w.flags)
    xd = to_dev_features(w)
    want, scale = orc.aggregate(w.model, row_ptr, col, w.x, w.f, rows=rows, threads=orc.max_threads())
    for width in widths or w.chunk_widths:
        got = run_model(g, w, csr, xd, width).cpu().numpy()
        assert got.shape == (w.n, w.f)
        if rows is not None:
            got = got[rows]
        (assert_close_bf16 if w.dtype == "bf16" else assert_close_f32)(got, want, scale, "%s width %d" % (w.name, width))
    return csr


def test_config1_gcn(g):
    w = gg.config1()
    check_workload(g, w, widths=(4, 8, 16, 1, 3, 5, 100))


def test_config2_sage(g):
    w = gg.config2()
    check_workload(g, w)


def test_config4_scaled_gcn_with_hub_rows_and_padding(g):
    w = gg.scaled("config4", 0.05)
    w.x[:, w.f:] = np.nan                      # padding columns must never reach a result
    csr = check_workload(g, w, widths=(32, 64, 128, 602, 7))
    assert csr.bin_count[4] > 0, "the scaled workload should still contain hub rows"


@pytest.mark.parametrize("f", [256, 8, 16, 32, 64])
def test_config5_scaled_gcn_bf16(g, f):
    w = gg.scaled("config5_f%d" % f, 1.0 / 64)
    check_workload(g, w, widths=w.chunk_widths + (4,))


def test_bf16_output_and_sage_on_bf16(g):
    w = gg.scaled("config5_f64", 1.0 / 256)
    row_ptr, col, _ = orc.build_csr(w.n, w.src, w.dst, w.flags)
    csr = g.build_csr(w.n, dev(w.src), dev(w.dst), w.flags)
    xd = to_dev_features(w)
    for model, fn in (("gcn", g.aggregate_gcn), ("sage", g.aggregate_sage)):
        want, scale = orc.aggregate(model, row_ptr, col, w.x, w.f)
        out = fn(csr, xd, f=w.f, chunk_width=16, out_dtype=torch.bfloat16)
        assert out.dtype == torch.bfloat16
        got = out.float().cpu().numpy()
        err = np.abs(got - want)
        assert (err <= 2.0 ** -8 * np.abs(want) + 1e-2 * np.abs(want) + 1e-5 * scale + 1e-6).all()


@pytest.mark.parametrize("model", ["gcn", "sage"])
def test_unaligned_layouts_take_the_narrow_path(g, model):
    n, f = 5000, 13
    src, dst = gg.powerlaw_graph(n, 60_000, 2.1, None, 4)
    x = gg.features_f32(n, f + 1, dist="normal", p0=0, p1=1, seed=4)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    csr = g.build_csr(n, dev(src), dev(dst), SL)
    xd = dev(x)
    view = xd[:, 1:]                            # 4-byte aligned base, odd leading dimension
    ref = np.ascontiguousarray(x[:, 1:])
    want, scale = orc.aggregate(model, row_ptr, col, ref, f)
    fn = g.aggregate_gcn if model == "gcn" else g.aggregate_sage
    out_buf = torch.full((n, f + 2), -5.0, device="cuda")
    for width in (13, 4, 8, 1):
        out = fn(csr, view, f=f, chunk_width=width, out=out_buf[:, 1:f + 1])
        got = out.cpu().numpy()
        assert_close_f32(got, want, scale, "%s unaligned width %d" % (model, width))
        assert (out_buf[:, 0] == -5.0).all() and (out_buf[:, f + 1] == -5.0).all()


def test_results_are_bit_identical_from_run_to_run(g):
    w = gg.scaled("config4", 0.03)
    csr = g.build_csr(w.n, dev(w.src), dev(w.dst), w.flags)
    csr2 = g.build_csr(w.n, dev(w.src), dev(w.dst), w.flags)
    assert torch.equal(csr.col_idx, csr2.col_idx) and torch.equal(csr.perm, csr2.perm)
    xd = to_dev_features(w)
    a = g.aggregate_gcn(csr, xd, f=w.f, chunk_width=64)
    b = g.aggregate_gcn(csr2, xd, f=w.f, chunk_width=64)
    assert torch.equal(a, b)


def test_launch_counter_and_kernel_timing(g):
    w = gg.config1()
    before = g.launch_count()
    csr = g.build_csr(w.n, dev(w.src), dev(w.dst), w.flags)
    g.kernel_timing_enable(True)
    try:
        g.aggregate_gcn(csr, dev(w.x), f=w.f, chunk_width=8)
        torch.cuda.synchronize()
        timing = g.kernel_timing_read()
    finally:
        g.kernel_timing_enable(False)
    assert g.launch_count() > before
    assert "gather_aggregate_gcn" in timing and timing["gather_aggregate_gcn"][1] == 1
    assert timing["gather_aggregate_gcn"][0] > 0


# ------------------------------------------------------------------ GAT

def test_config3_gat_and_edge_softmax(g):
    w = gg.config3()
    csr, (row_ptr, col, _) = check_csr(g, w.n, w.src, w.dst, w.flags)
    zd = dev(w.x)
    a_src, a_dst = dev(w.a_src), dev(w.a_dst)
    threads = orc.max_threads()
    want, scale = orc.aggregate_gat(row_ptr, col, w.x, w.a_src, w.a_dst, w.heads, w.dim, w.negative_slope,
                                    threads=threads)
    for width in (8, 64, 16, 4, 24):
        got = g.aggregate_gat(csr, zd, a_src, a_dst, w.heads, w.dim, w.negative_slope, chunk_width=width)
        assert_close_f32(got.cpu().numpy(), want, scale, "gat width %d" % width)
    # scores and the materialised softmax
    s_src, s_dst = g.gat_scores(zd, a_src, a_dst, w.heads, w.dim)
    o_src, o_dst = orc.gat_scores(w.x, w.a_src, w.a_dst, w.heads, w.dim)
    zz = np.abs(w.x.astype(np.float64)).reshape(w.n, w.heads, w.dim)
    s_scale = np.einsum("nhd,hd->nh", zz, np.abs(w.a_src.astype(np.float64)))
    assert_close_f32(s_src.cpu().numpy(), o_src, s_scale, "s_src")
    d_scale = np.einsum("nhd,hd->nh", zz, np.abs(w.a_dst.astype(np.float64)))
    assert_close_f32(s_dst.cpu().numpy(), o_dst, d_scale, "s_dst")
    assert np.abs(o_src - o_dst).max() > 1e-2          # the two score sets differ, so a mix-up would show
    alpha = g.edge_softmax(csr, s_src, s_dst, w.negative_slope).cpu().numpy()
    want_alpha = orc.edge_softmax(row_ptr, col, s_src.cpu().numpy(), s_dst.cpu().numpy(), w.negative_slope)
    assert (np.abs(alpha - want_alpha) <= 1e-5 * want_alpha + 1e-7).all()
    sums = np.add.reduceat(alpha.astype(np.float64), row_ptr[:-1], axis=0)
    assert np.abs(sums - 1.0).max() <= 1e-5


@pytest.mark.parametrize("heads,dim", [(3, 5), (1, 7), (4, 4), (2, 64)])
def test_gat_general_shapes_with_hub_rows(g, heads, dim):
    n = 6000
    src, dst = gg.powerlaw_graph(n, 90_000, 2.1, None, heads)
    dst[:5000] = 17                     # guarantees a row above the hub threshold
    f = heads * dim
    z = gg.features_f32(n, f, dist="normal", p0=0, p1=1, seed=heads)
    a_src = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.3, seed=heads, stream=5)
    a_dst = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.3, seed=heads, stream=6)
    csr, (row_ptr, col, _) = check_csr(g, n, src, dst, SL)
    assert csr.bin_count[4] > 0
    want, scale = orc.aggregate_gat(row_ptr, col, z, a_src, a_dst, heads, dim, 0.2, threads=orc.max_threads())
    for width in sorted({f, dim, 4, 3}):
        got = g.aggregate_gat(csr, dev(z), dev(a_src), dev(a_dst), heads, dim, 0.2, chunk_width=width)
        assert_close_f32(got.cpu().numpy(), want, scale, "gat %dx%d width %d" % (heads, dim, width))
    s_src, s_dst = g.gat_scores(dev(z), dev(a_src), dev(a_dst), heads, dim)
    alpha = g.edge_softmax(csr, s_src, s_dst, 0.2).cpu().numpy()
    want_alpha = orc.edge_softmax(row_ptr, col, s_src.cpu().numpy(), s_dst.cpu().numpy(), 0.2)
    assert (np.abs(alpha - want_alpha) <= 1e-5 * want_alpha + 1e-7).all()


def test_hub_rows_cut_at_source_ranges(g):
    """More vertices than one source range holds: hub rows are cut at the range boundaries and their pieces are
    launched range by range; partial results still combine per row in ascending source order."""
    n = 3 * g.HUB_RANGE_ROWS + 1234                   # four source ranges, the last one nearly empty
    src, dst = gg.uniform_graph(n, 400_000, seed=12)
    rng = np.random.default_rng(12)
    for i, (v, k) in enumerate(((5, 9000), (n - 1, 2500), (70_000, 3000))):
        dst[i * 10_000:i * 10_000 + k] = v            # hub rows whose sources fall in every range
    src[25_000:28_000] = rng.integers(0, 40_000, 3000)          # ... and one whose sources all lie in range 0
    dst[25_000:28_000] = 99_999
    csr, (row_ptr, col, _) = check_csr(g, n, src, dst, SL)
    assert csr.bin_count[4] == 4 and csr.n_segments > 4 * 3
    f, heads, dim = 16, 2, 8
    x = gg.features_f32(n, f, dist="normal", p0=0, p1=1, seed=12)
    threads = orc.max_threads()
    for model, fn in (("gcn", g.aggregate_gcn), ("sage", g.aggregate_sage)):
        want, scale = orc.aggregate(model, row_ptr, col, x, f, threads=threads)
        for width in (f, 4):
            assert_close_f32(fn(csr, dev(x), f=f, chunk_width=width).cpu().numpy(), want, scale, model)
    a_src = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.3, seed=12, stream=5)
    a_dst = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.3, seed=12, stream=6)
    want, scale = orc.aggregate_gat(row_ptr, col, x, a_src, a_dst, heads, dim, 0.2, threads=threads)
    got = g.aggregate_gat(csr, dev(x), dev(a_src), dev(a_dst), heads, dim, 0.2, chunk_width=8)
    assert_close_f32(got.cpu().numpy(), want, scale, "gat")
    s_src, s_dst = g.gat_scores(dev(x), dev(a_src), dev(a_dst), heads, dim)
    alpha = g.edge_softmax(csr, s_src, s_dst, 0.2).cpu().numpy()
    want_alpha = orc.edge_softmax(row_ptr, col, s_src.cpu().numpy(), s_dst.cpu().numpy(), 0.2)
    assert (np.abs(alpha - want_alpha) <= 1e-5 * want_alpha + 1e-7).all()


def test_gat_bf16_features(g):
    n, heads, dim = 4000, 4, 8
    src, dst = gg.powerlaw_graph(n, 50_000, 2.1, None, 9)
    bits = gg.to_bf16_bits(gg.features_f32(n, heads * dim, dist="normal", p0=0, p1=1, seed=9))
    a_src = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.1, seed=9, stream=5)
    a_dst = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.1, seed=9, stream=6)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    csr = g.build_csr(n, dev(src), dev(dst), SL)
    zd = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    want, scale = orc.aggregate_gat(row_ptr, col, bits, a_src, a_dst, heads, dim, 0.2)
    for width in (8, 32, 2):
        got = g.aggregate_gat(csr, zd, dev(a_src), dev(a_dst), heads, dim, 0.2, chunk_width=width)
        assert_close_bf16(got.cpu().numpy(), want, scale, "gat bf16 width %d" % width)


# ------------------------------------------------------------------ host-buffer front end

def test_host_pipeline_matches_direct_calls(g):
    from paper_2104_03058_b200.host import HostPipeline
    n, f, ld = 3000, 20, 24
    jobs = []
    for seed in range(4):
        src, dst = gg.powerlaw_graph(n, 30_000, 2.1, None, seed)
        x = gg.features_f32(n, f, ld=ld, dist="normal", p0=0, p1=1, seed=seed)
        jobs.append((torch.from_numpy(src).pin_memory(), torch.from_numpy(dst).pin_memory(),
                     torch.from_numpy(x).pin_memory()))
    max_e = max(j[0].numel() for j in jobs)
    pipe = HostPipeline(n, max_e, f, ld, SL, 8)
    outs = [torch.zeros((n, ld)).pin_memory() for _ in jobs]
    for i, job in enumerate(jobs):
        pipe.submit(*job, outs[i], next_job=jobs[i + 1] if i + 1 < len(jobs) else None)
    pipe.finish()
    torch.cuda.synchronize()
    for (h_src, h_dst, h_x), out in zip(jobs, outs):
        csr = g.build_csr(n, h_src.cuda(), h_dst.cuda(), SL)
        want = g.aggregate_gcn(csr, h_x.cuda(), f=f, chunk_width=8)
        assert torch.equal(out[:, :f], want.cpu())


def test_host_pipeline_grows_its_workspace_for_a_graph_with_more_hub_rows(g):
    from paper_2104_03058_b200.host import HostPipeline
    n, f, e = 3000, 12, 40_000
    jobs = []
    for hubs in ((), (5,), (7, 1200, 2999)):                 # 0, 1 and 3 rows above the hub threshold
        src, dst = gg.uniform_graph(n, e, seed=len(hubs))
        for i, v in enumerate(hubs):
            dst[i * 5000:(i + 1) * 5000] = v
        x = gg.features_f32(n, f, dist="normal", p0=0, p1=1, seed=len(hubs))
        jobs.append((torch.from_numpy(src).pin_memory(), torch.from_numpy(dst).pin_memory(),
                     torch.from_numpy(x).pin_memory()))
    pipe = HostPipeline(n, e, f, f, 0, 4)
    outs = [torch.zeros((n, f)).pin_memory() for _ in jobs]
    for i, job in enumerate(jobs):
        csr = pipe.submit(*job, outs[i])
        assert csr.bin_count[4] == (0, 1, 3)[i]
    pipe.finish()
    torch.cuda.synchronize()
    for (h_src, h_dst, h_x), out in zip(jobs, outs):
        csr = g.build_csr(n, h_src.cuda(), h_dst.cuda(), 0)
        assert torch.equal(out, g.aggregate_gcn(csr, h_x.cuda(), f=f, chunk_width=4).cpu())


def test_binding_refuses_bad_operands_before_any_launch(g):
    n, f = 500, 8
    src, dst = gg.uniform_graph(n, 4000, seed=3)
    csr = g.build_csr(n, dev(src), dev(dst), SL)
    x = torch.zeros((n, f), device="cuda")
    out = torch.zeros((n, f), device="cuda")
    a = torch.zeros((2, 4), device="cuda")
    s = torch.zeros((n, 2), device="cuda")
    before = g.launch_count()
    for call in (lambda: g.aggregate_gcn(csr, x[:n - 1], f=f, out=out),            # x too short
                 lambda: g.aggregate_sage(csr, x, f=f, out=out[:10]),               # out too short
                 lambda: g.aggregate_gcn(csr, x, f=f, out=x),                       # in place
                 lambda: g.aggregate_gcn(csr, x.cpu(), f=f),                        # wrong device
                 lambda: g.aggregate_gat(csr, x[:100], a, a, 2, 4, out=out),        # z too short
                 lambda: g.aggregate_gat(csr, x, a[:1], a, 2, 4, out=out),          # attention vector too short
                 lambda: g.edge_softmax(csr, s[:n - 3], s[:n - 3]),                 # scores too short
                 lambda: g.edge_softmax(csr, s, s, out=torch.zeros((csr.nnz - 1, 2), device="cuda")),
                 lambda: g.aggregate_gcn_static(csr, x[:n - 1], f=f, out=out)):
        with pytest.raises(ValueError):
            call()
    assert g.launch_count() == before
    # a non-default stream: scratch and temporaries are taken under that stream
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    x.normal_()
    torch.cuda.synchronize()
    want = g.aggregate_gcn(csr, x, f=f)
    got = g.aggregate_gcn(csr, x, f=f, stream=side)
    side.synchronize()
    assert torch.equal(got, want)


def test_chunk_width_tuner_picks_a_candidate_and_leaves_a_valid_result(g):
    w = gg.scaled("config4", 0.05)
    row_ptr, col, _ = orc.build_csr(w.n, w.src, w.dst, w.flags)
    csr = g.build_csr(w.n, dev(w.src), dev(w.dst), w.flags)
    xd = dev(w.x)
    out = torch.empty((w.n, w.f), device="cuda")
    cands = g.default_chunk_candidates(w.f)
    width, ms = g.tune_chunk_width(csr, xd, "gcn", f=w.f, candidates=cands, out=out)
    assert width in cands and ms > 0
    want, scale = orc.aggregate("gcn", row_ptr, col, w.x, w.f, threads=orc.max_threads())
    assert_close_f32(out.cpu().numpy(), want, scale, "tuner leaves the last candidate's result")
    width_sage, _ = g.tune_chunk_width(csr, xd, "sage", f=w.f, candidates=[64, 602])
    assert width_sage in (64, 602)
    with pytest.raises(g.GnnfdError):
        g.tune_chunk_width(csr, xd, "gcn", f=w.f, candidates=[0])


# ------------------------------------------------------------------ degenerate shapes

def test_degenerate_shapes(g):
    # a single vertex with a self-loop, one feature column
    one = np.zeros(1, np.int32)
    csr = g.build_csr(1, dev(one), dev(one), 0)
    x = torch.tensor([[2.5]], device="cuda")
    assert g.aggregate_gcn(csr, x, f=1, chunk_width=1).item() == 2.5
    assert g.aggregate_sage(csr, x, f=1, chunk_width=7).item() == 2.5
    # no edges at all: every row is empty and the output is zero, not stale memory
    empty = np.zeros(0, np.int32)
    csr = g.build_csr(9, dev(empty), dev(empty), 0)
    out = torch.full((9, 5), 3.0, device="cuda")
    g.aggregate_gcn(csr, torch.ones((9, 5), device="cuda"), f=5, chunk_width=2, out=out)
    assert bool((out == 0).all())
    a = torch.ones((1, 5), device="cuda")
    out.fill_(3.0)
    g.aggregate_gat(csr, torch.ones((9, 5), device="cuda"), a, a, 1, 5, 0.2, chunk_width=5, out=out)
    assert bool((out == 0).all())
    assert g.edge_softmax(csr, torch.zeros((9, 2), device="cuda"), torch.zeros((9, 2), device="cuda")).shape == (0, 2)


@pytest.mark.parametrize("width", [1, 2, 5])
def test_chunk_width_one_and_odd_widths(g, width):
    n, f = 2000, 5
    src, dst = gg.powerlaw_graph(n, 20_000, 2.1, None, 11)
    x = gg.features_f32(n, f, dist="normal", p0=0, p1=1, seed=11)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    csr = g.build_csr(n, dev(src), dev(dst), SL)
    for model, fn in (("gcn", g.aggregate_gcn), ("sage", g.aggregate_sage)):
        want, scale = orc.aggregate(model, row_ptr, col, x, f)
        assert_close_f32(fn(csr, dev(x), f=f, chunk_width=width).cpu().numpy(), want, scale, "%s width %d" % (model, width))


@pytest.mark.parametrize("heads,dim", [(40, 2), (6, 1), (33, 4)])
def test_gat_many_and_odd_head_counts(g, heads, dim):
    n = 3000
    src, dst = gg.powerlaw_graph(n, 40_000, 2.1, None, heads)
    dst[:2500] = 9                      # a hub row
    f = heads * dim
    z = gg.features_f32(n, f, dist="normal", p0=0, p1=1, seed=heads)
    a_src = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.3, seed=heads, stream=5)
    a_dst = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.3, seed=heads, stream=6)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    csr = g.build_csr(n, dev(src), dev(dst), SL)
    want, scale = orc.aggregate_gat(row_ptr, col, z, a_src, a_dst, heads, dim, 0.2, threads=orc.max_threads())
    for width in (f, 8):
        got = g.aggregate_gat(csr, dev(z), dev(a_src), dev(a_dst), heads, dim, 0.2, chunk_width=width)
        assert_close_f32(got.cpu().numpy(), want, scale, "gat %dx%d width %d" % (heads, dim, width))
    s_src, s_dst = g.gat_scores(dev(z), dev(a_src), dev(a_dst), heads, dim)
    alpha = g.edge_softmax(csr, s_src, s_dst, 0.2).cpu().numpy()
    want_alpha = orc.edge_softmax(row_ptr, col, s_src.cpu().numpy(), s_dst.cpu().numpy(), 0.2)
    assert (np.abs(alpha - want_alpha) <= 1e-5 * want_alpha + 1e-7).all()


def test_more_chunks_than_one_launch_covers(g):
    """70,000 decomposition layers of one column each: a launch covers at most 65,535 chunks (grid y), so the
    aggregation goes out as two launches; every column must still come back right."""
    n, f = 40, 70_000
    src, dst = gg.uniform_graph(n, 200, seed=8)
    x = gg.features_f32(n, f, dist="normal", p0=0, p1=1, seed=8)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    csr = g.build_csr(n, dev(src), dev(dst), SL)
    before = g.launch_count()
    want, scale = orc.aggregate("gcn", row_ptr, col, x, f)
    got = g.aggregate_gcn(csr, dev(x), f=f, chunk_width=1)
    assert g.launch_count() - before == 2
    assert_close_f32(got.cpu().numpy(), want, scale, "gcn, 70,000 chunks")
    heads, dim = f // 8, 8
    a_src = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.3, seed=8, stream=5)
    a_dst = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.3, seed=8, stream=6)
    want, scale = orc.aggregate_gat(row_ptr, col, x, a_src, a_dst, heads, dim, 0.2)
    got = g.aggregate_gat(csr, dev(x), dev(a_src), dev(a_dst), heads, dim, 0.2, chunk_width=1)
    assert_close_f32(got.cpu().numpy(), want, scale, "gat, 70,000 chunks")


def test_int64_ids_beyond_int32_are_rejected(g):
    src = torch.tensor([0, 2 ** 31 + 5], dtype=torch.int64, device="cuda")
    dst = torch.tensor([1, 2], dtype=torch.int64, device="cuda")
    with pytest.raises(g.GnnfdError) as err:
        g.build_csr(10, src, dst, 0)
    assert err.value.status == g.BAD_INDEX


# ------------------------------------------------------------------ sort boundaries

@pytest.mark.parametrize("n,e,flags", [
    (4096, 4096, 0), (4097, 8191, DD), (255, 4095, SL | DD), (256, 4097, SY), (257, 12288, SY | DD | SL),
    (1, 5000, DD), (2, 4096 * 3 + 1, 0), (513, 511, SL),
    ((1 << 20) + 1, 3000, DD),            # 21 + 21 key bits, values packed beside them
    (1 << 22, 4000, SY),                  # 22 + 23 key bits, still one word
    (1 << 27, 2000, DD),                  # 27 + 28 key bits: keys and values travel separately
])
def test_csr_sort_boundaries(g, n, e, flags):
    src, dst = gg.uniform_graph(n, e, seed=n % 1000 + e)
    if n > 4:
        dst[: e // 3] = dst[0]            # a long run of equal destinations, with duplicates of (dst, src)
        src[: e // 6] = src[0]
    csr = g.build_csr(n, dev(src), dev(dst), flags)
    row_ptr, col, perm = orc.build_csr(n, src, dst, flags)
    assert csr.nnz == len(col)
    assert torch.equal(csr.row_ptr.cpu(), torch.from_numpy(row_ptr))
    assert torch.equal(csr.col_idx.cpu(), torch.from_numpy(col))
    assert torch.equal(csr.perm.cpu(), torch.from_numpy(perm))
    assert sum(csr.bin_count) == n



@pytest.mark.parametrize("f,width", [(64, 64), (130, 128), (20, 5), (8, 8)])
def test_long_runs_of_equal_terms_stay_inside_the_tolerance(g, f, width):
    """A hub row fed thousands of times by the same source with same-sign features: every addition of a
    plain fp32 chain then rounds in the same direction, so the error grows with the chain length.  The
    kernels sum in two levels; the row must still meet the per-element bound."""
    n, e = 3000, 60_000
    rng = np.random.default_rng(f)
    src = rng.integers(0, n, size=e).astype(np.int32)
    dst = rng.integers(0, n, size=e).astype(np.int32)
    dst[: e // 2] = 7                      # one row of ~30,000 entries ...
    src[: e // 3] = 11                     # ... two thirds of them copies of one edge
    x = (np.abs(gg.features_f32(n, f, dist="normal", p0=0, p1=1, seed=f)) + 0.5).astype(np.float32)
    row_ptr, col, _ = orc.build_csr(n, src, dst, 0)
    csr = g.build_csr(n, dev(src), dev(dst), 0)
    for model, fn in (("gcn", g.aggregate_gcn), ("sage", g.aggregate_sage)):
        want, scale = orc.aggregate(model, row_ptr, col, x, f)
        assert_close_f32(fn(csr, dev(x), f=f, chunk_width=width).cpu().numpy(), want, scale, "%s f %d" % (model, f))
    if f % 8 == 0:
        heads, dim = f // 8, 8
        a_src = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.2, seed=f, stream=5)
        a_dst = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.2, seed=f, stream=6)
        want, scale = orc.aggregate_gat(row_ptr, col, x, a_src, a_dst, heads, dim, 0.2)
        got = g.aggregate_gat(csr, dev(x), dev(a_src), dev(a_dst), heads, dim, 0.2, chunk_width=width)
        assert_close_f32(got.cpu().numpy(), want, scale, "gat f %d" % f)


def test_one_row_of_two_million_entries(g):
    """Nearly 2,000 hub segments in one row: the per-row merges of the segment results (sums, softmax
    denominators) must not become long fp32 chains either."""
    n, e, f = 100, 2_000_000, 8
    rng = np.random.default_rng(5)
    src = rng.integers(0, n, size=e).astype(np.int32)
    dst = np.full(e, 7, np.int32)
    dst[:1000] = rng.integers(0, n, size=1000)
    x = (np.abs(gg.features_f32(n, f, dist="normal", p0=0, p1=1, seed=5)) + 0.5).astype(np.float32)
    row_ptr, col, _ = orc.build_csr(n, src, dst, 0)
    csr = g.build_csr(n, dev(src), dev(dst), 0)
    assert csr.max_degree > 1_990_000
    for model, fn in (("gcn", g.aggregate_gcn), ("sage", g.aggregate_sage)):
        want, scale = orc.aggregate(model, row_ptr, col, x, f)
        assert_close_f32(fn(csr, dev(x), f=f, chunk_width=f).cpu().numpy(), want, scale, model)
    a_src = gg.features_f32(1, f, dist="normal", p0=0, p1=0.2, seed=5, stream=5)
    a_dst = gg.features_f32(1, f, dist="normal", p0=0, p1=0.2, seed=5, stream=6)
    want, scale = orc.aggregate_gat(row_ptr, col, x, a_src, a_dst, 1, f, 0.2)
    got = g.aggregate_gat(csr, dev(x), dev(a_src), dev(a_dst), 1, f, 0.2, chunk_width=f)
    assert_close_f32(got.cpu().numpy(), want, scale, "gat")
    s_src, s_dst = g.gat_scores(dev(x), dev(a_src), dev(a_dst), 1, f)
    alpha = g.edge_softmax(csr, s_src, s_dst, 0.2).cpu().numpy()
    want_alpha = orc.edge_softmax(row_ptr, col, s_src.cpu().numpy(), s_dst.cpu().numpy(), 0.2)
    assert (np.abs(alpha - want_alpha) <= 1e-5 * want_alpha + 1e-7).all()
    sums = np.add.reduceat(alpha.astype(np.float64), row_ptr[:-1][np.diff(row_ptr) > 0], axis=0)
    assert np.abs(sums - 1.0).max() <= 1e-5
