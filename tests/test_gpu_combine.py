"""Combination ahead of aggregation (gnnfd_combine, tf32 tensor-core product) against the fp64 oracle.

Two bars.  Against the exact product: |z - exact| <= 2^-9 * sum|x w| + 1e-6, the bound that follows from
cutting both operands to tf32.  Against the oracle's tf32 reading (operands cut to 10 mantissa bits, exact
products, fp64 sums) only the fp32 summation order differs, so the aggregation tolerance
1e-5 * sum|x w| + 1e-6 applies; a wrong tile, a swapped operand or a missed K slice fails it by orders of
magnitude."""
import numpy as np
import pytest

import graphgen as gg
import oracle as orc

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def g():
    import paper_2104_03058_b200 as g
    g.lib()
    return g


def run_combine(g, x, w_t, f_in):
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((x.shape[0], w_t.shape[0]), float("nan"), device="cuda")
    g.combine(torch.from_numpy(x).cuda()[:, :f_in], torch.from_numpy(w_t).cuda()[:, :f_in], out=out, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out.cpu().numpy().astype(np.float64)


def check(got, x, w_t):
    exact, scale = orc.combine(x, w_t)
    cut, _ = orc.combine(x, w_t, tf32=True)
    assert not np.isnan(got).any()
    assert (np.abs(got - exact) <= 2.0 ** -9 * scale + 1e-6).all()
    assert (np.abs(got - cut) <= 1e-5 * scale + 1e-6).all()


# several row tiles and a ragged last one, K tails (f_in not a multiple of 32, padded rows), narrow and wide
# outputs, two column tiles (f_out > 256), a matrix smaller than one tile
@pytest.mark.parametrize("n,f_in,ld,f_out", [
    (1000, 602, 608, 64), (130, 40, 40, 24), (257, 33, 36, 8), (300, 128, 128, 256), (129, 64, 64, 300),
    (5, 7, 8, 3), (128, 32, 32, 16), (4096, 16, 16, 16), (777, 100, 100, 40), (2, 256, 260, 512),
])
def test_combine_matches_oracle(g, n, f_in, ld, f_out):
    x = gg.features_f32(n, ld, dist="normal", p0=0.0, p1=1.0, seed=n + f_out)
    w_t = gg.features_f32(f_out, ld, dist="normal", p0=0.0, p1=0.5, seed=n + f_out, stream=8)
    check(run_combine(g, x, w_t, f_in), x[:, :f_in], w_t[:, :f_in])


def test_combine_is_exact_on_tf32_representable_inputs(g):
    rng = np.random.default_rng(3)
    n, f_in, f_out = 700, 96, 48
    x = (rng.integers(-256, 257, size=(n, f_in)) / 64.0).astype(np.float32)
    w_t = (rng.integers(-256, 257, size=(f_out, f_in)) / 64.0).astype(np.float32)
    exact, _ = orc.combine(x, w_t)
    # every product and every partial sum is a multiple of 2^-12 below 2^12: fp32 holds them exactly
    assert np.array_equal(run_combine(g, x, w_t, f_in), exact)


def test_combine_identity_and_padding_columns_untouched(g):
    n, f = 300, 64
    x = gg.features_f32(n, f, dist="uniform", p0=-1.0, p1=1.0, seed=5)
    eye = np.eye(f, dtype=np.float32)
    out = torch.full((n, f + 8), 7.0, device="cuda")
    g.combine(torch.from_numpy(x).cuda(), torch.from_numpy(eye).cuda(), out=out[:, :f])
    got = out.cpu().numpy()
    cut = (x.view(np.uint32) & np.uint32(0xFFFFE000)).view(np.float32)
    assert np.array_equal(got[:, :f], cut) and (got[:, f:] == 7.0).all()


def test_combine_rejects_unaligned_and_bad_arguments(g):
    x = torch.zeros((8, 10), device="cuda")          # rows of 40 bytes: not a multiple of 16
    w = torch.zeros((4, 10), device="cuda")
    with pytest.raises(g.GnnfdError) as err:
        g.combine(x, w)
    assert err.value.status == g.UNSUPPORTED
    with pytest.raises(ValueError):
        g.combine(torch.zeros((8, 8), device="cuda"), torch.zeros((4, 16), device="cuda"))


def test_combine_then_aggregate_is_a_gcn_layer(g):
    """Section III's order of the two phases: transform first, aggregate the narrow result."""
    w = gg.scaled("config4", 0.02)
    row_ptr, col, _ = orc.build_csr(w.n, w.src, w.dst, w.flags)
    csr = g.build_csr(w.n, torch.from_numpy(w.src).cuda(), torch.from_numpy(w.dst).cuda(), w.flags)
    f_out = 32
    w_t = gg.features_f32(f_out, w.ld, dist="normal", p0=0.0, p1=0.05, seed=1, stream=8)
    z = g.combine(torch.from_numpy(w.x).cuda()[:, :w.f], torch.from_numpy(w_t).cuda()[:, :w.f])
    out = g.aggregate_gcn(csr, z, f=f_out, chunk_width=f_out).cpu().numpy()
    z_cut, z_scale = orc.combine(w.x[:, :w.f], w_t[:, :w.f], tf32=True)
    want, _ = orc.aggregate("gcn", row_ptr, col, z_cut.astype(np.float32), f_out)
    bound, _ = orc.aggregate("gcn", row_ptr, col, z_scale.astype(np.float32), f_out)
    assert (np.abs(out - want) <= 2e-5 * bound + 2e-6).all()


def _bf16(a):
    """bf16 bit patterns (uint16), the same values widened to float32, and a torch bfloat16 device tensor"""
    bits = gg.to_bf16_bits(a)
    wide = (bits.astype(np.uint32) << 16).view(np.float32)
    dev = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    return bits, wide, dev


@pytest.mark.parametrize("n,f_in,ld,f_out", [(1000, 256, 256, 64), (333, 100, 104, 24), (130, 64, 64, 8), (260, 72, 72, 272)])
def test_combine_bf16_operands(g, n, f_in, ld, f_out):
    """bf16 inputs are used as they are: products are exact in fp32, so only the summation order differs
    from the oracle run on the widened values."""
    x = gg.features_f32(n, ld, dist="uniform", p0=-1.0, p1=1.0, seed=n)
    w_t = gg.features_f32(f_out, ld, dist="normal", p0=0.0, p1=0.3, seed=n, stream=8)
    _, xw, xd = _bf16(x)
    _, ww, wd = _bf16(w_t)
    exact, scale = orc.combine(xw[:, :f_in], ww[:, :f_in])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = g.combine(xd[:, :f_in], wd[:, :f_in], status=status).cpu().numpy().astype(np.float64)
    assert int(status.item()) == 0
    assert (np.abs(got - exact) <= 1e-5 * scale + 1e-6).all()
    # bf16 output: the fp32 result rounded to nearest even (8 significant bits: half an ulp is at most 2^-8 relative)
    got16 = g.combine(xd[:, :f_in], wd[:, :f_in], out_dtype=torch.bfloat16).float().cpu().numpy().astype(np.float64)
    assert (np.abs(got16 - exact) <= 2.0 ** -8 * np.abs(exact) + 1e-5 * scale + 1e-6).all()


def test_combine_fp32_inputs_bf16_output(g):
    n, f_in, f_out = 500, 96, 40
    x = gg.features_f32(n, f_in, dist="normal", p0=0.0, p1=1.0, seed=21)
    w_t = gg.features_f32(f_out, f_in, dist="normal", p0=0.0, p1=0.5, seed=21, stream=8)
    cut, scale = orc.combine(x, w_t, tf32=True)
    got = g.combine(torch.from_numpy(x).cuda(), torch.from_numpy(w_t).cuda(), out_dtype=torch.bfloat16)
    got = got.float().cpu().numpy().astype(np.float64)
    assert (np.abs(got - cut) <= 2.0 ** -8 * np.abs(cut) + 1e-5 * scale + 1e-6).all()


# ------------------------------------------------------------------ fp32-faithful mode (three tf32 products)

@pytest.mark.parametrize("n,f_in,ld,f_out", [
    (1000, 602, 608, 64), (130, 40, 40, 24), (257, 33, 36, 8), (300, 128, 128, 256), (129, 64, 64, 300), (5, 7, 8, 3),
    (4096, 16, 16, 16), (2, 256, 260, 512),
])
def test_combine_fp32_mode_meets_the_fp32_bar_against_the_exact_product(g, n, f_in, ld, f_out):
    x = gg.features_f32(n, ld, dist="normal", p0=0.0, p1=1.0, seed=n + f_out)
    w_t = gg.features_f32(f_out, ld, dist="normal", p0=0.0, p1=0.5, seed=n + f_out, stream=8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((n, f_out), float("nan"), device="cuda")
    g.combine(torch.from_numpy(x).cuda()[:, :f_in], torch.from_numpy(w_t).cuda()[:, :f_in], out=out, status=status, mode="fp32")
    got = out.cpu().numpy().astype(np.float64)
    assert int(status.item()) == 0 and not np.isnan(got).any()
    exact, scale = orc.combine(x[:, :f_in], w_t[:, :f_in])               # the exact product, nothing cut
    err = np.abs(got - exact)
    assert (err <= 1e-5 * scale + 1e-6).all(), "worst %.3e of its scale" % (err / (scale + 1e-30)).max()
    # and it is really better than the one-product mode: the tf32 cut alone moves results by more than this bar
    cut, _ = orc.combine(x[:, :f_in], w_t[:, :f_in], tf32=True)
    if f_in >= 32:
        assert np.abs(cut - exact).max() > 10 * err.max()


def test_combine_fp32_mode_same_sign_terms(g):
    """All products positive: truncation errors of the cut operands cannot cancel, the bar must still hold."""
    n, f_in, f_out = 600, 602, 64
    x = np.abs(gg.features_f32(n, 608, dist="normal", p0=0.0, p1=1.0, seed=3)) + 0.1
    w_t = np.abs(gg.features_f32(f_out, 608, dist="normal", p0=0.0, p1=0.5, seed=3, stream=8)) + 0.1
    got = g.combine(torch.from_numpy(x).cuda()[:, :f_in], torch.from_numpy(w_t).cuda()[:, :f_in], mode="fp32")
    exact, scale = orc.combine(x[:, :f_in], w_t[:, :f_in])
    assert (np.abs(got.cpu().numpy().astype(np.float64) - exact) <= 1e-5 * scale + 1e-6).all()


# ------------------------------------------------------------------ scores from the epilogue, whole layers

@pytest.mark.parametrize("heads,dim,zdt", [(8, 8, "f32"), (3, 5, "f32"), (1, 64, "f32"), (40, 8, "f32"), (8, 8, "bf16"),
                                           (4, 16, "bf16")])
@pytest.mark.parametrize("mode", ["tf32", "fp32"])
def test_scores_from_the_epilogue_equal_a_scores_pass_over_z(g, heads, dim, zdt, mode):
    n, f_in = 777, 96
    f_out = heads * dim
    x = gg.features_f32(n, f_in, dist="normal", p0=0.0, p1=1.0, seed=heads)
    w_t = gg.features_f32(f_out, f_in, dist="normal", p0=0.0, p1=0.3, seed=heads, stream=8)
    a_src = gg.features_f32(heads, dim, dist="normal", p0=0.0, p1=0.3, seed=heads, stream=5)
    a_dst = gg.features_f32(heads, dim, dist="normal", p0=0.0, p1=0.3, seed=heads, stream=6)
    dt = torch.bfloat16 if zdt == "bf16" else torch.float32
    z, s_src, s_dst = g.combine(torch.from_numpy(x).cuda(), torch.from_numpy(w_t).cuda(), out_dtype=dt, mode=mode,
                                a_src=torch.from_numpy(a_src).cuda(), a_dst=torch.from_numpy(a_dst).cuda(), heads=heads, dim=dim)
    # z itself is what the plain call gives
    assert torch.equal(z, g.combine(torch.from_numpy(x).cuda(), torch.from_numpy(w_t).cuda(), out_dtype=dt, mode=mode))
    # the oracle's scores of the stored z (bf16 widened exactly)
    z_host = z.float().cpu().numpy()
    o_src, o_dst = orc.gat_scores(z_host, a_src, a_dst, heads, dim)
    zz = np.abs(z_host.astype(np.float64)).reshape(n, heads, dim)
    for got, want, a in ((s_src, o_src, a_src), (s_dst, o_dst, a_dst)):
        scale = np.einsum("nhd,hd->nh", zz, np.abs(a.astype(np.float64)))
        assert (np.abs(got.cpu().numpy().astype(np.float64) - want) <= 1e-5 * scale + 1e-6).all()
    # and the same bits as the library's own scores pass over the stored z
    p_src, p_dst = g.gat_scores(z, torch.from_numpy(a_src).cuda(), torch.from_numpy(a_dst).cuda(), heads, dim)
    assert torch.equal(s_src, p_src) and torch.equal(s_dst, p_dst)


def test_scores_need_whole_heads_per_column_tile(g):
    x = torch.zeros((64, 32), device="cuda")
    w_t = torch.zeros((300, 32), device="cuda")          # two column tiles of 160: heads of 12 straddle them
    a = torch.zeros((25, 12), device="cuda")
    with pytest.raises(g.GnnfdError) as err:
        g.combine(x, w_t, a_src=a, a_dst=a, heads=25, dim=12)
    assert err.value.status == g.UNSUPPORTED
    with pytest.raises(ValueError):
        g.combine(x, w_t, a_src=a[:3], a_dst=a, heads=25, dim=12)


@pytest.mark.parametrize("model", ["gcn", "sage", "gat"])
@pytest.mark.parametrize("mode", ["tf32", "fp32"])
def test_layer_entry_points_against_the_oracle(g, model, mode):
    """Section III's order: transform, then aggregate the narrow result, in one call on a built CSR."""
    w = gg.scaled("config4", 0.05)
    row_ptr, col, _ = orc.build_csr(w.n, w.src, w.dst, w.flags)
    csr = g.build_csr(w.n, torch.from_numpy(w.src).cuda(), torch.from_numpy(w.dst).cuda(), w.flags)
    heads, dim = 8, 8
    f_out = heads * dim
    w_t = gg.features_f32(f_out, w.ld, dist="normal", p0=0.0, p1=0.05, seed=1, stream=8)
    a_src = gg.features_f32(heads, dim, dist="normal", p0=0.0, p1=0.3, seed=1, stream=5)
    a_dst = gg.features_f32(heads, dim, dist="normal", p0=0.0, p1=0.3, seed=1, stream=6)
    xd, wd = torch.from_numpy(w.x).cuda(), torch.from_numpy(w_t).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kw = dict(a_src=torch.from_numpy(a_src).cuda(), a_dst=torch.from_numpy(a_dst).cuda(), heads=heads, dim=dim) if model == "gat" else {}
    out = g.layer(csr, model, xd[:, :w.f], wd[:, :w.f], mode=mode, chunk_width=32, status=status, **kw).cpu().numpy()
    assert int(status.item()) == 0
    # the same two steps through the separate entry points give the same bits
    z = g.combine(xd[:, :w.f], wd[:, :w.f], mode=mode)
    if model == "gat":
        two = g.aggregate_gat(csr, z, kw["a_src"], kw["a_dst"], heads, dim, 0.2, chunk_width=32)
    else:
        two = (g.aggregate_gcn if model == "gcn" else g.aggregate_sage)(csr, z, f=f_out, chunk_width=32)
    assert np.array_equal(out, two.cpu().numpy())
    # against the oracle: aggregate the oracle's own transform; the transform's error (fp32 bar) passes through the
    # aggregation's non-negative weights, so the bound is the aggregated bound of z plus the aggregation's own
    z_ref, z_scale = orc.combine(w.x[:, :w.f], w_t[:, :w.f], tf32=(mode == "tf32"))
    z32 = z.cpu().numpy()
    assert (np.abs(z32.astype(np.float64) - z_ref) <= 1e-5 * z_scale + 1e-6).all()
    if model == "gat":
        want, scale = orc.aggregate_gat(row_ptr, col, z32, a_src, a_dst, heads, dim, 0.2)
    else:
        want, scale = orc.aggregate(model, row_ptr, col, z32, f_out)
    assert (np.abs(out.astype(np.float64) - want) <= 1e-5 * scale + 1e-6).all()


def test_layer_with_bf16_features(g):
    w = gg.scaled("config5_f64", 1 / 64)
    row_ptr, col, _ = orc.build_csr(w.n, w.src, w.dst, w.flags)
    csr = g.build_csr(w.n, torch.from_numpy(w.src).cuda(), torch.from_numpy(w.dst).cuda(), w.flags)
    f_out = 16
    w_t = gg.features_f32(f_out, w.f, dist="normal", p0=0.0, p1=0.2, seed=2, stream=8)
    _, ww, wd = _bf16(w_t)
    xd = torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16)
    out = g.layer(csr, "gcn", xd, wd).cpu().numpy()
    z = g.combine(xd, wd, out_dtype=torch.bfloat16)
    zb = z.view(torch.int16).cpu().numpy().view(np.uint16)
    want, scale = orc.aggregate("gcn", row_ptr, col, zb, f_out)
    assert (np.abs(out.astype(np.float64) - want) <= 1e-5 * scale + 1e-6).all()


# ------------------------------------------------------------------ the give-up path, drilled without a fault

@pytest.mark.parametrize("mode", ["tf32", "fp32"])
@pytest.mark.parametrize("skip", [0, 3, 18])
def test_a_block_that_never_gets_its_tile_gives_up_and_the_next_call_is_fine(g, mode, skip):
    """The drill leaves one K block's loads out (nothing is in flight for it) and shortens every wait to a
    millisecond: the lanes that wait for that tile run out of time, every block reports through the status word,
    frees its tensor memory and returns.  The device stays usable: the following ordinary call is correct."""
    n, f_in, f_out = 1000, 602, 64                       # 19 K blocks of 32 columns, more than the ring holds
    x = gg.features_f32(n, 608, dist="normal", p0=0.0, p1=1.0, seed=9)
    w_t = gg.features_f32(f_out, 608, dist="normal", p0=0.0, p1=0.5, seed=9, stream=8)
    xd, wd = torch.from_numpy(x).cuda()[:, :f_in], torch.from_numpy(w_t).cuda()[:, :f_in]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    g.debug_combine_fault(1_000_000, skip)
    g.combine(xd, wd, status=status, mode=mode)
    torch.cuda.synchronize()
    assert int(status.item()) == 1
    # the drill is one-shot: the next call is an ordinary one and meets its bar
    status.zero_()
    got = g.combine(xd, wd, status=status, mode=mode).cpu().numpy().astype(np.float64)
    assert int(status.item()) == 0
    ref, scale = orc.combine(x[:, :f_in], w_t[:, :f_in], tf32=(mode == "tf32"))
    assert (np.abs(got - ref) <= 1e-5 * scale + 1e-6).all()


def test_bench_size_transform_with_two_column_tiles(g):
    """The config-4 feature matrix [232,965, 602] into 320 columns (two column tiles of 160): sampled rows against
    the exact product, every element written."""
    w = gg.config4()
    f_out = 320
    w_t = gg.features_f32(f_out, w.ld, dist="normal", p0=0.0, p1=0.05, seed=4, stream=8)
    xd, wd = torch.from_numpy(w.x).cuda()[:, :w.f], torch.from_numpy(w_t).cuda()[:, :w.f]
    rows = np.sort(np.random.default_rng(0).choice(w.n, 4096, replace=False))
    rows[-1] = w.n - 1                                   # the ragged last row tile
    for mode in ("tf32", "fp32"):
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = torch.full((w.n, f_out), float("nan"), device="cuda")
        g.combine(xd, wd, out=out, status=status, mode=mode)
        assert int(status.item()) == 0 and not bool(torch.isnan(out).any())
        ref, scale = orc.combine(w.x[rows, :w.f], w_t[:, :w.f], tf32=(mode == "tf32"))
        got = out[torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.float64)
        assert (np.abs(got - ref) <= 1e-5 * scale + 1e-6).all(), mode
