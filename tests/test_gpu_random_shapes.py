"""Seeded random shapes against the oracle: vertex and edge counts, build flags, id width, feature width,
leading dimension, chunk width, heads x dim, LeakyReLU slope (0, 1, negative and above 1 included) and the
shape of the dense transform are all drawn; half of the graphs get a hub row made of repeated edges.  Every
case checks the CSR bit for bit and each aggregator, the edge softmax and the transform element by element."""
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


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("seed", range(24))
def test_random_case(g, seed):
    rng = np.random.default_rng(1000 + seed)
    n = int(rng.integers(1, 6000))
    e = int(rng.integers(0, 120_000))
    flags = int(rng.integers(0, 8))
    src = rng.integers(0, n, size=e).astype(np.int32)
    dst = rng.integers(0, n, size=e).astype(np.int32)
    if e > 10 and seed % 2 == 0:
        dst[: e // 2] = dst[0]
        src[: e // 8] = src[1]
    wide_ids = seed % 3 == 0
    csr = g.build_csr(n, dev(src.astype(np.int64) if wide_ids else src), dev(dst.astype(np.int64) if wide_ids else dst), flags)
    row_ptr, col, perm = orc.build_csr(n, src, dst, flags)
    assert csr.nnz == len(col)
    assert np.array_equal(csr.row_ptr.cpu().numpy(), row_ptr)
    assert np.array_equal(csr.col_idx.cpu().numpy(), col)
    assert np.array_equal(csr.perm.cpu().numpy(), perm)

    f = int(rng.integers(1, 70))
    ld = f + int(rng.integers(0, 5))
    width = int(rng.integers(1, f + 3))
    x = rng.standard_normal((n, ld)).astype(np.float32)
    bits = gg.to_bf16_bits(x)
    x16 = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    for model, fn in (("gcn", g.aggregate_gcn), ("sage", g.aggregate_sage)):
        want, scale = orc.aggregate(model, row_ptr, col, x, f)
        got = fn(csr, dev(x), f=f, chunk_width=width).cpu().numpy()
        assert (np.abs(got - want) <= 1e-5 * scale + 1e-6).all(), (model, "f32")
        want, scale = orc.aggregate(model, row_ptr, col, bits, f)
        got = fn(csr, x16, f=f, chunk_width=width).cpu().numpy()
        assert (np.abs(got - want) <= 1e-5 * scale + 1e-6).all(), (model, "bf16")

    heads, dim = int(rng.integers(1, 10)), int(rng.integers(1, 10))
    z = rng.standard_normal((n, heads * dim)).astype(np.float32)
    a_src = (rng.standard_normal((heads, dim)) * 0.3).astype(np.float32)
    a_dst = (rng.standard_normal((heads, dim)) * 0.3).astype(np.float32)
    slope = float(rng.choice([0.2, 0.0, 1.0, -0.5, 2.0]))
    want, scale = orc.aggregate_gat(row_ptr, col, z, a_src, a_dst, heads, dim, slope)
    got = g.aggregate_gat(csr, dev(z), dev(a_src), dev(a_dst), heads, dim, slope,
                          chunk_width=int(rng.integers(1, heads * dim + 2))).cpu().numpy()
    assert (np.abs(got - want) <= 1e-5 * scale + 1e-6).all(), "gat"
    if csr.nnz > 0:
        s_src = (rng.standard_normal((n, heads)) * 4).astype(np.float32)
        s_dst = (rng.standard_normal((n, heads)) * 4).astype(np.float32)
        alpha = g.edge_softmax(csr, dev(s_src), dev(s_dst), slope).cpu().numpy()
        want_alpha = orc.edge_softmax(row_ptr, col, s_src, s_dst, slope)
        assert (np.abs(alpha - want_alpha) <= 1e-5 * want_alpha + 1e-7).all(), "edge softmax"

    f_in, f_out = int(rng.integers(1, 200)), int(rng.integers(1, 300))
    ldc = (f_in + 3) // 4 * 4
    xc = rng.standard_normal((n, ldc)).astype(np.float32)
    wc = rng.standard_normal((f_out, ldc)).astype(np.float32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    zc = g.combine(dev(xc)[:, :f_in], dev(wc)[:, :f_in], status=status).cpu().numpy()
    cut, sc = orc.combine(xc[:, :f_in], wc[:, :f_in], tf32=True)
    assert int(status.item()) == 0 and (np.abs(zc - cut) <= 1e-5 * sc + 1e-6).all(), "combine"
    csr.destroy()


def _close(got, want, scale):
    return bool((np.abs(got.astype(np.float64) - want) <= 1e-5 * scale + 1e-6).all())


@pytest.mark.parametrize("seed", range(10))
def test_random_case_light_build_oneshot_and_layers(g, seed):
    """The same kind of draw for the later entry points: the input-order build (rows compared as multisets), the
    one-shot calls, the transform in a drawn precision with scores from its epilogue, and whole layers."""
    rng = np.random.default_rng(5000 + seed)
    n = int(rng.integers(1, 5000))
    e = int(rng.integers(0, 90_000))
    flags = int(rng.choice([0, 1, 4, 5]))
    src = rng.integers(0, n, size=e).astype(np.int32)
    dst = rng.integers(0, n, size=e).astype(np.int32)
    if e > 10 and seed % 2 == 0:
        dst[: e // 2] = dst[0]
    row_ptr, col, _ = orc.build_csr(n, src, dst, flags)
    csr = g.build_csr(n, dev(src), dev(dst), flags | g.CSR_INPUT_ORDER)
    rows = np.repeat(np.arange(n), np.diff(row_ptr))
    got_col = csr.col_idx.cpu().numpy()
    order = np.lexsort((got_col, rows))
    assert np.array_equal(csr.row_ptr.cpu().numpy(), row_ptr) and np.array_equal(got_col[order], col)
    f = int(rng.integers(1, 40))
    cw = int(rng.integers(1, f + 3))
    x = rng.standard_normal((n, f)).astype(np.float32)
    for model, fn in (("gcn", g.aggregate_gcn), ("sage", g.aggregate_sage)):
        want, scale = orc.aggregate(model, row_ptr, col, x, f)
        assert _close(fn(csr, dev(x), f=f, chunk_width=cw).cpu().numpy(), want, scale), model
        assert _close(g.oneshot(model, n, dev(src), dev(dst), dev(x), flags=flags, chunk_width=cw).cpu().numpy(), want, scale)
    heads, dim = int(rng.integers(1, 6)), int(rng.integers(1, 9))
    a_src = (rng.standard_normal((heads, dim)) * 0.3).astype(np.float32)
    a_dst = (rng.standard_normal((heads, dim)) * 0.3).astype(np.float32)
    f_in = int(rng.integers(1, 120))
    ld = (f_in + 3) // 4 * 4
    xc = rng.standard_normal((n, ld)).astype(np.float32)
    wc = (rng.standard_normal((heads * dim, ld)) * 0.3).astype(np.float32)
    mode = "fp32" if seed % 3 else "tf32"
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    z, s_src, s_dst = g.combine(dev(xc)[:, :f_in], dev(wc)[:, :f_in], status=status, mode=mode, a_src=dev(a_src),
                                a_dst=dev(a_dst), heads=heads, dim=dim)
    ref, ref_scale = orc.combine(xc[:, :f_in], wc[:, :f_in], tf32=(mode == "tf32"))
    zh = z.cpu().numpy()
    assert int(status.item()) == 0 and _close(zh, ref, ref_scale)
    slope = float(rng.choice([0.2, 0.0, 1.0]))
    cwz = int(rng.integers(1, heads * dim + 2))
    out = g.layer(csr, "gat", dev(xc)[:, :f_in], dev(wc)[:, :f_in], mode=mode, chunk_width=cwz, a_src=dev(a_src),
                  a_dst=dev(a_dst), heads=heads, dim=dim, negative_slope=slope, status=status).cpu().numpy()
    want, scale = orc.aggregate_gat(row_ptr, col, zh, a_src, a_dst, heads, dim, slope)
    assert int(status.item()) == 0 and _close(out, want, scale)
    if csr.nnz:
        # alpha comes in the slot order of this CSR (edge-id order inside a row): bring it into the oracle's order
        alpha = g.edge_softmax(csr, s_src, s_dst, slope).cpu().numpy()[order]
        want_alpha = orc.edge_softmax(row_ptr, col, s_src.cpu().numpy(), s_dst.cpu().numpy(), slope)
        assert (np.abs(alpha - want_alpha) <= 1e-5 * want_alpha + 1e-7).all()
