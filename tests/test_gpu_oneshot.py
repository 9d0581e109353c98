"""The light build (rows in edge-id order, destination-only sort) and the one-shot COO entry points against the
CPU oracle.  The oracle's CSR lists a row's sources in ascending order; the light build lists the same sources in
edge-id order, so rows are compared as multisets (and exactly, through perm) and sums within the fp32 bar."""
import numpy as np
import pytest

import graphgen as gg
import oracle as orc

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

SL, DD, SY, IO = 1, 2, 4, 8


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def close(got, want, scale):
    return (np.abs(got.astype(np.float64) - want) <= 1e-5 * scale + 1e-6).all()


@pytest.mark.parametrize("flags", [0, SL, SY, SY | SL])
@pytest.mark.parametrize("itype", [np.int32, np.int64])
def test_input_order_build_has_the_oracles_rows_in_edge_id_order(flags, itype):
    import paper_2104_03058_b200 as g
    n, e = 3000, 60_000
    src, dst = gg.powerlaw_graph(n, e, 2.1, None, flags + 1)
    src, dst = src.astype(itype), dst.astype(itype)
    src[:50] = dst[:50]                                  # some input loops
    src[100:140] = src[60:100]; dst[100:140] = dst[60:100]      # some multi-edges
    e = len(src)
    row_ptr, col, perm = orc.build_csr(n, src, dst, flags)
    csr = g.build_csr(n, dev(src), dev(dst), flags | IO)
    assert csr.nnz == len(col)
    np.testing.assert_array_equal(csr.row_ptr.cpu().numpy(), row_ptr)          # same rows, same lengths
    got_col, got_perm = csr.col_idx.cpu().numpy(), csr.perm.cpu().numpy()
    rows = np.repeat(np.arange(n), np.diff(row_ptr))
    # every slot maps back to the input edge that produced it
    inp = got_perm >= 0
    fwd = inp & (got_perm < e)
    rev = inp & (got_perm >= e)
    assert (src[got_perm[fwd]] == got_col[fwd]).all() and (dst[got_perm[fwd]] == rows[fwd]).all()
    assert (dst[got_perm[rev] - e] == got_col[rev]).all() and (src[got_perm[rev] - e] == rows[rev]).all()
    assert (got_col[~inp] == rows[~inp]).all()
    # inside a row: ascending edge id, the added loop (-1) last; and the same multiset of sources as the oracle
    same_row = rows[1:] == rows[:-1]
    a, b = got_perm[:-1][same_row], got_perm[1:][same_row]
    assert ((a < b) | (b == -1)).all() and (a != -1).all()
    order = np.lexsort((got_col, rows))
    np.testing.assert_array_equal(got_col[order], col)
    deg, dinv, rdeg = orc.degree_norm(row_ptr)
    np.testing.assert_array_equal(csr.dinv_sqrt.cpu().numpy(), dinv.astype(np.float32))
    # the handle serves every aggregator
    x = gg.features_f32(n, 24, dist="normal", p0=0, p1=1, seed=3)
    for model, fn in (("gcn", g.aggregate_gcn), ("sage", g.aggregate_sage)):
        want, scale = orc.aggregate(model, row_ptr, col, x, 24)
        assert close(fn(csr, dev(x), f=24, chunk_width=8).cpu().numpy(), want, scale)
    a_src = gg.features_f32(3, 8, dist="normal", p0=0, p1=0.3, seed=1, stream=5)
    a_dst = gg.features_f32(3, 8, dist="normal", p0=0, p1=0.3, seed=1, stream=6)
    want, scale = orc.aggregate_gat(row_ptr, col, x, a_src, a_dst, 3, 8, 0.2)
    assert close(g.aggregate_gat(csr, dev(x), dev(a_src), dev(a_dst), 3, 8, 0.2).cpu().numpy(), want, scale)


def test_input_order_excludes_duplicate_removal():
    import paper_2104_03058_b200 as g
    src, dst = gg.uniform_graph(100, 500, seed=1)
    with pytest.raises(g.GnnfdError) as err:
        g.build_csr(100, dev(src), dev(dst), DD | IO)
    assert err.value.status == g.INVALID_ARG


@pytest.mark.parametrize("model", ["gcn", "sage"])
@pytest.mark.parametrize("flags", [SL, 0, SY | DD | SL])
def test_oneshot_matches_the_oracle_and_is_repeatable(model, flags):
    import paper_2104_03058_b200 as g
    w = gg.scaled("config4", 0.05)                       # hub rows included
    f = 32
    x = np.ascontiguousarray(w.x[:, :f])
    row_ptr, col, _ = orc.build_csr(w.n, w.src, w.dst, flags)
    want, scale = orc.aggregate(model, row_ptr, col, x, f)
    src, dst, xd = dev(w.src), dev(w.dst), dev(x)
    outs = []
    for width in (f, 8):
        out = torch.full((w.n, f), float("nan"), device="cuda")
        g.oneshot(model, w.n, src, dst, xd, flags=flags, chunk_width=width, out=out)
        assert close(out.cpu().numpy(), want, scale), (model, flags, width)
        outs.append(out)
    again = g.oneshot(model, w.n, src, dst, xd, flags=flags, chunk_width=f)
    assert torch.equal(again, outs[0])                   # no atomics: the same bits every time
    # bf16 features
    bits = gg.to_bf16_bits(x)
    xb = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    want16, scale16 = orc.aggregate(model, row_ptr, col, bits, f)
    assert close(g.oneshot(model, w.n, src, dst, xb, flags=flags).cpu().numpy(), want16, scale16)


@pytest.mark.parametrize("flags", [SL, SY | DD | SL])
def test_oneshot_gat_matches_the_oracle(flags):
    import paper_2104_03058_b200 as g
    w = gg.scaled("config4", 0.05)                       # hub rows included
    heads, dim = 4, 8
    z = np.ascontiguousarray(w.x[:, :heads * dim])
    a_src = gg.features_f32(heads, dim, dist="normal", p0=0.0, p1=0.3, seed=2, stream=5)
    a_dst = gg.features_f32(heads, dim, dist="normal", p0=0.0, p1=0.3, seed=2, stream=6)
    row_ptr, col, _ = orc.build_csr(w.n, w.src, w.dst, flags)
    want, scale = orc.aggregate_gat(row_ptr, col, z, a_src, a_dst, heads, dim, 0.2)
    for width in (heads * dim, dim):
        got = g.oneshot_gat(w.n, dev(w.src), dev(w.dst), dev(z), dev(a_src), dev(a_dst), heads, dim, 0.2, flags=flags,
                            chunk_width=width)
        assert close(got.cpu().numpy(), want, scale), (flags, width)


def test_oneshot_reports_bad_ids_and_small_buffers():
    import paper_2104_03058_b200 as g
    n, f = 50, 8
    src = torch.tensor([0, 1, 50], dtype=torch.int32, device="cuda")
    dst = torch.tensor([1, 2, 3], dtype=torch.int32, device="cuda")
    x = torch.zeros((n, f), device="cuda")
    with pytest.raises(g.GnnfdError) as err:
        g.oneshot("gcn", n, src, dst, x)
    assert err.value.status == g.BAD_INDEX
    need = g.oneshot_workspace_bytes(n, 3, 0, f)
    with pytest.raises(g.GnnfdError) as err:
        g.oneshot("gcn", n, src[:2], dst[:2], x, scratch=torch.empty(need - 256, dtype=torch.uint8, device="cuda"))
    assert err.value.status == g.WORKSPACE_TOO_SMALL
    empty = torch.zeros(0, dtype=torch.int32, device="cuda")
    out = g.oneshot("sage", n, empty, empty, x + 1.0, flags=SL)           # only the added loops: out = x
    assert torch.equal(out, x + 1.0)
