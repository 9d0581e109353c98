"""Pins for the CPU oracle: checks that do not go through the oracle's own code path.

Dense adjacency products (numpy), closed forms on star / regular / identity graphs, the
hand-computed Fig. 2 example, and invariants the method guarantees (the paper's exactness claim in
Section I: aggregation is element-wise over features, so decomposition does not change results).
"""
import os

import numpy as np
import pytest

import graphgen as gg
import oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
SL, DD, SY = orc.ADD_SELF_LOOPS, orc.DEDUP, orc.SYMMETRIZE


# ------------------------------------------------------------------ dense reference (numpy only)

def dense_adjacency(n, src, dst, flags):
    """A[v, u] = multiplicity of edge u -> v after the build flags, as a dense matrix."""
    a = np.zeros((n, n), np.float64)
    for s, d in zip(src.tolist(), dst.tolist()):
        a[d, s] += 1
    if flags & SY:
        off = a - np.diag(np.diag(a))
        a = a + off.T
    if flags & SL:
        np.fill_diagonal(a, 1.0)
    if flags & DD:
        a = np.minimum(a, 1.0)
    return a


def dense_gcn(a, x):
    deg = a.sum(axis=1)
    dinv = np.where(deg > 0, 1.0 / np.sqrt(np.maximum(deg, 1)), 0.0)
    return (dinv[:, None] * a * dinv[None, :]) @ x


def dense_sage(a, x):
    deg = a.sum(axis=1)
    rdeg = np.where(deg > 0, 1.0 / np.maximum(deg, 1), 0.0)
    return (rdeg[:, None] * a) @ x


def dense_gat(a, z, a_src, a_dst, heads, dim, slope, with_abs=False):
    n = a.shape[0]
    zz = z.reshape(n, heads, dim)
    s_src = np.einsum("nhd,hd->nh", zz, a_src.astype(np.float64))
    s_dst = np.einsum("nhd,hd->nh", zz, a_dst.astype(np.float64))
    out = np.zeros((n, heads, dim))
    out_abs = np.zeros((n, heads, dim))
    for h in range(heads):
        e = s_dst[:, h][:, None] + s_src[:, h][None, :]          # e[v, u]
        e = np.where(e >= 0, e, slope * e)
        e = np.where(a > 0, e, -np.inf)
        m = e.max(axis=1, keepdims=True)
        m = np.where(np.isfinite(m), m, 0.0)
        p = a * np.exp(e - m)
        den = p.sum(axis=1, keepdims=True)
        alpha = np.divide(p, den, out=np.zeros_like(p), where=den > 0)
        out[:, h, :] = alpha @ zz[:, h, :]
        out_abs[:, h, :] = alpha @ np.abs(zz[:, h, :])
    if with_abs:
        return out.reshape(n, heads * dim), out_abs.reshape(n, heads * dim)
    return out.reshape(n, heads * dim)


SIZES = [8, 13, 16, 33, 64]
FLAGSETS = [0, SL, DD, SY, SL | DD, SY | DD | SL, SY | SL]


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("flags", FLAGSETS)
def test_gcn_sage_match_dense_product(n, flags):
    src, dst = gg.uniform_graph(n, 3 * n, seed=n + 100 * flags)
    dst[dst == 1] = 0                       # leaves vertex 1 without in-edges when no self-loops
    x = gg.features_f32(n, 5, dist="normal", p0=0.0, p1=1.0, seed=n)
    a = dense_adjacency(n, src, dst, flags)
    row_ptr, col, perm = orc.build_csr(n, src, dst, flags)
    assert row_ptr[-1] == int(a.sum())
    for model, dense in (("gcn", dense_gcn), ("sage", dense_sage)):
        want = dense(a, x.astype(np.float64))
        got, ab = orc.aggregate(model, row_ptr, col, x, 5)
        np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)
        # the tolerance scale sum |w x| is the same product on absolute values (all weights are >= 0):
        # pinned by equality, since every GPU bound is a multiple of it
        want_ab = dense(a, np.abs(x.astype(np.float64)))
        np.testing.assert_allclose(ab, want_ab, rtol=1e-12, atol=1e-13)
        assert (ab >= np.abs(got) - 1e-12).all()


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("flags", [0, SL, SY | DD | SL])
def test_gat_matches_dense_masked_softmax(n, flags):
    heads, dim = 3, 4
    src, dst = gg.uniform_graph(n, 3 * n, seed=7 * n + flags)
    dst[dst == 2] = 0
    z = gg.features_f32(n, heads * dim, dist="normal", p0=0.0, p1=1.0, seed=n + 1)
    a_src = gg.features_f32(heads, dim, dist="normal", p0=0.0, p1=0.7, seed=n, stream=5)
    a_dst = gg.features_f32(heads, dim, dist="normal", p0=0.0, p1=0.7, seed=n, stream=6)
    a = dense_adjacency(n, src, dst, flags)
    row_ptr, col, _ = orc.build_csr(n, src, dst, flags)
    want, want_ab = dense_gat(a, z.astype(np.float64), a_src, a_dst, heads, dim, 0.2, with_abs=True)
    got, ab = orc.aggregate_gat(row_ptr, col, z, a_src, a_dst, heads, dim, 0.2)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(ab, want_ab, rtol=1e-12, atol=1e-13)       # the tolerance scale sum |alpha z|
    for width in (1, 5, heads * dim):                                     # ... for every decomposition too
        _, ab_w = orc.aggregate_gat(row_ptr, col, z, a_src, a_dst, heads, dim, 0.2, chunk_width=width)
        np.testing.assert_array_equal(ab_w, ab)
    # alpha written out: rows sum to one, and alpha-weighted sum reproduces the aggregation
    s_src, s_dst = orc.gat_scores(z, a_src, a_dst, heads, dim)
    alpha = orc.edge_softmax(row_ptr, col, s_src, s_dst, 0.2)
    for v in range(n):
        b, e = row_ptr[v], row_ptr[v + 1]
        if e > b:
            np.testing.assert_allclose(alpha[b:e].sum(axis=0), 1.0, rtol=0, atol=1e-14)
            zz = z[col[b:e]].astype(np.float64).reshape(e - b, heads, dim)
            np.testing.assert_allclose((alpha[b:e, :, None] * zz).sum(axis=0).reshape(-1), got[v],
                                       rtol=1e-12, atol=1e-13)
        else:
            assert (got[v] == 0).all()


def dense_alpha(a, s_src, s_dst, slope):
    """alpha[v, u, h]: masked row softmax of LeakyReLU(s_src[u, h] + s_dst[v, h]) over the in-neighbours u of v;
    multi-edges share the value (each copy is one softmax term, so the denominator counts it a[v, u] times)."""
    e = s_dst[:, None, :] + s_src[None, :, :]
    e = np.where(e >= 0, e, slope * e)
    e = np.where(a[:, :, None] > 0, e, -np.inf)
    m = e.max(axis=1, keepdims=True)
    m = np.where(np.isfinite(m), m, 0.0)
    p = np.exp(e - m)
    den = (a[:, :, None] * p).sum(axis=1, keepdims=True)
    return np.divide(p, den, out=np.zeros_like(p), where=den > 0)


@pytest.mark.parametrize("n", [8, 33, 64])
@pytest.mark.parametrize("flags", [0, SL, SY | DD | SL])
def test_edge_softmax_with_fp32_scores_matches_dense_softmax(n, flags):
    """The entry the GPU tests use: scores arrive as float32 (as the library's caller supplies them).  The
    source and destination scores are drawn differently, so a wrapper that swaps or reuses them fails."""
    heads = 3
    src, dst = gg.uniform_graph(n, 4 * n, seed=3 * n + flags)
    dst[dst == 2] = 0
    s_src = gg.features_f32(n, heads, dist="normal", p0=0.5, p1=1.5, seed=n, stream=5)
    s_dst = gg.features_f32(n, heads, dist="normal", p0=-1.0, p1=0.7, seed=n, stream=6)
    assert s_src.dtype == np.float32 and s_dst.dtype == np.float32
    a = dense_adjacency(n, src, dst, flags)
    row_ptr, col, _ = orc.build_csr(n, src, dst, flags)
    got = orc.edge_softmax(row_ptr, col, s_src, s_dst, 0.2)
    assert got.dtype == np.float64 and got.shape == (len(col), heads)
    want = dense_alpha(a, s_src.astype(np.float64), s_dst.astype(np.float64), 0.2)
    rows = np.repeat(np.arange(n), np.diff(row_ptr))
    np.testing.assert_allclose(got, want[rows, col, :], rtol=1e-12, atol=1e-15)
    # the float64 entry on the widened values is the same computation
    np.testing.assert_array_equal(got, orc.edge_softmax(row_ptr, col, s_src.astype(np.float64),
                                                        s_dst.astype(np.float64), 0.2))
    # and it is not what the swapped scores give
    swapped = orc.edge_softmax(row_ptr, col, s_dst, s_src, 0.2)
    assert np.abs(swapped - got).max() > 1e-3


# ------------------------------------------------------------------ CSR structure

@pytest.mark.parametrize("flags", FLAGSETS)
@pytest.mark.parametrize("itype", [np.int32, np.int64])
def test_csr_structure_and_perm(flags, itype):
    n, e = 50, 400
    src, dst = gg.uniform_graph(n, e, seed=flags + 11)
    row_ptr, col, perm = orc.build_csr(n, src.astype(itype), dst.astype(itype), flags)
    nnz = len(col)
    assert row_ptr[0] == 0 and row_ptr[-1] == nnz and (np.diff(row_ptr) >= 0).all()
    rows = np.repeat(np.arange(n), np.diff(row_ptr))
    key = rows.astype(np.int64) * n + col
    if flags & DD:
        assert (np.diff(key) > 0).all()
    else:
        assert (np.diff(key) >= 0).all()
    # perm maps every CSR slot back to the input edge that produced it
    for k in range(nnz):
        p = perm[k]
        if p < 0:
            assert flags & SL and col[k] == rows[k]
        elif p < e:
            assert (src[p], dst[p]) == (col[k], rows[k])
        else:
            assert flags & SY and (dst[p - e], src[p - e]) == (col[k], rows[k])
    kept = perm[perm >= 0]
    assert len(np.unique(kept)) == len(kept)
    if not (flags & DD):
        # ties keep ascending edge id
        same = np.diff(key) == 0
        assert (np.diff(perm)[same] > 0).all()
    if flags == 0:
        np.testing.assert_array_equal(np.diff(row_ptr), np.bincount(dst, minlength=n))
        assert sorted(perm.tolist()) == list(range(e))


def test_csr_input_order_invariance():
    n, e = 40, 300
    src, dst = gg.uniform_graph(n, e, seed=5)
    key = dst.astype(np.int64) * n + src
    keep = np.unique(key, return_index=True)[1]          # distinct edges: result is order-free
    src, dst = src[keep], dst[keep]
    rp0, col0, perm0 = orc.build_csr(n, src, dst, 0)
    shuffle = np.random.default_rng(0).permutation(len(src))
    rp1, col1, perm1 = orc.build_csr(n, src[shuffle], dst[shuffle], 0)
    np.testing.assert_array_equal(rp0, rp1)
    np.testing.assert_array_equal(col0, col1)
    np.testing.assert_array_equal(perm0, shuffle[perm1])


def test_csr_rejects_bad_ids():
    src = np.array([0, 5], np.int32)
    dst = np.array([1, 2], np.int32)
    with pytest.raises(orc.OracleError) as err:
        orc.build_csr(5, src, dst, 0)
    assert err.value.code == orc.ERR_BAD_INDEX
    with pytest.raises(orc.OracleError):
        orc.build_csr(5, np.array([-1], np.int32), np.array([0], np.int32), 0)


def test_degree_norm_values():
    row_ptr = np.array([0, 0, 1, 5, 14], np.int32)
    deg, dinv, rdeg = orc.degree_norm(row_ptr)
    np.testing.assert_array_equal(deg, [0, 1, 4, 9])
    np.testing.assert_allclose(dinv, [0, 1, 0.5, 1 / 3], rtol=1e-15)
    np.testing.assert_allclose(rdeg, [0, 1, 0.25, 1 / 9], rtol=1e-15)


# ------------------------------------------------------------------ closed forms

def test_fig2_toy_golden():
    vals = {}
    with open(os.path.join(GOLDEN, "fig2_toy.txt")) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                k, *v = line.split()
                vals[k] = np.array([float(t) for t in v])
    x = np.stack([vals["hA"], vals["hB"], vals["hC"], vals["hD"]]).astype(np.float32)
    src = np.array([1, 2, 3, 0, 0, 0], np.int32)
    dst = np.array([0, 0, 0, 1, 2, 3], np.int32)
    row_ptr, col, _ = orc.build_csr(4, src, dst, 0)
    for width in (4, 2, 1, 3):                         # P = 1, 2 (the figure), 4, and a ragged split
        got, _ = orc.aggregate("gcn", row_ptr, col, x, 4, width)
        for i, name in enumerate("ABCD"):
            np.testing.assert_allclose(got[i], vals["gcn_" + name], rtol=1e-15)
        got, _ = orc.aggregate("sage", row_ptr, col, x, 4, width)
        np.testing.assert_allclose(got[0], vals["sage_A"], rtol=1e-15)
        np.testing.assert_allclose(got[1], vals["sage_B"], rtol=1e-15)


def test_regular_graph_constant_feature():
    n, d = 30, 4                                       # ring lattice: d in-neighbours each, plus self-loop
    src = np.array([(v + k) % n for v in range(n) for k in range(1, d + 1)], np.int32)
    dst = np.array([v for v in range(n) for _ in range(d)], np.int32)
    x = np.full((n, 3), 2.5, np.float32)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    got, _ = orc.aggregate("gcn", row_ptr, col, x, 3)
    np.testing.assert_allclose(got, 2.5, rtol=1e-14)   # each of the d+1 weights is 1/(d+1)
    got, _ = orc.aggregate("sage", row_ptr, col, x, 3)
    np.testing.assert_allclose(got, 2.5, rtol=1e-14)


def test_star_graph_closed_form():
    n_leaf = 6
    n = n_leaf + 1
    src = np.array(list(range(1, n)) + [0] * n_leaf, np.int32)
    dst = np.array([0] * n_leaf + list(range(1, n)), np.int32)
    x = gg.features_f32(n, 3, dist="uniform", p0=-1, p1=1, seed=3)
    xd = x.astype(np.float64)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    got, _ = orc.aggregate("gcn", row_ptr, col, x, 3)
    centre = xd[0] / (n_leaf + 1) + xd[1:].sum(axis=0) / np.sqrt(2.0 * (n_leaf + 1))
    np.testing.assert_allclose(got[0], centre, rtol=1e-13)
    for leaf in range(1, n):
        np.testing.assert_allclose(got[leaf], xd[leaf] / 2 + xd[0] / np.sqrt(2.0 * (n_leaf + 1)), rtol=1e-13)


def test_identity_graph_returns_input():
    n = 9
    x = gg.features_f32(n, 4, seed=2)
    e = np.zeros(0, np.int32)
    row_ptr, col, perm = orc.build_csr(n, e, e, SL)
    np.testing.assert_array_equal(col, np.arange(n))
    assert (perm == -1).all()
    for model in ("gcn", "sage"):
        got, _ = orc.aggregate(model, row_ptr, col, x, 4)
        np.testing.assert_array_equal(got, x.astype(np.float64))
    a = gg.features_f32(2, 2, seed=1, stream=5)
    got, _ = orc.aggregate_gat(row_ptr, col, x, a, a, 2, 2)
    np.testing.assert_array_equal(got, x.astype(np.float64))     # single-entry rows: alpha = 1


def test_gat_zero_attention_is_mean():
    n, heads, dim = 40, 2, 3
    src, dst = gg.uniform_graph(n, 200, seed=9)
    z = gg.features_f32(n, heads * dim, seed=4)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    zero = np.zeros((heads, dim), np.float32)
    got, _ = orc.aggregate_gat(row_ptr, col, z, zero, zero, heads, dim)
    want, _ = orc.aggregate("sage", row_ptr, col, z, heads * dim)
    np.testing.assert_allclose(got, want, rtol=1e-13, atol=1e-15)


def test_gat_slope_one_ignores_destination_score():
    n, heads, dim = 25, 2, 4
    src, dst = gg.uniform_graph(n, 120, seed=10)
    z = gg.features_f32(n, heads * dim, dist="normal", p0=0, p1=1, seed=5)
    a_src = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.5, seed=5, stream=5)
    a_dst = gg.features_f32(heads, dim, dist="normal", p0=0, p1=0.5, seed=5, stream=6)
    row_ptr, col, _ = orc.build_csr(n, src, dst, 0)
    one, _ = orc.aggregate_gat(row_ptr, col, z, a_src, a_dst, heads, dim, slope=1.0)
    two, _ = orc.aggregate_gat(row_ptr, col, z, a_src, 3 * a_dst, heads, dim, slope=1.0)
    np.testing.assert_allclose(one, two, rtol=1e-12, atol=1e-14)
    # with the usual slope the destination term does matter
    three, _ = orc.aggregate_gat(row_ptr, col, z, a_src, a_dst, heads, dim, slope=0.2)
    four, _ = orc.aggregate_gat(row_ptr, col, z, a_src, 3 * a_dst, heads, dim, slope=0.2)
    assert np.abs(three - four).max() > 1e-3


def test_gat_two_neighbour_closed_form():
    # one destination (2) with in-neighbours 0 and 1, one head of width 1
    z = np.array([[1.0], [-2.0], [0.5]], np.float32)
    a_src = np.array([[0.7]], np.float32)
    a_dst = np.array([[-0.3]], np.float32)
    src = np.array([0, 1], np.int32)
    dst = np.array([2, 2], np.int32)
    row_ptr, col, _ = orc.build_csr(3, src, dst, 0)
    got, _ = orc.aggregate_gat(row_ptr, col, z, a_src, a_dst, 1, 1, slope=0.2)
    as_, ad = float(np.float32(0.7)), float(np.float32(-0.3))
    e0 = as_ * 1.0 + ad * 0.5                     # 0.55  -> positive branch
    e1 = 0.2 * (as_ * -2.0 + ad * 0.5)            # negative branch scaled by the slope
    w0, w1 = np.exp(e0), np.exp(e1)
    np.testing.assert_allclose(got[2, 0], (w0 * 1.0 + w1 * -2.0) / (w0 + w1), rtol=1e-14)
    assert got[0, 0] == 0 and got[1, 0] == 0


# ------------------------------------------------------------------ invariants

def _small_workload(seed=0):
    n = 300
    src, dst = gg.powerlaw_graph(n, 3000, 2.1, None, seed)
    return n, src, dst


def test_chunked_equals_unchunked_bitwise():
    n, src, dst = _small_workload()
    f = 13
    x = gg.features_f32(n, f, dist="normal", p0=0, p1=1, seed=1)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    for model in ("gcn", "sage"):
        full, _ = orc.aggregate(model, row_ptr, col, x, f, f)
        for width in range(1, f + 1):
            got, _ = orc.aggregate(model, row_ptr, col, x, f, width)
            np.testing.assert_array_equal(got, full)
    heads, dim = 2, 6
    z = gg.features_f32(n, heads * dim, dist="normal", p0=0, p1=1, seed=2)
    a_src = gg.features_f32(heads, dim, seed=1, stream=5)
    a_dst = gg.features_f32(heads, dim, seed=1, stream=6)
    full, _ = orc.aggregate_gat(row_ptr, col, z, a_src, a_dst, heads, dim)
    for width in range(1, heads * dim + 1):
        got, _ = orc.aggregate_gat(row_ptr, col, z, a_src, a_dst, heads, dim, chunk_width=width)
        np.testing.assert_array_equal(got, full)


def test_mean_of_constant_and_linearity():
    n, src, dst = _small_workload(1)
    row_ptr, col, _ = orc.build_csr(n, src, dst, 0)
    deg = np.diff(row_ptr)
    const = np.full((n, 2), -1.75, np.float32)
    got, _ = orc.aggregate("sage", row_ptr, col, const, 2)
    np.testing.assert_allclose(got[deg > 0], -1.75, rtol=1e-14)
    assert (got[deg == 0] == 0).all()
    x = gg.features_f32(n, 6, seed=3)
    y = gg.features_f32(n, 6, seed=4)
    comb = (np.float32(2.0) * x + np.float32(0.5) * y).astype(np.float32)
    for model in ("gcn", "sage"):
        ax, _ = orc.aggregate(model, row_ptr, col, x, 6)
        ay, _ = orc.aggregate(model, row_ptr, col, y, 6)
        ac, ab = orc.aggregate(model, row_ptr, col, comb, 6)
        assert (np.abs(ac - (2.0 * ax + 0.5 * ay)) <= 1e-6 * ab + 1e-9).all()


def test_rows_subset_matches_full():
    n, src, dst = _small_workload(2)
    x = gg.features_f32(n, 7, seed=5)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    rows = np.array([0, 17, 299, 5, 5], np.int64)
    for model in ("gcn", "sage"):
        full, fab = orc.aggregate(model, row_ptr, col, x, 7, 3)
        sub, sab = orc.aggregate(model, row_ptr, col, x, 7, 3, rows=rows)
        np.testing.assert_array_equal(sub, full[rows])
        np.testing.assert_array_equal(sab, fab[rows])
    a = gg.features_f32(1, 7, seed=1, stream=5)
    full, _ = orc.aggregate_gat(row_ptr, col, x, a, a, 1, 7)
    sub, _ = orc.aggregate_gat(row_ptr, col, x, a, a, 1, 7, rows=rows)
    np.testing.assert_array_equal(sub, full[rows])


def test_relabelling_equivariance():
    n, src, dst = _small_workload(3)
    x = gg.features_f32(n, 4, dist="normal", p0=0, p1=1, seed=6)
    pi = np.random.default_rng(1).permutation(n).astype(np.int32)       # old id -> new id
    xp = np.empty_like(x)
    xp[pi] = x
    rp0, c0, _ = orc.build_csr(n, src, dst, SL)
    rp1, c1, _ = orc.build_csr(n, pi[src], pi[dst], SL)
    for model in ("gcn", "sage"):
        a0, ab = orc.aggregate(model, rp0, c0, x, 4)
        a1, _ = orc.aggregate(model, rp1, c1, xp, 4)
        assert (np.abs(a1[pi] - a0) <= 1e-12 * ab + 1e-15).all()


def test_bf16_inputs_are_widened_exactly():
    n, src, dst = _small_workload(4)
    x = gg.features_f32(n, 8, seed=7)
    bits = gg.to_bf16_bits(x)
    widened = gg.bf16_bits_to_f32(bits)
    assert np.abs(widened - x).max() <= 2.0 ** -8 and not np.array_equal(widened, x)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    a, _ = orc.aggregate("gcn", row_ptr, col, bits, 8)
    b, _ = orc.aggregate("gcn", row_ptr, col, widened, 8)
    np.testing.assert_array_equal(a, b)


def test_row_parallel_oracle_is_identical():
    n, src, dst = _small_workload(5)
    x = gg.features_f32(n, 9, seed=8)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    one, _ = orc.aggregate("gcn", row_ptr, col, x, 9, 4, threads=1)
    many, _ = orc.aggregate("gcn", row_ptr, col, x, 9, 4, threads=4)
    np.testing.assert_array_equal(one, many)


def test_leading_dimension_padding_is_ignored():
    n, src, dst = _small_workload(6)
    x = gg.features_f32(n, 6, ld=8, seed=9, pad=np.nan)
    row_ptr, col, _ = orc.build_csr(n, src, dst, SL)
    a, _ = orc.aggregate("sage", row_ptr, col, x, 6, 4)
    b, _ = orc.aggregate("sage", row_ptr, col, np.ascontiguousarray(x[:, :6]), 6, 4)
    np.testing.assert_array_equal(a, b)


# ------------------------------------------------------------------ Combination (dense transform ahead of aggregation)

def test_combine_against_triple_loop_and_closed_forms():
    rng = np.random.default_rng(11)
    x = rng.standard_normal((7, 5)).astype(np.float32)
    w_t = rng.standard_normal((3, 5)).astype(np.float32)
    z, scale = orc.combine(x, w_t)
    for v in range(7):
        for j in range(3):
            acc = sum(float(x[v, k]) * float(w_t[j, k]) for k in range(5))
            assert abs(z[v, j] - acc) <= 1e-12 * (1 + abs(acc))
            assert abs(scale[v, j] - sum(abs(float(x[v, k]) * float(w_t[j, k])) for k in range(5))) <= 1e-12 * scale[v, j]
    # a transposed weight matrix must fail: w_t is [f_out, f_in], so x @ w_t.T, never x @ w_t
    sq = rng.standard_normal((5, 5)).astype(np.float32)
    assert not np.allclose(orc.combine(x, sq)[0], x.astype(np.float64) @ sq.astype(np.float64))
    # identity weights return x; all-ones weights return the row sums
    assert np.array_equal(orc.combine(x, np.eye(5, dtype=np.float32))[0], x.astype(np.float64))
    np.testing.assert_allclose(orc.combine(x, np.ones((2, 5), np.float32))[0],
                               np.repeat(x.astype(np.float64).sum(1)[:, None], 2, 1), rtol=1e-13)


def test_combine_tf32_reading_cuts_thirteen_mantissa_bits():
    one = np.float32(1.0)
    ulp_tf32 = np.float32(2.0 ** -10)
    x = np.array([[one + np.float32(2.0 ** -11), one + ulp_tf32, -(one + np.float32(2.0 ** -11)) - np.float32(2.0 ** -12)]],
                 np.float32)
    z, _ = orc.combine(x, np.eye(3, dtype=np.float32), tf32=True)
    # below the last kept bit: dropped (towards zero, for either sign); the last kept bit itself stays
    assert z[0, 0] == 1.0 and z[0, 1] == float(one + ulp_tf32) and z[0, 2] == -1.0
    # the cut never moves a value by more than 2^-10 relative, so a product by less than 2^-9
    rng = np.random.default_rng(12)
    a = rng.standard_normal((40, 30)).astype(np.float32)
    b = rng.standard_normal((20, 30)).astype(np.float32)
    exact, scale = orc.combine(a, b)
    cut, _ = orc.combine(a, b, tf32=True)
    assert (np.abs(cut - exact) <= 2.0 ** -9 * scale).all() and np.abs(cut - exact).max() > 0
