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
