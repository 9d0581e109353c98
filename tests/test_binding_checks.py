"""Host-side operand checks of the Python binding: they must refuse, before any kernel is launched, the
shapes, devices and overlaps that would make a gather read or write outside its allocation.  The helper
functions take plain tensors, so they are exercised here on CPU tensors with a stand-in for the CSR handle."""
from types import SimpleNamespace

import pytest

torch = pytest.importorskip("torch")

from paper_2104_03058_b200 import binding as b  # noqa: E402


def fake_csr(n=10, nnz=30):
    return SimpleNamespace(n=n, nnz=nnz, device=torch.device("cpu"))


def test_too_few_rows_are_refused():
    csr = fake_csr(10)
    x, out = torch.zeros(10, 4), torch.zeros(10, 4)
    b._check_aggregate_operands(csr, x, out, 4)                      # exact fit passes
    with pytest.raises(ValueError, match="x has 9 rows"):
        b._check_aggregate_operands(csr, x[:9], out, 4)
    with pytest.raises(ValueError, match="out has 7 rows"):
        b._check_aggregate_operands(csr, x, out[:7], 4)
    with pytest.raises(ValueError, match="z has 3 rows"):
        b._check_aggregate_operands(csr, x[:3], out, 4, "z")


def test_other_device_is_refused():
    csr = SimpleNamespace(n=4, nnz=4, device=torch.device("cuda", 0))
    with pytest.raises(ValueError, match="x is on cpu but the CSR is on cuda:0"):
        b._check_aggregate_operands(csr, torch.zeros(4, 2), torch.zeros(4, 2), 2)
    b._same_device(torch.device("cpu"), a=torch.zeros(1), nothing=None)       # None operands are skipped


def test_overlapping_input_and_output_are_refused():
    csr = fake_csr(6)
    buf = torch.zeros(6, 16)
    with pytest.raises(ValueError, match="overlap"):
        b._check_aggregate_operands(csr, buf, buf, 16)                         # in place
    with pytest.raises(ValueError, match="overlap"):
        b._check_aggregate_operands(csr, buf[:, :8], buf[:, 4:12], 8)          # shifted column views
    # disjoint column ranges of one buffer interleave row by row without sharing an element: allowed
    b._check_aggregate_operands(csr, buf[:, :8], buf[:, 8:], 8)
    b._check_aggregate_operands(csr, buf[:, 10:16], buf[:, 2:10], 6)
    with pytest.raises(ValueError, match="overlap"):
        b._check_aggregate_operands(csr, buf[:, 10:16], buf[:, 2:11], 6)
    with pytest.raises(ValueError, match="overlap"):                           # same columns, rows shifted by one
        b._no_overlap(buf[:5, :8], buf[1:, :8], "x", "out")
    flat = torch.zeros(2 * 6 * 8)
    b._check_aggregate_operands(csr, flat[:48].view(6, 8), flat[48:].view(6, 8), 8)   # back to back: fine


def test_extent_of_strided_views():
    t = torch.zeros(5, 12)
    lo, hi = b._extent(t[:, 2:6])
    assert lo == t.data_ptr() + 2 * 4 and hi == t.data_ptr() + (4 * 12 + 5 + 1) * 4
    e = torch.zeros(0, 3)
    assert b._extent(e)[0] == b._extent(e)[1]


def test_attention_vector_shape_is_checked():
    with pytest.raises(ValueError, match="heads\\*dim = 6"):
        b._attention_vectors(torch.zeros(2, 2), torch.zeros(2, 3), 2, 3, torch.device("cpu"), None)
    a, c = b._attention_vectors(torch.zeros(2, 3, dtype=torch.float64), torch.ones(2, 3), 2, 3, torch.device("cpu"), None)
    assert a.dtype == torch.float32 and c.dtype == torch.float32
