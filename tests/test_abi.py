"""The C-ABI library builds for sm_100a, loads without a GPU and exports what include/gnnfd.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gnnfd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gnnfd_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2104_03058_b200 import build
    path = build.build_library()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert len(names) >= 15 and "gnnfd_build_csr" in names and "gnnfd_edge_softmax" in names
    for name in names:
        assert hasattr(lib, name), name


def test_host_only_entry_points_work_without_a_device():
    import paper_2104_03058_b200 as g
    assert g.lib().gnnfd_status_string(0) == b"ok"
    assert b"range" in g.lib().gnnfd_status_string(g.BAD_INDEX)
    pb, sb = g.csr_workspace_bytes(1000, 10_000, g.CSR_ADD_SELF_LOOPS | g.CSR_SYMMETRIZE)
    m = 2 * 10_000 + 1000
    assert pb >= 3 * 4 * m and sb >= 2 * 8 * m          # col_idx, perm, weights; two buffers of 64-bit sort words
    try:
        g.csr_workspace_bytes(10, -1, 0)
    except g.GnnfdError as err:
        assert err.status == g.INVALID_ARG
    else:
        raise AssertionError("negative edge count accepted")
    assert g.launch_count() >= 0


def test_header_constants_match_binding():
    import paper_2104_03058_b200 as g
    text = open(os.path.join(ROOT, "include", "gnnfd.h")).read()
    assert int(re.search(r"#define GNNFD_HUB_DEGREE (\d+)", text).group(1)) == g.HUB_DEGREE
    assert int(re.search(r"#define GNNFD_HUB_SEGMENT (\d+)", text).group(1)) == g.HUB_SEGMENT
    for name, val in (("ADD_SELF_LOOPS", 1), ("DEDUP", 2), ("SYMMETRIZE", 4)):
        assert int(re.search(r"GNNFD_CSR_%s = (\d+)" % name, text).group(1)) == val == getattr(g, "CSR_" + name)


def test_default_chunk_candidates_are_host_only():
    import torch

    import paper_2104_03058_b200 as g
    assert g.default_chunk_candidates(602) == [602, 256, 128, 64, 32, 16, 8]
    assert g.default_chunk_candidates(64) == [64, 32, 16, 8]
    assert g.default_chunk_candidates(8, torch.bfloat16) == [8]
    assert g.default_chunk_candidates(256, torch.bfloat16) == [256, 128, 64, 32, 16]
