"""The C-ABI library loads without a GPU and exports every function that
include/muon.h declares; the Python binding lists the same names."""

import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "muon.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(muon_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2502_16982_b200 import binding, build

    build.build()
    names = declared_functions()
    assert "muon_init" in names and "muon_step" in names and "muon_destroy" in names
    L = ctypes.CDLL(binding.LIB_PATH)
    for name in names:
        assert hasattr(L, name), name
    assert sorted(binding.EXPORTED) == names


def test_host_only_calls_work_without_a_gpu():
    """muon_workspace_bytes is pure host arithmetic; bad descriptors are
    rejected with a message and nothing else happens."""
    from paper_2502_16982_b200 import binding as b

    groups = b.shape_only_groups([(2048, 1408, 4, b.MUON_DTYPE_BF16, b.MUON_DTYPE_BF16)])
    nbytes = b.muon_workspace_bytes(groups, 1)
    # two X buffers and A, B for four matrices at least
    assert nbytes >= 4 * (2 * 1408 * 2048 + 2 * 1408 * 1408) * 2
    bad = b.shape_only_groups([(0, 5, 1, b.MUON_DTYPE_BF16, b.MUON_DTYPE_BF16)])
    try:
        b.muon_workspace_bytes(bad, 1)
        raise AssertionError("expected an error")
    except b.MuonError as e:
        assert e.code == b.MUON_ERR_INVALID_ARG
        assert "positive" in str(e)
