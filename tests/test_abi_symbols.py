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


def test_workspace_plan_properties_on_the_host():
    """The shape-bucketed planner is pure host arithmetic: both orientations of
    one (min, max) share a bucket, buckets share the chunk buffers (the
    workspace follows the largest bucket, not the sum), and a bucket above the
    chunk limit is cut into chunks that reuse them."""
    from paper_2502_16982_b200 import binding as b

    bf = b.MUON_DTYPE_BF16

    def ws(shapes):
        return b.muon_workspace_bytes(b.shape_only_groups(shapes), len(shapes))

    one = ws([(2048, 1408, 8, bf, bf)])
    both = ws([(2048, 1408, 4, bf, bf), (1408, 2048, 4, bf, bf)])
    assert abs(both - one) <= 4096  # same bucket of 8 matrices (one more group header at most)
    small = ws([(256, 256, 8, bf, bf)])
    mixed = ws([(2048, 1408, 8, bf, bf), (256, 256, 8, bf, bf)])
    assert mixed < one + small and mixed >= one  # chunk buffers shared, per-matrix tables added
    per_matrix = (2 * 1408 * 2048 + 2 * 1408 * 1408) * 2
    assert one >= 8 * per_matrix
    prev = b.muon_debug_set_chunk_bytes(2 * per_matrix + 1024)
    try:
        chunked = ws([(2048, 1408, 8, bf, bf)])
    finally:
        b.muon_debug_set_chunk_bytes(prev)
    assert chunked < 4 * per_matrix  # two matrices per chunk instead of eight
    # fp32 and bf16 weights of one shape are different buckets but still share the buffers
    assert ws([(512, 512, 2, b.MUON_DTYPE_FP32, bf), (512, 512, 2, bf, bf)]) < 2 * ws([(512, 512, 2, bf, bf)])


def test_bucket_plan_groups_by_sides_and_dtypes_on_the_host():
    """muon_plan_buckets: matrices share a bucket exactly when short side, long
    side and both dtypes agree, whatever their orientation; numbering is dense."""
    from paper_2502_16982_b200 import binding as b

    BF, FP = b.MUON_DTYPE_BF16, b.MUON_DTYPE_FP32
    shapes = [(2048, 1408, 4, BF, BF), (512, 4096, 2, BF, BF), (1408, 2048, 3, BF, BF),
              (2048, 1408, 1, FP, BF), (4096, 512, 1, BF, FP), (2048, 2048, 2, BF, BF)]
    bucket_of, n = b.muon_plan_buckets(shapes)
    keys = []
    for r, c, cnt, wd, gd in shapes:
        keys += [(min(r, c), max(r, c), wd, gd)] * cnt
    assert len(bucket_of) == len(keys) and sorted(set(bucket_of)) == list(range(n))
    assert n == len(set(keys)) == 5
    for i in range(len(keys)):
        for j in range(len(keys)):
            assert (bucket_of[i] == bucket_of[j]) == (keys[i] == keys[j])
    assert b.muon_plan_buckets(shapes) == (bucket_of, n)


def test_planned_flops_follow_the_pairing_policy_on_the_host():
    """muon_plan_flops: 3 m^2 n + m^3 per iteration as the algorithmic count; the
    planned count replaces every two iterations of a wide matrix by
    3 m^2 n + 5 m^3; the knob switches the pairing off and on."""
    from paper_2502_16982_b200 import binding as b

    prev = b.muon_debug_set_pair_fold(0)
    try:
        one = lambda m, n: 3.0 * m * m * n + float(m) ** 3
        two = lambda m, n: 3.0 * m * m * n + 5.0 * float(m) ** 3
        shapes = [(2048, 8192, 2), (1408, 2048, 3), (8192, 2048, 1), (128, 4096, 1), (2048, 2048, 2)]
        alg, planned = b.muon_plan_flops(shapes, 5)
        assert alg == 5 * (3 * one(2048, 8192) + 3 * one(1408, 2048) + one(128, 4096) + 2 * one(2048, 2048))
        # default: from 256 rows and a long side of 1.25 x the short side, the first two iterations
        first_pair = lambda m, n: two(m, n) + 3 * one(m, n)
        assert planned == 3 * first_pair(2048, 8192) + 3 * first_pair(1408, 2048) + 5 * (one(128, 4096) + 2 * one(2048, 2048))
        b.muon_debug_set_pair_fold(1)
        assert b.muon_plan_flops([(2048, 8192, 2)], 5) == (10 * one(2048, 8192), 10 * one(2048, 8192))
        b.muon_debug_set_pair_fold(2)
        assert b.muon_plan_flops([(64, 64, 1)], 4)[1] == two(64, 64) + 2 * one(64, 64)
        b.muon_debug_set_pair_fold(3)   # wide: every pair; the others as by default
        assert b.muon_plan_flops([(2048, 8192, 1)], 5)[1] == 2 * two(2048, 8192) + one(2048, 8192)
        assert b.muon_plan_flops([(1408, 2048, 1)], 5)[1] == first_pair(1408, 2048)
        b.muon_debug_set_pair_fold(4)
        assert b.muon_plan_flops([(1408, 2048, 1)], 4)[1] == 2 * two(1408, 2048)
        assert b.muon_plan_flops([(1408, 2048, 1)], 1)[1] == one(1408, 2048)
        b.muon_debug_set_pair_fold(0)
        # pairs keep two more symmetric buffers per matrix
        BF = b.MUON_DTYPE_BF16
        shapes = b.shape_only_groups([(512, 2048, 4, BF, BF)])
        paired_bytes = b.muon_workspace_bytes(shapes, 1)
        b.muon_debug_set_pair_fold(1)
        plain_bytes = b.muon_workspace_bytes(shapes, 1)
        assert paired_bytes - plain_bytes >= 2 * 4 * 512 * 512 * 2
    finally:
        b.muon_debug_set_pair_fold(prev)
