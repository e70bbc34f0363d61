"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, validates arguments before any launch, and plans decompositions."""
import ctypes
import os
import re

import pytest

from paper_2407_02891_b200 import binding as bq
from paper_2407_02891_b200 import build as bq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    bq_build.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "bcq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bcq_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert len(names) >= 15
    L = ctypes.CDLL(bq.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(bq.SIGNATURES), "binding and header disagree"
    assert bq.lib().bcq_version() == 220


def test_status_strings():
    for s in (0, -1, -2, -3, -4, -5):
        assert bq.lib().bcq_status_string(s)
    assert bq.lib().bcq_status_string(-99) == b"unknown status"


def test_desc_validation_and_sizes():
    d = bq.desc(7168, 7168, 3, 128, bq.LAYOUT_TILED)
    assert bq.check_desc(d) == bq.OK
    assert bq.packed_bytes(d) == 3 * 7168 * 7168 // 8 + 2 * 4 * 7168 * 56     # tiles carry the scales
    assert bq.packed_bytes(d.with_layout(bq.LAYOUT_CANONICAL)) == 3 * 7168 * 7168 // 8
    assert bq.packed_bytes(bq.desc(64, 1024, 2, 0, bq.LAYOUT_TILED)) == 2 * 64 * 1024 // 8
    assert bq.alpha_elems(d) == 3 * 7168 * 56 and bq.offset_elems(d) == 7168 * 56
    assert bq.offset_elems(bq.desc(16, 32, 3, 0)) == 16
    for g in (64, 32):                                                           # smaller groups: more scales in the tiles
        assert bq.packed_bytes(bq.desc(64, 1024, 3, g, bq.LAYOUT_TILED)) == 3 * 64 * 1024 // 8 + 2 * 4 * 64 * (1024 // g)
    bad = [(0, 32, 3, 32, 0, bq.ERR_INVALID_ARG), (16, 32, 0, 32, 0, bq.ERR_INVALID_ARG),
           (16, 32, 5, 32, 0, bq.ERR_INVALID_ARG), (16, 32, 3, 32, 7, bq.ERR_INVALID_ARG),
           (16, 40, 3, 0, 0, bq.ERR_UNSUPPORTED_SHAPE), (16, 96, 3, 64, 0, bq.ERR_UNSUPPORTED_SHAPE),
           (16, 96, 3, 48, 0, bq.ERR_UNSUPPORTED_SHAPE), (16, 256, 3, 128, 1, bq.ERR_UNSUPPORTED_SHAPE),
           (12, 512, 3, 128, 1, bq.ERR_UNSUPPORTED_SHAPE), (16, 512, 3, 256, 1, bq.ERR_UNSUPPORTED_SHAPE)]
    for N, K, q, g, lay, want in bad:
        d = bq.desc(N, K, q, g, lay)
        assert bq.check_desc(d) == want, (N, K, q, g, lay)
        assert bq.packed_bytes(d) == 0 and bq.alpha_elems(d) == 0 and bq.offset_elems(d) == 0


def test_null_and_misaligned_pointers_are_rejected_before_any_launch():
    L = bq.lib()
    d = bq.desc(64, 512, 3, 128, bq.LAYOUT_CANONICAL)
    plan = bq.Plan(0, 8, 1, 0)
    ok = ctypes.c_void_p(0x10000)   # never dereferenced: every call below fails validation first
    odd = ctypes.c_void_p(0x10004)
    call = lambda *ptrs: L.bcq_gemv_plan(ctypes.byref(d), ctypes.byref(plan), *ptrs, None, 0, None)
    assert call(None, ok, ok, ok, ok) == bq.ERR_INVALID_ARG
    assert call(ok, None, ok, ok, ok) == bq.ERR_INVALID_ARG      # canonical operands need alpha and z
    assert call(ok, ok, ok, ok, None) == bq.ERR_INVALID_ARG
    assert call(odd, ok, ok, ok, ok) == bq.ERR_MISALIGNED
    assert call(ok, ok, ok, odd, ok) == bq.ERR_MISALIGNED
    assert L.bcq_gemv_plan(ctypes.byref(d), None, ok, ok, ok, ok, ok, None, 0, None) == bq.ERR_INVALID_ARG
    # a lookup-table plan on a canonical descriptor is invalid
    lut = bq.Plan(1, 1, 1, 0)
    assert L.bcq_gemv_plan(ctypes.byref(d), ctypes.byref(lut), ok, ok, ok, ok, ok, None, 0, None) == bq.ERR_INVALID_ARG
    # split-K without (enough) workspace
    dt = bq.desc(64, 1024, 3, 128, bq.LAYOUT_TILED)
    split = bq.Plan(1, 1, 2, 0)
    need = bq.workspace_bytes(dt, 1, split)
    assert need == 64 * 8                    # one 64-bit split-K word per row
    args = (ctypes.byref(dt), ctypes.byref(split), ok, ok, ok, ok, ok)
    assert L.bcq_gemv_plan(*args, None, 0, None) == bq.ERR_INVALID_ARG
    assert L.bcq_gemv_plan(*args, ok, need - 1, None) == bq.ERR_WORKSPACE_TOO_SMALL
    assert L.bcq_gemv_plan(*args, odd, need, None) == bq.ERR_MISALIGNED
    # plans that break the limits
    for p in (bq.Plan(1, 0, 1, 0), bq.Plan(1, 9, 1, 0), bq.Plan(1, 1, 3, 0), bq.Plan(2, 1, 1, 0)):
        assert L.bcq_gemv_plan(ctypes.byref(dt), ctypes.byref(p), ok, ok, ok, ok, ok, ok, 1 << 20, None) == bq.ERR_INVALID_ARG
    big = bq.desc(2048, 512, 3, 128, bq.LAYOUT_TILED)     # 256 units in one row block > 184
    p = bq.Plan(1, 1, 1, 0)
    assert L.bcq_gemv_plan(ctypes.byref(big), ctypes.byref(p), ok, ok, ok, ok, ok, None, 0, None) == bq.ERR_INVALID_ARG
    # batch limits
    assert L.bcq_gemm_smallbatch(ctypes.byref(d), ok, ok, ok, ok, ok, 17, None, 0, None) == bq.ERR_INVALID_ARG
    assert L.bcq_gemm_smallbatch(ctypes.byref(d), ok, ok, ok, ok, ok, 0, None, 0, None) == bq.ERR_INVALID_ARG
    assert L.bcq_gemm_smallbatch(ctypes.byref(d), ok, ok, ok, odd, ok, 2, None, 0, None) == bq.ERR_MISALIGNED


def test_merge_and_pack_argument_checks():
    L = bq.lib()
    d = bq.desc(16, 32, 3, 32)
    ok = ctypes.c_void_p(0x10000)
    b2p = (ctypes.c_uint8 * 4)(0, 1, 2, 2)
    bp = ctypes.cast(b2p, ctypes.c_void_p)
    m = lambda dd, n_bits, table: L.bcq_merge_linear(ctypes.byref(dd), ok, ok, ok, n_bits, table, ok, ok, ok, None)
    assert m(d, 9, bp) == bq.ERR_INVALID_ARG
    assert m(d, 2, bp) == bq.ERR_INVALID_ARG                       # q > n_bits
    assert m(d, 4, None) == bq.ERR_INVALID_ARG
    unused = (ctypes.c_uint8 * 4)(0, 0, 2, 2)                      # plane 1 has no bit
    assert m(d, 4, ctypes.cast(unused, ctypes.c_void_p)) == bq.ERR_INVALID_ARG
    toobig = (ctypes.c_uint8 * 4)(0, 1, 2, 3)
    assert m(d, 4, ctypes.cast(toobig, ctypes.c_void_p)) == bq.ERR_INVALID_ARG
    assert L.bcq_pack(ctypes.byref(d), None, None, None, ok, None, None, None) == bq.ERR_INVALID_ARG
    assert L.bcq_pack(ctypes.byref(d), ok, ok, None, ok, ok, ok, None) == bq.ERR_INVALID_ARG
    d2 = bq.desc(16, 64, 3, 32)
    assert L.bcq_repack(ctypes.byref(d), ok, None, None, ctypes.byref(d2), ok, None, None, None) == bq.ERR_INVALID_ARG
    assert L.bcq_repack(ctypes.byref(d), ok, None, None, ctypes.byref(d), ok, None, None, None) == bq.ERR_INVALID_ARG  # in place
    dc, dtl = bq.desc(64, 512, 3, 128), bq.desc(64, 512, 3, 128, bq.LAYOUT_TILED)
    ok2 = ctypes.c_void_p(0x20000)
    # a tiled operand cannot be made without its scales; bcq_pack needs them too
    assert L.bcq_repack(ctypes.byref(dc), ok, None, None, ctypes.byref(dtl), ok2, None, None, None) == bq.ERR_INVALID_ARG
    assert L.bcq_pack(ctypes.byref(dtl), ok, None, None, ok2, None, None, None) == bq.ERR_INVALID_ARG


@pytest.mark.parametrize("N,K", [(7168, 7168), (28672, 7168), (7168, 28672), (1024, 1024), (4096, 4096),
                                 (16384, 4096), (4096, 16384), (9216, 9216), (36864, 9216), (9216, 36864),
                                 (8192, 8192), (2048, 8192), (28672, 8192), (8192, 28672), (8, 512)])
def test_default_plan_is_valid_and_fills_the_gpu(N, K):
    d = bq.desc(N, K, 3, 128, bq.LAYOUT_TILED)
    p = bq.plan_default(d, 1, 148)
    assert p.kernel == 1
    U, W = N // 8, K // 512
    assert 1 <= p.row_blocks <= U and 1 <= p.k_splits <= W
    assert -(-U // p.row_blocks) <= 184 and -(-W // p.k_splits) <= 32
    blocks = p.row_blocks * p.k_splits
    if U * W >= 148 * 8:
        assert blocks >= 0.7 * 148
    assert bq.workspace_bytes(d, 1, p) == (0 if p.k_splits == 1 else N * 8)   # lookup-table kernel: a word per row
    # canonical descriptors and batches > 1 use the generic kernel
    assert bq.plan_default(bq.desc(N, K, 3, 128), 1, 148).kernel == 0
    for B in (2, 3, 4):                                    # up to four columns: the lookup-table kernel on column pairs
        p2 = bq.plan_default(d, B, 148)                    # (its own decomposition: the pair kernel has other rings)
        assert p2.kernel == 1 and 1 <= p2.row_blocks <= U and 1 <= p2.k_splits <= W
        assert -(-U // p2.row_blocks) <= 184 and -(-W // p2.k_splits) <= 32
    for B in (5, 8, 16):                                   # more: one pass of the tensor-core kernel
        pb = bq.plan_default(d, B, 148)
        assert pb.kernel == 2
        assert 1 <= pb.row_blocks <= U and 1 <= pb.k_splits <= W
        assert -(-U // pb.row_blocks) <= 176 and -(-W // pb.k_splits) <= 32
        assert bq.workspace_bytes(d, B, pb) == (0 if pb.k_splits == 1 else 4096 * 4 + pb.k_splits * B * N * 4)
        # a lookup-table plan runs the columns two at a time: partial sums of two columns
        assert bq.workspace_bytes(d, B, p) == (0 if p.k_splits == 1 else 2 * N * 8)   # a word per row and column
    assert bq.workspace_bytes(d, 1, bq.plan_default(d, 8, 148)) == 0        # the small-batch kernel needs B >= 2
    assert bq.plan_default(bq.desc(N, K, 2, 0, bq.LAYOUT_TILED), 4, 148).kernel == 2    # one scale per row: no column pairs
    assert bq.plan_default(bq.desc(N, K, 2, 0, bq.LAYOUT_TILED), 1, 148).kernel == 1     # one scale per row


def test_default_plans_are_remembered_consistently():
    """bcq_plan_default keeps its last plans in a small table: more shapes than the table holds, asked
    twice in different orders and for different batches, always give the same plan."""
    shapes = [(512 * k, 4096) for k in range(1, 50)]
    first = {}
    for B in (1, 8):
        for (N, K) in shapes:
            p = bq.plan_default(bq.desc(N, K, 3, 128, bq.LAYOUT_TILED), B, 148)
            first[(N, K, B)] = (p.kernel, p.row_blocks, p.k_splits)
    for (N, K) in reversed(shapes):
        for B in (8, 1):
            p = bq.plan_default(bq.desc(N, K, 3, 128, bq.LAYOUT_TILED), B, 148)
            assert first[(N, K, B)] == (p.kernel, p.row_blocks, p.k_splits)
    # a different GPU size is a different entry
    a = bq.plan_default(bq.desc(7168, 7168, 3, 128, bq.LAYOUT_TILED), 1, 148)
    b = bq.plan_default(bq.desc(7168, 7168, 3, 128, bq.LAYOUT_TILED), 1, 64)
    assert a.row_blocks * a.k_splits <= 148 and b.row_blocks * b.k_splits <= 2 * 64
    assert (a.row_blocks, a.k_splits) != (b.row_blocks, b.k_splits)


def test_multi_row_blocks_are_shared_in_proportion():
    d = bq.desc(7168 * 3, 7168, 3, 128, bq.LAYOUT_TILED)
    assert bq.multi_row_blocks(d, bq.Plan(1, 60, 7, 0), [7168, 7168, 7168]) == [20, 20, 20]
    assert bq.multi_row_blocks(d, bq.Plan(1, 61, 7, 0), [7168, 7168, 7168]) == [21, 20, 20]
    d = bq.desc(8192 + 2048, 8192, 3, 128, bq.LAYOUT_TILED)          # a query projection and a fused k/v (GQA)
    assert bq.multi_row_blocks(d, bq.Plan(1, 20, 7, 0), [8192, 2048]) == [16, 4]
    assert bq.multi_row_blocks(d, bq.Plan(1, 18, 7, 0), [8192, 2048]) == [14, 4]      # 14.4 and 3.6: the remainder goes to 3.6
    with pytest.raises(bq.BcqError):                                  # rows do not add up to desc.N
        bq.multi_row_blocks(d, bq.Plan(1, 20, 7, 0), [8192, 1024])
    with pytest.raises(bq.BcqError):                                  # 1024 row units in 5 row blocks: more than 184 each
        bq.multi_row_blocks(d, bq.Plan(1, 6, 7, 0), [8192, 2048])
    with pytest.raises(bq.BcqError):                                  # fewer row blocks than operands
        bq.multi_row_blocks(d, bq.Plan(1, 1, 7, 0), [8192, 2048])


def test_search_host_helpers_agree_with_the_oracle():
    """The enumeration of bit partitions and the scale-factor grid are host code: compared with the
    oracle's own enumeration (written independently) without touching a GPU."""
    import numpy as np
    import oracle
    for (n, q) in [(1, 1), (2, 1), (3, 2), (4, 3), (5, 3), (5, 2), (4, 4), (6, 4), (8, 2)]:
        got = bq.partitions(n, q)
        want = np.array(oracle.set_partitions(n, q))
        assert got.shape == want.shape and (got == want).all()
    assert bq.lib().bcq_partition_count(3, 4) == 0 and bq.lib().bcq_partition_count(9, 2) == 0
    for n in (2, 3, 4, 5):
        np.testing.assert_allclose(bq.reexplore_factors(n, 7), oracle.reexplore_factors(n, 7), rtol=1e-15)
    d = bq.desc(256, 512, 3, 128)
    L = bq.lib()
    assert L.bcq_grid_search_workspace(ctypes.byref(d), 64, 4, 6, 3, 1) > 256 * 512
    assert L.bcq_grid_search_workspace(ctypes.byref(d), 24, 4, 6, 3, 1) == 0      # T not a multiple of 16
    assert L.bcq_grid_search_workspace(ctypes.byref(d), 64, 7, 6, 3, 1) == 0      # more than 6 step-1 bits
    assert L.bcq_grid_search_workspace(ctypes.byref(bq.desc(256, 512, 3, 96)), 64, 4, 6, 3, 1) == 0


def test_default_plans_are_valid_for_every_layout_variant():
    """Seeded sweep over shapes, plane counts, scaling units and batches: the planner's choice always passes
    the library's own plan check (workspace query non-failing, limits respected).  Host logic only."""
    import numpy as np
    rng = np.random.default_rng(7)
    for _ in range(300):
        N = 8 * int(rng.integers(1, 6000))
        K = 512 * int(rng.integers(1, 80))
        q = int(rng.integers(1, 5))
        group = int(rng.choice([0, 32, 64, 128]))
        B = int(rng.choice([1, 2, 3, 4, 5, 8, 16]))
        d = bq.desc(N, K, q, group, bq.LAYOUT_TILED)
        assert bq.check_desc(d) == bq.OK
        p = bq.plan_default(d, B, 148)
        U, W = N // 8, K // 512
        assert p.kernel in (1, 2) and 1 <= p.row_blocks <= U and 1 <= p.k_splits <= W
        assert -(-W // p.k_splits) <= 32
        if group in (32, 64):
            assert p.kernel == 1                              # no tensor-core kernel for the small groups
        need = bq.workspace_bytes(d, B, p)
        assert (need == 0) == (p.k_splits == 1)
        if p.kernel == 1:
            cols = 2 if (group == 128 and B >= 2) else 1
            assert need in (0, cols * N * 8)
