"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs.  Integer / byte work must be bit-exact; products must satisfy
max|y_gpu - y_ref| <= 5e-3 * max|y_ref|."""
import numpy as np
import pytest
import torch

import oracle
from helpers import lut_max_units, TOL, make_layer, rel_err, tiled_operands
from paper_2407_02891_b200 import binding as bq
from paper_2407_02891_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def gpu_layer(N, K, q, group, layout, codes, alpha, z):
    return bq.pack_layer(N, K, q, group, layout, dev(codes), dev(alpha), dev(z))


def run_gemv(layer, x, plan=None):
    y = torch.full((layer.d.N,), float("nan"), dtype=torch.float16, device=DEV)
    xd = dev(x.reshape(-1))
    if plan is None:
        ws = bq.new_workspace(layer.d, 1)
        bq.gemv(layer.d, layer.packed, layer.alpha, layer.z, xd, y, ws)
    else:
        ws = bq.new_workspace(layer.d, 1, plan)
        bq.gemv_plan(layer.d, plan, layer.packed, layer.alpha, layer.z, xd, y, ws)
    torch.cuda.synchronize()
    return y.cpu().numpy().astype(np.float64)


# ---------------------------------------------------------------------------------------
# packing / repacking: bit-exact
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("N,K,q,group", [(16, 32, 3, 32), (16, 32, 3, 0), (40, 1024, 3, 128), (24, 512, 2, 128),
                                         (8, 1536, 4, 128), (72, 512, 1, 0), (13, 96, 3, 32)])
def test_pack_canonical_bit_exact(N, K, q, group):
    p, codes, alpha, z, _ = make_layer(f"pack/{N}x{K}", N, K, q, group)
    L = gpu_layer(N, K, q, group, bq.LAYOUT_CANONICAL, codes, alpha, z)
    assert np.array_equal(L.packed.cpu().numpy(), oracle.pack_canonical(codes, q).ravel())
    assert np.array_equal(L.alpha.cpu().numpy().view(np.uint16), alpha.ravel().view(np.uint16))
    assert np.array_equal(L.z.cpu().numpy().view(np.uint16), z.ravel().view(np.uint16))


@pytest.mark.parametrize("N,K,q,group", [(40, 1024, 3, 128), (24, 512, 2, 128), (8, 1536, 4, 128), (72, 512, 1, 0),
                                         (296, 2048, 3, 128), (64, 1024, 2, 0), (40, 1024, 3, 64), (24, 512, 2, 32),
                                         (8, 1536, 4, 32), (72, 512, 1, 64), (296, 2048, 3, 32), (64, 1024, 4, 64)])
def test_pack_tiled_and_repack_bit_exact(N, K, q, group):
    p, codes, alpha, z, _ = make_layer(f"tile/{N}x{K}", N, K, q, group)
    canon = oracle.pack_canonical(codes, q)
    want_p, want_a, want_z = tiled_operands(canon, alpha, z, group)
    T = gpu_layer(N, K, q, group, bq.LAYOUT_TILED, codes, alpha, z)
    assert T.packed.numel() == want_p.size == bq.packed_bytes(T.d)
    assert np.array_equal(T.packed.cpu().numpy(), want_p)
    if group == 0:
        assert np.array_equal(T.alpha.cpu().numpy().view(np.uint16), want_a.view(np.uint16))
        assert np.array_equal(T.z.cpu().numpy().view(np.uint16), want_z.view(np.uint16))
    else:
        assert T.alpha is None and T.z is None
    # canonical -> tiled via repack gives the same bytes; tiled -> canonical is the inverse
    C = gpu_layer(N, K, q, group, bq.LAYOUT_CANONICAL, codes, alpha, z)
    p2, a2, z2 = bq.empty_operands(T.d, DEV)
    p2.zero_()
    bq.repack(C.d, C.packed, C.alpha, C.z, T.d, p2, a2, z2)
    assert torch.equal(p2, T.packed)
    if group == 0:
        assert torch.equal(a2.view(torch.int16), T.alpha.view(torch.int16))
        assert torch.equal(z2.view(torch.int16), T.z.view(torch.int16))
    p3, a3, z3 = torch.zeros_like(C.packed), torch.zeros_like(C.alpha), torch.zeros_like(C.z)
    bq.repack(T.d, p2, a2, z2, C.d, p3, a3, z3)
    assert np.array_equal(p3.cpu().numpy(), canon.ravel())
    assert np.array_equal(a3.cpu().numpy().view(np.uint16), alpha.ravel().view(np.uint16))
    assert np.array_equal(z3.cpu().numpy().view(np.uint16), z.ravel().view(np.uint16))


# ---------------------------------------------------------------------------------------
# linear-int -> merged binary code: bit-exact codes, alpha, z
# ---------------------------------------------------------------------------------------

def _partitions(n, q):
    out = []

    def rec(i, assign, used):
        if i == n:
            if used == q:
                out.append(list(assign))
            return
        for j in range(min(used + 1, q)):
            rec(i + 1, assign + [j], max(used, j + 1))

    rec(0, [], 0)
    return out


@pytest.mark.parametrize("N,K,group,n,q", [(16, 32, 32, 4, 3), (16, 32, 0, 4, 3), (16, 32, 32, 5, 3),
                                           (64, 512, 128, 5, 2), (16, 32, 32, 3, 2), (24, 256, 64, 4, 4)])
def test_merge_linear_bit_exact(N, K, group, n, q):
    w, S, qbias = synth.linear_int_case(f"merge/n{n}", N, K, group, n)
    d = bq.desc(N, K, q, group)
    G = d.G
    for b2p in _partitions(n, q):
        codes = torch.zeros((N, K), dtype=torch.uint8, device=DEV)
        alpha = torch.zeros((q, N, G), dtype=torch.float16, device=DEV)
        z = torch.zeros((N, G), dtype=torch.float16, device=DEV)
        bq.merge_linear(d, dev(w), dev(S), dev(qbias), n, b2p, codes, alpha, z)
        rc, ra, rz = oracle.merge_linear(w, S, qbias, group, n, b2p)
        assert np.array_equal(codes.cpu().numpy(), rc)
        assert np.array_equal(alpha.cpu().numpy().view(np.uint16), ra.view(np.uint16))
        assert np.array_equal(z.cpu().numpy().view(np.uint16), rz.view(np.uint16))


def test_merge_linear_rounds_general_scales_like_the_oracle():
    """S, qbias with full 11-bit significands: alpha and z need a real rounding to fp16."""
    N, K, group, n, q = 32, 256, 64, 5, 3
    w, _, _ = synth.linear_int_case("merge/general", N, K, group, n)
    G = K // group
    S = (0.002 + 0.03 * synth.uniform("merge/general/S", 0, N * G)).astype(np.float16).reshape(N, G)
    qbias = (synth.normal("merge/general/b", 0, N * G) * 0.1).astype(np.float16).reshape(N, G)
    d = bq.desc(N, K, q, group)
    b2p = [0, 1, 1, 2, 2]
    codes = torch.zeros((N, K), dtype=torch.uint8, device=DEV)
    alpha = torch.zeros((q, N, G), dtype=torch.float16, device=DEV)
    z = torch.zeros((N, G), dtype=torch.float16, device=DEV)
    bq.merge_linear(d, dev(w), dev(S), dev(qbias), n, b2p, codes, alpha, z)
    rc, ra, rz = oracle.merge_linear(w, S, qbias, group, n, b2p)
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(alpha.cpu().numpy().view(np.uint16), ra.view(np.uint16))
    assert np.array_equal(z.cpu().numpy().view(np.uint16), rz.view(np.uint16))


def test_tiny_case_end_to_end():
    """16 x 32, 4-bit linear codes -> 3 planes -> pack -> product, against the oracle chain."""
    N, K, group, n, q = 16, 32, 32, 4, 3
    w, S, qbias = synth.linear_int_case("tiny/e2e", N, K, group, n)
    x = synth.activations("tiny/e2e", 1, K)
    d = bq.desc(N, K, q, group)
    for b2p in _partitions(n, q):
        codes = torch.zeros((N, K), dtype=torch.uint8, device=DEV)
        alpha = torch.zeros((q, N, 1), dtype=torch.float16, device=DEV)
        z = torch.zeros((N, 1), dtype=torch.float16, device=DEV)
        bq.merge_linear(d, dev(w), dev(S), dev(qbias), n, b2p, codes, alpha, z)
        L = bq.pack_layer(N, K, q, group, bq.LAYOUT_CANONICAL, codes, alpha, z)
        y = run_gemv(L, x)
        rc, ra, rz = oracle.merge_linear(w, S, qbias, group, n, b2p)
        ref = oracle.forward_dequant(rc, ra, rz, x, group)[0]
        assert rel_err(y, ref) <= TOL


# ---------------------------------------------------------------------------------------
# products
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("N,K,q,group", [(16, 32, 3, 32), (13, 96, 3, 32), (50, 256, 2, 64), (33, 1024, 4, 0),
                                         (1024, 1024, 3, 128), (7, 2048, 1, 128)])
def test_gemv_generic_kernel(N, K, q, group):
    p, codes, alpha, z, x = make_layer(f"gen/{N}x{K}", N, K, q, group)
    ref = oracle.forward_planes(p, alpha, z, x, group)[0]
    L = gpu_layer(N, K, q, group, bq.LAYOUT_CANONICAL, codes, alpha, z)
    assert rel_err(run_gemv(L, x), ref) <= TOL


LUT_SHAPES = [(1024, 1024, 3, 128), (8, 512, 3, 128), (296, 2048, 3, 128), (1000, 1536, 2, 128),
              (520, 3584, 3, 128), (64, 1024, 1, 128), (136, 1024, 4, 128), (4096, 4096, 3, 128),
              # one scale per row (the paper's granularity)
              (1024, 1024, 2, 0), (8, 512, 3, 0), (296, 2048, 2, 0), (520, 3584, 3, 0), (136, 1024, 4, 0),
              (64, 1024, 1, 0), (2304, 9216, 2, 0)]


@pytest.mark.parametrize("N,K,q,group", LUT_SHAPES)
def test_gemv_lut_kernel_default_plan(N, K, q, group):
    p, codes, alpha, z, x = make_layer(f"lut/{N}x{K}", N, K, q, group)
    ref = oracle.forward_planes(p, alpha, z, x, group)[0]
    L = gpu_layer(N, K, q, group, bq.LAYOUT_TILED, codes, alpha, z)
    assert bq.plan_default(L.d).kernel == 1
    assert rel_err(run_gemv(L, x), ref) <= TOL


@pytest.mark.parametrize("group", [128, 0])
@pytest.mark.parametrize("N,K,q,rb,ks", [(520, 3584, 3, 2, 1), (520, 3584, 3, 2, 7), (520, 3584, 3, 3, 2),
                                         (520, 3584, 3, 65, 3), (520, 3584, 3, 5, 4), (512, 1024, 2, 1, 1),
                                         (512, 1024, 2, 1, 2), (1000, 1536, 2, 125, 3), (1000, 1536, 2, 2, 1),
                                         (1472, 1024, 3, 1, 2), (4000, 512, 2, 3, 1)])
def test_gemv_lut_kernel_explicit_plans(N, K, q, rb, ks, group):
    """Ragged row blocks, one and several windows per block, with and without split-K."""
    p, codes, alpha, z, x = make_layer(f"lutp/{N}x{K}", N, K, q, group)
    ref = oracle.forward_planes(p, alpha, z, x, group)[0]
    L = gpu_layer(N, K, q, group, bq.LAYOUT_TILED, codes, alpha, z)
    assert rel_err(run_gemv(L, x, bq.Plan(1, rb, ks, 0)), ref) <= TOL


def test_gemv_workspace_is_reusable_and_result_deterministic():
    N, K, q = 520, 3584, 3
    p, codes, alpha, z, x = make_layer("lut/reuse", N, K, q, 128)
    L = gpu_layer(N, K, q, 128, bq.LAYOUT_TILED, codes, alpha, z)
    plan = bq.Plan(1, 3, 7, 0)
    ws = bq.new_workspace(L.d, 1, plan)
    xd = dev(x.reshape(-1))
    ys = []
    for _ in range(3):
        y = torch.zeros(N, dtype=torch.float16, device=DEV)
        bq.gemv_plan(L.d, plan, L.packed, L.alpha, L.z, xd, y, ws)
        ys.append(y)
    torch.cuda.synchronize()
    assert torch.equal(ys[0].view(torch.int16), ys[1].view(torch.int16))
    assert torch.equal(ys[0].view(torch.int16), ys[2].view(torch.int16))
    ref = oracle.forward_planes(p, alpha, z, x, 128)[0]
    assert rel_err(ys[2].cpu().numpy(), ref) <= TOL


@pytest.mark.parametrize("layout", [bq.LAYOUT_CANONICAL, bq.LAYOUT_TILED])
def test_gemv_structured_inputs(layout):
    N, K, q, group = 64, 1024, 3, 128
    p, codes, alpha, z, x = make_layer("struct", N, K, q, group)
    W = oracle.dequant(codes, alpha, z, group)
    L = gpu_layer(N, K, q, group, layout, codes, alpha, z)
    # unit vectors return columns of the dequantised matrix (rounded to fp16 once)
    for k in (0, 7, 8, 15, 16, 127, 128, 511, 512, 1023):
        e = np.zeros((1, K), np.float16)
        e[0, k] = 1.0
        y = run_gemv(L, e)
        assert np.abs(y - W[:, k]).max() <= 2.0 ** -10 * np.abs(W[:, k]).max() + 1e-7
    # all planes +1
    ones = np.full_like(codes, (1 << q) - 1)
    L1 = gpu_layer(N, K, q, group, layout, ones, alpha, z)
    ref = oracle.forward_dequant(ones, alpha, z, x, group)[0]
    assert rel_err(run_gemv(L1, x), ref) <= TOL
    # alpha = 0: only the offsets remain
    L0 = gpu_layer(N, K, q, group, layout, codes, np.zeros_like(alpha), z)
    ref = oracle.forward_dequant(codes, np.zeros_like(alpha), z, x, group)[0]
    assert rel_err(run_gemv(L0, x), ref) <= TOL
    # a single non-zero group
    xg = np.zeros((1, K), np.float16)
    xg[0, 384:512] = x[0, 384:512]
    ref = oracle.forward_dequant(codes, alpha, z, xg, group)[0]
    assert rel_err(run_gemv(L, xg), ref) <= TOL
    # negative and zero scales are legal
    a2 = alpha.copy()
    a2[1] = -a2[1]
    a2[2, ::2] = 0
    L2 = gpu_layer(N, K, q, group, layout, codes, a2, z)
    ref = oracle.forward_dequant(codes, a2, z, x, group)[0]
    assert rel_err(run_gemv(L2, x), ref) <= TOL


@pytest.mark.parametrize("layout,N,K,q,group", [(bq.LAYOUT_CANONICAL, 50, 256, 3, 64), (bq.LAYOUT_TILED, 264, 1024, 3, 128),
                                                (bq.LAYOUT_CANONICAL, 16, 32, 3, 32), (bq.LAYOUT_TILED, 64, 512, 2, 0)])
@pytest.mark.parametrize("B", [1, 2, 3, 4, 8, 16])
def test_gemm_smallbatch(layout, N, K, q, group, B):
    p, codes, alpha, z, X = make_layer(f"sb/{N}x{K}", N, K, q, group, B)
    ref = oracle.forward_planes(p, alpha, z, X, group)
    L = gpu_layer(N, K, q, group, layout, codes, alpha, z)
    Y = torch.full((B, N), float("nan"), dtype=torch.float16, device=DEV)
    ws = bq.new_workspace(L.d, B)
    bq.gemm_smallbatch(L.d, L.packed, L.alpha, L.z, dev(X), Y, B, ws)
    torch.cuda.synchronize()
    Yh = Y.cpu().numpy()
    assert rel_err(Yh, ref) <= TOL
    if B > 1:
        # permuting the batch permutes the result bit for bit
        perm = np.roll(np.arange(B), 1)
        Y2 = torch.zeros_like(Y)
        bq.gemm_smallbatch(L.d, L.packed, L.alpha, L.z, dev(X[perm]), Y2, B, ws)
        torch.cuda.synchronize()
        assert np.array_equal(Y2.cpu().numpy().view(np.uint16), Yh[perm].view(np.uint16))


@pytest.mark.parametrize("N,K,q,group,rb,ks,B", [
    (264, 1024, 3, 128, 1, 1, 2),      # 33 units: an odd number, the last pair is a single tile
    (264, 1024, 3, 128, 1, 2, 8),      # split-K, both windows apart
    (264, 2048, 3, 128, 3, 2, 16),     # 11 units per block, two windows per split, wide
    (1408, 1536, 3, 128, 1, 1, 5),     # 176 units: every warp four pairs, three windows
    (1408, 1536, 3, 128, 1, 3, 9),
    (776, 2560, 2, 128, 2, 1, 4),      # 97 units -> 48 + 49
    (776, 2560, 2, 0, 2, 5, 16),       # one scale per row
    (512, 1024, 1, 128, 4, 1, 3),
    (512, 1024, 4, 128, 4, 2, 12),
    (512, 1024, 4, 0, 1, 1, 7),
    (8, 512, 3, 128, 1, 1, 2),         # one unit, one window
    (16, 16384, 3, 128, 1, 1, 16),     # 32 windows in one block
])
def test_small_batch_kernel_explicit_plans(N, K, q, group, rb, ks, B):
    """The tensor-core small-batch kernel under decompositions chosen by the caller."""
    p, codes, alpha, z, X = make_layer(f"mma/{N}x{K}q{q}g{group}", N, K, q, group, B)
    ref = oracle.forward_planes(p, alpha, z, X, group)
    L = gpu_layer(N, K, q, group, bq.LAYOUT_TILED, codes, alpha, z)
    plan = bq.Plan(2, rb, ks, 0)
    ws = bq.new_workspace(L.d, B, plan)
    Y = torch.full((B, N), float("nan"), dtype=torch.float16, device=DEV)
    for _ in range(2):   # the second call finds the counters as the first one left them
        bq.gemm_smallbatch_plan(L.d, plan, L.packed, L.alpha, L.z, dev(X), Y, B, ws)
    torch.cuda.synchronize()
    bq.poll_status()
    assert rel_err(Y.cpu().numpy(), ref) <= TOL
    # through the lookup-table kernel (two columns per pass with group 128, one with per-row scales):
    # the same numbers up to rounding
    p1 = bq.plan_default(L.d, 1)
    Y1 = torch.zeros_like(Y)
    bq.gemm_smallbatch_plan(L.d, p1, L.packed, L.alpha, L.z, dev(X), Y1, B, bq.new_workspace(L.d, B, p1))
    torch.cuda.synchronize()
    bq.poll_status()
    assert rel_err(Y1.cpu().numpy(), ref) <= TOL


@pytest.mark.parametrize("N,K,q,rb,ks,B", [
    (264, 1024, 3, 1, 1, 2),       # 33 units, both windows in one block
    (264, 1024, 3, 1, 2, 2),       # split-K
    (1472, 1536, 3, 1, 3, 2),      # 184 units: every consumer warp eight units
    (776, 2560, 2, 2, 5, 3),       # a pair and a single column
    (512, 1024, 1, 4, 1, 4),
    (512, 1024, 4, 4, 2, 5),
    (8, 512, 3, 1, 1, 2),          # one unit, one window
    (16, 16384, 3, 1, 1, 2),       # 32 windows in one block
])
def test_lookup_kernel_on_column_pairs(N, K, q, rb, ks, B):
    """Plan kernel 1 with group 128 runs two columns per launch (both columns' sums in one table entry)."""
    group = 128
    p, codes, alpha, z, X = make_layer(f"pair/{N}x{K}q{q}", N, K, q, group, B)
    ref = oracle.forward_planes(p, alpha, z, X, group)
    L = gpu_layer(N, K, q, group, bq.LAYOUT_TILED, codes, alpha, z)
    plan = bq.Plan(1, rb, ks, 0)
    ws = bq.new_workspace(L.d, B, plan)
    Y = torch.full((B, N), float("nan"), dtype=torch.float16, device=DEV)
    for _ in range(2):   # the second call finds the counters as the first one left them
        bq.gemm_smallbatch_plan(L.d, plan, L.packed, L.alpha, L.z, dev(X), Y, B, ws)
    torch.cuda.synchronize()
    bq.poll_status()
    Yh = Y.cpu().numpy()
    assert rel_err(Yh, ref) <= TOL
    # each column equals the batch-1 product of that column bit for bit (same table values, same order of sums)
    y1 = torch.zeros(N, dtype=torch.float16, device=DEV)
    ws1 = bq.new_workspace(L.d, 1, plan)
    for b in range(B):
        bq.gemv_plan(L.d, plan, L.packed, L.alpha, L.z, dev(X[b]), y1, ws1)
        torch.cuda.synchronize()
        assert np.array_equal(y1.cpu().numpy().view(np.uint16), Yh[b].view(np.uint16))


def test_small_batch_kernel_structured_inputs():
    """Unit activations pick out single weights: exact values, every (row, k) position distinguishable."""
    N, K, q, group, B = 64, 1024, 3, 128, 16
    p, codes, alpha, z, _ = make_layer("mma/struct", N, K, q, group, B)
    L = gpu_layer(N, K, q, group, bq.LAYOUT_TILED, codes, alpha, z)
    rng = np.random.default_rng(5)
    ks = rng.choice(K, size=B, replace=False)
    X = np.zeros((B, K), np.float16)
    X[np.arange(B), ks] = 1.0
    ref = oracle.forward_planes(p, alpha, z, X, group)     # = column ks[b] of the dequantised matrix
    Y = torch.zeros((B, N), dtype=torch.float16, device=DEV)
    bq.gemm_smallbatch(L.d, L.packed, L.alpha, L.z, dev(X), Y, B, bq.new_workspace(L.d, B))
    torch.cuda.synchronize()
    got = Y.cpu().numpy().astype(np.float64)
    assert np.abs(got - ref).max() <= 2.0 ** -10 * np.abs(ref).max()


def test_gemv_host_buffers():
    N, K, q, group = 520, 3584, 3, 128
    p, codes, alpha, z, x = make_layer("host", N, K, q, group)
    L = gpu_layer(N, K, q, group, bq.LAYOUT_TILED, codes, alpha, z)
    xh = torch.from_numpy(x.reshape(-1).copy()).pin_memory()
    yh = torch.zeros(N, dtype=torch.float16).pin_memory()
    xs = torch.zeros(K, dtype=torch.float16, device=DEV)
    ys = torch.zeros(N, dtype=torch.float16, device=DEV)
    ws = bq.new_workspace(L.d, 1)
    bq.gemv_host(L.d, L.packed, L.alpha, L.z, xh, yh, xs, ys, ws)
    torch.cuda.synchronize()
    ref = oracle.forward_planes(p, alpha, z, x, group)[0]
    assert rel_err(yh.numpy(), ref) <= TOL
    # pageable host buffers take the staged path
    yp = torch.zeros(N, dtype=torch.float16)
    ys.zero_()
    bq.gemv_host(L.d, L.packed, L.alpha, L.z, torch.from_numpy(x.reshape(-1).copy()), yp, xs, ys, ws)
    torch.cuda.synchronize()
    assert np.array_equal(yp.numpy().view(np.uint16), yh.numpy().view(np.uint16))
    assert np.array_equal(ys.cpu().numpy().view(np.uint16), yh.numpy().view(np.uint16))   # staged through y_stage


def test_device_errors_are_reported_not_raised_as_faults():
    """Bad arguments come back as status codes through the binding, with the GPU untouched."""
    d = bq.desc(64, 1000, 3, 128)
    t = torch.zeros(64, dtype=torch.float16, device=DEV)
    with pytest.raises(bq.BcqError) as e:
        bq.gemv(d, t, t, t, t, t)
    assert e.value.status == bq.ERR_UNSUPPORTED_SHAPE
    bq.poll_status()        # no bounded wait ran out in any kernel launched so far


def test_random_shapes_batches_and_plans():
    """Seeded random cases over every kernel of the tiled layout: shapes (1..260 row units, 1..11 windows),
    q, scale granularity, batch, and decompositions (given and default), each against the oracle."""
    rng = np.random.default_rng(240702891)
    for case in range(48):
        q = int(rng.integers(1, 5))
        group = int(rng.choice([0, 128]))
        U, W = int(rng.integers(1, 260)), int(rng.integers(1, 12))
        N, K = 8 * U, 512 * W
        B = int(rng.choice([1, 1, 2, 3, 4, 5, 8, 9, 16]))
        kernel = int(rng.choice([1, 2])) if B >= 2 else 1
        ks = int(rng.integers(1, W + 1))
        rb_min = -(-U // (lut_max_units(q, group, B) if kernel == 1 else 176))
        rb = int(rng.integers(rb_min, min(U, rb_min + 6) + 1))
        p, codes, alpha, z, X = make_layer(f"random/{case}", N, K, q, group, B)
        ref = oracle.forward_planes(p, alpha, z, X, group)
        L = gpu_layer(N, K, q, group, bq.LAYOUT_TILED, codes, alpha, z)
        Y = torch.empty((B, N), dtype=torch.float16, device=DEV)
        for plan in (bq.Plan(kernel, rb, ks, 0), bq.plan_default(L.d, B)):
            ws = bq.new_workspace(L.d, B, plan)
            Y.fill_(float("nan"))
            for _ in range(2):
                bq.gemm_smallbatch_plan(L.d, plan, L.packed, L.alpha, L.z, dev(X), Y, B, ws)
            torch.cuda.synchronize()
            bq.poll_status()
            assert rel_err(Y.cpu().numpy(), ref) <= TOL, (case, N, K, q, group, B, plan.kernel, plan.row_blocks, plan.k_splits)


def _heavy_tailed(kind, K, name):
    """Activations with the outliers LLM hidden states have: fp16, the bulk N(0,1)."""
    x = synth.normal(name + "/x", 0, K)
    u = synth.uniform(name + "/pick", 0, K)
    if kind == "outliers_x50":               # one value in a hundred is fifty times larger
        x = np.where(u < 0.01, 50.0 * x, x)
    elif kind == "spikes_1e2_1e4":           # a few spikes of 1e2 .. 1e4 in every window of 512
        for w in range(K // 512):
            for j, mag in enumerate((1e2, -1e3, 1e4)):
                x[512 * w + int(u[512 * w + j] * 512)] = mag
    elif kind == "near_table_limit":         # one chunk of eight same-sign values whose sum is just below the
        x[8 * 37:8 * 37 + 8] = 8000.0        # largest finite fp16 (64000 < 65504), another with the opposite sign
        x[8 * 101:8 * 101 + 8] = -8000.0
    elif kind == "cancelling":               # large values that cancel inside a chunk: the table entry is small,
        x[8 * 5:8 * 5 + 8] = [3000.0, -3000.0, 2000.0, -2000.0, 1000.0, -1000.0, 0.5, -0.25]   # its terms are not
    return x.astype(np.float16).reshape(1, K)


@pytest.mark.parametrize("group", [128, 0])
@pytest.mark.parametrize("kind", ["outliers_x50", "spikes_1e2_1e4", "near_table_limit", "cancelling"])
def test_gemv_heavy_tailed_activations(kind, group):
    """The lookup tables hold fp16 sums of 8 activations (one rounding each, relative 2^-11): the product
    must stay inside the stated tolerance when the activations have outliers, up to the documented limit
    (every 8-activation sum finite in fp16)."""
    N, K, q = 1024, 4096, 3
    p, codes, alpha, z, _ = make_layer(f"tails/{group}", N, K, q, group)
    x = _heavy_tailed(kind, K, f"tails/{kind}")
    ref = oracle.forward_planes(p, alpha, z, x, group)[0]
    L = gpu_layer(N, K, q, group, bq.LAYOUT_TILED, codes, alpha, z)
    assert bq.plan_default(L.d).kernel == 1
    y = run_gemv(L, x)
    assert np.isfinite(y).all()
    assert rel_err(y, ref) <= TOL
    # two columns per launch build their tables the same way
    if group:
        X = np.concatenate([x, synth.activations("tails/col1", 1, K)])
        Y = torch.zeros((2, N), dtype=torch.float16, device=DEV)
        bq.gemm_smallbatch(L.d, L.packed, L.alpha, L.z, dev(X), Y, 2, bq.new_workspace(L.d, 2))
        torch.cuda.synchronize()
        assert rel_err(Y.cpu().numpy(), oracle.forward_planes(p, alpha, z, X, group)) <= TOL


def test_operands_rewritten_in_place_between_two_products():
    """The products fetch packed operands before they wait for the kernel in front of them; operands
    written by the library's own calls must still be complete.  Pack layer A, multiply, pack layer B into
    the SAME buffers, multiply again at once: the second result is B's, for each way of writing operands."""
    N, K, q, group = 2048, 4096, 3, 128
    pa, ca, aa, za, x = make_layer("inplace/A", N, K, q, group)
    pb, cb, ab, zb, _ = make_layer("inplace/B", N, K, q, group)
    ref_b = oracle.forward_planes(pb, ab, zb, x, group)[0]
    d = bq.desc(N, K, q, group, bq.LAYOUT_TILED)
    dc = d.with_layout(bq.LAYOUT_CANONICAL)
    packed, _, _ = bq.empty_operands(d, DEV)
    xd = dev(x.reshape(-1))
    ws = bq.new_workspace(d, 1)
    ya = torch.zeros(N, dtype=torch.float16, device=DEV)
    yb = torch.zeros(N, dtype=torch.float16, device=DEV)
    codes_a, codes_b = dev(ca), dev(cb)
    canon_b = dev(pb.reshape(-1))
    for how in ("pack", "repack"):
        for _ in range(3):
            bq.pack(d, codes_a, dev(aa), dev(za), packed, None, None)
            bq.gemv(d, packed, None, None, xd, ya, ws)
            if how == "pack":
                bq.pack(d, codes_b, dev(ab), dev(zb), packed, None, None)
            else:
                bq.repack(dc, canon_b, dev(ab), dev(zb), d, packed, None, None)
            bq.gemv(d, packed, None, None, xd, yb, ws)          # no synchronisation in between
        torch.cuda.synchronize()
        bq.poll_status()
        assert rel_err(yb.cpu().numpy(), ref_b) <= TOL, how
