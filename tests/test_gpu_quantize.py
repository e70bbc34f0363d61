"""bcq_quantize_rtn against the oracle: step-1 integers, S, qbias, packed planes and fused scales,
all bit for bit (the integer is decided in fp64 on both sides, from the stored fp16 S)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import TOL, rel_err, tiled_operands
from paper_2407_02891_b200 import binding as bq
from paper_2407_02891_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def weights(name, N, K, scale=0.05):
    return (scale * synth.normal(name + "/W", 0, N * K)).reshape(N, K).astype(np.float16)


def run(W, q, group, layout, n_bits, b2p, s_factor=1.0, want_int=True):
    N, K = W.shape
    d = bq.desc(N, K, q, group, layout)
    G = 1 if group == 0 else K // group
    Wd = torch.from_numpy(W).to(DEV)
    S = torch.zeros(N * G, dtype=torch.float16, device=DEV)
    qb = torch.zeros(N * G, dtype=torch.float16, device=DEV)
    wi = torch.full((N * K,), 255, dtype=torch.uint8, device=DEV) if want_int else None
    packed, a, z = bq.empty_operands(d, DEV)
    packed.fill_(0xA5)
    bq.quantize_rtn(d, Wd, n_bits, b2p, S, qb, wi, packed, a, z, s_factor)
    torch.cuda.synchronize()
    cpu = lambda t: None if t is None else t.cpu().numpy()
    return cpu(S), cpu(qb), cpu(wi), cpu(packed), cpu(a), cpu(z)


def expected(W, q, group, layout, n_bits, b2p, s_factor=1.0):
    w_int, S, qb = oracle.quantize_rtn(W, group, n_bits, s_factor)
    codes, alpha, z = oracle.merge_linear(w_int, S, qb, group, n_bits, b2p)
    planes = oracle.pack_canonical(codes, q)
    if layout == bq.LAYOUT_TILED:
        packed, a, zz = tiled_operands(planes, alpha, z, group)
    else:
        packed, a, zz = planes.reshape(-1), alpha.reshape(-1), z.reshape(-1)
    return w_int, S, qb, packed, a, zz, (codes, alpha, z)


def same(a, b):
    return np.array_equal(np.asarray(a).reshape(-1).view(np.uint8), np.asarray(b).reshape(-1).view(np.uint8))


@pytest.mark.parametrize("N,K,q,group,layout,n_bits,b2p,s_factor", [
    (16, 32, 3, 32, bq.LAYOUT_CANONICAL, 4, [0, 1, 2, 2], 1.0),          # the tiny 4-bit -> 3-plane case
    (16, 32, 3, 0, bq.LAYOUT_CANONICAL, 4, [0, 1, 1, 2], 1.0),
    (50, 256, 3, 64, bq.LAYOUT_CANONICAL, 4, [0, 1, 2, 2], 1.0),
    (40, 1024, 3, 128, bq.LAYOUT_TILED, 4, [0, 1, 2, 2], 1.0),
    (264, 1536, 3, 128, bq.LAYOUT_TILED, 5, [0, 0, 1, 1, 2], 0.8),       # a re-explored scale: the top clamps
    (264, 1536, 2, 128, bq.LAYOUT_TILED, 5, [0, 0, 1, 1, 1], 1.3),
    (72, 512, 2, 0, bq.LAYOUT_TILED, 3, [0, 1, 1], 1.0),                 # one scale per row
    (24, 4096, 4, 128, bq.LAYOUT_TILED, 4, [0, 1, 2, 3], 1.0),           # q = n: plain linear quantisation
    (13, 96, 1, 32, bq.LAYOUT_CANONICAL, 2, [0, 0], 0.55),
    (8, 36864, 3, 0, bq.LAYOUT_CANONICAL, 8, [0, 0, 0, 1, 1, 1, 2, 2], 1.0),   # long rows, 8-bit step 1
])
def test_quantize_rtn_bit_exact(N, K, q, group, layout, n_bits, b2p, s_factor):
    W = weights(f"q/{N}x{K}/{group}", N, K)
    S, qb, wi, packed, a, z = run(W, q, group, layout, n_bits, b2p, s_factor)
    e_wi, e_S, e_qb, e_packed, e_a, e_z, _ = expected(W, q, group, layout, n_bits, b2p, s_factor)
    assert same(S, e_S) and same(qb, e_qb)
    assert same(wi, e_wi)
    assert same(packed, e_packed)
    if a is not None:
        assert same(a, e_a) and same(z, e_z)


def test_quantize_rtn_structured_weights():
    """Constant groups (S = 0), exact half-way points (ties to even), zeros of both signs."""
    N, K, q, group = 8, 512, 3, 128
    W = weights("q/struct", N, K)
    W[0, :128] = np.float16(0.375)                       # constant group
    W[1, :] = 0.0
    W[1, 5] = np.float16(-0.0)                           # a zero row with a negative zero
    W[2, :8] = [0.0, 7.0, 0.5, 1.5, 2.5, 3.5, 4.5, 6.5]  # with n = 3, S = 1: ties
    W[2, 8:128] = 3.0
    for layout in (bq.LAYOUT_CANONICAL, bq.LAYOUT_TILED):
        S, qb, wi, packed, a, z = run(W, q, group, layout, 3, [0, 1, 2])
        e_wi, e_S, e_qb, e_packed, e_a, e_z, _ = expected(W, q, group, layout, 3, [0, 1, 2])
        assert same(S, e_S) and same(qb, e_qb) and same(wi, e_wi) and same(packed, e_packed)
        if a is not None:
            assert same(a, e_a) and same(z, e_z)
        assert wi.reshape(N, K)[2, :8].tolist() == [0, 7, 0, 2, 2, 4, 4, 6]
        assert np.all(wi.reshape(N, K)[0, :128] == 0) and np.all(wi.reshape(N, K)[1] == 0)


def test_quantize_rtn_without_integer_output_and_product():
    """w_int is optional; the operand that comes out multiplies like the oracle's dequantised matrix."""
    N, K, q, group, n_bits, b2p = 520, 2048, 3, 128, 4, [0, 0, 1, 2]
    W = weights("q/prod", N, K)
    d = bq.desc(N, K, q, group, bq.LAYOUT_TILED)
    S, qb, wi, packed, a, z = run(W, q, group, bq.LAYOUT_TILED, n_bits, b2p, want_int=False)
    assert wi is None
    _, _, _, e_packed, _, _, (codes, alpha, zz) = expected(W, q, group, bq.LAYOUT_TILED, n_bits, b2p)
    assert same(packed, e_packed)
    x = synth.activations("q/prod", 1, K)
    y = torch.zeros(N, dtype=torch.float16, device=DEV)
    bq.gemv(d, torch.from_numpy(packed).to(DEV), None, None, torch.from_numpy(x.reshape(-1)).to(DEV), y,
            bq.new_workspace(d, 1))
    torch.cuda.synchronize()
    ref = oracle.forward_dequant(codes, alpha, zz, x, group)[0]
    assert rel_err(y.cpu().numpy(), ref) <= TOL
    # and stays within the method's own error of the unquantised product.  Per weight: half a step of
    # step 1 (S/2: the range scale reaches both ends of the group exactly), half the largest gap between
    # reachable integers in the rounding of Eq. round (S * gap / 2), and the fp16 rounding of the fused
    # scales (2^-11 of sum_j alpha_j + |z|).  Per row that sums, at worst, against |x|.
    _, reach = oracle.bcchoice(n_bits, b2p)
    gap = float(np.diff(np.sort(reach)).max())
    _, e_S, _ = oracle.quantize_rtn(W, group, n_bits)
    Sd = e_S.astype(np.float64)                                          # [N][G]
    per_weight = 0.5 * Sd * (1.0 + gap) + 2.0 ** -11 * (np.abs(alpha.astype(np.float64)).sum(0) + np.abs(zz.astype(np.float64)))
    ax = np.abs(x[0].astype(np.float64)).reshape(-1, group).sum(1)        # sum |x| per group
    bound = per_weight @ ax
    exact = W.astype(np.float64) @ x[0].astype(np.float64)
    assert (np.abs(ref - exact) <= bound).all()


def test_quantize_rtn_full_size_sampled_rows():
    """OPT-30B projection size: S, qbias of all rows, integers and planes of sampled rows."""
    N, K, q, group, n_bits, b2p = 7168, 7168, 3, 128, 4, [0, 1, 2, 2]
    W = weights("q/full", N, K)
    d = bq.desc(N, K, q, group, bq.LAYOUT_CANONICAL)
    S, qb, wi, packed, a, z = run(W, q, group, bq.LAYOUT_CANONICAL, n_bits, b2p)
    rows = np.array([0, 1, 7, 3583, 3584, 7160, 7167])
    e_wi, e_S, e_qb = oracle.quantize_rtn(W[rows], group, n_bits)
    G = K // group
    assert same(S.reshape(N, G)[rows], e_S) and same(qb.reshape(N, G)[rows], e_qb)
    assert same(wi.reshape(N, K)[rows], e_wi)
    codes, alpha, zz = oracle.merge_linear(e_wi, e_S, e_qb, group, n_bits, b2p)
    planes = oracle.pack_canonical(codes, q)
    assert same(packed.reshape(q, N, K // 8)[:, rows], planes)
    assert same(a.reshape(q, N, G)[:, rows], alpha) and same(z.reshape(N, G)[rows], zz)
    # every row: S is one fp16 rounding away from the range formula, qbias is the minimum
    Wd = W.astype(np.float64).reshape(N, G, group)
    assert np.array_equal(qb.reshape(N, G).astype(np.float64), Wd.min(axis=2))
    exact_S = (Wd.max(axis=2) - Wd.min(axis=2)) / 15
    assert np.all(np.abs(S.reshape(N, G).astype(np.float64) - exact_S) <= exact_S * 2.0 ** -11)


def test_quantize_rtn_rejects_bad_arguments():
    d = bq.desc(16, 64, 3, 32, bq.LAYOUT_CANONICAL)
    t16 = torch.zeros(16 * 64, dtype=torch.float16, device=DEV)
    t8 = torch.zeros(3 * 16 * 8, dtype=torch.uint8, device=DEV)
    sc = torch.zeros(3 * 16 * 2, dtype=torch.float16, device=DEV)
    for kwargs in (dict(n_bits=2, b2p=[0, 1]),            # fewer bits than planes
                   dict(n_bits=4, b2p=[0, 1, 1, 1]),      # plane 2 empty
                   dict(n_bits=4, b2p=[0, 1, 2, 3])):     # plane index out of range
        with pytest.raises(bq.BcqError):
            bq.quantize_rtn(d, t16, kwargs["n_bits"], kwargs["b2p"], sc, sc, None, t8, sc, sc)
    with pytest.raises(bq.BcqError):
        bq.quantize_rtn(d, t16, 4, [0, 1, 2, 2], sc, sc, None, t8, sc, sc, s_factor=0.0)
    with pytest.raises(bq.BcqError):
        bq.quantize_rtn(d, t16, 4, [0, 1, 2, 2], sc, sc, None, t8, None, None)   # canonical needs alpha and z
