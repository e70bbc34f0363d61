"""Pins of the CPU oracle against what the paper prints and what the mathematics fixes.

None of these tests needs a GPU and none touches the CUDA library.  Each check is
independent of the oracle's own code: printed values (tests/golden/), bit-level
characterisations, exhaustive enumeration, numpy library routines.
"""
import itertools

import numpy as np
import pytest

import oracle
from conftest import load_golden
from paper_2407_02891_b200 import synth


# ---------------------------------------------------------------------------------------
# fp16 <-> fp64 conversion: numpy's float16 is the independent reference
# ---------------------------------------------------------------------------------------

def test_half_to_double_all_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float64)
    got = np.array([oracle.half_to_double(int(b)) for b in bits])
    finite = np.isfinite(ref)
    assert np.array_equal(got[finite], ref[finite])
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    assert np.array_equal(np.isinf(got), np.isinf(ref))
    assert np.array_equal(np.signbit(got[finite]), np.signbit(ref[finite]))


def test_double_to_half_matches_numpy():
    rng = np.random.default_rng(7)
    vals = np.concatenate([
        rng.standard_normal(20000) * 10.0 ** rng.integers(-9, 5, 20000),
        # exact ties between neighbouring halves, and the subnormal / overflow edges
        np.arange(1, 4096, dtype=np.float64) * 2.0 ** -25,
        (np.arange(2048, 4096, dtype=np.float64) + 0.5) * 2.0 ** -3,
        [0.0, -0.0, 65504.0, 65519.99, 65520.0, 1e9, -1e9, 2.0 ** -24, 2.0 ** -25, 2.0 ** -26],
    ])
    with np.errstate(over="ignore"):
        ref = vals.astype(np.float16).view(np.uint16)
    got = np.array([oracle.double_to_half_bits(v) for v in vals], dtype=np.uint16)
    assert np.array_equal(got, ref)


# ---------------------------------------------------------------------------------------
# Eq. fuse_step1 / fuse_step2: which integers a merged code reaches
# ---------------------------------------------------------------------------------------

def set_partitions(n, q):
    """All assignments bit -> plane (surjective, planes numbered by first appearance)."""
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


def test_partition_counts():
    # Stirling numbers of the second kind: S(4,3)=6, S(5,3)=25, S(5,2)=15
    assert len(set_partitions(4, 3)) == 6
    assert len(set_partitions(5, 3)) == 25
    assert len(set_partitions(5, 2)) == 15


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 6])
def test_step1_identity_reaches_every_integer(n):
    """Eq. fuse_step1: with one plane per bit, sign pattern c reaches the integer c."""
    m, value = oracle.bcchoice(n, list(range(n)))
    assert np.array_equal(m, 2.0 ** (np.arange(n) - 1))
    assert np.array_equal(value, np.arange(1 << n, dtype=np.float64))


def test_step1_printed_values():
    g = load_golden("eq_fuse.txt")
    n = int(g["step1_n_bits"][0])
    m, value = oracle.bcchoice(n, list(range(n)))
    assert list(m) == g["step1_alpha"]
    assert sorted(value) == g["step1_reaches"]
    # the printed offset: all-minus pattern reaches offset - sum(alpha) = 0
    assert g["step1_offset"][0] - sum(g["step1_alpha"]) == value[0]


def test_step2_printed_values():
    g = load_golden("eq_fuse.txt")
    r = load_golden("eq_round.txt")
    b2p = [int(v) for v in g["step2_bit_to_plane"]]
    m, value = oracle.bcchoice(3, b2p)
    assert list(m) == g["step2_alpha"]
    assert sorted(value) == r["bcchoice"]          # the two passages agree: {0,1,6,7}
    off = g["step2_offset"][0]
    signs = list(itertools.product([-1, 1], repeat=2))
    assert sorted(off + s0 * m[0] + s1 * m[1] for s0, s1 in signs) == r["bcchoice"]


@pytest.mark.parametrize("n,q", [(2, 1), (3, 2), (4, 2), (4, 3), (4, 4), (5, 2), (5, 3), (5, 4)])
def test_reachable_values_bit_characterisation(n, q):
    """A merged code reaches exactly the integers whose binary digits agree inside each plane:
    digit (i-1) of value[c] equals bit bit_to_plane[i-1] of c."""
    for b2p in set_partitions(n, q):
        _, value = oracle.bcchoice(n, b2p)
        assert len(set(value)) == 1 << q
        for c, v in enumerate(value):
            assert v == int(v) and 0 <= v < (1 << n)
            for i in range(n):
                assert (int(v) >> i) & 1 == (c >> b2p[i]) & 1


def test_bcchoice_rejects_unused_plane():
    with pytest.raises(ValueError):
        oracle.bcchoice(3, [0, 2, 2])           # plane 1 has no bit


# ---------------------------------------------------------------------------------------
# Eq. round: nearest reachable value
# ---------------------------------------------------------------------------------------

def test_round_printed_vector():
    r = load_golden("eq_round.txt")
    w = np.array(r["w_int"], np.uint8)
    wq, codes = oracle.round_to_bcchoice(w, int(r["n_bits"][0]), [int(v) for v in r["bit_to_plane"]])
    assert list(wq) == r["w_q"]
    _, value = oracle.bcchoice(3, [int(v) for v in r["bit_to_plane"]])
    assert np.array_equal(value[codes], wq)


@pytest.mark.parametrize("n,q", [(3, 2), (4, 3), (5, 3), (5, 2), (4, 4)])
def test_round_is_nearest_brute_force(n, q):
    w = np.arange(1 << n, dtype=np.uint8)
    for b2p in set_partitions(n, q):
        _, value = oracle.bcchoice(n, b2p)
        wq, codes = oracle.round_to_bcchoice(w, n, b2p)
        for t in range(1 << n):
            best = min(abs(t - v) for v in value)
            assert abs(int(wq[t]) - t) == best           # minimal distance (unique part)
            assert wq[t] in value and value[codes[t]] == wq[t]
            ties = [v for v in value if abs(t - v) == best]
            assert wq[t] == min(ties)                    # documented reading: smaller value on ties
        wq2, codes2 = oracle.round_to_bcchoice(w, n, b2p)
        assert np.array_equal(wq, wq2) and np.array_equal(codes, codes2)


def test_round_rejects_out_of_range():
    with pytest.raises(ValueError):
        oracle.round_to_bcchoice(np.array([8], np.uint8), 3, [0, 1, 1])


# ---------------------------------------------------------------------------------------
# Eq. fuse_step3: fused alpha, z; exact reconstruction of the linear-quantised weights
# ---------------------------------------------------------------------------------------

def test_step3_printed_closed_form():
    g = load_golden("eq_fuse.txt")
    S, qbias = np.float16(0.01171875), np.float16(-0.1171875)       # 3 * 2^-8, -10 S
    w = np.arange(8, dtype=np.uint8).reshape(1, 8)
    codes, alpha, z = oracle.merge_linear(w, [[S]], [[qbias]], 0, 3, [0, 1, 1])
    assert [float(a) / float(S) for a in alpha[:, 0, 0]] == g["step3_alpha_over_S"]
    assert float(z[0, 0]) == g["step3_offset_S_coeff"][0] * float(S) + float(qbias)


def test_linear2_printed_closed_form():
    """Eq. linear_eql_bcq: 2-bit linear quantisation == binary coding with alpha = (S, S/2)."""
    g = load_golden("eq_fuse.txt")
    S = np.float16(0.0625)
    w = np.arange(4, dtype=np.uint8).reshape(1, 4)
    _, alpha, _ = oracle.merge_linear(w, [[S]], [[np.float16(0)]], 0, 2, [0, 1])
    assert sorted((float(a) / float(S) for a in alpha[:, 0, 0]), reverse=True) == g["linear2_alpha_over_S"]


@pytest.mark.parametrize("n,q,group", [(4, 3, 32), (4, 3, 0), (5, 3, 32), (5, 2, 0), (3, 2, 32), (4, 4, 32)])
def test_merge_reconstructs_linear_quantised_weights_exactly(n, q, group):
    """Tiny 16 x 32 case: sum_j alpha_j b_j + z == S * W_q + qbias exactly, from the fp16 arrays."""
    N, K = 16, 32
    w, S, qbias = synth.linear_int_case(f"tiny/n{n}", N, K, group, n)
    assert set(np.unique(w)) == set(range(1 << n))          # every step-1 value occurs
    G = 1 if group == 0 else K // group
    L = K // G
    seen = set()
    for b2p in set_partitions(n, q):
        codes, alpha, z = oracle.merge_linear(w, S, qbias, group, n, b2p)
        wq, codes_r = oracle.round_to_bcchoice(w, n, b2p)
        assert np.array_equal(codes, codes_r)
        W = oracle.dequant(codes, alpha, z, group)
        Sx = np.repeat(S.astype(np.float64), L, axis=1)
        Bx = np.repeat(qbias.astype(np.float64), L, axis=1)
        assert np.array_equal(W, Sx * wq.astype(np.float64) + Bx)
        seen |= set(np.unique(codes))
    assert seen == set(range(1 << q))                        # every code occurs


# ---------------------------------------------------------------------------------------
# canonical packing: numpy's packbits is the independent reference
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("N,K,q", [(16, 32, 3), (5, 64, 2), (3, 128, 4), (1, 8, 1)])
def test_pack_matches_numpy_packbits(N, K, q):
    rng = np.random.default_rng(N * K + q)
    codes = rng.integers(0, 1 << q, (N, K), dtype=np.uint8)
    planes = oracle.pack_canonical(codes, q)
    assert planes.shape == (q, N, K // 8)
    for i in range(q):
        ref = np.packbits((codes >> i) & 1, axis=1, bitorder="little")
        assert np.array_equal(planes[i], ref)
        assert int(np.unpackbits(planes[i]).sum()) == int(((codes >> i) & 1).sum())
    assert np.array_equal(oracle.unpack_canonical(planes), codes)


def test_pack_layout_constants():
    """Bit (k mod 8) of byte (k div 8), LSB = lowest k, plane-major then row-major."""
    N, K, q = 4, 32, 3
    codes = np.zeros((N, K), np.uint8)
    codes[2, 13] = 0b101
    planes = oracle.pack_canonical(codes, q)
    expect = np.zeros((q, N, K // 8), np.uint8)
    expect[0, 2, 1] = 1 << 5
    expect[2, 2, 1] = 1 << 5
    assert np.array_equal(planes, expect)


# ---------------------------------------------------------------------------------------
# forward
# ---------------------------------------------------------------------------------------

def _layer(name, N, K, q, group, B):
    p = synth.planes(name, N, K, q)
    alpha, z = synth.scale_rows(name, N, K, q, group)
    x = synth.activations(name, B, K)
    return p, synth.codes_from_planes(p), alpha, z, x


@pytest.mark.parametrize("N,K,q,group,B", [(16, 32, 3, 32, 1), (24, 256, 3, 128, 2), (8, 512, 2, 0, 3),
                                           (40, 384, 4, 64, 1)])
def test_forward_two_forms_agree_and_match_numpy_matmul(N, K, q, group, B):
    p, codes, alpha, z, x = _layer(f"fw/{N}x{K}", N, K, q, group, B)
    y1 = oracle.forward_planes(p, alpha, z, x, group)
    y2 = oracle.forward_dequant(codes, alpha, z, x, group)
    W = oracle.dequant(codes, alpha, z, group)
    y3 = x.astype(np.float64) @ W.T                      # library routine
    scale = np.abs(y3).max()
    assert np.abs(y1 - y2).max() <= 1e-12 * scale
    assert np.abs(y1 - y3).max() <= 1e-12 * scale
    assert np.abs(y2 - y3).max() <= 1e-12 * scale


@pytest.mark.parametrize("n,group", [(2, 0), (3, 32), (4, 64)])
def test_q_equals_n_is_plain_linear_quantised_matvec(n, group):
    """Special case q = n (Eq. linear_eql_bcq): the BCQ layer equals (S * W_int + qbias) x."""
    N, K = 12, 128
    w, S, qbias = synth.linear_int_case(f"lin/n{n}", N, K, group, n)
    codes, alpha, z = oracle.merge_linear(w, S, qbias, group, n, list(range(n)))
    x = synth.activations(f"lin/n{n}", 2, K)
    L = K if group == 0 else group
    Wlin = np.repeat(S.astype(np.float64), L, axis=1) * w + np.repeat(qbias.astype(np.float64), L, axis=1)
    ref = x.astype(np.float64) @ Wlin.T
    for y in (oracle.forward_planes(oracle.pack_canonical(codes, n), alpha, z, x, group),
              oracle.forward_dequant(codes, alpha, z, x, group)):
        assert np.abs(y - ref).max() <= 1e-12 * np.abs(ref).max()


def test_forward_unit_vector_returns_column_of_w():
    N, K, q, group = 8, 256, 3, 128
    p, codes, alpha, z, _ = _layer("fw/unit", N, K, q, group, 1)
    W = oracle.dequant(codes, alpha, z, group)
    for k in (0, 7, 8, 127, 128, 255):
        x = np.zeros((1, K), np.float16)
        x[0, k] = 1.0
        assert np.array_equal(oracle.forward_planes(p, alpha, z, x, group)[0], W[:, k])
        assert np.array_equal(oracle.forward_dequant(codes, alpha, z, x, group)[0], W[:, k])


def test_forward_structured_cases():
    N, K, q, group = 8, 256, 3, 128
    p, codes, alpha, z, x = _layer("fw/struct", N, K, q, group, 1)
    xd = x.astype(np.float64)[0]
    gs = xd.reshape(-1, group).sum(axis=1)                                  # group sums of x
    a64, z64 = alpha.astype(np.float64), z.astype(np.float64)
    # all planes +1: y[n] = sum_g (sum_i alpha + z) * sum_{k in g} x
    ones = np.full_like(p, 0xFF)
    y = oracle.forward_planes(ones, alpha, z, x, group)[0]
    assert np.allclose(y, ((a64.sum(axis=0) + z64) * gs).sum(axis=1), rtol=1e-12, atol=1e-12)
    # alpha = 0: only the offset term remains
    y = oracle.forward_planes(p, np.zeros_like(alpha), z, x, group)[0]
    assert np.allclose(y, (z64 * gs).sum(axis=1), rtol=1e-12, atol=1e-12)
    # flipping a plane and negating its alpha changes nothing
    p2, a2 = p.copy(), alpha.copy()
    p2[1] ^= 0xFF
    a2[1] = -a2[1]
    y0 = oracle.forward_planes(p, alpha, z, x, group)
    assert np.allclose(oracle.forward_planes(p2, a2, z, x, group), y0, rtol=1e-12, atol=1e-12)
    # linearity in x (inputs chosen so that the fp16 sum is exact)
    xa = (np.round(xd * 8) / 8).astype(np.float16)[None]
    xb = np.roll(xa, 5, axis=1)
    xs = (xa.astype(np.float64) + xb.astype(np.float64)).astype(np.float16)
    ya, yb, ys = (oracle.forward_planes(p, alpha, z, v, group) for v in (xa, xb, xs))
    assert np.allclose(ya + yb, ys, rtol=1e-11, atol=1e-11)
    # batch columns are independent products
    xB = np.concatenate([xa, xb, xs])
    assert np.array_equal(oracle.forward_planes(p, alpha, z, xB, group), np.concatenate([ya, yb, ys]))


def test_group_boundaries_matter():
    """A scale belongs to its own group only: moving alpha to the other group changes the result."""
    N, K, q, group = 2, 256, 1, 128
    p = np.zeros((q, N, K // 8), np.uint8)
    p[0, :, :16] = 0xFF                       # +1 in group 0, -1 in group 1
    alpha = np.array([[[1.0, 2.0], [1.0, 2.0]]], np.float16)
    z = np.array([[0.5, -0.25], [0.5, -0.25]], np.float16)
    x = np.ones((1, K), np.float16)
    y = oracle.forward_planes(p, alpha, z, x, group)
    assert np.array_equal(y[0], np.full(N, 128 * (1.0 + 0.5) + 128 * (-2.0 - 0.25)))


# ---------------------------------------------------------------------------------------
# Eq. gptqt step 1: linear quantisation of fp16 weights (oracle.quantize_rtn)
# ---------------------------------------------------------------------------------------

def _weights(name, N, K, scale=0.05):
    return (scale * synth.normal(name + "/W", 0, N * K)).reshape(N, K).astype(np.float16)


def test_rtn_exact_grid_is_recovered():
    """Weights that lie on a grid qbias + S k (S a power of two) quantise to k, S and qbias exactly
    (section "Re-explore Scaling Factor": S = (Wmax - Wmin)/(2^n - 1), qbias = Wmin)."""
    for n in (2, 3, 4, 5):
        top = 2 ** n - 1
        rng = np.random.default_rng(n)
        k = rng.integers(0, top + 1, size=(6, 64)).astype(np.float64)
        k[:, 0], k[:, 1] = 0, top                                   # both ends occur in every group of 32
        k[:, 32], k[:, 33] = 0, top
        for S, b in ((2.0 ** -6, -0.75), (2.0 ** -9, 0.125)):
            W = (b + S * k).astype(np.float16)
            assert np.array_equal(W.astype(np.float64), b + S * k)  # representable: the case is exact
            for group in (0, 32):
                w_int, S_h, q_h = oracle.quantize_rtn(W, group, n)
                assert np.array_equal(w_int, k.astype(np.uint8))
                assert np.all(S_h.astype(np.float64) == S) and np.all(q_h.astype(np.float64) == b)


@pytest.mark.parametrize("n,group", [(3, 0), (4, 128), (5, 64), (8, 32)])
def test_rtn_is_the_nearest_grid_point_by_brute_force(n, group):
    """Against enumeration of every level: the chosen integer minimises |W - (S k + qbias)|, the ends
    of the range map to 0 and 2^n - 1, the error is at most S/2, and S is the range formula."""
    N, K = 5, 256
    W = _weights(f"rtn/{n}/{group}", N, K)
    w_int, S_h, q_h = oracle.quantize_rtn(W, group, n)
    L = K if group == 0 else group
    Wd = W.astype(np.float64).reshape(N, K // L, L)
    S = S_h.astype(np.float64)[:, :, None]
    b = q_h.astype(np.float64)[:, :, None]
    assert np.array_equal(b[:, :, 0], Wd.min(axis=2))
    exact_S = (Wd.max(axis=2) - Wd.min(axis=2)) / (2 ** n - 1)
    assert np.all(np.abs(S[:, :, 0] - exact_S) <= exact_S * 2.0 ** -11)       # one fp16 rounding
    levels = np.arange(2 ** n, dtype=np.float64)
    dist = np.abs(Wd[..., None] - (S[..., None] * levels + b[..., None]))     # [N, G, L, 2^n]
    chosen = np.take_along_axis(dist, w_int.reshape(N, K // L, L, 1).astype(np.int64), axis=3)[..., 0]
    assert np.all(chosen <= dist.min(axis=3) * (1 + 1e-12))
    # the top of the range may sit half an fp16 rounding of S outside the grid, never more
    assert np.all(chosen <= S / 2 + (2 ** n - 1) * exact_S[:, :, None] * 2.0 ** -11)
    wi = w_int.reshape(N, K // L, L)
    assert np.all(wi[Wd == Wd.min(axis=2, keepdims=True)] == 0)
    assert np.all(wi[Wd == Wd.max(axis=2, keepdims=True)] == 2 ** n - 1)
    # monotone: a larger weight never gets a smaller integer
    order = np.argsort(Wd, axis=2, kind="stable")
    assert np.all(np.diff(np.take_along_axis(wi.astype(np.int64), order, axis=2), axis=2) >= 0)


def test_rtn_ties_go_to_even_and_clamp():
    """Half-way points (exactly representable) round to the even integer; a re-explored, smaller S
    (Eq. reexplore) pushes large weights past the grid and they clamp to 2^n - 1."""
    n = 3
    W = np.array([[0.0, 7.0, 0.5, 1.5, 2.5, 3.5, 4.5, 6.5]], np.float16)
    w_int, S, b = oracle.quantize_rtn(W, 0, n)
    assert float(S[0, 0]) == 1.0 and float(b[0, 0]) == 0.0
    assert w_int.tolist() == [[0, 7, 0, 2, 2, 4, 4, 6]]
    w2, S2, _ = oracle.quantize_rtn(W, 0, n, s_factor=0.5)         # S = 0.5: 3.5 -> 7, everything above clamps
    assert float(S2[0, 0]) == 0.5
    assert w2.tolist() == [[0, 7, 1, 3, 5, 7, 7, 7]]
    w3, S3, _ = oracle.quantize_rtn(W, 0, n, s_factor=2.0)         # S = 2: half-way points 1, 3, 5, 7 do not occur
    assert float(S3[0, 0]) == 2.0 and w3.tolist() == [[0, 4, 0, 1, 1, 2, 2, 3]]


def test_rtn_constant_group_and_errors():
    W = np.full((2, 64), 0.375, np.float16)
    W[1, 32:] = [0.25] * 16 + [0.5] * 16
    w_int, S, b = oracle.quantize_rtn(W, 32, 4)
    assert np.all(w_int[0] == 0) and np.all(S[0] == 0) and np.all(b[0] == np.float16(0.375))
    assert np.all(w_int[1, :32] == 0) and w_int[1, 32:].tolist() == [0] * 16 + [15] * 16
    # S = 0 dequantises the constant group exactly through the merge as well
    codes, alpha, z = oracle.merge_linear(w_int, S, b, 32, 4, [0, 1, 2, 2])
    Wq = oracle.dequant(codes, alpha, z, 32)
    assert np.array_equal(Wq[0], np.full(64, 0.375))
    bad = W.copy()
    bad[0, 3] = np.inf
    with pytest.raises(Exception):
        oracle.quantize_rtn(bad, 32, 4)
    with pytest.raises(Exception):
        oracle.quantize_rtn(W, 32, 4, s_factor=0.0)


@pytest.mark.parametrize("n,q,b2p", [(4, 3, [0, 1, 2, 2]), (3, 3, [0, 1, 2]), (5, 2, [0, 0, 1, 1, 1])])
def test_rtn_then_merge_reconstruction_error_bound(n, q, b2p):
    """End to end (step 1, Eq. round, Eq. fuse_step3): the dequantised weight differs from the fp16
    weight by at most S/2 (step 1) + S * the largest gap/2 of the reachable set (Eq. round)."""
    N, K, group = 4, 256, 128
    W = _weights(f"rtnmerge/{n}/{q}", N, K)
    w_int, S, qb = oracle.quantize_rtn(W, group, n)
    codes, alpha, z = oracle.merge_linear(w_int, S, qb, group, n, b2p)
    Wq = oracle.dequant(codes, alpha, z, group)
    _, values = oracle.bcchoice(n, b2p)
    reach = np.sort(np.asarray(values, np.float64))
    half_gap = max(np.diff(reach).max() / 2, reach[0], (2 ** n - 1) - reach[-1])
    Sd = np.repeat(S.astype(np.float64), group, axis=1)
    slack = (np.abs(W.astype(np.float64)).max() + 1) * 2.0 ** -9     # fp16 rounding of alpha and z
    assert np.all(np.abs(Wq - W.astype(np.float64)) <= Sd * (0.5 + half_gap) + slack)
    if q == n:
        assert np.all(np.abs(Wq - W.astype(np.float64)) <= Sd * 0.5 + slack)


def test_rtn_zero_minimum_is_stored_as_plus_zero_whichever_zero_comes_first():
    """A group whose minimum is zero: -0.0 and +0.0 compare equal, so which of the two the minimum search
    ends on depends on the order of the weights; the stored qbias must not.  Both orders give the bit
    pattern 0x0000, the same S and the same integers; a strictly negative minimum keeps its sign."""
    neg0, pos0 = np.uint16(0x8000).view(np.float16), np.float16(0.0)
    top = np.float16(0.75)
    first = np.array([[neg0, np.float16(0.25), pos0, top]], np.float16)      # -0 met first
    last = np.array([[pos0, np.float16(0.25), top, neg0]], np.float16)       # -0 met last
    only = np.array([[neg0, np.float16(0.25), np.float16(0.5), top]], np.float16)   # no +0 in the group at all
    for W in (first, last, only):
        w_int, S, qb = oracle.quantize_rtn(W, 0, 2)
        assert qb.view(np.uint16).tolist() == [[0x0000]]
        assert S.view(np.uint16).tolist() == np.array([[0.25]], np.float16).view(np.uint16).tolist()   # 0.75 / 3
        zero_at = [i for i in range(4) if W[0, i] == 0]
        assert all(w_int[0, i] == 0 for i in zero_at) and w_int[0].max() == 3
    # the offset that merge derives from it is then S * centre exactly (no -0 leaking into z)
    _, alpha, z = oracle.merge_linear(oracle.quantize_rtn(first, 0, 2)[0], *oracle.quantize_rtn(first, 0, 2)[1:], 0, 2, [0, 1])
    assert z.view(np.uint16).tolist() == np.array([[0.375]], np.float16).view(np.uint16).tolist()
    # a negative minimum is kept as it is
    W = np.array([[np.float16(-0.5), neg0, np.float16(0.25), np.float16(1.0)]], np.float16)
    assert oracle.quantize_rtn(W, 0, 2)[2].view(np.uint16).tolist() == np.array([[-0.5]], np.float16).view(np.uint16).tolist()
