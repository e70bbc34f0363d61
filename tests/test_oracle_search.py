"""Pins of the oracle's search over BCchoice and the re-explored scale (sections "Quantize Weight Twice",
Eq. gptqt step 2, Eq. round, and "Re-explore Scale Factor", Eq. reexplore).  CPU only."""
import itertools

import numpy as np
import pytest

import oracle


def test_set_partitions_counts_are_stirling_numbers():
    # Stirling numbers of the second kind: the number of ways to split n bits into q non-empty planes
    stirling = {(1, 1): 1, (2, 1): 1, (2, 2): 1, (3, 2): 3, (4, 2): 7, (4, 3): 6, (4, 4): 1, (5, 2): 15, (5, 3): 25,
                (5, 4): 10, (6, 3): 90}
    for (n, q), want in stirling.items():
        ps = oracle.set_partitions(n, q)
        assert len(ps) == want
        as_sets = set()
        for b2p in ps:
            assert b2p.shape == (n,) and set(b2p.tolist()) == set(range(q))       # every plane used
            as_sets.add(frozenset(frozenset(np.flatnonzero(b2p == p).tolist()) for p in range(q)))
        assert len(as_sets) == want                                              # each split once
        assert [tuple(p) for p in ps] == sorted(tuple(p) for p in ps)            # lexicographic


def test_set_partitions_against_brute_force():
    for n, q in [(3, 2), (4, 3), (5, 2)]:
        brute = set()
        for assign in itertools.product(range(q), repeat=n):
            if len(set(assign)) == q:
                brute.add(frozenset(frozenset(i for i in range(n) if assign[i] == p) for p in range(q)))
        got = {frozenset(frozenset(np.flatnonzero(b == p).tolist()) for p in range(q)) for b in oracle.set_partitions(n, q)}
        assert got == brute


def test_reexplore_factors_lie_inside_the_interval_of_eq_reexplore():
    for n in (2, 3, 4, 5):
        s = oracle.reexplore_factors(n, 9)
        full = 2.0 ** n - 1
        # S_hat = s (Wmax - Wmin)/(2^n - 1) must lie strictly between the n+1-bit and the n-1-bit step
        assert np.all(s / full > 1.0 / (2.0 ** (n + 1) - 1)) and np.all(s / full < 1.0 / (2.0 ** (n - 1) - 1))
        assert np.all(np.diff(s) > 0) and np.allclose(np.diff(s), np.diff(s)[0])
    # n = 4: the interval is (15/31, 15/7); one interior point is its middle
    assert oracle.reexplore_factors(4, 1)[0] == pytest.approx((15 / 31 + 15 / 7) / 2)


def test_hand_computed_case():
    # one row [0, 1, 2, 3], two step-1 bits, per-row scale: S = 1, qbias = 0, W_int = W.
    W = np.array([[0, 1, 2, 3]], np.float16)
    X = np.array([[1, 2, 3, 4], [1, 1, 1, 1]], np.float16)
    both = np.array([0, 0], np.uint8)         # one plane holds both bits: BCchoice {0, 3}
    apart = np.array([0, 1], np.uint8)        # two planes: BCchoice {0, 1, 2, 3}
    rows, err, best = oracle.grid_search(W, X, 0, 2, [both, apart], [1.0, 2.0])
    # s = 1, {0,3}: W_q = [0,0,3,3], dW = [0,-1,1,0]; outputs 1 and 0           -> 1
    # s = 1, identity: exact                                                  -> 0
    # s = 2: S = 2, W_int = rint([0, .5, 1, 1.5]) = [0,0,1,2];
    #        {0,3}: W_q = [0,0,0,3] -> W_hat = [0,0,0,6], dW = [0,-1,-2,3]; outputs 4 and 0  -> 16
    #        identity: W_hat = [0,0,2,4], dW = [0,-1,0,1]; outputs 2 and 0                   -> 4
    assert err.tolist() == [[1.0, 0.0], [16.0, 4.0]]
    assert rows.shape == (2, 2, 1) and best == (0, 1)


def _search_inputs(N=24, K=256, T=16, seed=5):
    rng = np.random.default_rng(seed)
    W = (0.05 * rng.standard_normal((N, K))).astype(np.float16)
    X = rng.standard_normal((T, K)).astype(np.float16)
    return W, X


@pytest.mark.parametrize("group", [0, 128])
def test_identity_calibration_gives_the_plain_squared_error(group):
    # with X = I the output error is the weight error itself: an independent route through dequant()
    W, _ = _search_inputs(K=128 if group == 0 else 256)
    N, K = W.shape
    X = np.eye(K, dtype=np.float16)
    parts = oracle.set_partitions(4, 3)
    rows, err, _ = oracle.grid_search(W, X, group, 4, parts, [1.0, 0.8])
    for si, s in enumerate([1.0, 0.8]):
        w_int, S, qb = oracle.quantize_rtn(W, group, 4, s)
        G = S.shape[1]
        for pi, b2p in enumerate(parts):
            _, value = oracle.bcchoice(4, b2p)
            near = value[np.abs(w_int[..., None].astype(np.float64) - value).argmin(axis=-1)]    # some nearest value
            # |W_int - nearest| is unique even where the nearest value is not; here distances decide the error
            # only up to ties, so compare through the rounding the oracle itself documents (ties to smaller)
            tie = np.sort(np.abs(w_int[..., None].astype(np.float64) - value), axis=-1)
            has_tie = tie[..., 0] == tie[..., 1]
            near = np.where(has_tie, np.minimum(near, w_int - tie[..., 0]), near)
            Wh = np.repeat(S.astype(np.float64), K // G, axis=1) * near + np.repeat(qb.astype(np.float64), K // G, axis=1)
            want = ((Wh - W.astype(np.float64)) ** 2).sum(axis=1)
            np.testing.assert_allclose(rows[si, pi], want, rtol=1e-12, atol=0)


def test_all_bits_apart_leaves_the_step_one_residual():
    # q = n: BCchoice holds every integer, step 2 changes nothing
    W, X = _search_inputs()
    ident = np.arange(3, dtype=np.uint8)
    rows, err, _ = oracle.grid_search(W, X, 128, 3, [ident], [1.0, 1.3])
    for si, s in enumerate([1.0, 1.3]):
        w_int, S, qb = oracle.quantize_rtn(W, 128, 3, s)
        R = np.repeat(S.astype(np.float64), 128, axis=1) * w_int + np.repeat(qb.astype(np.float64), 128, axis=1) - W.astype(np.float64)
        want = np.einsum("nk,tk->nt", R, X.astype(np.float64))
        np.testing.assert_allclose(rows[si, 0], (want ** 2).sum(axis=1), rtol=1e-12)


def test_scaling_and_permutation_properties_and_the_argmin():
    W, X = _search_inputs()
    parts = oracle.set_partitions(4, 2)
    s = oracle.reexplore_factors(4, 5)
    rows, err, best = oracle.grid_search(W, X, 128, 4, parts, s)
    assert err[best] == err.min() and np.all(err >= 0)
    flat = err.reshape(-1)
    assert best == divmod(int(np.flatnonzero(flat == flat.min())[0]), len(parts))       # the first of the minima
    rows2, err2, _ = oracle.grid_search(W, (2 * X.astype(np.float32)).astype(np.float16), 128, 4, parts, s)
    np.testing.assert_array_equal(rows2, 4 * rows)                                      # exact: a power of two
    perm = np.random.default_rng(1).permutation(W.shape[0])
    rows3, _, _ = oracle.grid_search(W[perm], X, 128, 4, parts, s)
    np.testing.assert_array_equal(rows3, rows[:, :, perm])                              # rows are independent
    rows4, _, _ = oracle.grid_search(W, X[::-1].copy(), 128, 4, parts, s)
    np.testing.assert_allclose(rows4, rows, rtol=1e-12)                                 # a sum over tokens


def test_exactly_representable_weights_have_zero_error_at_their_own_candidate():
    # weights that already sit on S0 * BCchoice + qbias, with both end values present: s = 1 and that
    # BCchoice reproduce them exactly; another BCchoice does not
    parts = oracle.set_partitions(4, 3)
    b2p = parts[2]
    _, value = oracle.bcchoice(4, b2p)
    rng = np.random.default_rng(3)
    v = value[rng.integers(0, len(value), size=(8, 128))]
    v[:, 0], v[:, 1] = 0.0, 15.0
    W = (0.0078125 * v - 0.0625).astype(np.float16)          # exact in fp16
    assert np.array_equal(W.astype(np.float64), 0.0078125 * v - 0.0625)
    X = rng.standard_normal((8, 128)).astype(np.float16)
    rows, err, best = oracle.grid_search(W, X, 0, 4, parts, [0.9, 1.0])
    assert err[1, 2] == 0.0 and best == (1, 2)
    assert np.all(np.delete(err[1], 2) > 0)
