"""bcq_grid_search (the search over BCchoice and the re-explored scale, Eq. gptqt step 2 and Eq. reexplore)
against the fp64 oracle on the same seeded inputs."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("needs a GPU", allow_module_level=True)

import oracle
from paper_2407_02891_b200 import binding as bq
from paper_2407_02891_b200 import synth

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)
RTOL = 5e-3   # fp16 operands (one rounding of every weight difference), fp32 accumulation: about 1e-3 at worst


def _inputs(name, N, K, T):
    W = (0.05 * synth.normal(name + "/W", 0, N * K)).reshape(N, K).astype(np.float16)   # the quantiser tests' weights
    X = synth.activations(name + "/X", T, K)
    return W, X


def _check(N, K, T, q, group, n_bits, n_scales, name):
    W, X = _inputs(name, N, K, T)
    parts = bq.partitions(n_bits, q)
    s = bq.reexplore_factors(n_bits, n_scales)
    err, rows, best = bq.grid_search(N, K, q, group, torch.from_numpy(W).to(DEV), torch.from_numpy(X).to(DEV), n_bits, parts, s)
    torch.cuda.synchronize()
    assert bq.lib().bcq_poll_status() == bq.OK
    ref_rows, ref_err, ref_best = oracle.grid_search(W, X, group, n_bits, list(parts), s)
    got_rows = rows.cpu().numpy().astype(np.float64)
    got_err = err.cpu().numpy()
    scale = np.abs(ref_rows).max(axis=2, keepdims=True)
    assert np.abs(got_rows - ref_rows).max() <= RTOL * np.abs(ref_rows).max()
    assert (np.abs(got_rows - ref_rows) <= RTOL * scale + 1e-30).all()          # per candidate, against its largest row
    np.testing.assert_allclose(got_err, ref_err, rtol=RTOL)
    np.testing.assert_allclose(got_err, got_rows.sum(axis=2), rtol=1e-5)         # the totals are the sums of the rows
    si, pi = (int(v) for v in best.cpu().numpy())
    assert got_err[si, pi] == got_err.min()
    flat = got_err.reshape(-1)
    assert (si, pi) == divmod(int(np.flatnonzero(flat == flat.min())[0]), len(parts))   # the first minimum, in loop order
    assert ref_err[si, pi] <= ref_err.min() * (1 + 2 * RTOL)                     # a minimum of the oracle's errors too
    return got_err, ref_err


@pytest.mark.parametrize("N,K,T,q,group,n_bits,n_scales", [
    (256, 512, 64, 3, 128, 4, 3),      # two row tiles, six candidates in two groups of four
    (128, 256, 16, 2, 0, 3, 2),        # the smallest T, one scale per row
    (200, 512, 128, 3, 128, 4, 2),     # a ragged last row tile
    (384, 1024, 256, 3, 128, 4, 2),    # the most tokens one launch takes: two candidates per block
    (256, 512, 32, 2, 64, 5, 2),       # 15 candidates, scaling units of 64
    (136, 576, 48, 3, 0, 5, 1),        # 25 candidates, K = 9 slices, T = 48
    (128, 128, 64, 1, 128, 2, 3),      # one plane
    (128, 256, 32, 4, 128, 6, 1),      # six step-1 bits into four planes: 65 candidates, tables of 64 entries
    (200, 256, 32, 2, 128, 3, 11),     # more scale factors than one launch takes (8 + 3), ragged row tiles between them
    (256, 256, 528, 3, 128, 4, 2),     # more tokens than one launch takes: three pieces of 176
    (128, 512, 272, 2, 0, 4, 9),       # two pieces of 144 and 128 tokens, two launches of scale factors
])
def test_grid_search_matches_the_oracle(N, K, T, q, group, n_bits, n_scales):
    _check(N, K, T, q, group, n_bits, n_scales, f"search/{N}x{K}x{T}")


def test_grid_search_repeats_bit_identically_and_validates_arguments():
    N, K, T = 256, 512, 64
    W, X = _inputs("search/repeat", N, K, T)
    Wd, Xd = torch.from_numpy(W).to(DEV), torch.from_numpy(X).to(DEV)
    parts, s = bq.partitions(4, 3), bq.reexplore_factors(4, 3)
    a = bq.grid_search(N, K, 3, 128, Wd, Xd, 4, parts, s)
    b = bq.grid_search(N, K, 3, 128, Wd, Xd, 4, parts, s)
    torch.cuda.synchronize()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])
    c = bq.grid_search(N, K, 3, 128, Wd, Xd, 4, parts, s, want_rows=False)        # without the per-row output
    torch.cuda.synchronize()
    assert torch.equal(a[0], c[0]) and torch.equal(a[2], c[2]) and c[1] is None
    with pytest.raises(bq.BcqError):
        bq.grid_search(N, K, 3, 128, Wd, Xd[:24].contiguous(), 4, parts, s)      # T = 24 is not a multiple of 16
    with pytest.raises(bq.BcqError):
        bq.grid_search(N, K, 3, 96, Wd, Xd, 4, parts, s)                         # scaling units of 96 cut a slice of 64
    bad = parts.copy()
    bad[0, :] = 0                                                                # planes 1 and 2 left empty
    with pytest.raises(bq.BcqError):
        bq.grid_search(N, K, 3, 128, Wd, Xd, 4, bad, s)


def test_grid_search_exact_candidate_has_zero_error():
    # weights that already sit on one candidate's grid: that candidate's error is exactly zero and it is chosen
    parts = bq.partitions(4, 3)
    _, value = oracle.bcchoice(4, parts[2])
    rng = np.random.default_rng(3)
    v = value[rng.integers(0, len(value), size=(128, 256))]
    v[:, 0], v[:, 1] = 0.0, 15.0
    W = (0.0078125 * v - 0.0625).astype(np.float16)
    X = synth.activations("search/exact/X", 32, 256)
    err, rows, best = bq.grid_search(128, 256, 3, 0, torch.from_numpy(W).to(DEV), torch.from_numpy(X).to(DEV), 4, parts,
                                     np.array([0.9, 1.0]))
    torch.cuda.synchronize()
    e = err.cpu().numpy()
    assert e[1, 2] == 0.0 and tuple(best.cpu().numpy()) == (1, 2)
    assert (np.delete(e[1], 2) > 0).all()


@pytest.mark.parametrize("T", [128, 256])
def test_grid_search_fullsize_sampled_rows(T):
    # the configuration bench.py --search times (7168 x 7168, 25 candidates x 8 scale factors in one launch): rows
    # are independent, so the oracle recomputes a seeded sample of them
    N = K = 7168
    W, X = _inputs("search/full", N, K, T)
    parts, s = bq.partitions(5, 3), bq.reexplore_factors(5, 8)
    err, rows_out, best = bq.grid_search(N, K, 3, 128, torch.from_numpy(W).to(DEV), torch.from_numpy(X).to(DEV), 5, parts, s)
    torch.cuda.synchronize()
    assert bq.lib().bcq_poll_status() == bq.OK
    rows = np.unique(synth.u64("search/full/rows", 0, 12) % np.uint64(N)).astype(np.int64)
    rows = np.concatenate([rows, [0, N - 1]])
    ref_rows, _, _ = oracle.grid_search(W[rows], X, 128, 5, list(parts), s)
    got = rows_out.cpu().numpy().astype(np.float64)
    assert np.abs(got[:, :, rows] - ref_rows).max() <= RTOL * np.abs(ref_rows).max()
    e = err.cpu().numpy()
    np.testing.assert_allclose(e, got.sum(axis=2), rtol=1e-5)
    si, pi = (int(v) for v in best.cpu().numpy())
    assert e[si, pi] == e.min()
