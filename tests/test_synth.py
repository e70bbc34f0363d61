"""The seeded input generators: determinism, random access, host/torch agreement, distributions."""
import numpy as np
import torch

from paper_2407_02891_b200 import synth


def test_streams_are_deterministic_and_distinct():
    a = synth.u64("a", 0, 16)
    assert np.array_equal(a, synth.u64("a", 0, 16))
    assert np.array_equal(a[5:9], synth.u64("a", 5, 4))          # counter-based: random access
    assert not np.array_equal(a, synth.u64("b", 0, 16))
    assert not np.array_equal(a, synth.u64("a", 0, 16, seed=1))


def test_plane_rows_match_full_tensor():
    for (N, K, q) in [(16, 32, 3), (40, 512, 2), (24, 1024, 3)]:
        full = synth.planes("t", N, K, q)
        rows = [0, 3, N - 1]
        assert np.array_equal(synth.plane_rows("t", N, K, q, rows), full[:, rows, :])


def test_planes_device_matches_host():
    for (N, K, q) in [(16, 32, 3), (24, 1024, 3)]:
        host = synth.planes("t", N, K, q)
        dev = synth.planes_device("t", N, K, q, torch.device("cpu")).numpy()
        assert np.array_equal(host, dev)


def test_scale_rows_random_access_and_ranges():
    N, K, q, group = 64, 1024, 3, 128
    alpha, z = synth.scale_rows("t", N, K, q, group)
    assert alpha.shape == (q, N, 8) and z.shape == (N, 8)
    a2, z2 = synth.scale_rows("t", N, K, q, group, rows=[5, 63])
    assert np.array_equal(a2, alpha[:, [5, 63]]) and np.array_equal(z2, z[[5, 63]])
    a = alpha.astype(np.float64)
    assert a[0].min() >= 0.0099 and a[0].max() <= 0.0501
    for i in (1, 2):
        r = a[i] / (a[0] * 2.0 ** -i)
        assert r.min() >= 0.79 and r.max() <= 1.21
    assert abs(z.astype(np.float64).std() - synth.Z_STD) < 0.002
    ap, _ = synth.scale_rows("t", N, K, q, 0)
    assert ap.shape == (q, N, 1)


def test_bits_and_activations_look_right():
    p = synth.planes("t2", 64, 4096, 3)
    frac = np.unpackbits(p).mean()
    assert abs(frac - 0.5) < 0.005
    x = synth.activations("t2", 4, 4096).astype(np.float64)
    assert abs(x.mean()) < 0.03 and abs(x.std() - 1.0) < 0.03
    codes = synth.codes_from_planes(p)
    assert codes.max() == 7 and codes.shape == (64, 4096)


def test_linear_int_case_is_fp16_exact():
    for n in (3, 4, 5):
        w, S, qbias = synth.linear_int_case("t3", 16, 32, 32, n)
        assert w.max() == (1 << n) - 1
        S64, b64 = S.astype(np.float64), qbias.astype(np.float64)
        k = 2.0 * b64 / S64
        assert np.array_equal(k, np.round(k)) and k.min() >= -48 and k.max() <= 15
        centre = ((1 << n) - 1) / 2.0
        zz = S64 * centre + b64
        assert np.array_equal(zz.astype(np.float16).astype(np.float64), zz)
