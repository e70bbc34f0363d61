"""Seeded synthetic inputs for the BCQ linear layer -- data only, none of the method's arithmetic.

Every tensor is a pure function of (seed, stream name, element index): a counter-based
SplitMix64 generator, so any slice (a few rows of a 28672 x 7168 layer, one layer out of
a 48-layer stack) can be regenerated on its own, on the host with numpy or -- for the
integer-only bit-planes -- on the device with torch integer ops, with identical bits.

The value distributions are those of the synthetic workloads this repository is
measured on; they stand in for the OPT / Llama-2 checkpoints the paper quantises
(only the layer shapes are taken from those model families):
    bits     uniform random
    alpha_0  ~ U(0.01, 0.05) per (row, group)
    alpha_i  = alpha_0 * 2^-i * (1 + U(-0.2, 0.2)),  i >= 1
    z        ~ N(0, std 0.01) per (row, group)
    x        ~ N(0, 1)
all rounded to fp16.  Floating-point draws are always made on the host in fp64.
"""
from __future__ import annotations

import numpy as np

SEED = 240702891
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
Z_STD = 0.01


def stream_key(name: str, seed: int = SEED) -> int:
    """64-bit key of a named stream (FNV-1a of the name, mixed with the seed)."""
    h = 0xCBF29CE484222325
    for ch in name.encode():
        h = ((h ^ ch) * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    v = np.array([(h ^ (seed * 0x9E3779B97F4A7C15)) & 0xFFFFFFFFFFFFFFFF], np.uint64)
    return int(_mix_np(v)[0])


def _mix_np(z: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def u64(name: str, start: int, count: int, seed: int = SEED) -> np.ndarray:
    """Draws start .. start+count-1 of the named stream as uint64."""
    key = np.uint64(stream_key(name, seed))
    with np.errstate(over="ignore"):
        idx = np.arange(start + 1, start + count + 1, dtype=np.uint64)
        return _mix_np(key + idx * _GOLDEN)


def uniform(name: str, start: int, count: int, seed: int = SEED) -> np.ndarray:
    """U[0,1) in fp64 (53 random bits)."""
    return (u64(name, start, count, seed) >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def normal(name: str, start: int, count: int, seed: int = SEED) -> np.ndarray:
    """N(0,1) in fp64 by Box-Muller; draw t uses counters 2t and 2t+1."""
    u = uniform(name, 2 * start, 2 * count, seed).reshape(count, 2)
    return np.sqrt(-2.0 * np.log1p(-u[:, 0])) * np.cos(2.0 * np.pi * u[:, 1])


# ---------------------------------------------------------------------------------------
# tensors of one linear layer; `name` identifies the layer (config / layer / projection)
# ---------------------------------------------------------------------------------------

def n_groups(K: int, group: int) -> int:
    return 1 if group == 0 else K // group


def plane_rows(name: str, N: int, K: int, q: int, rows) -> np.ndarray:
    """Canonical packed bit-planes of selected rows: uint8 [q, len(rows), K//8].

    The full tensor is uint8 [q, N, K//8] whose bytes are the little-endian bytes of the
    stream's uint64 draws in linear order.
    """
    rows = np.asarray(rows, np.int64)
    rb = K // 8
    out = np.empty((q, rows.size, rb), np.uint8)
    for i in range(q):
        for j, n in enumerate(rows):
            lo = (i * N + int(n)) * rb
            w0, w1 = lo // 8, (lo + rb + 7) // 8
            b = u64(name + "/planes", w0, w1 - w0).view(np.uint8)
            out[i, j] = b[lo - 8 * w0: lo - 8 * w0 + rb]
    return out


def planes(name: str, N: int, K: int, q: int) -> np.ndarray:
    """All canonical packed bit-planes, uint8 [q, N, K//8] (host)."""
    total = q * N * (K // 8)
    b = u64(name + "/planes", 0, (total + 7) // 8).view(np.uint8)[:total]
    return b.reshape(q, N, K // 8).copy()


def planes_device(name: str, N: int, K: int, q: int, device):
    """The same bytes as `planes`, produced on `device` with torch integer ops only."""
    import torch

    total = q * N * (K // 8)
    words = (total + 7) // 8

    def s64(v: int) -> int:  # uint64 constant as the int64 with the same bits
        return v - (1 << 64) if v >= (1 << 63) else v

    def lsr(t, s):  # logical shift right on int64
        return (t >> s) & ((1 << (64 - s)) - 1)

    key = s64(stream_key(name + "/planes"))
    out = torch.empty(words, dtype=torch.int64, device=device)
    step = 1 << 24
    for w0 in range(0, words, step):
        w1 = min(words, w0 + step)
        z = torch.arange(w0 + 1, w1 + 1, dtype=torch.int64, device=device) * s64(int(_GOLDEN)) + key
        z = (z ^ lsr(z, 30)) * s64(int(_M1))
        z = (z ^ lsr(z, 27)) * s64(int(_M2))
        out[w0:w1] = z ^ lsr(z, 31)
    return out.view(torch.uint8)[:total].reshape(q, N, K // 8)


def codes_from_planes(p: np.ndarray) -> np.ndarray:
    """uint8 [N, K] codes whose bit i is plane i's bit (pure re-indexing of the random bits)."""
    q, N, rb = p.shape
    bits = np.unpackbits(p, axis=2, bitorder="little")  # [q, N, K]
    codes = np.zeros((N, rb * 8), np.uint8)
    for i in range(q):
        codes |= (bits[i] << i).astype(np.uint8)
    return codes


def scale_rows(name: str, N: int, K: int, q: int, group: int, rows=None):
    """(alpha [q, R, G] f16, z [R, G] f16) for selected rows (all rows when rows is None)."""
    G = n_groups(K, group)
    rows = np.arange(N, dtype=np.int64) if rows is None else np.asarray(rows, np.int64)
    contiguous = rows.size == N
    alpha = np.empty((q, rows.size, G), np.float64)
    z = np.empty((rows.size, G), np.float64)

    def draw(fn, stream, per_row, out):
        if contiguous:
            out[...] = fn(stream, 0, N * per_row).reshape(out.shape)
        else:
            for j, n in enumerate(rows):
                out[j] = fn(stream, int(n) * per_row, per_row)

    a0 = np.empty((rows.size, G), np.float64)
    draw(uniform, name + "/alpha0", G, a0)
    alpha[0] = 0.01 + 0.04 * a0
    for i in range(1, q):
        j = np.empty((rows.size, G), np.float64)
        draw(uniform, f"{name}/jitter{i}", G, j)
        alpha[i] = alpha[0] * 2.0 ** (-i) * (1.0 + (0.4 * j - 0.2))
    draw(normal, name + "/z", G, z)
    return alpha.astype(np.float16), (Z_STD * z).astype(np.float16)


def activations(name: str, B: int, K: int) -> np.ndarray:
    """x ~ N(0,1), fp16 [B, K]."""
    return normal(name + "/x", 0, B * K).reshape(B, K).astype(np.float16)


def linear_int_case(name: str, N: int, K: int, group: int, n_bits: int):
    """Inputs of the linear-int -> binary-code conversion: (w_int u8 [N,K], S f16 [N,G], qbias f16 [N,G]).

    S has 5 significant bits and qbias is a multiple k * S/2 with -48 <= k <= 15, so that S,
    qbias and the fused alpha and z (for n_bits <= 5) all fit fp16's 11-bit significand exactly.
    """
    G = n_groups(K, group)
    w = (u64(name + "/w_int", 0, N * K) % np.uint64(1 << n_bits)).astype(np.uint8).reshape(N, K)
    mant = 16 + (u64(name + "/S_mant", 0, N * G) % np.uint64(16)).astype(np.float64)      # 16..31
    expo = (u64(name + "/S_exp", 0, N * G) % np.uint64(4)).astype(np.float64)             # 0..3
    S = (mant * 2.0 ** (-10 - expo)).reshape(N, G)                                        # ~[0.002, 0.03]
    kq = (u64(name + "/qbias", 0, N * G) % np.uint64(64)).astype(np.float64).reshape(N, G) - 48.0
    qbias = kq * S / 2.0
    return w, S.astype(np.float16), qbias.astype(np.float16)
