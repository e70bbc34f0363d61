"""CPU oracle for the BCQ linear layer of GPTQT -- TEST INFRASTRUCTURE ONLY.

Thin ctypes access to ``bcq_oracle.c`` (plain C, fp64).  Only the tests, the smoke
check and the benchmark's CPU-baseline leg may import this package; the product
library never does, and nothing here imports the product.

Array conventions (numpy, C-contiguous):
    w_int, codes  uint8  [N, K]
    S, qbias, z   float16 [N, G]      G = K // group, or 1 when group == 0 (per row)
    alpha         float16 [q, N, G]
    planes        uint8  [q, N, K // 8]
    x             float16 [B, K]
    y             float64 [B, N]
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bcq_oracle.c")
_LIB = os.path.join(_HERE, "libbcq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over output rows).  Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_half_to_double.restype = ctypes.c_double
        _lib.orc_half_to_double.argtypes = [ctypes.c_uint16]
        _lib.orc_double_to_half.restype = ctypes.c_uint16
        _lib.orc_double_to_half.argtypes = [ctypes.c_double]
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle rejected the arguments of {what}")


def num_threads() -> int:
    return int(_load().orc_num_threads())


def half_to_double(bits: int) -> float:
    return float(_load().orc_half_to_double(int(bits)))


def double_to_half_bits(v: float) -> int:
    return int(_load().orc_double_to_half(float(v)))


def bcchoice(n_bits: int, bit_to_plane) -> tuple[np.ndarray, np.ndarray]:
    """Eq. fuse_step1/2.  Returns (m[q], value[2**q]); value[c] is what sign pattern c reaches."""
    b2p = _c(bit_to_plane, np.uint8)
    q = int(b2p.max()) + 1 if b2p.size else 0
    m = np.zeros(8, np.float64)
    value = np.zeros(256, np.float64)
    rc = _load().orc_bcchoice(ctypes.c_int(n_bits), ctypes.c_int(q), _p(b2p), _p(m), _p(value))
    _check(rc, "bcchoice")
    return m[:q].copy(), value[: 1 << q].copy()


def round_to_bcchoice(w_int, n_bits: int, bit_to_plane) -> tuple[np.ndarray, np.ndarray]:
    """Eq. round.  Returns (W_q, codes), both uint8 with the shape of w_int."""
    w = _c(w_int, np.uint8)
    b2p = _c(bit_to_plane, np.uint8)
    q = int(b2p.max()) + 1
    wq = np.empty_like(w)
    codes = np.empty_like(w)
    rc = _load().orc_round_to_bcchoice(_p(w), ctypes.c_size_t(w.size), ctypes.c_int(n_bits),
                                       ctypes.c_int(q), _p(b2p), _p(wq), _p(codes))
    _check(rc, "round_to_bcchoice")
    return wq, codes


def quantize_rtn(W, group: int, n_bits: int, s_factor: float = 1.0):
    """Eq. gptqt step 1 with S = s_factor (Wmax - Wmin)/(2^n - 1), qbias = Wmin per (row, group).
    W fp16 [N, K].  Returns (w_int [N,K] u8, S [N,G] f16, qbias [N,G] f16)."""
    W = _c(W, np.float16)
    N, K = W.shape
    G = 1 if group == 0 else K // group
    w_int = np.empty((N, K), np.uint8)
    S = np.empty((N, G), np.float16)
    qbias = np.empty((N, G), np.float16)
    rc = _load().orc_quantize_rtn(_p(W), ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group), ctypes.c_int(n_bits),
                                  ctypes.c_double(s_factor), _p(w_int), _p(S), _p(qbias))
    _check(rc, "quantize_rtn")
    return w_int, S, qbias


def merge_linear(w_int, S, qbias, group: int, n_bits: int, bit_to_plane):
    """Eq. fuse_step3.  Returns (codes [N,K] u8, alpha [q,N,G] f16, z [N,G] f16)."""
    w = _c(w_int, np.uint8)
    N, K = w.shape
    G = 1 if group == 0 else K // group
    S = _c(S, np.float16).reshape(N, G)
    qbias = _c(qbias, np.float16).reshape(N, G)
    b2p = _c(bit_to_plane, np.uint8)
    q = int(b2p.max()) + 1
    codes = np.empty((N, K), np.uint8)
    alpha = np.empty((q, N, G), np.float16)
    z = np.empty((N, G), np.float16)
    rc = _load().orc_merge_linear(_p(w), _p(S), _p(qbias), ctypes.c_int(N), ctypes.c_int(K),
                                  ctypes.c_int(group), ctypes.c_int(n_bits), ctypes.c_int(q),
                                  _p(b2p), _p(codes), _p(alpha), _p(z))
    _check(rc, "merge_linear")
    return codes, alpha, z


def pack_canonical(codes, q: int) -> np.ndarray:
    c = _c(codes, np.uint8)
    N, K = c.shape
    planes = np.empty((q, N, K // 8), np.uint8)
    rc = _load().orc_pack_canonical(_p(c), ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(q), _p(planes))
    _check(rc, "pack_canonical")
    return planes


def unpack_canonical(planes) -> np.ndarray:
    p = _c(planes, np.uint8)
    q, N, KB = p.shape
    codes = np.empty((N, KB * 8), np.uint8)
    rc = _load().orc_unpack_canonical(_p(p), ctypes.c_int(N), ctypes.c_int(KB * 8), ctypes.c_int(q), _p(codes))
    _check(rc, "unpack_canonical")
    return codes


def _scales(alpha, z, N, K, group):
    G = 1 if group == 0 else K // group
    alpha = _c(alpha, np.float16)
    q = alpha.shape[0]
    alpha = alpha.reshape(q, N, G)
    z = _c(z, np.float16).reshape(N, G)
    return alpha, z, q


def dequant(codes, alpha, z, group: int) -> np.ndarray:
    """Eq. bcw dequantisation plus the fused offset: W[n,k] = sum_i alpha_i b_i + z (fp64)."""
    c = _c(codes, np.uint8)
    N, K = c.shape
    alpha, z, q = _scales(alpha, z, N, K, group)
    W = np.empty((N, K), np.float64)
    rc = _load().orc_dequant(_p(c), _p(alpha), _p(z), ctypes.c_int(N), ctypes.c_int(K),
                             ctypes.c_int(q), ctypes.c_int(group), _p(W))
    _check(rc, "dequant")
    return W


def forward_dequant(codes, alpha, z, x, group: int) -> np.ndarray:
    """y = W x with W dequantised element by element (fp64).  x [B,K] or [K]."""
    c = _c(codes, np.uint8)
    N, K = c.shape
    alpha, z, q = _scales(alpha, z, N, K, group)
    x = _c(x, np.float16).reshape(-1, K)
    B = x.shape[0]
    y = np.empty((B, N), np.float64)
    rc = _load().orc_forward_dequant(_p(c), _p(alpha), _p(z), _p(x), ctypes.c_int(N), ctypes.c_int(K),
                                     ctypes.c_int(q), ctypes.c_int(group), ctypes.c_int(B), _p(y))
    _check(rc, "forward_dequant")
    return y


def forward_planes(planes, alpha, z, x, group: int) -> np.ndarray:
    """y = sum_g ( sum_i alpha_i (B_i x)_g + z (sum x)_g ) from packed bit-planes (fp64)."""
    p = _c(planes, np.uint8)
    q, N, KB = p.shape
    K = KB * 8
    alpha, z, q2 = _scales(alpha, z, N, K, group)
    if q2 != q:
        raise ValueError("alpha and planes disagree on q")
    x = _c(x, np.float16).reshape(-1, K)
    B = x.shape[0]
    y = np.empty((B, N), np.float64)
    rc = _load().orc_forward_planes(_p(p), _p(alpha), _p(z), _p(x), ctypes.c_int(N), ctypes.c_int(K),
                                    ctypes.c_int(q), ctypes.c_int(group), ctypes.c_int(B), _p(y))
    _check(rc, "forward_planes")
    return y


# ---- the search over BCchoice and the re-explored scale (sections "Quantize Weight Twice" and
# ---- "Re-explore Scale Factor") -------------------------------------------------------------------

def set_partitions(n_bits: int, q: int):
    """Every way of dealing the n step-1 bits into q non-empty planes (the BCchoice candidates of Eq. round
    built as Eq. fuse_step2 builds them), each once, as bit_to_plane arrays: planes are numbered in the
    order of their lowest bit, and the arrays come in lexicographic order."""
    out = []

    def grow(prefix, used):
        if len(prefix) == n_bits:
            if used == q:
                out.append(np.array(prefix, np.uint8))
            return
        for p in range(min(used + 1, q)):
            grow(prefix + [p], max(used, p + 1))

    grow([], 0)
    return out


def reexplore_factors(n_bits: int, count: int) -> np.ndarray:
    """`count` evenly spaced scale factors strictly inside the interval of Eq. reexplore, as multiples s of the
    step-1 scale (Wmax - Wmin)/(2^n - 1):  s in ((2^n - 1)/(2^(n+1) - 1), (2^n - 1)/(2^(n-1) - 1))."""
    lo = (2.0 ** n_bits - 1.0) / (2.0 ** (n_bits + 1) - 1.0)
    hi = (2.0 ** n_bits - 1.0) / (2.0 ** (n_bits - 1) - 1.0)
    return lo + (hi - lo) * (np.arange(count, dtype=np.float64) + 1.0) / (count + 1.0)


def grid_search(W, X, group: int, n_bits: int, partitions, s_factors):
    """Eq. gptqt step 2 searched as the section "Re-explore Scale Factor" says: for every scale factor (outer
    loop) and every BCchoice (inner loop) quantise W by step 1 with that scale, round to the BCchoice, and
    measure the output error on the calibration inputs,  sum_t || (S W_q + qbias - W) x_t ||^2  (fp64).
    W fp16 [N, K]; X fp16 [T, K].  Returns (err_rows [S, P, N], err [S, P], (si, pi)) where (si, pi) is the
    first candidate, in loop order, whose error is below all earlier ones."""
    W = _c(W, np.float16)
    X = _c(X, np.float16)
    N, K = W.shape
    G = 1 if group == 0 else K // group
    glen = K // G
    Wd, Xd = W.astype(np.float64), X.astype(np.float64)
    err_rows = np.zeros((len(s_factors), len(partitions), N), np.float64)
    for si, s in enumerate(s_factors):
        w_int, S, qbias = quantize_rtn(W, group, n_bits, float(s))
        Sd = np.repeat(S.astype(np.float64), glen, axis=1)
        qd = np.repeat(qbias.astype(np.float64), glen, axis=1)
        for pi, b2p in enumerate(partitions):
            wq, _ = round_to_bcchoice(w_int, n_bits, b2p)
            dW = Sd * wq.astype(np.float64) + qd - Wd           # dequantised minus original weights
            E = dW @ Xd.T                                        # [N, T]: the error of every output
            err_rows[si, pi] = (E * E).sum(axis=1)
    err = err_rows.sum(axis=2)
    best, best_err = (0, 0), np.inf
    for si in range(len(s_factors)):
        for pi in range(len(partitions)):
            if err[si, pi] < best_err:
                best, best_err = (si, pi), err[si, pi]
    return err_rows, err, best
