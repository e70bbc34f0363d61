"""ctypes binding of the C ABI in include/bcq.h -- argument marshalling only.

Every function takes torch CUDA tensors (device memory) and forwards their data pointers and
the current torch CUDA stream to the library entry point of the same name.  There is no
fallback: if libbcq.so is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbcq.so")

LAYOUT_CANONICAL = 0
LAYOUT_TILED = 1

OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED_SHAPE = -2
ERR_MISALIGNED = -3
ERR_WORKSPACE_TOO_SMALL = -4
ERR_CUDA = -5
ERR_SCRATCH_LIMIT = -6
ERR_TIMEOUT = -7
NOALLOC_SCRATCH_BYTES = 2 << 20
PLAN_TEST_SHORT_WAITS = 1      # bcq_plan.reserved bits used by the library's own tests (see include/bcq.h)
PLAN_TEST_WITHHOLD_TABLE = 2


class Desc(ctypes.Structure):
    """bcq_desc"""
    _fields_ = [("N", ctypes.c_int32), ("K", ctypes.c_int32), ("q", ctypes.c_int32),
                ("group", ctypes.c_int32), ("layout", ctypes.c_int32)]

    def with_layout(self, layout: int) -> "Desc":
        return Desc(self.N, self.K, self.q, self.group, layout)

    @property
    def G(self) -> int:
        return 1 if self.group == 0 else self.K // self.group


class Plan(ctypes.Structure):
    """bcq_plan"""
    _fields_ = [("kernel", ctypes.c_int32), ("row_blocks", ctypes.c_int32),
                ("k_splits", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class Operand(ctypes.Structure):
    """bcq_operand"""
    _fields_ = [("packed_dev", ctypes.c_void_p), ("alpha_dev", ctypes.c_void_p), ("z_dev", ctypes.c_void_p),
                ("y_dev", ctypes.c_void_p), ("N", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class Epilogue(ctypes.Structure):
    """bcq_epilogue"""
    _fields_ = [("bias_dev", ctypes.c_void_p), ("residual_dev", ctypes.c_void_p), ("activation", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]


ACT_NONE, ACT_RELU, ACT_GELU, ACT_SILU = 0, 1, 2, 3


class BcqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        msg = lib().bcq_status_string(status).decode()
        if status == ERR_CUDA:
            msg += ": " + lib().bcq_last_cuda_error().decode()
        super().__init__(f"{what}: {msg} ({status})")


_lib = None
_vp, _sz, _i = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
_dp, _pp = ctypes.POINTER(Desc), ctypes.POINTER(Plan)

SIGNATURES = {
    "bcq_version": (_i, []),
    "bcq_status_string": (ctypes.c_char_p, [_i]),
    "bcq_last_cuda_error": (ctypes.c_char_p, []),
    "bcq_check_desc": (_i, [_dp]),
    "bcq_packed_bytes": (_sz, [_dp]),
    "bcq_alpha_elems": (_sz, [_dp]),
    "bcq_offset_elems": (_sz, [_dp]),
    "bcq_plan_default": (_i, [_dp, _i, _i, _pp]),
    "bcq_workspace_bytes": (_sz, [_dp, _i, _pp]),
    "bcq_workspace_init": (_i, [_vp, _sz, _vp]),
    "bcq_merge_linear": (_i, [_dp, _vp, _vp, _vp, _i, _vp, _vp, _vp, _vp, _vp]),
    "bcq_quantize_rtn": (_i, [_dp, _vp, _i, _vp, ctypes.c_double, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "bcq_pack": (_i, [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "bcq_repack": (_i, [_dp, _vp, _vp, _vp, _dp, _vp, _vp, _vp, _vp]),
    "bcq_gemv": (_i, [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "bcq_gemv_plan": (_i, [_dp, _pp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "bcq_gemv_bf16": (_i, [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "bcq_gemv_dequant": (_i, [_dp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "bcq_gemv_fused": (_i, [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "bcq_gemv_multi": (_i, [_dp, _vp, _i, _vp, _vp, _sz, _vp]),
    "bcq_gemv_multi_plan": (_i, [_dp, _pp, _vp, _i, _vp, _vp, _sz, _vp]),
    "bcq_multi_row_blocks": (_i, [_dp, _pp, _vp, _i, _vp]),
    "bcq_gemm_smallbatch": (_i, [_dp, _vp, _vp, _vp, _vp, _vp, _i, _vp, _sz, _vp]),
    "bcq_gemm_smallbatch_plan": (_i, [_dp, _pp, _vp, _vp, _vp, _vp, _vp, _i, _vp, _sz, _vp]),
    "bcq_gemv_host": (_i, [_dp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "bcq_gemv_noalloc": (_i, [_dp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "bcq_poll_status": (_i, []),
    "bcq_grid_search_workspace": (_sz, [_dp, _i, _i, _i, _i, _i]),
    "bcq_grid_search": (_i, [_dp, _vp, _vp, _i, _i, _vp, _i, _vp, _i, _vp, _vp, _vp, _vp, _sz, _vp]),
    "bcq_partition_count": (_i, [_i, _i]),
    "bcq_partition_get": (_i, [_i, _i, _i, _vp]),
    "bcq_reexplore_factors": (_i, [_i, _i, _vp]),
}


def lib() -> ctypes.CDLL:
    """Load libbcq.so (built in-tree by paper_2407_02891_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2407_02891_b200.build`; "
                               "there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _dev(*ts):
    for t in ts:
        if t is not None and not t.is_cuda:
            raise ValueError("expected a CUDA tensor")


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc: int, what: str):
    if rc != OK:
        raise BcqError(rc, what)


def desc(N: int, K: int, q: int, group: int, layout: int = LAYOUT_CANONICAL) -> Desc:
    return Desc(N, K, q, group, layout)


def check_desc(d: Desc) -> int:
    return lib().bcq_check_desc(ctypes.byref(d))


def packed_bytes(d: Desc) -> int:
    return lib().bcq_packed_bytes(ctypes.byref(d))


def alpha_elems(d: Desc) -> int:
    return lib().bcq_alpha_elems(ctypes.byref(d))


def offset_elems(d: Desc) -> int:
    return lib().bcq_offset_elems(ctypes.byref(d))


def plan_default(d: Desc, B: int = 1, sm_count: int = 0) -> Plan:
    p = Plan()
    _check(lib().bcq_plan_default(ctypes.byref(d), B, sm_count, ctypes.byref(p)), "bcq_plan_default")
    return p


def workspace_bytes(d: Desc, B: int = 1, plan: Plan | None = None) -> int:
    return lib().bcq_workspace_bytes(ctypes.byref(d), B, ctypes.byref(plan) if plan is not None else None)


def workspace_init(ws: torch.Tensor):
    _dev(ws)
    _check(lib().bcq_workspace_init(_ptr(ws), ws.numel() * ws.element_size(), _stream()), "bcq_workspace_init")


def new_workspace(d: Desc, B: int = 1, plan: Plan | None = None, device="cuda") -> torch.Tensor | None:
    """Allocate (torch) and zero-fill a workspace for the plan; None when none is needed."""
    n = workspace_bytes(d, B, plan)
    if n == 0:
        return None
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    workspace_init(ws)
    return ws


def _ws_args(ws):
    if ws is None:
        return None, 0
    _dev(ws)
    return _ptr(ws), ws.numel() * ws.element_size()


def merge_linear(d: Desc, w_int, S, qbias, n_bits: int, bit_to_plane, codes, alpha, z):
    _dev(w_int, S, qbias, codes, alpha, z)
    b2p = (ctypes.c_uint8 * len(bit_to_plane))(*[int(v) for v in bit_to_plane])
    if len(bit_to_plane) != n_bits:
        raise ValueError("bit_to_plane needs n_bits entries")
    _check(lib().bcq_merge_linear(ctypes.byref(d), _ptr(w_int), _ptr(S), _ptr(qbias), n_bits,
                                  ctypes.cast(b2p, ctypes.c_void_p), _ptr(codes), _ptr(alpha), _ptr(z),
                                  _stream()), "bcq_merge_linear")


def quantize_rtn(d: Desc, W, n_bits: int, bit_to_plane, S, qbias, w_int, packed, alpha, z, s_factor: float = 1.0):
    """bcq_quantize_rtn: fp16 weights W [N, K] -> S, qbias, (w_int), packed, alpha, z in d's layout."""
    _dev(W, S, qbias, w_int, packed, alpha, z)
    if len(bit_to_plane) != n_bits:
        raise ValueError("bit_to_plane needs n_bits entries")
    b2p = (ctypes.c_uint8 * len(bit_to_plane))(*[int(v) for v in bit_to_plane])
    _check(lib().bcq_quantize_rtn(ctypes.byref(d), _ptr(W), n_bits, ctypes.cast(b2p, ctypes.c_void_p), float(s_factor),
                                  _ptr(S), _ptr(qbias), _ptr(w_int), _ptr(packed), _ptr(alpha), _ptr(z), _stream()),
           "bcq_quantize_rtn")


def pack(d: Desc, codes, alpha_in, z_in, packed_out, alpha_out, z_out):
    _dev(codes, alpha_in, z_in, packed_out, alpha_out, z_out)
    _check(lib().bcq_pack(ctypes.byref(d), _ptr(codes), _ptr(alpha_in), _ptr(z_in), _ptr(packed_out),
                          _ptr(alpha_out), _ptr(z_out), _stream()), "bcq_pack")


def repack(src: Desc, packed_src, alpha_src, z_src, dst: Desc, packed_dst, alpha_dst, z_dst):
    _dev(packed_src, alpha_src, z_src, packed_dst, alpha_dst, z_dst)
    _check(lib().bcq_repack(ctypes.byref(src), _ptr(packed_src), _ptr(alpha_src), _ptr(z_src),
                            ctypes.byref(dst), _ptr(packed_dst), _ptr(alpha_dst), _ptr(z_dst), _stream()),
           "bcq_repack")


def gemv(d: Desc, packed, alpha, z, x, y, workspace=None):
    _dev(packed, alpha, z, x, y)
    wp, wn = _ws_args(workspace)
    _check(lib().bcq_gemv(ctypes.byref(d), _ptr(packed), _ptr(alpha), _ptr(z), _ptr(x), _ptr(y), wp, wn,
                          _stream()), "bcq_gemv")


def gemv_bf16(d: Desc, packed, alpha, z, x, y, bias=None, residual=None, activation=ACT_NONE, workspace=None):
    """bcq_gemv_bf16: x, y (and bias, residual) are torch.bfloat16 tensors."""
    _dev(packed, alpha, z, x, y, bias, residual)
    wp, wn = _ws_args(workspace)
    ep = None
    if bias is not None or residual is not None or activation != ACT_NONE:
        ep = ctypes.byref(Epilogue(None if bias is None else bias.data_ptr(), None if residual is None else residual.data_ptr(),
                                   activation, 0))
    _check(lib().bcq_gemv_bf16(ctypes.byref(d), _ptr(packed), _ptr(alpha), _ptr(z), _ptr(x), _ptr(y), ep, wp, wn, _stream()),
           "bcq_gemv_bf16")


def gemv_dequant(d: Desc, packed, alpha, z, x, y):
    """The ablation without lookup tables (bcq_gemv_dequant)."""
    _dev(packed, alpha, z, x, y)
    _check(lib().bcq_gemv_dequant(ctypes.byref(d), _ptr(packed), _ptr(alpha), _ptr(z), _ptr(x), _ptr(y), _stream()),
           "bcq_gemv_dequant")


def gemv_fused(d: Desc, packed, alpha, z, x, y, bias=None, residual=None, activation=ACT_NONE, workspace=None):
    """y = act(W x + bias) + residual (bcq_gemv_fused)."""
    _dev(packed, alpha, z, x, y, bias, residual)
    wp, wn = _ws_args(workspace)
    ep = Epilogue(None if bias is None else bias.data_ptr(), None if residual is None else residual.data_ptr(), activation, 0)
    _check(lib().bcq_gemv_fused(ctypes.byref(d), _ptr(packed), _ptr(alpha), _ptr(z), _ptr(x), _ptr(y), ctypes.byref(ep),
                                wp, wn, _stream()), "bcq_gemv_fused")


def gemv_plan(d: Desc, plan: Plan, packed, alpha, z, x, y, workspace=None):
    _dev(packed, alpha, z, x, y)
    wp, wn = _ws_args(workspace)
    _check(lib().bcq_gemv_plan(ctypes.byref(d), ctypes.byref(plan), _ptr(packed), _ptr(alpha), _ptr(z), _ptr(x),
                               _ptr(y), wp, wn, _stream()), "bcq_gemv_plan")


def _operands(layers, ys):
    arr = (Operand * len(layers))()
    for o, (L, y) in enumerate(zip(layers, ys)):
        _dev(L.packed, L.alpha, L.z, y)
        arr[o] = Operand(_ptr(L.packed), _ptr(L.alpha), _ptr(L.z), _ptr(y), L.d.N, 0)
    return arr


def gemv_multi(d: Desc, layers, x, ys, workspace=None, plan: Plan | None = None):
    """bcq_gemv_multi(_plan): the layers (Layer objects that share K, q, group) times one x; d.N = sum of rows."""
    _dev(x)
    arr = _operands(layers, ys)
    wp, wn = _ws_args(workspace)
    if plan is None:
        _check(lib().bcq_gemv_multi(ctypes.byref(d), ctypes.cast(arr, ctypes.c_void_p), len(layers), _ptr(x), wp, wn,
                                    _stream()), "bcq_gemv_multi")
    else:
        _check(lib().bcq_gemv_multi_plan(ctypes.byref(d), ctypes.byref(plan), ctypes.cast(arr, ctypes.c_void_p),
                                         len(layers), _ptr(x), wp, wn, _stream()), "bcq_gemv_multi_plan")


def multi_row_blocks(d: Desc, plan: Plan, Ns) -> list[int]:
    n = (ctypes.c_int32 * len(Ns))(*[int(v) for v in Ns])
    out = (ctypes.c_int32 * len(Ns))()
    _check(lib().bcq_multi_row_blocks(ctypes.byref(d), ctypes.byref(plan), ctypes.cast(n, ctypes.c_void_p), len(Ns),
                                      ctypes.cast(out, ctypes.c_void_p)), "bcq_multi_row_blocks")
    return list(out)


def gemm_smallbatch(d: Desc, packed, alpha, z, X, Y, B: int, workspace=None):
    _dev(packed, alpha, z, X, Y)
    wp, wn = _ws_args(workspace)
    _check(lib().bcq_gemm_smallbatch(ctypes.byref(d), _ptr(packed), _ptr(alpha), _ptr(z), _ptr(X), _ptr(Y), B,
                                     wp, wn, _stream()), "bcq_gemm_smallbatch")


def gemm_smallbatch_plan(d: Desc, plan: Plan, packed, alpha, z, X, Y, B: int, workspace=None):
    _dev(packed, alpha, z, X, Y)
    wp, wn = _ws_args(workspace)
    _check(lib().bcq_gemm_smallbatch_plan(ctypes.byref(d), ctypes.byref(plan), _ptr(packed), _ptr(alpha), _ptr(z), _ptr(X),
                                          _ptr(Y), B, wp, wn, _stream()), "bcq_gemm_smallbatch_plan")


def gemv_host(d: Desc, packed, alpha, z, x_host, y_host, x_stage, y_stage, workspace=None):
    """x_host / y_host are CPU tensors (pinned for asynchronous copies); the caller synchronises."""
    _dev(packed, alpha, z, x_stage, y_stage)
    if x_host.is_cuda or y_host.is_cuda:
        raise ValueError("x_host and y_host must be host tensors")
    wp, wn = _ws_args(workspace)
    _check(lib().bcq_gemv_host(ctypes.byref(d), _ptr(packed), _ptr(alpha), _ptr(z), _ptr(x_host), _ptr(y_host),
                               _ptr(x_stage), _ptr(y_stage), wp, wn, _stream()), "bcq_gemv_host")


def poll_status():
    """bcq_poll_status: synchronise and raise if a bounded device-side wait ran out since the last poll."""
    _check(lib().bcq_poll_status(), "bcq_poll_status")


def gemv_noalloc(d: Desc, packed, alpha, z, x, y):
    """bcq_gemv_noalloc: no workspace argument; the library's built-in scratch array is used.

    For callers that cannot allocate device memory.  All calls on a device share that array, so
    only issue them on one stream (or otherwise ordered); see include/bcq.h for the limits.
    """
    _dev(packed, alpha, z, x, y)
    _check(lib().bcq_gemv_noalloc(ctypes.byref(d), _ptr(packed), _ptr(alpha), _ptr(z), _ptr(x), _ptr(y),
                                  _stream()), "bcq_gemv_noalloc")


@dataclass
class Layer:
    """Device-resident operands of one packed layer (a convenience holder, no arithmetic)."""
    d: Desc
    packed: torch.Tensor
    alpha: torch.Tensor | None
    z: torch.Tensor | None


def scales_in_tiles(d: Desc) -> bool:
    """True when the layout keeps alpha and z inside `packed` (tiled, group 128)."""
    return d.layout == LAYOUT_TILED and d.group != 0


def empty_operands(d: Desc, device):
    """Uninitialised torch tensors for (packed, alpha, z) of a descriptor; alpha/z are None when
    the scales live inside `packed`."""
    rc = check_desc(d)
    if rc != OK:
        raise BcqError(rc, "bcq_check_desc")
    packed = torch.empty(packed_bytes(d), dtype=torch.uint8, device=device)
    if scales_in_tiles(d):
        return packed, None, None
    return (packed, torch.empty(alpha_elems(d), dtype=torch.float16, device=device),
            torch.empty(offset_elems(d), dtype=torch.float16, device=device))


def pack_layer(N, K, q, group, layout, codes, alpha, z) -> Layer:
    """bcq_pack into freshly allocated torch tensors.  codes/alpha/z: canonical CUDA tensors."""
    d = desc(N, K, q, group, layout)
    packed, a, zz = empty_operands(d, codes.device)
    pack(d, codes, alpha, z, packed, a, zz)
    return Layer(d, packed, a, zz)


def partitions(n_bits: int, q: int):
    """All bit_to_plane arrays of bcq_partition_get, as a uint8 numpy array [P, n_bits]."""
    import numpy as np
    P = lib().bcq_partition_count(n_bits, q)
    out = np.zeros((P, n_bits), np.uint8)
    for i in range(P):
        _check(lib().bcq_partition_get(n_bits, q, i, out[i].ctypes.data_as(ctypes.c_void_p)), "bcq_partition_get")
    return out


def reexplore_factors(n_bits: int, count: int):
    import numpy as np
    out = np.zeros(count, np.float64)
    _check(lib().bcq_reexplore_factors(n_bits, count, out.ctypes.data_as(ctypes.c_void_p)), "bcq_reexplore_factors")
    return out


def grid_search(N, K, q, group, W, X, n_bits, parts, s_factors, want_rows=True):
    """bcq_grid_search on torch CUDA tensors W [N, K], X [T, K] (fp16); parts: uint8 numpy [P, n_bits]; s_factors:
    float64 numpy.  Returns (err [S, P] float64 tensor, err_rows [S, P, N] float32 tensor or None, best [2] int32 tensor)."""
    import numpy as np
    _dev(W, X)
    d = desc(N, K, q, group, LAYOUT_CANONICAL)
    parts = np.ascontiguousarray(parts, np.uint8)
    s_factors = np.ascontiguousarray(s_factors, np.float64)
    P, S, T = parts.shape[0], s_factors.shape[0], X.shape[0]
    nbytes = lib().bcq_grid_search_workspace(ctypes.byref(d), T, n_bits, P, S, 1 if want_rows else 0)
    if nbytes == 0:
        raise BcqError(ERR_INVALID_ARG, "bcq_grid_search_workspace")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=W.device)
    err = torch.empty((S, P), dtype=torch.float64, device=W.device)
    rows = torch.empty((S, P, N), dtype=torch.float32, device=W.device) if want_rows else None
    best = torch.zeros(2, dtype=torch.int32, device=W.device)
    _check(lib().bcq_grid_search(ctypes.byref(d), _ptr(W), _ptr(X), T, n_bits, parts.ctypes.data_as(ctypes.c_void_p), P,
                                 s_factors.ctypes.data_as(ctypes.c_void_p), S, _ptr(err), _ptr(rows), _ptr(best), _ptr(ws),
                                 nbytes, _stream()), "bcq_grid_search")
    return err, rows, best
