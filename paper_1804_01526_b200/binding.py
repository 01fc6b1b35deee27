"""ctypes binding of ``libhbfp.so`` (the C ABI declared in ``include/hbfp.h``).

Argument marshalling only: every step of the path runs in the CUDA kernels of the library.
PyTorch supplies device memory and the current stream. There is no fallback: if the shared
library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, replace
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# HBFP_LIBRARY selects another build of the same library (e.g. one with debug checks).
LIB_PATH = os.environ.get("HBFP_LIBRARY") or os.path.join(_HERE, "libhbfp.so")

(OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT,
 ERR_STATIC_LIMIT, ERR_EXPONENT_RANGE) = range(9)
STATIC_WORKSPACE_BYTES = 16 << 20
GEMM_AUTO, GEMM_FORCE_SIMT, GEMM_FORCE_TENSOR, GEMM_FORCE_TENSOR_1SM, GEMM_FORCE_TENSOR_2SM, GEMM_FORCE_SMALL = 0, 1, 2, 3, 4, 5
ROUND_NEAREST_EVEN, ROUND_STOCHASTIC = 0, 1

EXPORTS = [
    "hbfp_status_string", "hbfp_packed_layout", "hbfp_packed_sizes", "hbfp_quantize",
    "hbfp_quantize_tiles", "hbfp_unpack", "hbfp_dequantize", "hbfp_gemm_workspace",
    "hbfp_gemm_q_workspace", "hbfp_gemm", "hbfp_gemm_q", "hbfp_gemm_block_partials",
    "hbfp_device_status", "hbfp_gemm_static", "hbfp_wide_quantize", "hbfp_wide_update", "hbfp_wide_narrow",
    "hbfp_im2col_packed", "hbfp_im2col_packed_t", "hbfp_wide_dequantize", "hbfp_selftest_bounded_wait", "hbfp_last_gemm_kernel", "hbfp_last_gemm_cycles", "hbfp_conv_forward", "hbfp_quantize_conv_weights", "hbfp_conv_dgrad_filters",
]


class HbfpError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


class _CFormat(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("mant_bits", ctypes.c_int32),
                ("block", ctypes.c_int32), ("tile", ctypes.c_int32), ("rounding", ctypes.c_int32),
                ("exp_mode", ctypes.c_int32), ("stream_id", ctypes.c_uint32),
                ("reserved", ctypes.c_uint32), ("seed", ctypes.c_uint64)]


class _CLayout(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in
                ("rows", "k", "b", "bp", "nkb", "kst", "planes", "plane_stride", "rs",
                 "mant_bytes", "exp_bytes")]


class _COperand(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("kind", ctypes.c_int32),
                ("data", ctypes.c_void_p), ("exps", ctypes.c_void_p), ("ld", ctypes.c_int64),
                ("trans", ctypes.c_int32), ("reserved", ctypes.c_int32), ("fmt", _CFormat)]


@dataclass(frozen=True)
class Format:
    """Mirror of ``hbfp_format``."""
    mant_bits: int = 8
    block: int = 32
    tile: int = 0
    rounding: int = 0
    exp_mode: int = 0
    seed: int = 0
    stream_id: int = 0

    def c(self) -> _CFormat:
        return _CFormat(ctypes.sizeof(_CFormat), self.mant_bits, self.block, self.tile, self.rounding,
                        self.exp_mode, self.stream_id, 0, self.seed)


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with "
                              "`python -m paper_1804_01526_b200.build` (there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        i64, p, i32, u32, sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_uint32, ctypes.c_size_t
        L.hbfp_status_string.restype = ctypes.c_char_p
        L.hbfp_status_string.argtypes = [i32]
        L.hbfp_packed_layout.argtypes = [i64, i64, p, p]
        L.hbfp_packed_sizes.argtypes = [i64, i64, p, p, p]
        L.hbfp_quantize.argtypes = [p, i64, i64, i64, i32, p, p, p, p]
        L.hbfp_quantize_tiles.argtypes = [p, i64, i64, i64, p, p, p, p, p, p, p]
        L.hbfp_wide_quantize.argtypes = [p, i64, i64, i64, p, p, p, p, p, p, p, p]
        L.hbfp_wide_update.argtypes = [p, p, p, i64, i64, i64, p, p, p, p, p, p]
        L.hbfp_wide_narrow.argtypes = [p, p, i64, i64, p, p, p, p, p, p]
        L.hbfp_im2col_packed.argtypes = [p, p, i64, i64, i64, i64, i32, i32, i32, p, p, p, p]
        L.hbfp_im2col_packed_t.argtypes = [p, i64, i64, i64, i64, i32, i32, i32, p, p, p, p]
        L.hbfp_unpack.argtypes = [p, p, i64, i64, p, p, p, p]
        L.hbfp_dequantize.argtypes = [p, p, i64, i64, p, p, i64, p]
        L.hbfp_gemm_workspace.argtypes = [i32, i32, i64, i64, i64, p, p, p]
        L.hbfp_gemm_q_workspace.argtypes = [i64, i64, i64, p, p, p]
        L.hbfp_gemm.argtypes = [i32, i32, i64, i64, i64, p, i64, p, i64, p, i64, p, p, p, sz, u32, p]
        L.hbfp_gemm_q.argtypes = [i64, i64, i64, p, p, p, i64, p, sz, u32, p]
        L.hbfp_gemm_static.argtypes = [i32, i32, i64, i64, i64, p, i64, p, i64, p, i64, p, p, u32, p]
        L.hbfp_gemm_block_partials.argtypes = [i64, i64, i64, p, p, p, u32, p]
        L.hbfp_device_status.argtypes = [p, p]
        L.hbfp_quantize_conv_weights.argtypes = [p, i64, i64, i64, i64, p, p, p, p, p, p, p]
        L.hbfp_conv_forward.argtypes = [p, p, i64, i64, i64, i64, i32, i32, i32, p, p, i64, p, i64, p]
        L.hbfp_conv_dgrad_filters.argtypes = [p, p, i32, i32, i64, i64, p, p, p, p]
        L.hbfp_wide_dequantize.argtypes = [p, p, i64, i64, i32, p, i64, p]
        L.hbfp_selftest_bounded_wait.argtypes = [i64, i32, p, p]
        L.hbfp_last_gemm_cycles.argtypes = [p]
        L.hbfp_last_gemm_kernel.restype = ctypes.c_char_p
        L.hbfp_last_gemm_kernel.argtypes = []
        for name in EXPORTS[1:]:
            if name != "hbfp_last_gemm_kernel":
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().hbfp_status_string(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != OK:
        raise HbfpError(code, where)


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dptr(t: Optional[torch.Tensor]) -> ctypes.c_void_p:
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def packed_layout(rows: int, k: int, fmt: Format) -> dict:
    out = _CLayout()
    cf = fmt.c()
    _check(lib().hbfp_packed_layout(rows, k, ctypes.byref(cf), ctypes.byref(out)), "hbfp_packed_layout")
    return {n: getattr(out, n) for n, _ in _CLayout._fields_}


def packed_sizes(rows: int, k: int, fmt: Format) -> Tuple[int, int]:
    mb, eb = ctypes.c_size_t(), ctypes.c_size_t()
    cf = fmt.c()
    _check(lib().hbfp_packed_sizes(rows, k, ctypes.byref(cf), ctypes.byref(mb), ctypes.byref(eb)),
           "hbfp_packed_sizes")
    return mb.value, eb.value


@dataclass
class Packed:
    """A quantised GEMM operand held on the device (see "Packed operand layout" in hbfp.h)."""
    mant: torch.Tensor     # int8, mant_bytes
    exps: torch.Tensor     # int8, exp_bytes
    rows: int
    k: int
    fmt: Format

    def operand(self) -> _COperand:
        return _COperand(ctypes.sizeof(_COperand), 1, self.mant.data_ptr(), self.exps.data_ptr(), 0, 0, 0,
                         self.fmt.c())


def alloc_packed(rows: int, k: int, fmt: Format, device="cuda") -> Packed:
    mb, eb = packed_sizes(rows, k, fmt)
    return Packed(torch.empty(mb, dtype=torch.int8, device=device),
                  torch.empty(eb, dtype=torch.int8, device=device), rows, k, fmt)


def _check_f32(x: torch.Tensor, name: str) -> None:
    if not (x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and (x.shape[1] <= 1 or x.stride(1) == 1)):
        raise ValueError(f"{name} must be a 2-D float32 CUDA tensor with contiguous rows")


def _ld(x: torch.Tensor) -> int:
    return x.stride(0) if x.shape[0] > 1 else max(x.shape[1], 1)


def quantize(x: torch.Tensor, contract_axis: int, fmt: Format, out: Optional[Packed] = None) -> Packed:
    """hbfp_quantize: blocks along ``contract_axis`` of the 2-D float32 CUDA tensor ``x``."""
    _check_f32(x, "x")
    d0, d1 = x.shape
    rows, k = (d0, d1) if contract_axis == 1 else (d1, d0)
    if out is None:
        out = alloc_packed(rows, k, fmt, x.device)
    cf = fmt.c()
    _check(lib().hbfp_quantize(_dptr(x), d0, d1, _ld(x), contract_axis, ctypes.byref(cf), _dptr(out.mant),
                               _dptr(out.exps), _stream()), "hbfp_quantize")
    return out


def quantize_tiles(w: torch.Tensor, fmt: Format, out: Optional[Tuple[Packed, Packed]] = None,
                   want_grid: bool = True):
    """hbfp_quantize_tiles: both packed views of ``w`` (``c0``: contraction down the rows of w,
    ``c1``: along them) and the tile exponent grid."""
    _check_f32(w, "w")
    d0, d1 = w.shape
    c0, c1 = out if out is not None else (alloc_packed(d1, d0, fmt, w.device), alloc_packed(d0, d1, fmt, w.device))
    t = max(fmt.tile, 1)
    grid = torch.empty(((d0 + t - 1) // t, (d1 + t - 1) // t), dtype=torch.int8, device=w.device) if want_grid else None
    cf = fmt.c()
    _check(lib().hbfp_quantize_tiles(_dptr(w), d0, d1, _ld(w), ctypes.byref(cf), _dptr(c0.mant), _dptr(c0.exps),
                                     _dptr(c1.mant), _dptr(c1.exps), _dptr(grid), _stream()),
           "hbfp_quantize_tiles")
    return c0, c1, grid


class Wide:
    """Wide weight storage of ``w [d0][d1]``: int16 mantissas ``[d0][d1]`` and int8 tile exponents
    ``[ceil(d0/t)][ceil(d1/t)]`` (device tensors)."""

    def __init__(self, mant: torch.Tensor, exps: torch.Tensor, tile: int):
        self.mant, self.exps, self.tile = mant, exps, tile


def _alloc_views(d0: int, d1: int, fmt: Format, device) -> Tuple[Packed, Packed]:
    return alloc_packed(d1, d0, fmt, device), alloc_packed(d0, d1, fmt, device)


def _view_args(views: Optional[Tuple[Packed, Packed]]):
    if views is None:
        return [ctypes.c_void_p(0)] * 4
    c0, c1 = views
    return [_dptr(c0.mant), _dptr(c0.exps), _dptr(c1.mant), _dptr(c1.exps)]


def wide_quantize(w: torch.Tensor, fmt: Format, out: Optional[Wide] = None, views: Optional[Tuple[Packed, Packed]] = None,
                  want_views: bool = True):
    """hbfp_wide_quantize: FP32 weights -> wide storage and (unless ``want_views`` is false) the two
    packed narrow views of ``fmt.mant_bits`` bits. Returns ``(wide, (c0, c1) or None)``."""
    _check_f32(w, "w")
    d0, d1 = w.shape
    t = fmt.tile
    if out is None:
        out = Wide(torch.empty((d0, d1), dtype=torch.int16, device=w.device),
                   torch.empty((-(-d0 // t), -(-d1 // t)), dtype=torch.int8, device=w.device), t)
    if views is None and want_views:
        views = _alloc_views(d0, d1, fmt, w.device)
    f = fmt.c()
    _check(lib().hbfp_wide_quantize(_dptr(w), d0, d1, _ld(w), ctypes.byref(f), _dptr(out.mant), _dptr(out.exps),
                                    *_view_args(views), _stream()), "hbfp_wide_quantize")
    return out, views


def wide_update(wide: Wide, delta: torch.Tensor, fmt: Format, views: Optional[Tuple[Packed, Packed]] = None,
                want_views: bool = True):
    """hbfp_wide_update: ``wide <- Q16(float32(wide + delta))`` in place; returns the narrow views."""
    _check_f32(delta, "delta")
    d0, d1 = wide.mant.shape
    if tuple(delta.shape) != (d0, d1):
        raise ValueError("delta must have the shape of the weights")
    if views is None and want_views:
        views = _alloc_views(d0, d1, fmt, delta.device)
    f = fmt.c()
    _check(lib().hbfp_wide_update(_dptr(wide.mant), _dptr(wide.exps), _dptr(delta), d0, d1, _ld(delta), ctypes.byref(f),
                                  *_view_args(views), _stream()), "hbfp_wide_update")
    return views


def wide_narrow(wide: Wide, fmt: Format, views: Optional[Tuple[Packed, Packed]] = None) -> Tuple[Packed, Packed]:
    """hbfp_wide_narrow: the two packed views of the top ``fmt.mant_bits`` bits of the wide mantissas."""
    d0, d1 = wide.mant.shape
    if views is None:
        views = _alloc_views(d0, d1, fmt, wide.mant.device)
    f = fmt.c()
    _check(lib().hbfp_wide_narrow(_dptr(wide.mant), _dptr(wide.exps), d0, d1, ctypes.byref(f), *_view_args(views),
                                  _stream()), "hbfp_wide_narrow")
    return views


def wide_dequantize(wide: Wide, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """hbfp_wide_dequantize: the FP32 value ``mant * 2^exps`` of the wide copy (exact)."""
    d0, d1 = wide.mant.shape
    if out is None:
        out = torch.empty((d0, d1), dtype=torch.float32, device=wide.mant.device)
    _check_f32(out, "out")
    _check(lib().hbfp_wide_dequantize(_dptr(wide.mant), _dptr(wide.exps), d0, d1, wide.tile, _dptr(out), _ld(out),
                                      _stream()), "hbfp_wide_dequantize")
    return out


def selftest_bounded_wait(limit_cycles: int = 20000, code: int = 777) -> int:
    """hbfp_selftest_bounded_wait: one warp runs the kernels' bounded barrier wait on a barrier nobody
    arrives on; returns the outcome word (2 = the wait was abandoned)."""
    outcome = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check(lib().hbfp_selftest_bounded_wait(limit_cycles, code, _dptr(outcome), _stream()), "hbfp_selftest_bounded_wait")
    return int(outcome.item())


def im2col_packed(px: Packed, n: int, h: int, w: int, c: int, kh: int, kw: int, pad: int,
                  out: Optional[Packed] = None) -> Packed:
    """hbfp_im2col_packed: the packed convolution operand ``[n*ho*wo][kh*kw*c]`` gathered from the
    packed pixels ``px`` (``quantize(x.view(n*h*w, c), 1, fmt)`` with ``fmt.block == c``)."""
    ho, wo = h + 2 * pad - kh + 1, w + 2 * pad - kw + 1
    if out is None:
        out = alloc_packed(n * ho * wo, kh * kw * c, px.fmt, px.mant.device)
    f = px.fmt.c()
    _check(lib().hbfp_im2col_packed(_dptr(px.mant), _dptr(px.exps), n, h, w, c, kh, kw, pad, ctypes.byref(f),
                                    _dptr(out.mant), _dptr(out.exps), _stream()), "hbfp_im2col_packed")
    return out


def quantize_conv_weights(w: torch.Tensor, taps: int, fmt: Format, want_grid: bool = False, out=None):
    """hbfp_quantize_conv_weights: convolution weights ``w [taps * c_in][c_out]`` with one exponent per tile of
    ``t`` input maps x ``t`` output maps over all taps. Returns ``(c0, c1, grid or None)``."""
    _check_f32(w, "w")
    d0, d1 = w.shape
    c_in = d0 // taps
    c0, c1 = out if out is not None else _alloc_views(d0, d1, fmt, w.device)
    t = fmt.tile
    grid = torch.empty((c_in // t, -(-d1 // t)), dtype=torch.int8, device=w.device) if want_grid else None
    f = fmt.c()
    _check(lib().hbfp_quantize_conv_weights(_dptr(w), taps, c_in, d1, _ld(w), ctypes.byref(f), _dptr(c0.mant), _dptr(c0.exps),
                                            _dptr(c1.mant), _dptr(c1.exps), _dptr(grid) if grid is not None else None,
                                            _stream()), "hbfp_quantize_conv_weights")
    return c0, c1, grid


def conv_dgrad_filters(c1: Packed, kh: int, kw: int, c_in: int, c_out: int, out: Optional[Packed] = None) -> Packed:
    """hbfp_conv_dgrad_filters: the filter operand of the backward-data convolution (rows = c_in, k = kh*kw*c_out)
    from view ``c1`` of ``quantize_conv_weights``: the forward pass's mantissas and tile exponents, taps reversed."""
    if out is None:
        out = alloc_packed(c_in, kh * kw * c_out, c1.fmt, c1.mant.device)
    f = c1.fmt.c()
    _check(lib().hbfp_conv_dgrad_filters(_dptr(c1.mant), _dptr(c1.exps), kh, kw, c_in, c_out, ctypes.byref(f), _dptr(out.mant),
                                         _dptr(out.exps), _stream()), "hbfp_conv_dgrad_filters")
    return out


def conv_forward(px: Packed, filters: Packed, n: int, h: int, w: int, c: int, kh: int, kw: int, pad: int,
                 out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """hbfp_conv_forward: the convolution ``[n*h*w][filters]`` of packed pixels ``px`` (block = c) with the
    packed filters ``filters`` (rows = filters, k = kh*kw*c) as one implicit GEMM. Raises ``HbfpError``
    (ERR_UNSUPPORTED) for shapes the kernel does not cover."""
    nf = filters.rows
    if out is None:
        out = torch.empty((n * h * w, nf), dtype=torch.float32, device=px.mant.device)
    _check_f32(out, "out")
    fx = px.fmt.c()
    op = filters.operand()
    _check(lib().hbfp_conv_forward(_dptr(px.mant), _dptr(px.exps), n, h, w, c, kh, kw, pad, ctypes.byref(fx), ctypes.byref(op),
                                   nf, _dptr(out), _ld(out), _stream()), "hbfp_conv_forward")
    return out


def im2col_packed_t(x: torch.Tensor, kh: int, kw: int, pad: int, fmt: Format, out: Optional[Packed] = None) -> Packed:
    """hbfp_im2col_packed_t: the packed backward-weight operand ``[kh*kw*c][n*h*w]`` (blocks of
    ``fmt.block`` consecutive output pixels) straight from FP32 activations ``x [n][h][w][c]``."""
    if not (x.is_cuda and x.dtype == torch.float32 and x.dim() == 4 and x.is_contiguous()):
        raise ValueError("x must be a contiguous float32 CUDA tensor [n][h][w][c]")
    n, h, w, c = x.shape
    if out is None:
        out = alloc_packed(kh * kw * c, n * h * w, fmt, x.device)
    f = fmt.c()
    _check(lib().hbfp_im2col_packed_t(_dptr(x), n, h, w, c, kh, kw, pad, ctypes.byref(f), _dptr(out.mant),
                                      _dptr(out.exps), _stream()), "hbfp_im2col_packed_t")
    return out


def unpack(p: Packed) -> Tuple[torch.Tensor, torch.Tensor]:
    """hbfp_unpack: canonical ``q [rows][k]`` int16 and ``s [rows][nkb]`` int8."""
    lay = packed_layout(p.rows, p.k, p.fmt)
    q = torch.empty((p.rows, p.k), dtype=torch.int16, device=p.mant.device)
    s = torch.empty((p.rows, lay["nkb"]), dtype=torch.int8, device=p.mant.device)
    cf = p.fmt.c()
    _check(lib().hbfp_unpack(_dptr(p.mant), _dptr(p.exps), p.rows, p.k, ctypes.byref(cf), _dptr(q), _dptr(s),
                             _stream()), "hbfp_unpack")
    return q, s


def dequantize(p: Packed) -> torch.Tensor:
    out = torch.empty((p.rows, p.k), dtype=torch.float32, device=p.mant.device)
    cf = p.fmt.c()
    _check(lib().hbfp_dequantize(_dptr(p.mant), _dptr(p.exps), p.rows, p.k, ctypes.byref(cf), _dptr(out),
                                 max(p.k, 1), _stream()), "hbfp_dequantize")
    return out


def gemm_workspace(transA: int, transB: int, M: int, N: int, K: int, fmtA: Format, fmtB: Format) -> int:
    b = ctypes.c_size_t()
    fa, fb = fmtA.c(), fmtB.c()
    _check(lib().hbfp_gemm_workspace(transA, transB, M, N, K, ctypes.byref(fa), ctypes.byref(fb), ctypes.byref(b)),
           "hbfp_gemm_workspace")
    return b.value


def _gemm_dims(transA, transB, A, B):
    M, K = (A.shape[1], A.shape[0]) if transA else A.shape
    K2, N = (B.shape[1], B.shape[0]) if transB else B.shape
    if K != K2:
        raise ValueError("contraction extents differ")
    return M, N, K


def gemm(transA: int, transB: int, A: torch.Tensor, B: torch.Tensor, fmtA: Format, fmtB: Format,
         out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
         flags: int = GEMM_AUTO) -> torch.Tensor:
    """hbfp_gemm: ``C = op(A) op(B)`` with both FP32 operands quantised by the call."""
    _check_f32(A, "A")
    _check_f32(B, "B")
    M, N, K = _gemm_dims(transA, transB, A, B)
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=A.device)
    if workspace is None:
        workspace = torch.empty(max(gemm_workspace(transA, transB, M, N, K, fmtA, fmtB), 1), dtype=torch.int8,
                                device=A.device)
    fa, fb = fmtA.c(), fmtB.c()
    _check(lib().hbfp_gemm(transA, transB, M, N, K, _dptr(A), _ld(A), _dptr(B), _ld(B), _dptr(out), _ld(out),
                           ctypes.byref(fa), ctypes.byref(fb), _dptr(workspace), workspace.numel(), flags,
                           _stream()), "hbfp_gemm")
    return out


def gemm_static(transA: int, transB: int, A: torch.Tensor, B: torch.Tensor, fmtA: Format, fmtB: Format,
                out: Optional[torch.Tensor] = None, flags: int = GEMM_AUTO) -> torch.Tensor:
    """hbfp_gemm_static: hbfp_gemm on the library's built-in scratch, for callers that cannot
    allocate device memory. Pass ``out`` if the output, too, must come from memory you already
    own; problems larger than the built-in scratch raise ``HbfpError`` (ERR_STATIC_LIMIT)."""
    _check_f32(A, "A")
    _check_f32(B, "B")
    M, N, K = _gemm_dims(transA, transB, A, B)
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=A.device)
    fa, fb = fmtA.c(), fmtB.c()
    _check(lib().hbfp_gemm_static(transA, transB, M, N, K, _dptr(A), _ld(A), _dptr(B), _ld(B), _dptr(out),
                                  _ld(out), ctypes.byref(fa), ctypes.byref(fb), flags, _stream()),
           "hbfp_gemm_static")
    return out


def _as_operand(x, trans: int, fmt: Optional[Format]):
    if isinstance(x, Packed):
        return x.operand()
    _check_f32(x, "operand")
    return _COperand(ctypes.sizeof(_COperand), 0, x.data_ptr(), 0, _ld(x), trans, 0, fmt.c())


def gemm_q_workspace(M: int, N: int, K: int, a, b, transA=0, transB=0, fmtA=None, fmtB=None) -> int:
    oa, ob = _as_operand(a, transA, fmtA), _as_operand(b, transB, fmtB)
    n = ctypes.c_size_t()
    _check(lib().hbfp_gemm_q_workspace(M, N, K, ctypes.byref(oa), ctypes.byref(ob), ctypes.byref(n)),
           "hbfp_gemm_q_workspace")
    return n.value


def gemm_q(M: int, N: int, K: int, a, b, transA: int = 0, transB: int = 0, fmtA: Optional[Format] = None,
           fmtB: Optional[Format] = None, out: Optional[torch.Tensor] = None,
           workspace: Optional[torch.Tensor] = None, flags: int = GEMM_AUTO) -> torch.Tensor:
    """hbfp_gemm_q: each operand is an FP32 tensor (with its trans flag and format) or a ``Packed``."""
    oa, ob = _as_operand(a, transA, fmtA), _as_operand(b, transB, fmtB)
    dev = a.mant.device if isinstance(a, Packed) else a.device
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = torch.empty(max(gemm_q_workspace(M, N, K, a, b, transA, transB, fmtA, fmtB), 1),
                                dtype=torch.int8, device=dev)
    _check(lib().hbfp_gemm_q(M, N, K, ctypes.byref(oa), ctypes.byref(ob), _dptr(out), _ld(out), _dptr(workspace),
                             workspace.numel(), flags, _stream()), "hbfp_gemm_q")
    return out


def gemm_block_partials(a: Packed, b: Packed, impl: int = GEMM_FORCE_SIMT) -> torch.Tensor:
    """hbfp_gemm_block_partials: int32 ``P [M][N][nkb]``."""
    M, N, K = a.rows, b.rows, a.k
    nkb = packed_layout(M, K, a.fmt)["nkb"]
    P = torch.empty((M, N, nkb), dtype=torch.int32, device=a.mant.device)
    oa, ob = a.operand(), b.operand()
    _check(lib().hbfp_gemm_block_partials(M, N, K, ctypes.byref(oa), ctypes.byref(ob), _dptr(P), impl, _stream()),
           "hbfp_gemm_block_partials")
    return P


def last_gemm_cycles() -> int:
    """hbfp_last_gemm_cycles: SM cycles of the longest CTA of the most recent paired-SM GEMM launch (synchronises)."""
    out = ctypes.c_uint64(0)
    _check(lib().hbfp_last_gemm_cycles(ctypes.byref(out)), "hbfp_last_gemm_cycles")
    return int(out.value)


def last_gemm_kernel() -> str:
    """hbfp_last_gemm_kernel: the GEMM kernel this thread's last GEMM call launched."""
    return lib().hbfp_last_gemm_kernel().decode()


def device_status() -> int:
    """hbfp_device_status: synchronises the current stream, returns and clears the status word."""
    return device_status_rc()[1]


def device_status_rc():
    """hbfp_device_status as (return code, recorded code): (OK, 0), (ERR_TIMEOUT, code below 900) or
    (ERR_EXPONENT_RANGE, code 900-999)."""
    v = ctypes.c_int32()
    rc = lib().hbfp_device_status(_stream(), ctypes.byref(v))
    return rc, v.value
