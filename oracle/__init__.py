"""ctypes front end of the HBFP oracle (``hbfp_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: the test-suite, the smoke check and the benchmark's CPU-baseline
leg may import this package; the CUDA library and its Python binding never do, and nothing
here imports them. The arithmetic lives in the C++ file; this module only builds the shared
object with plain ``g++ -O2 -fopenmp`` and marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hbfp_oracle.cpp")
_LIB = os.path.join(_HERE, "libhbfp_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["g++", "-std=c++17", "-O2", "-fopenmp", "-fPIC", "-shared",
               "-fno-fast-math", "-o", tmp, _SRC]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


class _Format(ctypes.Structure):
    _fields_ = [("mant_bits", ctypes.c_int32), ("block", ctypes.c_int32),
                ("tile", ctypes.c_int32), ("rounding", ctypes.c_int32),
                ("exp_mode", ctypes.c_int32), ("stream_id", ctypes.c_uint32),
                ("seed", ctypes.c_uint64), ("idx_row_off", ctypes.c_int64),
                ("idx_col_off", ctypes.c_int64), ("idx_cols", ctypes.c_int64)]


@dataclass(frozen=True)
class Format:
    """Block-floating-point format: m-bit mantissas (sign + m-1 bits), block/tile geometry,
    rounding (0 nearest-even, 1 stochastic), exponent rule and the random stream."""
    mant_bits: int = 8
    block: int = 32
    tile: int = 0
    rounding: int = 0
    exp_mode: int = 0
    seed: int = 0
    stream_id: int = 0
    idx_row_off: int = 0
    idx_col_off: int = 0
    idx_cols: int = 0

    def _c(self) -> _Format:
        return _Format(self.mant_bits, self.block, self.tile, self.rounding, self.exp_mode,
                       self.stream_id, self.seed, self.idx_row_off, self.idx_col_off,
                       self.idx_cols)


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        L = _lib
        i64, p = ctypes.c_int64, ctypes.c_void_p
        L.oracle_num_threads.restype = ctypes.c_int
        L.oracle_set_threads.argtypes = [ctypes.c_int]
        L.oracle_philox4x32_10.argtypes = [p, p, p]
        L.oracle_sr_draw.restype = ctypes.c_uint32
        L.oracle_sr_draw.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint64]
        L.oracle_block_exponent.restype = ctypes.c_int
        L.oracle_block_exponent.argtypes = [ctypes.c_double, ctypes.c_int, ctypes.c_int]
        L.oracle_round_rne.restype = ctypes.c_int32
        L.oracle_round_rne.argtypes = [ctypes.c_float, ctypes.c_int, ctypes.c_int]
        L.oracle_round_sr.restype = ctypes.c_int32
        L.oracle_round_sr.argtypes = [ctypes.c_float, ctypes.c_int, ctypes.c_int, ctypes.c_uint32]
        L.oracle_quantize.restype = ctypes.c_int
        L.oracle_quantize.argtypes = [p, i64, i64, i64, ctypes.c_int, p, p, p]
        L.oracle_gemm.restype = ctypes.c_int
        L.oracle_gemm.argtypes = [i64, i64, i64, i64, p, p, p, p, p, p, p, p, ctypes.c_int]
        L.oracle_quantize_indexed.restype = ctypes.c_int
        L.oracle_quantize_indexed.argtypes = [p, i64, i64, i64, ctypes.c_int, p, p, p, p]
        L.oracle_quantize_conv_weights.restype = ctypes.c_int
        L.oracle_quantize_conv_weights.argtypes = [p, i64, i64, i64, i64, ctypes.c_int, p, p, p]
        L.oracle_wide_narrow.restype = ctypes.c_int
        L.oracle_wide_narrow.argtypes = [p, p, i64, i64, ctypes.c_int, p, p]
        L.oracle_wide_update.restype = ctypes.c_int
        L.oracle_wide_update.argtypes = [p, p, p, i64, i64, i64, p]
        L.oracle_hbfp_gemm.restype = ctypes.c_int
        L.oracle_hbfp_gemm.argtypes = [ctypes.c_int, ctypes.c_int, i64, i64, i64, p, i64, p, i64,
                                       p, p, p, p, p]
    return _lib


def num_threads() -> int:
    return lib().oracle_num_threads()


def set_threads(n: int) -> None:
    lib().oracle_set_threads(int(n))


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def sr_draw(seed: int, stream_id: int, L: int) -> int:
    return int(lib().oracle_sr_draw(seed, stream_id, L))


def block_exponent(amax: float, mant_bits: int, exp_mode: int = 0) -> int:
    return int(lib().oracle_block_exponent(float(amax), mant_bits, exp_mode))


def round_rne(x: float, s: int, mant_bits: int) -> int:
    return int(lib().oracle_round_rne(float(np.float32(x)), s, mant_bits))


def round_sr(x: float, s: int, mant_bits: int, r: int) -> int:
    return int(lib().oracle_round_sr(float(np.float32(x)), s, mant_bits, r))


def n_blocks(k: int, block: int) -> int:
    b = block if block > 0 else max(k, 1)
    return (k + b - 1) // b


def quantize(x: np.ndarray, contract_axis: int, fmt: Format):
    """Quantise a 2-D float32 array with blocks along ``contract_axis``.

    Returns ``(q, s)``: ``q`` int16 ``[rows][k]`` and ``s`` int8 ``[rows][nkb]`` with ``k`` the
    contraction extent and ``rows`` the other one (so for ``contract_axis == 0`` the result is
    laid out as the transpose of ``x``)."""
    assert x.dtype == np.float32 and x.ndim == 2
    if x.strides[1] != 4:
        x = np.ascontiguousarray(x)
    ld = x.strides[0] // 4 if x.shape[0] > 1 else x.shape[1]
    d0, d1 = x.shape
    k, rows = (d1, d0) if contract_axis == 1 else (d0, d1)
    nkb = n_blocks(k, fmt.block)
    q = np.zeros((rows, k), dtype=np.int16)
    s = np.zeros((rows, nkb), dtype=np.int8)
    cf = fmt._c()
    rc = lib().oracle_quantize(_ptr(x), d0, d1, max(ld, d1), contract_axis, ctypes.byref(cf),
                               _ptr(q), _ptr(s))
    if rc:
        raise ValueError(f"oracle_quantize failed: {rc}")
    return q, s


def dequantize(q: np.ndarray, s: np.ndarray, block: int) -> np.ndarray:
    """Eq. 1 on canonical arrays: value = q * 2^s (float64)."""
    rows, k = q.shape
    b = block if block > 0 else max(k, 1)
    sc = np.repeat(np.ldexp(1.0, s.astype(np.int64)), b, axis=1)[:, :k]
    return q.astype(np.float64) * sc


def gemm(qA, sA, qB, sB, block: int, want_partials: bool = False, exact_p: bool = False):
    """BFP product of canonical operands ``qA [M][K]``, ``qB [N][K]``.

    Returns a dict with ``c_ref`` (float32), ``a_mag`` (float64), ``c_seq`` (float32) and, if
    asked, ``P`` (int32 ``[M][N][nkb]``)."""
    M, K = qA.shape
    N, K2 = qB.shape
    assert K == K2
    nkb = n_blocks(K, block)
    assert sA.shape == (M, nkb) and sB.shape == (N, nkb)
    qA = np.ascontiguousarray(qA, dtype=np.int16)
    qB = np.ascontiguousarray(qB, dtype=np.int16)
    sA = np.ascontiguousarray(sA, dtype=np.int8)
    sB = np.ascontiguousarray(sB, dtype=np.int8)
    c_ref = np.zeros((M, N), dtype=np.float32)
    a_mag = np.zeros((M, N), dtype=np.float64)
    c_seq = np.zeros((M, N), dtype=np.float32)
    P = np.zeros((M, N, nkb), dtype=np.int32) if want_partials else None
    rc = lib().oracle_gemm(M, N, K, block, _ptr(qA), _ptr(sA), _ptr(qB), _ptr(sB),
                           _ptr(c_ref), _ptr(a_mag), _ptr(c_seq), _ptr(P), int(exact_p))
    if rc:
        raise ValueError(f"oracle_gemm failed: {rc}")
    out = {"c_ref": c_ref, "a_mag": a_mag, "c_seq": c_seq}
    if want_partials:
        out["P"] = P
    return out


def hbfp_gemm(transA: int, transB: int, A: np.ndarray, B: np.ndarray, fmtA: Format, fmtB: Format):
    """Quantise op(A), op(B) along the contraction axis, then the BFP product."""
    A = np.ascontiguousarray(A, dtype=np.float32)
    B = np.ascontiguousarray(B, dtype=np.float32)
    M, K = (A.shape[1], A.shape[0]) if transA else A.shape
    K2, N = (B.shape[1], B.shape[0]) if transB else B.shape
    assert K == K2
    c_ref = np.zeros((M, N), dtype=np.float32)
    a_mag = np.zeros((M, N), dtype=np.float64)
    c_seq = np.zeros((M, N), dtype=np.float32)
    fa, fb = fmtA._c(), fmtB._c()
    rc = lib().oracle_hbfp_gemm(transA, transB, M, N, K, _ptr(A), A.shape[1], _ptr(B), B.shape[1],
                                ctypes.byref(fa), ctypes.byref(fb), _ptr(c_ref), _ptr(a_mag),
                                _ptr(c_seq))
    if rc:
        raise ValueError(f"oracle_hbfp_gemm failed: {rc}")
    return {"c_ref": c_ref, "a_mag": a_mag, "c_seq": c_seq}


def quantize_indexed(x: np.ndarray, contract_axis: int, fmt: Format, index: np.ndarray):
    """``quantize`` with the stochastic-rounding draw of element ``(i, j)`` taken at ``index[i, j]`` (its
    position in the tensor it is a copy of; negative = structural zero, no draw)."""
    assert x.dtype == np.float32 and x.ndim == 2 and index.shape == x.shape
    x = np.ascontiguousarray(x)
    index = np.ascontiguousarray(index, dtype=np.int64)
    d0, d1 = x.shape
    k, rows = (d1, d0) if contract_axis == 1 else (d0, d1)
    q = np.zeros((rows, k), dtype=np.int16)
    s = np.zeros((rows, n_blocks(k, fmt.block)), dtype=np.int8)
    cf = fmt._c()
    rc = lib().oracle_quantize_indexed(_ptr(x), d0, d1, d1, contract_axis, ctypes.byref(cf), _ptr(index), _ptr(q), _ptr(s))
    if rc:
        raise ValueError(f"oracle_quantize_indexed failed: {rc}")
    return q, s


def quantize_conv_weights(w: np.ndarray, taps: int, contract_axis: int, fmt: Format):
    """Convolution weights ``w [taps * c_in][c_out]`` with one exponent per tile of ``t`` input maps x ``t``
    output maps across all filter taps (``fmt.tile``). Returns ``(q, s)`` laid out like ``quantize``."""
    assert w.dtype == np.float32 and w.ndim == 2 and w.shape[0] % taps == 0
    w = np.ascontiguousarray(w)
    d0, d1 = w.shape
    c_in = d0 // taps
    k, rows = (d1, d0) if contract_axis == 1 else (d0, d1)
    q = np.zeros((rows, k), dtype=np.int16)
    s = np.zeros((rows, n_blocks(k, fmt.tile)), dtype=np.int8)
    cf = fmt._c()
    rc = lib().oracle_quantize_conv_weights(_ptr(w), taps, c_in, d1, d1, contract_axis, ctypes.byref(cf), _ptr(q), _ptr(s))
    if rc:
        raise ValueError(f"oracle_quantize_conv_weights failed: {rc}")
    return q, s


def wide_quantize(w: np.ndarray, fmt: Format):
    """Wide weight storage of a stored weight matrix ``w [d0][d1]``: 16-bit mantissas ``q16 [d0][d1]``
    and canonical exponents ``s16 [d0][ceil(d1/t)]``, one exponent per ``t x t`` tile (``fmt.tile``)."""
    f16 = Format(**{**fmt.__dict__, "mant_bits": 16})
    return quantize(w, 1, f16)


def wide_narrow(q16: np.ndarray, s16: np.ndarray, mant_bits: int):
    """The narrow copy the passes read: the ``mant_bits`` most significant bits of every mantissa."""
    q16 = np.ascontiguousarray(q16, dtype=np.int16)
    s16 = np.ascontiguousarray(s16, dtype=np.int8)
    qm, sm = np.zeros_like(q16), np.zeros_like(s16)
    rc = lib().oracle_wide_narrow(_ptr(q16), _ptr(s16), q16.size, s16.size, int(mant_bits), _ptr(qm), _ptr(sm))
    if rc:
        raise ValueError(f"oracle_wide_narrow failed: {rc}")
    return qm, sm


def wide_update(q16: np.ndarray, s16: np.ndarray, delta: np.ndarray, fmt: Format):
    """``w = float32(q16 * 2^s16 + delta)`` re-quantised to wide storage; returns new ``(q16, s16)``."""
    assert delta.dtype == np.float32 and delta.shape == q16.shape
    q = np.ascontiguousarray(q16, dtype=np.int16).copy()
    s = np.ascontiguousarray(s16, dtype=np.int8).copy()
    delta = np.ascontiguousarray(delta)
    d0, d1 = q.shape
    cf = fmt._c()
    rc = lib().oracle_wide_update(_ptr(q), _ptr(s), _ptr(delta), d1, d0, d1, ctypes.byref(cf))
    if rc:
        raise ValueError(f"oracle_wide_update failed: {rc}")
    return q, s


def im2col(x: np.ndarray, kh: int, kw: int, pad: int) -> np.ndarray:
    """Convolution as a matrix product (the paper runs convolutions through the same BFP dot products,
    Sec. 5.1): ``x [n][h][w][c]`` -> ``[n*ho*wo][kh*kw*c]`` with ``ho = h + 2 pad - kh + 1`` (stride 1),
    row = output pixel, columns ordered tap-major ``(i, j, channel)``, zeros outside the image. With a
    block of ``c`` along the columns every block is the channel vector of one input pixel."""
    assert x.ndim == 4
    n, h, w, c = x.shape
    ho, wo = h + 2 * pad - kh + 1, w + 2 * pad - kw + 1
    out = np.zeros((n, ho, wo, kh, kw, c), dtype=x.dtype)
    for i in range(kh):
        for j in range(kw):
            for oy in range(ho):
                iy = oy + i - pad
                if iy < 0 or iy >= h:
                    continue
                for ox in range(wo):
                    ix = ox + j - pad
                    if 0 <= ix < w:
                        out[:, oy, ox, i, j, :] = x[:, iy, ix, :]
    return out.reshape(n * ho * wo, kh * kw * c)


def im2col_index(n: int, h: int, w: int, c: int, kh: int, kw: int, pad: int) -> np.ndarray:
    """For every element of ``im2col(x, kh, kw, pad)`` the row-major index in ``x [n][h][w][c]`` of the
    activation it is a copy of, -1 for the zeros outside the image (int64, same shape as the im2col matrix)."""
    ids = np.arange(1, n * h * w * c + 1, dtype=np.int64).reshape(n, h, w, c)
    return im2col(ids, kh, kw, pad) - 1
