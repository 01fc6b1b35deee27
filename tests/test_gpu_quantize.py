"""GPU parity of the quantiser: packed mantissas and exponents must equal the oracle's bit for bit,
stochastic rounding included, through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_1804_01526_b200 import workloads as wl
from tests.helpers import decode_packed, gfmt, ofmt, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hb():
    from paper_1804_01526_b200 import binding
    binding.lib()
    return binding


def _check(hb, x, axis, fd):
    """Quantise on both sides, compare canonical arrays (through hbfp_unpack and through a raw
    decode of the packed buffers, which also checks the zero padding)."""
    q_ref, s_ref = oracle.quantize(x, axis, ofmt(fd))
    p = hb.quantize(to_dev(x), axis, gfmt(fd))
    q, s = hb.unpack(p)
    assert np.array_equal(s.cpu().numpy(), s_ref), "exponents differ"
    assert np.array_equal(q.cpu().numpy(), q_ref), "mantissas differ"
    qd, sd = decode_packed(p, hb.packed_layout(p.rows, p.k, p.fmt))
    assert np.array_equal(qd, q_ref) and np.array_equal(sd, s_ref)
    assert hb.device_status() == 0
    return p


def F(m=8, b=32, tile=0, rounding=0, seed=0, sid=0, exp_mode=0):
    return dict(mant_bits=m, block=b, tile=tile, rounding=rounding, seed=seed, stream_id=sid, exp_mode=exp_mode)


ROW_CASES = [
    ((256, 256), "normal", F(8, 32)),                       # the 256^3 configuration's operand
    ((70, 520), "lognormal", F(8, 64, rounding=1, seed=5)),  # ragged rows, ragged last block
    ((33, 1024), "outliers", F(12, 128, rounding=1, seed=7, sid=3)),
    ((100, 1536), "lognormal", F(12, 256)),
    ((1000, 64), "half_normal", F(8, 32, rounding=1, seed=1)),
    ((128, 784), "half_normal", F(8, 24, rounding=1, seed=1)),   # generic path: b = 24
    ((5, 10), "normal", F(8, 24)),
    ((64, 300), "lognormal", F(8, 0)),                      # one exponent per row
    ((64, 300), "lognormal", F(12, 100, rounding=1, seed=2)),
    ((9, 1000), "grad", F(4, 16)),
    ((40, 512), "lognormal", F(8, 32, exp_mode=1)),
]


@pytest.mark.parametrize("shape,law,fd", ROW_CASES)
def test_row_blocks(hb, shape, law, fd):
    _check(hb, wl.draw(law, shape, seed=11), 1, fd)


# Row lengths that are not a multiple of 512 (the im2col widths 576 and 1152 among them) take the
# kernel that numbers 8-element groups through the whole matrix: warps straddle row ends, the packed
# rows carry padding up to the next multiple of 128, and the last CTA is ragged.
ROW_FLAT_CASES = [
    ((300, 576), "half_normal", F(8, 64)),
    ((257, 1152), "lognormal", F(12, 64, rounding=1, seed=5, sid=2)),
    ((64, 2176), "grad", F(8, 128, rounding=1, seed=6)),
    ((1000, 96), "outliers", F(8, 32)),
    ((3, 640), "normal", F(6, 128, exp_mode=1)),
    ((4099, 192), "lognormal", F(8, 64, rounding=1, seed=8)),
]


@pytest.mark.parametrize("shape,law,fd", ROW_FLAT_CASES)
def test_row_blocks_ragged_row_lengths(hb, shape, law, fd):
    _check(hb, wl.draw(law, shape, seed=16), 1, fd)


COL_CASES = [
    ((784, 128), "half_normal", F(8, 24, rounding=1, seed=1)),
    ((1000, 300), "lognormal", F(12, 64)),
    ((131, 77), "normal", F(8, 32, rounding=1, seed=9)),
    ((256, 256), "normal", F(8, 32)),
    ((512, 1024), "grad", F(8, 128, rounding=1, seed=3, sid=2)),
    ((200, 64), "lognormal", F(8, 0)),                      # generic: whole column
    ((600, 40), "outliers", F(12, 256, rounding=1, seed=4)),
    ((128, 10), "grad", F(8, 24, rounding=1, seed=1)),
]


@pytest.mark.parametrize("shape,law,fd", COL_CASES)
def test_column_blocks_transposed_output(hb, shape, law, fd):
    _check(hb, wl.draw(law, shape, seed=12), 0, fd)


# The streaming column kernel (128 x 64 tiles through a TMA pipeline) takes b in {32, 64, 128} with a
# 16-byte aligned pitch: several tiles per CTA, ragged last tiles in both directions, fewer rows than
# one tile, both plane counts, both rounding modes, every blocks-per-tile variant.
COL_STREAM_CASES = [
    ((4096, 2048), "lognormal", F(8, 128)),                                 # 1024 tiles: the persistent loop wraps
    ((3000, 1096), "grad", F(8, 64, rounding=1, seed=8, sid=1)),            # ragged K and N, N % 8 == 0
    ((1111, 520), "outliers", F(12, 32, rounding=1, seed=2)),               # two planes, stochastic
    ((90, 72), "normal", F(12, 128)),                                       # less than one tile
    ((640, 4), "half_normal", F(8, 64)),                                    # four output rows
    ((2048, 640), "lognormal", F(6, 32, rounding=1, seed=13, exp_mode=1)),
]


@pytest.mark.parametrize("shape,law,fd", COL_STREAM_CASES)
def test_column_blocks_streaming_kernel(hb, shape, law, fd):
    _check(hb, wl.draw(law, shape, seed=14), 0, fd)


# One exponent per column over the whole axis (block 0) with a column length that is a multiple of 128: column maxima
# in a first pass (scratch in the mantissa buffer), then the streaming kernel with the exponents given.
COL_WHOLE_AXIS_CASES = [
    ((1024, 200), "lognormal", F(8, 0, rounding=1, seed=6, sid=3)),         # ragged columns, stochastic
    ((2048, 1000), "outliers", F(8, 0, exp_mode=1)),                        # several bands of rows per column
    ((384, 72), "grad", F(12, 0, rounding=1, seed=2)),                      # two planes
    ((256, 8), "normal", F(4, 0)),                                          # eight output rows
]


@pytest.mark.parametrize("shape,law,fd", COL_WHOLE_AXIS_CASES)
def test_column_blocks_over_the_whole_axis(hb, shape, law, fd):
    _check(hb, wl.draw(law, shape, seed=16), 0, fd)


# The same for rows: one exponent per row over more than 256 columns (row maxima first, then the fast row kernel with
# the exponents given).
ROW_WHOLE_AXIS_CASES = [
    ((200, 1032), "lognormal", F(8, 0, rounding=1, seed=6, sid=3)),         # ragged last column tile, stochastic
    ((1000, 2048), "outliers", F(8, 0, exp_mode=1)),
    ((72, 384), "grad", F(12, 0, rounding=1, seed=2)),                      # two planes
    ((33, 264), "normal", F(4, 0)),                                         # ragged last row tile
    ((37, 4096), "lognormal", F(8, 0, rounding=1, seed=9, sid=1)),          # rows kept in registers: one pass
    ((5, 8192), "outliers", F(6, 0)),
    ((3, 16384), "lognormal", F(8, 0, rounding=1, seed=4)),
    ((64, 1536), "normal", F(8, 0)),                                        # not a multiple of 2048: two passes
]


@pytest.mark.parametrize("shape,law,fd", ROW_WHOLE_AXIS_CASES)
def test_row_blocks_over_the_whole_axis(hb, shape, law, fd):
    _check(hb, wl.draw(law, shape, seed=17), 1, fd)


def test_column_blocks_of_a_pitched_view(hb):
    # a 16-byte aligned column window of a wider matrix: the pitch differs from the logical width,
    # and the stochastic stream follows the logical index of the window
    base = wl.draw("lognormal", (700, 1024), seed=15)
    xd = to_dev(base)
    for sl in (np.s_[:, 256:896], np.s_[60:, 128:392]):
        ref = np.ascontiguousarray(base[sl])
        for fd in (F(8, 128, rounding=1, seed=3), F(12, 64)):
            q_ref, s_ref = oracle.quantize(ref, 0, ofmt(fd))
            p = hb.quantize(xd[sl], 0, gfmt(fd))
            q, s = hb.unpack(p)
            assert np.array_equal(q.cpu().numpy(), q_ref) and np.array_equal(s.cpu().numpy(), s_ref)
            qd, sd = decode_packed(p, hb.packed_layout(p.rows, p.k, p.fmt))
            assert np.array_equal(qd, q_ref) and np.array_equal(sd, s_ref)
    assert hb.device_status() == 0


def test_strided_and_unaligned_inputs(hb):
    import torch
    base = wl.draw("lognormal", (50, 203), seed=3)
    xd = to_dev(base)
    for sl in (np.s_[:, :200], np.s_[:, 1:201], np.s_[3:, 2:66]):
        view = xd[sl]
        ref = np.ascontiguousarray(base[sl])
        for axis, fd in ((1, F(8, 32, rounding=1, seed=6)), (0, F(8, 16)), (1, F(12, 64))):
            # the random stream follows the logical index inside the matrix as passed
            q_ref, s_ref = oracle.quantize(ref, axis, ofmt(fd))
            p = hb.quantize(view, axis, gfmt(fd))
            q, s = hb.unpack(p)
            assert np.array_equal(q.cpu().numpy(), q_ref) and np.array_equal(s.cpu().numpy(), s_ref)


def test_special_values(hb):
    x = np.zeros((8, 64), dtype=np.float32)
    x[1, :] = 2.0 ** -140                       # subnormal
    x[2, ::2] = 64.0                            # exact power of two as the maximum
    x[2, 1::2] = 63.5
    x[3, 0] = np.finfo(np.float32).max
    x[3, 1] = -1.0
    x[4, :] = np.ldexp(np.arange(64) - 32.0, -70)   # floored block
    x[5, :] = np.arange(64) + 0.5               # ties
    x[6, :] = -(np.arange(64) + 0.5)
    x[7, 5] = -3e-39
    for fd in (F(8, 32), F(8, 32, rounding=1, seed=1), F(12, 64), F(8, 32, exp_mode=1), F(8, 24), F(3, 32)):
        _check(hb, x, 1, fd)
        _check(hb, np.ascontiguousarray(x.T), 0, fd)


def test_empty_inputs(hb):
    import torch
    for shape in ((0, 64), (16, 0)):
        x = torch.empty(shape, dtype=torch.float32, device="cuda")
        for axis in (0, 1):
            p = hb.quantize(x, axis, hb.Format(8, 32))
            assert p.rows == shape[1 - axis] and p.k == shape[axis]


TILE_CASES = [
    ((100, 58), "normal", F(8, 24, 24, rounding=1, seed=1, sid=1)),
    ((784, 1024), "he_weight", F(8, 24, 24, rounding=1, seed=1, sid=1)),
    ((1024, 10), "he_weight", F(8, 24, 24, rounding=1, seed=1, sid=21)),
    ((1024, 256), "he_weight", F(12, 64, 64, rounding=1, seed=7, sid=1)),
    ((300, 200), "lognormal", F(8, 128, 128)),
]


@pytest.mark.parametrize("shape,law,fd", TILE_CASES)
def test_weight_tiles_share_mantissas_and_exponents(hb, shape, law, fd):
    kw = {"fan_in": shape[0]} if law == "he_weight" else {}
    w = wl.draw(law, shape, seed=13, **kw)
    c0, c1, grid = hb.quantize_tiles(to_dev(w), gfmt(fd))
    q0_ref, s0_ref = oracle.quantize(w, 0, ofmt(fd))
    q1_ref, s1_ref = oracle.quantize(w, 1, ofmt(fd))
    for p, q_ref, s_ref in ((c0, q0_ref, s0_ref), (c1, q1_ref, s1_ref)):
        qd, sd = decode_packed(p, hb.packed_layout(p.rows, p.k, p.fmt))
        assert np.array_equal(qd, q_ref) and np.array_equal(sd, s_ref)
    t = fd["tile"]
    assert np.array_equal(grid.cpu().numpy(), s1_ref[::t, :])
    # the single-view entry point gives the same bytes
    for axis, p_both in ((0, c0), (1, c1)):
        p = hb.quantize(to_dev(w), axis, gfmt(fd))
        lay = hb.packed_layout(p.rows, p.k, p.fmt)
        for pl in range(lay["planes"]):
            lo, hi = pl * lay["plane_stride"], pl * lay["plane_stride"] + p.rows * lay["kst"]
            assert np.array_equal(p.mant[lo:hi].cpu().numpy(), p_both.mant[lo:hi].cpu().numpy())
        qd, sd = decode_packed(p, lay)
        assert np.array_equal(sd, s0_ref if axis == 0 else s1_ref)


def test_large_tiles_take_the_generic_path(hb):
    w = wl.draw("lognormal", (300, 420), seed=14)
    fd = F(8, 200, 200, rounding=1, seed=3)
    for axis in (0, 1):
        _check(hb, w, axis, fd)


def test_dequantize_is_eq1(hb):
    x = wl.draw("lognormal", (40, 512), seed=15)
    fd = F(12, 64, rounding=1, seed=2)
    p = hb.quantize(to_dev(x), 1, gfmt(fd))
    q_ref, s_ref = oracle.quantize(x, 1, ofmt(fd))
    assert np.array_equal(hb.dequantize(p).cpu().numpy().astype(np.float64), oracle.dequantize(q_ref, s_ref, 64))


@pytest.mark.parametrize("m,b,rounding", [(8, 32, 0), (12, 128, 1)])
def test_full_size_one_gib_tensor(hb, m, b, rounding):
    """The standalone-quantiser workload (2^28 FP32 values as 16384 x 16384, log-normal
    magnitudes), compared in full against the oracle, slab by slab."""
    import torch
    n = 16384
    x = wl.draw("lognormal", (n, n), seed=3)
    fd = F(m, b, rounding=rounding, seed=3)
    p = hb.quantize(to_dev(x), 1, gfmt(fd))
    q, s = hb.unpack(p)
    q, s = q.cpu().numpy(), s.cpu().numpy()
    step = 2048
    for r0 in range(0, n, step):
        q_ref, s_ref = oracle.quantize(x[r0:r0 + step], 1, ofmt(fd, idx_row_off=r0, idx_cols=n))
        assert np.array_equal(s[r0:r0 + step], s_ref), r0
        assert np.array_equal(q[r0:r0 + step], q_ref), r0
    assert hb.device_status() == 0
