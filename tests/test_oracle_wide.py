"""Pins of the oracle's wide weight storage (Sec. 4.2): 16-bit quantisation against exact rational
rounding, the narrow copy as the top bits after half a narrow unit was added (nearest narrow value, ties
upward, checked in exact rationals), and the weight
update against a binary32 numpy restatement, its fixed point and exact integer steps."""
from fractions import Fraction
import math

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle
from oracle import Format

F32 = np.float32


def rational_exponent(values, m):
    amax = max(abs(Fraction(float(v))) for v in values)
    if amax == 0:
        return -63
    e = -200
    while Fraction(2) ** e <= amax:
        e += 1
    return max(e - (m - 1), -63)


def rational_nearest_even(v, s, m):
    qmax = 2 ** (m - 1) - 1
    k = round(Fraction(float(v)) / Fraction(2) ** s)      # Fraction rounds half to even, exactly
    return max(-qmax, min(qmax, k))


small_f32 = st.floats(min_value=-1e6, max_value=1e6, width=32)
finite_f32 = st.floats(width=32, allow_nan=False, allow_infinity=False)


@settings(max_examples=120, deadline=None)
@given(st.lists(st.one_of(small_f32, finite_f32), min_size=1, max_size=9))
def test_sixteen_bit_quantisation_matches_exact_rational_rounding(xs):
    x = np.array([xs], dtype=F32)
    q, s = oracle.wide_quantize(x, Format(block=16, tile=16))        # one tile holds the whole row
    s_ref = rational_exponent(xs, 16)
    assert int(s[0, 0]) == s_ref
    assert q[0].tolist() == [rational_nearest_even(v, s_ref, 16) for v in xs]


def test_one_exponent_per_tile_of_the_stored_matrix():
    rng = np.random.default_rng(5)
    d0, d1, t = 61, 100, 24
    w = (rng.standard_normal((d0, d1)) * np.exp(rng.standard_normal((d0, d1)) * 3)).astype(F32)
    w[30:48, 48:72] = 0                                              # an all-zero tile region (rows 30..47 only)
    q, s = oracle.wide_quantize(w, Format(block=t, tile=t))
    assert q.shape == (d0, d1) and s.shape == (d0, math.ceil(d1 / t))
    for u in range(math.ceil(d0 / t)):
        for v in range(math.ceil(d1 / t)):
            tile = w[u * t:(u + 1) * t, v * t:(v + 1) * t].astype(np.float64)
            amax = np.abs(tile).max()
            _, ex = np.frexp(amax)
            s_ref = max(int(ex) - 15, -63) if amax > 0 else -63
            assert (s[u * t:(u + 1) * t, v] == s_ref).all()
            ref = np.clip(np.rint(tile * 2.0 ** -s_ref), -32767, 32767)    # float64: exact scaling, ties to even
            assert np.array_equal(q[u * t:(u + 1) * t, v * t:(v + 1) * t], ref.astype(np.int16))


@pytest.mark.parametrize("m", [4, 8, 12, 16])
def test_narrow_copy_is_the_wide_value_rounded_to_the_narrow_grid(m):
    rng = np.random.default_rng(m)
    q16 = rng.integers(-32767, 32768, size=(40, 50)).astype(np.int16)
    half = (1 << (16 - m)) >> 1
    q16[0, :8] = [-1, 0, 1, -32767, 32767, -(1 << (16 - m)), half, -half]
    s16 = rng.integers(-63, 100, size=(40, 3)).astype(np.int8)
    qm, sm = oracle.wide_narrow(q16, s16, m)
    assert np.array_equal(sm.astype(int), s16.astype(int) + (16 - m))
    qmax = (1 << (m - 1)) - 1
    for i in range(0, 40, 7):
        for j in range(50):
            wide = Fraction(int(q16[i, j])) * Fraction(2) ** int(s16[i, 0])
            step = Fraction(2) ** int(sm[i, 0])
            narrow = Fraction(int(qm[i, j])) * step
            if abs(int(qm[i, j])) < qmax:
                assert -step / 2 <= wide - narrow < step / 2         # nearest point of the grid, ties upward
            else:
                assert abs(wide - narrow) < step                     # saturated at the top of the range
    if m < 15:
        assert int(qm[0, 0]) == 0 and int(qm[0, 2]) == 0             # +-1 of the wide grid round to 0 ...
    if m < 16:
        assert int(qm[0, 6]) == 1 and int(qm[0, 7]) == 0             # ... and exact halves go upward
    else:
        assert np.array_equal(qm, q16)                               # sixteen bits: the copy is the mantissa itself
    assert -qmax <= int(qm.min()) and int(qm.max()) <= qmax          # the symmetric range of every mantissa


@pytest.mark.parametrize("m", [8, 12])
def test_narrow_copy_has_no_systematic_offset(m):
    # truncating the mantissa would leave every weight half a narrow ULP low; rounded, the mean error over
    # many weights is a small fraction of an ULP
    rng = np.random.default_rng(20 + m)
    q16 = rng.integers(-30000, 30001, size=(200, 500)).astype(np.int16)
    s16 = np.zeros((200, 1), dtype=np.int8)
    qm, _ = oracle.wide_narrow(q16, s16, m)
    ulp = 1 << (16 - m)
    err = qm.astype(np.float64) * ulp - q16
    assert abs(err.mean()) < 0.04 * ulp and np.abs(err).max() <= ulp / 2      # (ties upward: +1/2 of a wide unit)


@pytest.mark.parametrize("m", [8, 12])
def test_weights_on_the_narrow_grid_survive_wide_storage_exactly(m):
    # every weight is k * 2^e with |k| < 2^(m-1) and the tile maximum pins the exponent: the wide
    # mantissa is k * 2^(16-m), its top bits are k again, and a direct m-bit quantisation agrees
    rng = np.random.default_rng(17 + m)
    t = 24
    k = rng.integers(-(2 ** (m - 1)) + 1, 2 ** (m - 1), size=(48, 72))
    k[::t, ::t] = 2 ** (m - 1) - 1                                    # the maximum of every tile
    e = rng.integers(-20, 20, size=(2, 3))
    w = (k * np.exp2(np.kron(e, np.ones((t, t))))).astype(F32)
    f = Format(mant_bits=m, block=t, tile=t)
    q16, s16 = oracle.wide_quantize(w, f)
    qm, sm = oracle.wide_narrow(q16, s16, m)
    assert np.array_equal(qm, k)
    assert np.array_equal(oracle.dequantize(qm, sm, t), w.astype(np.float64))
    qd, sd = oracle.quantize(w, 1, f)
    assert np.array_equal(qd, qm) and np.array_equal(sd, sm)


@pytest.mark.parametrize("rounding", [0, 1])
def test_zero_update_is_a_fixed_point(rounding):
    rng = np.random.default_rng(3)
    w = rng.standard_normal((50, 70)).astype(F32)
    f = Format(block=24, tile=24, rounding=rounding, seed=11, stream_id=2)
    q, s = oracle.wide_quantize(w, f)
    q2, s2 = oracle.wide_update(q, s, np.zeros_like(w), Format(block=24, tile=24, rounding=rounding, seed=99))
    assert np.array_equal(q2, q) and np.array_equal(s2, s)          # representable values never move


@pytest.mark.parametrize("rounding", [0, 1])
def test_update_matches_binary32_restatement(rounding):
    rng = np.random.default_rng(8)
    d0, d1, t = 70, 90, 24
    w = (rng.standard_normal((d0, d1)) * 0.05).astype(F32)
    f = Format(block=t, tile=t, rounding=rounding, seed=4, stream_id=1)
    q, s = oracle.wide_quantize(w, f)
    delta = (rng.standard_normal((d0, d1)) * 1e-3).astype(F32)
    delta[:, 5] = 0.5                                                # moves the maximum of a tile column
    q2, s2 = oracle.wide_update(q, s, delta, f)
    scale = np.exp2(np.repeat(s.astype(np.int32), t, axis=1)[:, :d1]).astype(F32)
    w32 = q.astype(F32) * scale                                      # exact: 15 bits times a power of two
    w32 = (w32 + delta).astype(F32)                                  # one binary32 rounding
    qr, sr = oracle.wide_quantize(w32, f)
    assert np.array_equal(q2, qr) and np.array_equal(s2, sr)
    assert not np.array_equal(s2, s)


def test_update_by_whole_units_of_the_last_place_is_exact():
    rng = np.random.default_rng(9)
    t = 16
    q = rng.integers(-20000, 20001, size=(32, 32)).astype(np.int16)
    q[::t, ::t] = 32767                                              # the maximum of every tile, left untouched
    s = np.array([[-10, -3]] * 16 + [[4, -20]] * 16, dtype=np.int8)
    k = rng.integers(-5000, 5001, size=(32, 32))
    k[::t, ::t] = 0
    delta = (k * np.exp2(np.repeat(s.astype(np.int32), t, axis=1))).astype(F32)
    q2, s2 = oracle.wide_update(q, s, delta, Format(block=t, tile=t))
    assert np.array_equal(s2, s) and np.array_equal(q2, q + k)


def test_stochastic_rounding_of_sixteen_bit_mantissas_near_the_top_of_the_range():
    # y = x * 2^(16-s) reaches 2^31 here: the floor form must be evaluated without 32-bit overflow
    s = -3
    for x, r in [(32767.25 * 2.0 ** s, 0), (32767.25 * 2.0 ** s, 65535), (-32767.75 * 2.0 ** s, 1),
                 (-32767.75 * 2.0 ** s, 65535), (12345.5 * 2.0 ** s, 32767), (12345.5 * 2.0 ** s, 32768)]:
        y = Fraction(float(F32(x))) * Fraction(2) ** (16 - s)
        want = math.floor((math.floor(y) + r) / Fraction(65536))
        want = max(-32767, min(32767, want))
        assert oracle.round_sr(float(F32(x)), s, 16, r) == want
