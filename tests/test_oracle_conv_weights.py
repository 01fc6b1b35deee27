"""Pins of the oracle's convolution-weight quantiser (Sec. 5.1: for convolutional layers the two outer,
feature-map dimensions of the weights are tiled): exact-rational brute force over whole tiles, the one-tap
case against the ordinary tile quantiser, and the structure of the exponent array."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import Format
from tests.test_oracle_quantize import brute_exponent, brute_nearest_even


def rand_w(taps, c_in, c_out, seed):
    rng = np.random.default_rng(seed)
    w = rng.standard_normal((taps * c_in, c_out)) * np.exp(2 * rng.standard_normal((taps * c_in, c_out)))
    return w.astype(np.float32)


@pytest.mark.parametrize("taps,c_in,c_out,t,m", [(9, 4, 5, 2, 8), (4, 6, 3, 3, 4), (1, 4, 4, 4, 12), (3, 2, 7, 2, 6)])
def test_tile_exponent_and_mantissas_match_rational_brute_force(taps, c_in, c_out, t, m):
    w = rand_w(taps, c_in, c_out, seed=5)
    w[0, 0] = 0.5          # an exact power of two in the first tile
    fmt = Format(mant_bits=m, block=t, tile=t)
    q0, s0 = oracle.quantize_conv_weights(w, taps, 0, fmt)
    q1, s1 = oracle.quantize_conv_weights(w, taps, 1, fmt)
    for u in range(c_in // t):
        for v in range(-(-c_out // t)):
            cols = range(v * t, min((v + 1) * t, c_out))
            group = [w[tap * c_in + ci, co] for tap in range(taps) for ci in range(u * t, (u + 1) * t) for co in cols]
            s_ref = brute_exponent(group, m)
            for tap in range(taps):
                for ci in range(u * t, (u + 1) * t):
                    i = tap * c_in + ci
                    for co in cols:
                        k = brute_nearest_even(w[i, co], s_ref, m)
                        assert q1[i, co] == k and q0[co, i] == k
                        assert s1[i, v] == s_ref and s0[co, i // t] == s_ref


def test_one_tap_is_the_ordinary_tile_quantiser():
    w = rand_w(1, 12, 10, seed=6)
    fmt = Format(mant_bits=8, block=4, tile=4)
    for axis in (0, 1):
        q, s = oracle.quantize_conv_weights(w, 1, axis, fmt)
        q_ref, s_ref = oracle.quantize(w, axis, fmt)
        assert np.array_equal(q, q_ref) and np.array_equal(s, s_ref)


def test_every_tap_of_a_tile_shares_the_exponent_of_the_largest_tap():
    taps, c_in, c_out, t = 9, 8, 8, 4
    w = rand_w(taps, c_in, c_out, seed=7)
    fmt = Format(mant_bits=8, block=t, tile=t)
    q, s = oracle.quantize_conv_weights(w, taps, 0, fmt)          # s [c_out][taps * c_in / t]
    s = s.reshape(c_out, taps, c_in // t)
    assert (s == s[:, :1, :]).all()
    # the shared exponent is the largest of the exponents the taps would take on their own
    per_tap = np.stack([oracle.quantize(w[tap * c_in:(tap + 1) * c_in], 0, fmt)[1] for tap in range(taps)], axis=1)
    assert np.array_equal(s[:, 0, :], per_tap.max(axis=1))
    # and no mantissa exceeds the symmetric range, while the largest weight of a tile uses the top bit
    assert np.abs(q).max() <= 127 and np.abs(q).max() >= 64


def test_stochastic_rounding_uses_the_index_in_the_weight_matrix():
    taps, c_in, c_out, t = 4, 4, 6, 2
    w = rand_w(taps, c_in, c_out, seed=8)
    fmt = Format(mant_bits=8, block=t, tile=t, rounding=1, seed=11, stream_id=3)
    q0, _ = oracle.quantize_conv_weights(w, taps, 0, fmt)
    q1, s1 = oracle.quantize_conv_weights(w, taps, 1, fmt)
    assert np.array_equal(q0, q1.T)                         # one draw per weight, whatever the view
    for i, j in ((0, 0), (5, 3), (15, 5)):
        r = oracle.sr_draw(11, 3, i * c_out + j)
        assert q1[i, j] == oracle.round_sr(w[i, j], int(s1[i, j // t]), 8, r)
