"""Pins of the oracle's quantiser: exact-rational brute force, a float64 restatement,
and the invariants a block-floating-point encoder must have (Eq. 1, Sec. 4.1, Sec. 5.3)."""
from fractions import Fraction

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle
from oracle import Format

F32 = np.float32


# ------------------------------------------------------------------ exact-rational brute force

def brute_exponent(xs, m, exp_mode=0):
    amax = max(abs(Fraction(float(v))) for v in xs)
    if amax == 0:
        return -63
    e = -200
    while Fraction(2) ** e <= amax:        # smallest e with amax < 2^e  == floor(log2 amax)+1
        e += 1
    if exp_mode == 1 and Fraction(2) ** (e - 1) == amax:
        e -= 1                              # literal ceil(log2 amax)
    return max(e - (m - 1), -63)


def brute_nearest_even(x, s, m):
    """Nearest point of the grid {k 2^s, |k| <= 2^(m-1)-1}; ties to the even k."""
    qmax = 2 ** (m - 1) - 1
    xv = Fraction(float(x))
    step = Fraction(2) ** s
    best, bestd = None, None
    for k in range(-qmax, qmax + 1):
        d = abs(xv - k * step)
        if bestd is None or d < bestd or (d == bestd and k % 2 == 0 and best % 2 != 0):
            best, bestd = k, d
    return best


finite_f32 = st.floats(width=32, allow_nan=False, allow_infinity=False)
small_f32 = st.floats(min_value=-1e6, max_value=1e6, width=32)


@settings(max_examples=150, deadline=None)
@given(st.lists(finite_f32, min_size=1, max_size=8), st.sampled_from([3, 4, 8]), st.sampled_from([0, 1]))
def test_rne_matches_rational_brute_force_any_float(xs, m, exp_mode):
    x = np.array([xs], dtype=F32)
    q, s = oracle.quantize(x, 1, Format(mant_bits=m, block=0, exp_mode=exp_mode))
    s_ref = brute_exponent(xs, m, exp_mode)
    assert int(s[0, 0]) == s_ref
    for j, v in enumerate(xs):
        assert int(q[0, j]) == brute_nearest_even(v, s_ref, m)


@settings(max_examples=25, deadline=None)
@given(st.lists(small_f32, min_size=1, max_size=6))
def test_rne_matches_rational_brute_force_m12(xs):
    x = np.array([xs], dtype=F32)
    q, s = oracle.quantize(x, 1, Format(mant_bits=12, block=0))
    s_ref = brute_exponent(xs, 12)
    assert int(s[0, 0]) == s_ref
    for j, v in enumerate(xs):
        assert int(q[0, j]) == brute_nearest_even(v, s_ref, 12)


def test_hand_worked_block():
    # amax = 5 -> floor(log2 5)+1 = 3 -> s = 3 - 7 = -4 -> grid step 1/16.
    x = np.array([[5.0, -0.03125, 0.09375, 1.0, -4.96875, 0.15625, 0.0, 3.3]], dtype=F32)
    q, s = oracle.quantize(x, 1, Format(8, 8))
    assert int(s[0, 0]) == -4
    # 5*16=80; -0.5 -> tie -> 0 (even); 1.5 -> tie -> 2; 16; -79.5 -> tie -> -80; 2.5 -> 2; 0; 52.8 -> 53
    assert q[0].tolist() == [80, 0, 2, 16, -80, 2, 0, 53]


def test_powers_of_two_and_literal_ceil_mode():
    x = np.array([[64.0, 1.0, -63.5, 0.25]], dtype=F32)
    q0, s0 = oracle.quantize(x, 1, Format(8, 4, exp_mode=0))
    assert int(s0[0, 0]) == 0 and q0[0].tolist() == [64, 1, -64, 0]       # e = 7
    q1, s1 = oracle.quantize(x, 1, Format(8, 4, exp_mode=1))
    # literal ceil(log2 64) = 6 -> s = -1 -> 64 would need mantissa 128: saturates at 127.
    assert int(s1[0, 0]) == -1 and q1[0].tolist() == [127, 2, -127, 0]    # 0.5 ties to even 0


def test_zero_block_subnormals_and_floor():
    z = np.zeros((1, 8), dtype=F32)
    q, s = oracle.quantize(z, 1, Format(8, 8))
    assert int(s[0, 0]) == -63 and not q.any()
    tiny = np.array([[1e-45, -3e-39, 2.0 ** -70, 2.0 ** -64]], dtype=F32)
    q, s = oracle.quantize(tiny, 1, Format(8, 4))
    assert int(s[0, 0]) == -63
    assert q[0].tolist() == [0, 0, 0, 0]       # 2^-64 / 2^-63 = 0.5 ties to even 0
    big = np.array([[np.finfo(F32).max, -1.0]], dtype=F32)
    q, s = oracle.quantize(big, 1, Format(8, 2))
    assert int(s[0, 0]) == 128 - 7 and q[0].tolist() == [127, 0]   # top value saturates (< 1 ULP)


# ------------------------------------------------------------------ float64 restatement at scale

@pytest.mark.parametrize("m,b", [(8, 32), (12, 64), (8, 24), (4, 16)])
def test_rne_matches_float64_restatement(m, b):
    rng = np.random.default_rng(m * 100 + b)
    x = (rng.standard_normal((512, 40 * b)) * np.exp(rng.standard_normal((512, 40 * b)) * 3)).astype(F32)
    x[rng.random(x.shape) < 0.05] = 0
    q, s = oracle.quantize(x, 1, Format(m, b))
    xb = x.reshape(512, 40, b).astype(np.float64)
    amax = np.abs(xb).max(axis=2)
    _, ex = np.frexp(amax)                             # amax = f * 2^ex, f in [0.5,1)
    s_ref = np.where(amax > 0, np.maximum(ex - (m - 1), -63), -63)
    assert np.array_equal(s.astype(np.int64), s_ref)
    qmax = 2 ** (m - 1) - 1
    q_ref = np.clip(np.rint(xb / np.ldexp(1.0, s_ref)[:, :, None]), -qmax, qmax)
    assert np.array_equal(q.reshape(512, 40, b).astype(np.float64), q_ref)


# ------------------------------------------------------------------ invariants

def _rand(shape, seed, spread=3.0):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal(shape) * np.exp(rng.standard_normal(shape) * spread)).astype(F32)


@pytest.mark.parametrize("rounding", [0, 1])
@pytest.mark.parametrize("m,b", [(8, 32), (12, 64), (8, 24)])
def test_idempotence(m, b, rounding):
    x = _rand((64, 5 * b + 7), 1)
    x[3, :b] = 0
    x[5] *= 1e-30                                     # floored blocks
    f = Format(m, b, rounding=rounding, seed=9, stream_id=2)
    q, s = oracle.quantize(x, 1, f)
    d = oracle.dequantize(q, s, b).astype(F32)
    assert np.array_equal(d.astype(np.float64), oracle.dequantize(q, s, b))   # D(Q(x)) is binary32
    q2, s2 = oracle.quantize(d, 1, Format(m, b, rounding=rounding, seed=1234, stream_id=7))
    # The largest element keeps a mantissa of at least 2^(m-2), so the exponent is re-derived
    # unchanged and every mantissa is already on the grid: Q(D(Q(x))) == Q(x) exactly.
    assert np.array_equal(s2, s) and np.array_equal(q2, q)


@pytest.mark.parametrize("rounding", [0, 1])
@pytest.mark.parametrize("m", [8, 12])
def test_exact_pass_through_of_representable_values(m, rounding):
    rng = np.random.default_rng(5)
    qmax = 2 ** (m - 1) - 1
    k = rng.integers(-qmax, qmax + 1, size=(32, 96))
    k[:, ::32] = qmax * rng.choice([-1, 1], size=(32, 3))      # pins every block's exponent
    c = rng.integers(-40, 40, size=(32, 3))
    x = (k * np.repeat(np.ldexp(1.0, c), 32, axis=1)).astype(F32)
    q, s = oracle.quantize(x, 1, Format(m, 32, rounding=rounding, seed=3))
    assert np.array_equal(s, c.astype(np.int8))
    assert np.array_equal(q, k.astype(np.int16))
    assert np.array_equal(oracle.dequantize(q, s, 32), x.astype(np.float64))


@pytest.mark.parametrize("m,b", [(8, 32), (12, 16)])
def test_power_of_two_equivariance_and_sign_symmetry(m, b):
    x = _rand((16, 4 * b), 2, spread=1.0)
    q, s = oracle.quantize(x, 1, Format(m, b))
    for j in (-20, 7):
        qj, sj = oracle.quantize(np.ldexp(x, j).astype(F32), 1, Format(m, b))
        assert np.array_equal(qj, q) and np.array_equal(sj.astype(int), s.astype(int) + j)
    qn, sn = oracle.quantize(-x, 1, Format(m, b))
    assert np.array_equal(qn, -q) and np.array_equal(sn, s)


@pytest.mark.parametrize("m,b", [(8, 32), (12, 64), (8, 24), (4, 8)])
def test_error_bounds(m, b):
    x = _rand((128, 6 * b), 3)
    qmax = 2 ** (m - 1) - 1
    xs = x.astype(np.float64)
    # nearest: |x - D(Q(x))| <= 1/2 ULP, except where the value rounds past the top mantissa
    # and saturates (then < 1 ULP).
    q, s = oracle.quantize(x, 1, Format(m, b))
    ulp = np.repeat(np.ldexp(1.0, s.astype(np.int64)), b, axis=1)
    err = np.abs(xs - oracle.dequantize(q, s, b))
    sat = np.abs(xs) / ulp >= qmax + 0.5
    assert (err[~sat] <= 0.5 * ulp[~sat]).all()
    assert (err[sat] < ulp[sat]).all()
    # the exponent is tight: ULP <= amax * 2^(2-m) (the top mantissa bit is used)
    amax = np.abs(xs).reshape(128, 6, b).max(axis=2)
    assert (np.ldexp(1.0, s.astype(np.int64)) <= amax * 2.0 ** (2 - m)).all()
    # stochastic: strictly less than one ULP, and the result is one of the two neighbours.
    q, s = oracle.quantize(x, 1, Format(m, b, rounding=1, seed=11))
    y = xs / ulp
    assert ((q == np.clip(np.floor(y), -qmax, qmax)) | (q == np.clip(np.floor(y) + 1, -qmax, qmax))).all()
    assert (np.abs(xs - oracle.dequantize(q, s, b)) < ulp).all()


# ------------------------------------------------------------------ stochastic rounding

def test_sr_exhaustive_mean_is_exact():
    for x, s, m in [(0.3, -7, 8), (-0.3, -7, 8), (5.6789, -4, 8), (-100.001, 0, 12), (1e-3, -12, 8)]:
        y16 = Fraction(float(F32(x))) * Fraction(2) ** (16 - s)
        Y = y16.numerator // y16.denominator                      # floor
        qs = np.array([oracle.round_sr(x, s, m, r) for r in range(65536)], dtype=np.int64)
        lo = Y // 65536
        assert set(np.unique(qs)) <= {lo, lo + 1}
        assert Fraction(int(qs.sum()), 65536) == Fraction(Y, 65536)       # mean = Y / 2^16 exactly
        assert (np.diff(qs) >= 0).all()                                   # monotone in r


def test_sr_representable_never_moves():
    for k in (-127, -1, 0, 1, 77, 127):
        for s in (-10, 0, 5):
            for r in (0, 1, 32768, 65535):
                assert oracle.round_sr(k * 2.0 ** s, s, 8, r) == k


def test_sr_unbiased_over_seeds():
    x = _rand((4, 64), 8, spread=0.5)
    S = 1500
    acc = np.zeros(x.shape, dtype=np.float64)
    ulp = None
    for seed in range(S):
        q, s = oracle.quantize(x, 1, Format(8, 32, rounding=1, seed=seed))
        acc += oracle.dequantize(q, s, 32)
        ulp = np.repeat(np.ldexp(1.0, s.astype(np.int64)), 32, axis=1)
    mean = acc / S
    # sd of one draw <= ULP/2; 5 sd of the mean, plus the 2^-16 ULP floor bias.
    assert (np.abs(mean - x.astype(np.float64)) <= 5 * 0.5 * ulp / np.sqrt(S) + ulp / 65536).all()


def test_sr_uses_linear_index_of_source_not_layout():
    x = _rand((24, 40), 4, spread=0.3)
    f = Format(8, 8, rounding=1, seed=77, stream_id=4)
    q, s = oracle.quantize(x, 1, f)
    for i in (0, 7, 23):
        for j in (0, 13, 39):
            r = oracle.sr_draw(77, 4, i * 40 + j)
            assert int(q[i, j]) == oracle.round_sr(x[i, j], int(s[i, j // 8]), 8, r)
    # a row slab passed as a view with its offset reproduces the same mantissas
    fv = Format(8, 8, rounding=1, seed=77, stream_id=4, idx_row_off=5, idx_cols=40)
    qv, sv = oracle.quantize(x[5:9], 1, fv)
    assert np.array_equal(qv, q[5:9]) and np.array_equal(sv, s[5:9])
    # blocks down the columns: the draw still follows the source index
    qc, sc = oracle.quantize(x, 0, f)
    for i in (0, 23):
        for j in (0, 39):
            r = oracle.sr_draw(77, 4, i * 40 + j)
            assert int(qc[j, i]) == oracle.round_sr(x[i, j], int(sc[j, i // 8]), 8, r)


# ------------------------------------------------------------------ geometry

def test_column_blocks_equal_row_blocks_of_transpose():
    x = _rand((50, 37), 6)
    qa, sa = oracle.quantize(x, 0, Format(8, 16))
    qb, sb = oracle.quantize(np.ascontiguousarray(x.T), 1, Format(8, 16))
    assert np.array_equal(qa, qb) and np.array_equal(sa, sb)


def test_ragged_last_block_and_whole_axis_block():
    x = _rand((3, 70), 7)
    q, s = oracle.quantize(x, 1, Format(8, 32))
    assert s.shape == (3, 3)
    q2, s2 = oracle.quantize(x[:, 64:], 1, Format(8, 32))
    assert np.array_equal(q[:, 64:], q2) and np.array_equal(s[:, 2:], s2)
    qw, sw = oracle.quantize(x, 1, Format(8, 0))
    assert sw.shape == (3, 1)
    q70, s70 = oracle.quantize(x, 1, Format(8, 70))
    assert np.array_equal(qw, q70) and np.array_equal(sw, s70)


def test_tiles_share_exponents_between_w_and_its_transpose():
    t = 24
    w = _rand((100, 58), 9)
    f = Format(8, t, tile=t)
    q0, s0 = oracle.quantize(w, 0, f)        # contraction down the rows:  [58][100]
    q1, s1 = oracle.quantize(w, 1, f)        # contraction along the rows: [100][58]
    assert np.array_equal(q0, q1.T)          # the very same mantissas
    g0 = s0[::t, :]                          # [ceil(58/t)][ceil(100/t)]
    g1 = s1[::t, :]                          # [ceil(100/t)][ceil(58/t)]
    assert np.array_equal(g0, g1.T)
    # each tile's exponent is that of its own maximum
    for u in range(0, 100, t):
        for v in range(0, 58, t):
            amax = float(np.abs(w[u:u + t, v:v + t]).max())
            assert int(s1[u, v // t]) == oracle.block_exponent(amax, 8)
            assert (s1[u:u + t, v // t] == s1[u, v // t]).all()
    # and a tile holding a large value gives coarser mantissas to its small entries than a 1-D block would
    assert np.array_equal(oracle.quantize(w, 1, Format(8, 100, tile=100))[1][:, 0],
                          np.full(100, oracle.block_exponent(float(np.abs(w).max()), 8), dtype=np.int8))
