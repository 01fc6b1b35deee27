"""Pins of the oracle's BFP matrix product (Eq. 2, tiled accumulation in floating point)."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import Format

F32 = np.float32


def _rand(shape, seed, spread=1.0):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal(shape) * np.exp(rng.standard_normal(shape) * spread)).astype(F32)


def _quant_pair(M, N, K, fa, fb, seed=0):
    A, B = _rand((M, K), seed), _rand((K, N), seed + 1)
    qA, sA = oracle.quantize(A, 1, fa)
    qB, sB = oracle.quantize(B, 0, fb)
    return A, B, qA, sA, qB, sB


# -------------------------------------------------------------- Eq. 2 against a library matmul

@pytest.mark.parametrize("m,b,K", [(8, 32, 256), (8, 24, 100), (8, 128, 300), (8, 0, 77), (4, 16, 64)])
def test_eq2_equals_fp64_matmul_of_dequantised_operands_m8(m, b, K):
    # The paper's own simulation method (Sec. 5.1): quantise, de-quantise, multiply natively.
    fa, fb = Format(m, b), Format(m, b)
    _, _, qA, sA, qB, sB = _quant_pair(33, 29, K, fa, fb)
    out = oracle.gemm(qA, sA, qB, sB, b, want_partials=True)
    ref = oracle.dequantize(qA, sA, b) @ oracle.dequantize(qB, sB, b).T
    mag = np.abs(oracle.dequantize(qA, sA, b)) @ np.abs(oracle.dequantize(qB, sB, b)).T
    # binary32(P) is exact for these widths, so only float64 summation and the final
    # rounding to binary32 separate the two.
    assert (np.abs(out["P"]) < 2 ** 24).all()
    assert np.abs(out["c_ref"].astype(np.float64) - ref).max() <= 2.0 ** -24 * np.abs(ref).max() * 1.01 + 1e-13 * mag.max()
    assert (np.abs(out["c_ref"].astype(np.float64) - ref) <= 2.0 ** -24 * np.abs(ref) + 1e-13 * mag).all()
    assert (out["a_mag"] <= mag * (1 + 1e-12)).all() and (out["a_mag"] >= np.abs(ref) * (1 - 1e-12)).all()


def test_eq2_m12_one_rounding_of_p_per_block():
    b = 128
    fa, fb = Format(12, b), Format(12, b)
    _, _, qA, sA, qB, sB = _quant_pair(17, 19, 512, fa, fb, seed=3)
    qA[:, :] = np.sign(qA) * 2047 + (qA == 0) * 2047      # drive |P| well past 2^24
    qB[:, :] = 2047
    ref = oracle.dequantize(qA, sA, b) @ oracle.dequantize(qB, sB, b).T
    ex = oracle.gemm(qA, sA, qB, sB, b, exact_p=True, want_partials=True)
    assert np.abs(ex["P"]).max() > 2 ** 24
    assert (np.abs(ex["c_ref"].astype(np.float64) - ref) <= 2.0 ** -24 * np.abs(ref) + 1e-13 * ex["a_mag"]).all()
    rn = oracle.gemm(qA, sA, qB, sB, b)
    assert (np.abs(rn["c_ref"].astype(np.float64) - ref) <= 2.0 ** -24 * np.abs(ref) + 2.0 ** -24 * rn["a_mag"]).all()


# -------------------------------------------------------------- exact rationals on tiny shapes

@pytest.mark.parametrize("m,b", [(8, 4), (12, 8), (8, 0)])
def test_exact_rational_sum_on_tiny_shapes(m, b):
    M, N, K = 3, 4, 19
    _, _, qA, sA, qB, sB = _quant_pair(M, N, K, Format(m, b), Format(m, b), seed=5)
    out = oracle.gemm(qA, sA, qB, sB, b, want_partials=True)
    bb = b if b else K
    for i in range(M):
        for j in range(N):
            tot = Fraction(0)
            for kb in range(out["P"].shape[2]):
                p = sum(int(qA[i, k]) * int(qB[j, k]) for k in range(kb * bb, min(K, (kb + 1) * bb)))
                assert p == int(out["P"][i, j, kb])
                tot += p * Fraction(2) ** (int(sA[i, kb]) + int(sB[j, kb]))
            # |P| < 2^24 here, so c_ref is the correctly rounded exact sum up to float64 noise.
            assert abs(Fraction(float(out["c_ref"][i, j])) - tot) <= abs(tot) * Fraction(1, 2 ** 23)
            d = sum(Fraction(float(oracle.dequantize(qA, sA, b)[i, k])) *
                    Fraction(float(oracle.dequantize(qB, sB, b)[j, k])) for k in range(K))
            assert d == tot                                       # Eq. 2, exactly


# -------------------------------------------------------------- closed forms

def test_constant_operands_closed_form():
    K, b = 96, 32
    A = np.full((5, K), 2.0 ** 3, dtype=F32)
    B = np.full((K, 6), 2.0 ** -5, dtype=F32)
    out = oracle.hbfp_gemm(0, 0, A, B, Format(8, b), Format(8, b))
    assert np.array_equal(out["c_ref"], np.full((5, 6), K * 2.0 ** -2, dtype=F32))
    assert np.array_equal(out["c_seq"], out["c_ref"])
    assert np.array_equal(out["a_mag"], np.full((5, 6), K * 2.0 ** -2))


def test_block_partial_closed_form_and_extremes_fit_int32():
    b, nkb = 128, 3
    qA = np.full((2, b * nkb), 127, dtype=np.int16)
    qB = np.full((2, b * nkb), -127, dtype=np.int16)
    s0 = np.zeros((2, nkb), dtype=np.int8)
    out = oracle.gemm(qA, s0, qB, s0, b, want_partials=True)
    assert (out["P"] == -127 * 127 * b).all()
    q12 = np.full((1, 512), 2047, dtype=np.int16)
    out = oracle.gemm(q12, np.zeros((1, 1), np.int8), q12, np.zeros((1, 1), np.int8), 512, want_partials=True)
    assert int(out["P"][0, 0, 0]) == 2047 * 2047 * 512 < 2 ** 31
    with pytest.raises(ValueError):
        q = np.full((1, 1024), 2047, dtype=np.int16)
        oracle.gemm(q, np.zeros((1, 1), np.int8), q, np.zeros((1, 1), np.int8), 1024)


def test_one_hot_rows_select_dequantised_rows_of_b():
    K, N, b = 64, 10, 16
    B = _rand((K, N), 11)
    A = np.zeros((K, K), dtype=F32)
    A[np.arange(K), np.arange(K)] = 4.0
    fa = fb = Format(8, b)
    out = oracle.hbfp_gemm(0, 0, A, B, fa, fb)
    qB, sB = oracle.quantize(B, 0, fb)
    want = 4.0 * oracle.dequantize(qB, sB, b).T
    assert np.array_equal(out["c_ref"].astype(np.float64), want)
    assert np.array_equal(out["c_seq"], out["c_ref"])


def test_wide_mantissa_whole_row_block_reproduces_plain_product():
    # Small integers are representable with a 12-bit mantissa and one exponent per row/column
    # (Sec. 4: "one exponent per row of A, one per column of B"): the BFP product is then exact.
    rng = np.random.default_rng(2)
    A = rng.integers(-500, 500, size=(12, 40)).astype(F32)
    B = rng.integers(-500, 500, size=(40, 9)).astype(F32)
    A[:, 0] = 1024
    B[0, :] = 1024
    out = oracle.hbfp_gemm(0, 0, A, B, Format(12, 0), Format(12, 0))
    assert np.array_equal(out["c_ref"].astype(np.float64), A.astype(np.float64) @ B.astype(np.float64))


# -------------------------------------------------------------- order of accumulation

def test_c_seq_is_sequential_binary32_accumulation():
    b = 8
    _, _, qA, sA, qB, sB = _quant_pair(6, 7, 20 * b, Format(8, b), Format(8, b), seed=8)
    out = oracle.gemm(qA, sA, qB, sB, b, want_partials=True)
    T = out["P"].astype(np.float64) * np.ldexp(1.0, sA.astype(int)[:, None, :] + sB.astype(int)[None, :, :])
    assert np.array_equal(T.astype(F32).astype(np.float64), T)          # every term is a binary32
    acc = np.zeros((6, 7), dtype=F32)
    for kb in range(T.shape[2]):
        acc = (acc + T[:, :, kb].astype(F32)).astype(F32)                # numpy binary32 add
    assert np.array_equal(acc, out["c_seq"])
    assert np.array_equal(T.sum(axis=2).astype(F32), out["c_ref"]) or \
        np.abs(T.sum(axis=2) - out["c_ref"]).max() <= 2.0 ** -23 * np.abs(T).sum(axis=2).max()
    assert (np.abs(out["c_seq"].astype(np.float64) - out["c_ref"]) <= 1e-6 * out["a_mag"]).all()


# -------------------------------------------------------------- trans flags and shared tiles

def test_trans_flags_equal_explicit_transposes():
    M, N, K, b = 20, 24, 72, 24
    A, B = _rand((M, K), 20), _rand((K, N), 21)
    fa, fb = Format(8, b, rounding=1, seed=5, stream_id=0), Format(8, b, rounding=0)
    base = oracle.hbfp_gemm(0, 0, A, B, fa, fb)
    # B handed as its transpose with transB=1 (nearest rounding: no dependence on the source index)
    tb = oracle.hbfp_gemm(0, 1, A, np.ascontiguousarray(B.T), fa, fb)
    assert np.array_equal(base["c_seq"], tb["c_seq"])
    # A handed as its transpose with transA=1: stochastic draws follow the stored index, so
    # compare against quantising the stored array down its columns.
    At = np.ascontiguousarray(A.T)
    ta = oracle.hbfp_gemm(1, 0, At, B, fa, fb)
    qA, sA = oracle.quantize(At, 0, fa)
    qB, sB = oracle.quantize(B, 0, fb)
    assert np.array_equal(ta["c_seq"], oracle.gemm(qA, sA, qB, sB, b)["c_seq"])


def test_backward_data_reuses_forward_weight_mantissas():
    # Y = X W and dX = dY W^T with W in shared t x t tiles: the second product must see the
    # transposed quantised W, never a re-quantisation with other exponents.
    t, batch, fin, fout = 24, 16, 100, 58
    X, W, dY = _rand((batch, fin), 30), _rand((fin, fout), 31), _rand((batch, fout), 32)
    fw = Format(8, t, tile=t, rounding=1, seed=1, stream_id=1)
    fx = Format(8, t, rounding=1, seed=1, stream_id=0)
    fg = Format(8, t, rounding=1, seed=1, stream_id=2)
    q_fwd, s_fwd = oracle.quantize(W, 0, fw)          # [fout][fin]
    q_bwd, s_bwd = oracle.quantize(W, 1, fw)          # [fin][fout]
    assert np.array_equal(q_fwd, q_bwd.T)
    Wd = oracle.dequantize(q_bwd, s_bwd, t)           # de-quantised W, [fin][fout]
    assert np.array_equal(oracle.dequantize(q_fwd, s_fwd, t), Wd.T)
    dg = oracle.hbfp_gemm(0, 1, dY, W, fg, fw)
    qg, sg = oracle.quantize(dY, 1, fg)
    ref = oracle.dequantize(qg, sg, t) @ Wd.T
    assert (np.abs(dg["c_ref"].astype(np.float64) - ref) <= 2.0 ** -24 * np.abs(ref) + 1e-13 * dg["a_mag"]).all()
    fw_out = oracle.hbfp_gemm(0, 0, X, W, fx, fw)
    qx, sx = oracle.quantize(X, 1, fx)
    ref = oracle.dequantize(qx, sx, t) @ Wd
    assert (np.abs(fw_out["c_ref"].astype(np.float64) - ref) <= 2.0 ** -24 * np.abs(ref) + 1e-13 * fw_out["a_mag"]).all()


def test_quantisation_error_of_the_product_is_within_the_derived_bound():
    # |C_bfp - A B| <= sum_k |a| db + |b| da + da db with da, db the half-ULP bounds (sanity only).
    M, N, K, b = 16, 16, 128, 32
    A, B, qA, sA, qB, sB = _quant_pair(M, N, K, Format(8, b), Format(8, b), seed=40)
    out = oracle.gemm(qA, sA, qB, sB, b)
    da = np.repeat(np.ldexp(0.5, sA.astype(int)), b, axis=1)           # [M][K]
    db = np.repeat(np.ldexp(0.5, sB.astype(int)), b, axis=1)           # [N][K]
    Ad, Bd = np.abs(A.astype(np.float64)), np.abs(B.astype(np.float64)).T
    bound = Ad @ db.T + da @ Bd.T + da @ db.T
    exact = A.astype(np.float64) @ B.astype(np.float64)
    assert (np.abs(out["c_ref"] - exact) <= bound * 1.000001 + 1e-30).all()
