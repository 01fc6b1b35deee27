"""Seeded random sweeps through the C ABI: shapes, pitches, block lengths, mantissa widths, rounding
modes and transposition flags drawn at random, every case compared with the oracle (quantiser:
mantissas and exponents bit-exact; GEMM: within 1e-6 of the accumulator magnitude, on both GPU paths)."""
import numpy as np
import pytest

import oracle
from tests.helpers import decode_packed

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hb():
    from paper_1804_01526_b200 import binding
    binding.lib()
    return binding


def lognormal(rng, shape, sigma):
    return (rng.standard_normal(shape) * np.exp(rng.standard_normal(shape) * sigma)).astype(np.float32)


@pytest.mark.parametrize("seed", [1, 2])
def test_random_quantiser_cases(hb, seed):
    import torch
    rng = np.random.default_rng(seed)
    done = 0
    for _ in range(70):
        d0, d1 = int(rng.integers(1, 700)), int(rng.integers(1, 700))
        if rng.random() < 0.3:
            d1 = int(rng.integers(1, 9)) * 64
        if rng.random() < 0.3:
            d0 = int(rng.integers(1, 9)) * 128
        b = int(rng.choice([0, 8, 16, 24, 32, 64, 128, 100, 256]))
        fd = dict(mant_bits=int(rng.choice([3, 4, 8, 8, 12])), block=b, tile=b if (rng.random() < 0.3 and 0 < b <= 128) else 0,
                  rounding=int(rng.integers(0, 2)), seed=int(rng.integers(0, 99)), stream_id=int(rng.integers(0, 5)))
        axis = int(rng.integers(0, 2))
        pitch = d1 + (int(rng.integers(0, 3)) * 4 if rng.random() < 0.4 else 0)
        buf = lognormal(rng, (d0, pitch), 3)
        if rng.random() < 0.2:
            buf[rng.random(buf.shape) < 0.6] = 0
        try:
            q_ref, s_ref = oracle.quantize(np.ascontiguousarray(buf[:, :d1]), axis, oracle.Format(**fd))
        except ValueError:
            continue                                   # a format whose block sums could overflow 32 bits
        try:
            p = hb.quantize(torch.from_numpy(buf).cuda()[:, :d1], axis, hb.Format(**fd))
        except hb.HbfpError as e:
            assert e.code == hb.ERR_UNSUPPORTED, (d0, d1, fd)
            continue
        q, s = decode_packed(p, hb.packed_layout(p.rows, p.k, p.fmt))
        assert np.array_equal(q, q_ref) and np.array_equal(s, s_ref), (d0, d1, pitch, axis, fd)
        done += 1
    assert hb.device_status() == 0 and done > 50


@pytest.mark.parametrize("seed", [1, 2])
def test_random_gemm_cases(hb, seed):
    import torch
    rng = np.random.default_rng(100 + seed)
    done = 0
    ran = {}
    for _ in range(45):
        M, N, K = (int(rng.integers(1, 600)) for _ in range(3))
        if rng.random() < 0.3:
            N = int(rng.integers(1, 40))
        if rng.random() < 0.2:
            K = int(rng.integers(600, 3000))
        m = int(rng.choice([3, 4, 6, 8, 8, 8, 10, 12, 12]))
        b = int(rng.choice([0, 8, 16, 24, 32, 48, 64, 64, 100, 128, 128, 200, 256]))
        if (2 ** (m - 1) - 1) ** 2 * (b if b > 0 else K) > 2 ** 31 - 1:
            continue
        tA, tB = int(rng.integers(0, 2)), int(rng.integers(0, 2))
        A = lognormal(rng, (K, M) if tA else (M, K), 2)
        B = lognormal(rng, (N, K) if tB else (K, N), 2)
        fa = dict(mant_bits=m, block=b, rounding=int(rng.integers(0, 2)), seed=int(rng.integers(0, 1000)), stream_id=0)
        fb = dict(fa, stream_id=1)
        ref = oracle.hbfp_gemm(tA, tB, A, B, oracle.Format(**fa), oracle.Format(**fb))
        for flags in (hb.GEMM_AUTO, hb.GEMM_FORCE_SIMT, hb.GEMM_FORCE_TENSOR, hb.GEMM_FORCE_SMALL):
            try:
                C = hb.gemm(tA, tB, torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), hb.Format(**fa), hb.Format(**fb),
                            flags=flags).cpu().numpy()
            except hb.HbfpError as e:
                # a forced kernel may not cover the format (two-plane operands on the small-problem kernel, ...)
                assert e.code == hb.ERR_UNSUPPORTED and flags in (hb.GEMM_FORCE_TENSOR, hb.GEMM_FORCE_SMALL), (M, N, K, m, b, flags)
                continue
            err = np.abs(C.astype(np.float64) - ref["c_ref"].astype(np.float64))
            assert (err <= 1e-6 * ref["a_mag"] + 1e-300).all(), (M, N, K, m, b, tA, tB, flags)
            if flags in (hb.GEMM_FORCE_SIMT, hb.GEMM_FORCE_SMALL):       # neither splits K: the sequential order
                assert np.array_equal(C, ref["c_seq"]), (M, N, K, m, b, tA, tB, flags)
            ran[flags] = ran.get(flags, 0) + 1
        done += 1
    assert hb.device_status() == 0 and done > 30
    assert ran.get(hb.GEMM_FORCE_TENSOR, 0) > 20 and ran.get(hb.GEMM_FORCE_SMALL, 0) > 15, ran
