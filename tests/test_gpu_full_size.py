"""Parity at the full benchmark sizes, in the launch configuration bench.py times, on sampled
outputs the oracle can compute one by one: pick rows of op(A) and columns of op(B), quantise just
those lines with the oracle (full contraction length, same random-stream positions), evaluate the
sampled entries of C, and compare with the GPU result of the whole GEMM."""
import numpy as np
import pytest

import oracle
from paper_1804_01526_b200 import workloads as wl
from tests.helpers import gfmt, ofmt, to_dev

pytestmark = pytest.mark.gpu
TOL = 1e-6


@pytest.fixture(scope="module")
def hb():
    from paper_1804_01526_b200 import binding
    binding.lib()
    return binding


def _lines(X, trans_is_lines_rows, idx, fd, block_cols=None):
    """Oracle-quantise selected lines (full contraction) of a stored matrix.

    trans_is_lines_rows: True if the lines are rows of X (contraction along axis 1), False if they
    are columns (contraction down axis 0). Returns canonical q [len(idx)][k], s [len(idx)][nkb]."""
    qs, ss = [], []
    for i in idx:
        if trans_is_lines_rows:
            view = X[i:i + 1, :]
            f = ofmt(fd, idx_row_off=int(i), idx_col_off=0, idx_cols=X.shape[1])
            q, s = oracle.quantize(np.ascontiguousarray(view), 1, f)
        else:
            view = X[:, i:i + 1]
            f = ofmt(fd, idx_row_off=0, idx_col_off=int(i), idx_cols=X.shape[1])
            q, s = oracle.quantize(np.ascontiguousarray(view), 0, f)
        qs.append(q[0]); ss.append(s[0])
    return np.stack(qs), np.stack(ss)


def _check_sampled(hb, sp, A, B, n_rows=24, n_cols=24, seed=0):
    rng = np.random.default_rng(seed)
    ri = np.sort(rng.choice(sp.M, size=min(n_rows, sp.M), replace=False))
    ci = np.sort(rng.choice(sp.N, size=min(n_cols, sp.N), replace=False))
    # include the corners and a tile boundary
    ri[0], ri[-1] = 0, sp.M - 1
    ci[0], ci[-1] = 0, sp.N - 1
    C = hb.gemm(sp.transA, sp.transB, to_dev(A), to_dev(B), gfmt(sp.fmt_a), gfmt(sp.fmt_b))
    assert hb.device_status() == 0
    Cs = C[ri][:, ci].cpu().numpy()
    # op(A) rows: rows of A if not transA, else columns of A. op(B) columns: columns of B if not transB, else rows of B.
    qA, sA = _lines(A, not sp.transA, ri, sp.fmt_a)
    qB, sB = _lines(B, bool(sp.transB), ci, sp.fmt_b)
    ref = oracle.gemm(qA, sA, qB, sB, sp.fmt_a["block"])
    err = np.abs(Cs.astype(np.float64) - ref["c_ref"].astype(np.float64))
    assert (err <= TOL * ref["a_mag"]).all(), float((err / np.maximum(ref["a_mag"], 1e-300)).max())
    return Cs, ref


def test_headline_sweep_gemm_16384_sampled(hb):
    """The configuration bench.py times: n = 16384, m = 8, b = 128, nearest-even, log-normal inputs."""
    n = 16384
    sp = wl.config_sweep(n, 8, 128, 0)[0]
    A = wl.draw("lognormal", (n, n), seed=3, salt=0)
    B = wl.draw("lognormal", (n, n), seed=3, salt=1)
    Cs, ref = _check_sampled(hb, sp, A, B)
    assert np.array_equal(Cs, ref["c_seq"])          # no split-K here: ascending-order accumulation, bit for bit


@pytest.mark.parametrize("m,b,rounding", [(8, 32, 1), (12, 64, 1)])
def test_sweep_gemm_4096_other_formats_sampled(hb, m, b, rounding):
    n = 4096
    sp = wl.config_sweep(n, m, b, rounding)[0]
    A = wl.draw("lognormal", (n, n), seed=5, salt=0)
    B = wl.draw("lognormal", (n, n), seed=5, salt=1)
    Cs, ref = _check_sampled(hb, sp, A, B, seed=1)
    assert np.array_equal(Cs, ref["c_seq"])


def test_resnet_im2col_full_batch_sampled(hb):
    """batch 128: M = 131072 / 32768 rows, skinny N, and the 131072-long backward-weight contraction (split-K)."""
    specs = wl.config_resnet_im2col(batch=128)
    t = wl.materialize(specs, seed=2)
    for sp in specs:
        _check_sampled(hb, sp, t[sp.a_key], t[sp.b_key], n_rows=12, n_cols=12, seed=2)


def test_transformer_full_size_tiled_weights_sampled(hb):
    """tokens 4096, hidden 1024: 12-bit planes, stochastic rounding; the tiled weight operand is sampled
    in whole 64-wide tile columns/rows so that the oracle sees complete tiles."""
    specs = wl.config_transformer()
    t = wl.materialize(specs, seed=7)
    for sp in specs:
        A, B = t[sp.a_key], t[sp.b_key]
        C = hb.gemm(sp.transA, sp.transB, to_dev(A), to_dev(B), gfmt(sp.fmt_a), gfmt(sp.fmt_b))
        assert hb.device_status() == 0
        rng = np.random.default_rng(11)
        ri = np.sort(rng.choice(sp.M, size=16, replace=False))
        qA, sA = _lines(A, not sp.transA, ri, sp.fmt_a)
        if sp.fmt_b["tile"] > 0:
            # a 64-line slab of the weight's non-contraction axis: complete tiles
            tile = sp.fmt_b["tile"]
            j0 = int(rng.integers(0, sp.N // tile)) * tile
            ci = np.arange(j0, j0 + tile)
            if sp.transB:      # stored [N][K]: lines are rows
                f = ofmt(sp.fmt_b, idx_row_off=j0, idx_col_off=0, idx_cols=B.shape[1])
                qB, sB = oracle.quantize(np.ascontiguousarray(B[j0:j0 + tile, :]), 1, f)
            else:              # stored [K][N]: lines are columns
                f = ofmt(sp.fmt_b, idx_row_off=0, idx_col_off=j0, idx_cols=B.shape[1])
                qB, sB = oracle.quantize(np.ascontiguousarray(B[:, j0:j0 + tile]), 0, f)
        else:
            ci = np.sort(rng.choice(sp.N, size=16, replace=False))
            qB, sB = _lines(B, bool(sp.transB), ci, sp.fmt_b)
        ref = oracle.gemm(qA, sA, qB, sB, sp.fmt_a["block"])
        Cs = C[ri][:, ci].cpu().numpy()
        err = np.abs(Cs.astype(np.float64) - ref["c_ref"].astype(np.float64))
        assert (err <= TOL * ref["a_mag"]).all(), sp.name
