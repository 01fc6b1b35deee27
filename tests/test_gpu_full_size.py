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


def _gathered_rows(hw, ids_q, q_rows, s_rows, pix, c):
    """im2col rows (3 x 3, one pixel of padding) of the sampled pixels `pix` from the canonical rows of the pixels
    they touch: ids_q maps a pixel id to its line in q_rows / s_rows. Pure index movement."""
    qa = np.zeros((len(pix), 9 * c), dtype=np.int16)
    sa = np.zeros((len(pix), 9), dtype=np.int8)
    for r, p in enumerate(pix):
        img, rem = divmod(int(p), hw * hw)
        y, x = divmod(rem, hw)
        for tap in range(9):
            yy, xx = y + tap // 3 - 1, x + tap % 3 - 1
            if 0 <= yy < hw and 0 <= xx < hw:
                k = ids_q[img * hw * hw + yy * hw + xx]
                qa[r, tap * c:(tap + 1) * c] = q_rows[k]
                sa[r, tap] = s_rows[k, 0]
    return qa, sa


@pytest.mark.parametrize("hw,c", [(32, 64), (16, 128)])
def test_convolutions_full_batch_sampled(hb, hw, c):
    """The two 3 x 3 convolutions of the ResNet configuration at batch 128 through the implicit-GEMM kernel,
    forward and backward-data, on sampled pixels (image corners and edges among them): bit-equal to the
    oracle's sequential GEMM on the gathered rows of oracle-quantised pixels."""
    from tests.helpers import dgrad_filters_view
    n, f = 128, c
    rows = n * hw * hw
    rng = np.random.default_rng(hw)
    pix = np.unique(np.concatenate([[0, hw - 1, hw * hw - 1, rows - 1, rows - hw, 5 * hw * hw + 7 * hw],
                                    rng.choice(rows, size=40, replace=False)]))
    need = sorted({int(p) // (hw * hw) * hw * hw + yy * hw + xx
                   for p in pix for yy in range(int(p) % (hw * hw) // hw - 1, int(p) % (hw * hw) // hw + 2)
                   for xx in range(int(p) % hw - 1, int(p) % hw + 2) if 0 <= yy < hw and 0 <= xx < hw})
    ids_q = {p: k for k, p in enumerate(need)}
    wt = wl.draw("he_weight", (9 * c, f), seed=52, fan_in=9 * c)
    fw = dict(mant_bits=8, block=c, tile=c, stream_id=1)
    c0, c1, _ = hb.quantize_conv_weights(to_dev(wt), 9, gfmt(fw))
    # forward
    x = wl.draw("half_normal", (rows, c), seed=51)
    fx = dict(mant_bits=8, block=c)
    px = hb.quantize(to_dev(x), 1, gfmt(fx))
    Y = hb.conv_forward(px, c0, n, hw, hw, c, 3, 3, 1)
    assert hb.device_status() == 0 and hb.last_gemm_kernel() == "conv_fwd_kernel"
    q_rows, s_rows = _lines(x, True, need, fx)
    qa, sa = _gathered_rows(hw, ids_q, q_rows, s_rows, pix, c)
    qb, sb = oracle.quantize_conv_weights(wt, 9, 0, ofmt(fw))
    ref = oracle.gemm(qa, sa, qb, sb, c)
    assert np.array_equal(Y[torch_index(pix)].cpu().numpy(), ref["c_seq"])
    # backward-data: the packed output gradient (stochastic rounding, draws keyed by its own index) against the
    # regrouped forward weights
    dy = (wl.draw("normal", (rows, f), seed=53) * np.float32(0.03)).astype(np.float32)
    fg = dict(mant_bits=8, block=f, rounding=1, seed=13, stream_id=2)
    pg = hb.quantize(to_dev(dy), 1, gfmt(fg))
    dX = hb.conv_forward(pg, hb.conv_dgrad_filters(c1, 3, 3, c, f), n, hw, hw, f, 3, 3, 1)
    assert hb.device_status() == 0
    q_rows, s_rows = _lines(dy, True, need, fg)
    qa, sa = _gathered_rows(hw, ids_q, q_rows, s_rows, pix, f)
    q1, s1 = oracle.quantize_conv_weights(wt, 9, 1, ofmt(fw))
    qb, sb = dgrad_filters_view(q1, s1, 9, c)
    ref = oracle.gemm(qa, sa, qb, sb, f)
    assert np.array_equal(dX[torch_index(pix)].cpu().numpy(), ref["c_seq"])


def torch_index(ids):
    import torch
    return torch.as_tensor(np.asarray(ids, dtype=np.int64), device="cuda")
