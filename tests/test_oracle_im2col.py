"""Pins of the oracle's convolution-as-matrix-product gather: against a direct evaluation of the
convolution sum, and the block structure the packed gather on the GPU relies on."""
import numpy as np
import pytest

import oracle
from oracle import Format
from tests.helpers import dgrad_filters_view


@pytest.mark.parametrize("n,h,w,c,kh,kw,pad,f", [(2, 5, 6, 3, 3, 3, 1, 4), (1, 4, 4, 2, 1, 1, 0, 3), (2, 6, 5, 4, 3, 3, 0, 2),
                                               (1, 5, 5, 2, 5, 3, 2, 3)])
def test_matrix_product_of_the_gather_is_the_convolution_sum(n, h, w, c, kh, kw, pad, f):
    rng = np.random.default_rng(n * 100 + h)
    x = rng.integers(-4, 5, size=(n, h, w, c)).astype(np.float64)
    wt = rng.integers(-3, 4, size=(kh, kw, c, f)).astype(np.float64)
    ho, wo = h + 2 * pad - kh + 1, w + 2 * pad - kw + 1
    direct = np.zeros((n, ho, wo, f))
    for b in range(n):
        for oy in range(ho):
            for ox in range(wo):
                for i in range(kh):
                    for j in range(kw):
                        iy, ix = oy + i - pad, ox + j - pad
                        if 0 <= iy < h and 0 <= ix < w:
                            direct[b, oy, ox] += x[b, iy, ix] @ wt[i, j]
    cols = oracle.im2col(x, kh, kw, pad)
    assert cols.shape == (n * ho * wo, kh * kw * c)
    assert np.array_equal((cols @ wt.reshape(kh * kw * c, f)).reshape(n, ho, wo, f), direct)


def test_blocks_of_the_gathered_matrix_are_blocks_of_the_pixels():
    # with a block of c along the columns, quantising the gathered matrix gives, block by block, the
    # quantised channel vector of the pixel the block was gathered from (and an all-zero block outside)
    rng = np.random.default_rng(3)
    n, h, w, c = 2, 6, 7, 16
    x = (rng.standard_normal((n, h, w, c)) * np.exp(rng.standard_normal((n, h, w, 1)) * 2)).astype(np.float32)
    f = Format(mant_bits=8, block=c)
    qp, sp = oracle.quantize(x.reshape(n * h * w, c), 1, f)
    cols = oracle.im2col(x, 3, 3, 1)
    qc, sc = oracle.quantize(cols, 1, f)
    qc = qc.reshape(n, h, w, 3, 3, c)
    sc = sc.reshape(n, h, w, 3, 3)
    qp = qp.reshape(n, h, w, c)
    sp = sp.reshape(n, h, w)
    for i in range(3):
        for j in range(3):
            for oy in range(h):
                for ox in range(w):
                    iy, ix = oy + i - 1, ox + j - 1
                    if 0 <= iy < h and 0 <= ix < w:
                        assert np.array_equal(qc[:, oy, ox, i, j], qp[:, iy, ix]) and np.array_equal(sc[:, oy, ox, i, j], sp[:, iy, ix])
                    else:
                        assert not qc[:, oy, ox, i, j].any() and (sc[:, oy, ox, i, j] == -63).all()


def test_indexed_quantiser_reduces_to_the_plain_one_and_draws_by_the_given_index():
    """oracle.quantize_indexed: with the identity index it is oracle.quantize; otherwise every element is
    rounded with the draw of the index it names (the scalar functions are pinned on their own)."""
    rng = np.random.default_rng(3)
    x = (rng.standard_normal((12, 20)) * np.exp(rng.standard_normal((12, 20)))).astype(np.float32)
    fmt = oracle.Format(mant_bits=8, block=4, rounding=1, seed=21, stream_id=5)
    ident = np.arange(x.size, dtype=np.int64).reshape(x.shape)
    for axis in (0, 1):
        q, s = oracle.quantize_indexed(x, axis, fmt, ident)
        q_ref, s_ref = oracle.quantize(x, axis, fmt)
        assert np.array_equal(q, q_ref) and np.array_equal(s, s_ref)
    perm = rng.permutation(x.size).astype(np.int64).reshape(x.shape)
    perm[0, 0] = -1
    x[0, 0] = 0.0                                         # a structural zero: no draw, stays zero
    q, s = oracle.quantize_indexed(x, 0, fmt, perm)       # q [20][12], blocks of 4 down the columns of x
    _, s_plain = oracle.quantize(x, 0, fmt)
    assert np.array_equal(s, s_plain)                     # exponents do not depend on the draws
    assert q[0, 0] == 0
    for (i, j) in ((3, 7), (11, 19), (5, 0)):
        r = oracle.sr_draw(21, 5, int(perm[i, j]))
        assert q[j, i] == oracle.round_sr(x[i, j], int(s[j, i // 4]), 8, r)


def test_im2col_index_names_the_activation_each_entry_copies():
    n, h, w, c = 2, 5, 4, 3
    x = np.random.default_rng(4).standard_normal((n, h, w, c)).astype(np.float32)
    cols = oracle.im2col(x, 3, 3, 1)
    idx = oracle.im2col_index(n, h, w, c, 3, 3, 1)
    assert idx.shape == cols.shape
    flat = x.reshape(-1)
    inside = idx >= 0
    assert np.array_equal(cols[inside], flat[idx[inside]])
    assert (cols[~inside] == 0).all() and (~inside).sum() > 0
    # every interior activation appears once per tap
    counts = np.bincount(idx[inside], minlength=flat.size).reshape(n, h, w, c)
    assert (counts[:, 1:-1, 1:-1, :] == 9).all()


@pytest.mark.parametrize("n,h,w,c,k,pad,f", [(2, 5, 6, 3, 3, 1, 4), (1, 6, 5, 2, 5, 2, 3), (2, 4, 4, 3, 1, 0, 2), (1, 7, 6, 2, 3, 0, 3),
                                             (1, 6, 6, 2, 3, 2, 2)])
def test_backward_data_is_the_gather_of_the_gradient_times_the_turned_filters(n, h, w, c, k, pad, f):
    """The index transform the backward-data convolution rests on: the gradient with respect to the input is the
    gather of the output gradient with padding k - 1 - pad times the filters with taps reversed and feature-map
    roles swapped. Checked against the library's own derivative of its convolution, in integers held in float64."""
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(17 * n + h)
    wt = rng.integers(-3, 4, size=(k * k * c, f)).astype(np.float64)
    ho, wo = h + 2 * pad - k + 1, w + 2 * pad - k + 1
    dy = rng.integers(-4, 5, size=(n, ho, wo, f)).astype(np.float64)
    x = torch.zeros(n, c, h, w, dtype=torch.float64, requires_grad=True)
    wt_t = torch.from_numpy(wt.reshape(k, k, c, f)).permute(3, 2, 0, 1).contiguous()      # [f][c][kh][kw]
    y = torch.nn.functional.conv2d(x, wt_t, padding=pad)
    y.backward(torch.from_numpy(dy).permute(0, 3, 1, 2).contiguous())
    want = x.grad.permute(0, 2, 3, 1).numpy()                                             # [n][h][w][c]
    turned, _ = dgrad_filters_view(wt, np.zeros((k * k * c, 1)), k * k, c)                # [c][taps * f]
    got = oracle.im2col(dy, k, k, k - 1 - pad) @ turned.T
    assert got.shape == (n * h * w, c)
    assert np.array_equal(got.reshape(n, h, w, c), want)
