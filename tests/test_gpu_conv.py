"""GPU parity of the packed im2col gather through the C ABI: the convolution operand built from
activations that were converted once per pixel is bit-identical to converting the FP32 im2col matrix,
and the convolution GEMM on it equals the GEMM on the FP32 im2col matrix."""
import numpy as np
import pytest

import oracle
from paper_1804_01526_b200 import workloads as wl
from tests.helpers import decode_packed, dgrad_filters_view, gfmt, ofmt, to_dev

pytestmark = pytest.mark.gpu

TOL = 1e-6


@pytest.fixture(scope="module")
def hb():
    from paper_1804_01526_b200 import binding
    binding.lib()
    return binding


CASES = [
    # n, h, w, c, kh, kw, pad, mantissa bits
    (2, 32, 32, 64, 3, 3, 1, 8),       # the 64-channel 3x3 convolution of the ResNet configuration, two images
    (1, 16, 16, 128, 3, 3, 1, 8),
    (3, 9, 7, 24, 3, 3, 1, 8),         # channel count below the padded block width
    (2, 8, 8, 64, 3, 3, 1, 12),        # two mantissa planes
    (2, 10, 11, 32, 5, 3, 0, 8),       # no padding, rectangular filter: the output is smaller than the input
    (1, 6, 6, 16, 1, 1, 0, 6),
]


@pytest.mark.parametrize("n,h,w,c,kh,kw,pad,m", CASES)
def test_gathered_operand_equals_quantised_im2col_matrix(hb, n, h, w, c, kh, kw, pad, m):
    x = wl.draw("half_normal", (n * h * w, c), seed=71).reshape(n, h, w, c)
    x *= np.exp(wl.draw("normal", (n * h * w, 1), seed=72)).reshape(n, h, w, 1).astype(np.float32)
    fd = dict(mant_bits=m, block=c, rounding=0, seed=0)
    px = hb.quantize(to_dev(x.reshape(n * h * w, c)), 1, gfmt(fd))
    pa = hb.im2col_packed(px, n, h, w, c, kh, kw, pad)
    assert hb.device_status() == 0
    cols = oracle.im2col(x, kh, kw, pad)
    q_ref, s_ref = oracle.quantize(cols, 1, ofmt(fd))
    q, s = decode_packed(pa, hb.packed_layout(pa.rows, pa.k, pa.fmt))
    assert np.array_equal(q, q_ref) and np.array_equal(s, s_ref)
    # byte for byte what converting the FP32 im2col matrix gives
    pb = hb.quantize(to_dev(cols), 1, gfmt(fd))
    lay = hb.packed_layout(pa.rows, pa.k, pa.fmt)
    for pl in range(lay["planes"]):
        lo, hi = pl * lay["plane_stride"], pl * lay["plane_stride"] + pa.rows * lay["kst"]
        assert np.array_equal(pa.mant[lo:hi].cpu().numpy(), pb.mant[lo:hi].cpu().numpy())
    ne = lay["nkb"] * lay["rs"]
    assert np.array_equal(pa.exps[:ne].cpu().numpy(), pb.exps[:ne].cpu().numpy())


def test_convolution_forward_gemm_on_the_gathered_operand(hb):
    n, h, w, c, f = 4, 32, 32, 64, 64
    x = wl.draw("half_normal", (n * h * w, c), seed=73).reshape(n, h, w, c)
    wt = wl.draw("he_weight", (9 * c, f), seed=74, fan_in=9 * c)
    fd = dict(mant_bits=8, block=c, rounding=0, seed=0)
    px = hb.quantize(to_dev(x.reshape(n * h * w, c)), 1, gfmt(fd))
    pa = hb.im2col_packed(px, n, h, w, c, 3, 3, 1)
    Y = hb.gemm_q(n * h * w, f, 9 * c, pa, to_dev(wt), fmtB=gfmt(fd)).cpu().numpy()
    assert hb.device_status() == 0
    cols = oracle.im2col(x, 3, 3, 1)
    ref = oracle.hbfp_gemm(0, 0, cols, wt, ofmt(fd), ofmt(fd))
    err = np.abs(Y.astype(np.float64) - ref["c_ref"].astype(np.float64))
    assert (err <= TOL * ref["a_mag"]).all()
    Y2 = hb.gemm(0, 0, to_dev(cols), to_dev(wt), gfmt(fd), gfmt(fd)).cpu().numpy()
    assert np.array_equal(Y, Y2)


def test_gather_argument_errors(hb):
    x = to_dev(wl.draw("normal", (64, 32), seed=1))
    px = hb.quantize(x, 1, hb.Format(mant_bits=8, block=16))
    with pytest.raises(hb.HbfpError) as e:               # the block must be the channel count
        hb.im2col_packed(px, 1, 8, 8, 32, 3, 3, 1)
    assert e.value.code == hb.ERR_INVALID_ARG


def test_gather_of_an_empty_batch_and_of_a_single_pixel(hb):
    import torch
    f = hb.Format(mant_bits=8, block=16)
    px = hb.quantize(torch.empty((0, 16), device="cuda"), 1, f)
    pa = hb.im2col_packed(px, 0, 4, 4, 16, 3, 3, 1)
    assert pa.rows == 0 and hb.device_status() == 0
    x = wl.draw("normal", (1, 16), seed=3)                      # a 1 x 1 image: eight of the nine taps lie outside
    px = hb.quantize(to_dev(x), 1, f)
    pa = hb.im2col_packed(px, 1, 1, 1, 16, 3, 3, 1)
    q, s = decode_packed(pa, hb.packed_layout(pa.rows, pa.k, pa.fmt))
    q_ref, s_ref = oracle.quantize(oracle.im2col(x.reshape(1, 1, 1, 16), 3, 3, 1), 1, oracle.Format(mant_bits=8, block=16))
    assert np.array_equal(q, q_ref) and np.array_equal(s, s_ref)


@pytest.mark.parametrize("n,hw,c,b,m,rounding", [(2, 32, 64, 64, 8, 0), (3, 16, 128, 64, 8, 0), (2, 8, 24, 32, 8, 0),
                                                 (1, 16, 32, 128, 12, 0), (2, 16, 16, 16, 6, 0)])
def test_backward_weight_operand_equals_column_quantised_im2col_matrix(hb, n, hw, c, b, m, rounding):
    x = wl.draw("half_normal", (n * hw * hw, c), seed=81).reshape(n, hw, hw, c)
    x *= np.exp(wl.draw("normal", (n * hw * hw, 1), seed=82)).reshape(n, hw, hw, 1).astype(np.float32)
    fd = dict(mant_bits=m, block=b, rounding=rounding, seed=0)
    pa = hb.im2col_packed_t(to_dev(x), 3, 3, 1, gfmt(fd))
    assert hb.device_status() == 0
    cols = oracle.im2col(x, 3, 3, 1)
    q_ref, s_ref = oracle.quantize(cols, 0, ofmt(fd))
    q, s = decode_packed(pa, hb.packed_layout(pa.rows, pa.k, pa.fmt))
    assert np.array_equal(q, q_ref) and np.array_equal(s, s_ref)


def test_convolution_backward_weight_gemm(hb):
    n, hw, c, f = 4, 32, 64, 64
    x = wl.draw("half_normal", (n * hw * hw, c), seed=83).reshape(n, hw, hw, c)
    dy = wl.draw("grad", (n * hw * hw, f), seed=84)
    fd = dict(mant_bits=8, block=64, rounding=0, seed=0)
    pa = hb.im2col_packed_t(to_dev(x), 3, 3, 1, gfmt(fd))
    dW = hb.gemm_q(9 * c, f, n * hw * hw, pa, to_dev(dy), fmtB=gfmt(fd)).cpu().numpy()
    assert hb.device_status() == 0
    cols = oracle.im2col(x, 3, 3, 1)
    ref = oracle.hbfp_gemm(1, 0, cols, dy, ofmt(fd), ofmt(fd))
    err = np.abs(dW.astype(np.float64) - ref["c_ref"].astype(np.float64))
    assert (err <= TOL * ref["a_mag"]).all()


def test_backward_weight_operand_refuses_what_it_does_not_cover(hb):
    import torch
    x = torch.zeros((1, 8, 8, 16), device="cuda")
    with pytest.raises(hb.HbfpError) as e:                 # a block that is not whole image rows
        hb.im2col_packed_t(x, 3, 3, 1, hb.Format(mant_bits=8, block=12))
    assert e.value.code == hb.ERR_UNSUPPORTED
    with pytest.raises(hb.HbfpError) as e:                 # an output smaller than the input
        hb.im2col_packed_t(x, 3, 3, 0, hb.Format(mant_bits=8, block=16))
    assert e.value.code == hb.ERR_UNSUPPORTED


@pytest.mark.parametrize("n,hw,c,b,m", [(2, 32, 64, 64, 8), (3, 16, 32, 128, 12), (2, 8, 16, 16, 8), (1, 16, 128, 32, 6)])
def test_backward_weight_operand_under_stochastic_rounding(hb, n, hw, c, b, m):
    """Every entry of the operand is a copy of an activation and is rounded with that activation's draw
    (index in x): the oracle's indexed quantiser on the im2col matrix, bit for bit."""
    x = wl.draw("half_normal", (n * hw * hw, c), seed=87).reshape(n, hw, hw, c)
    x *= np.exp(wl.draw("normal", (n * hw * hw, 1), seed=88)).reshape(n, hw, hw, 1).astype(np.float32)
    fd = dict(mant_bits=m, block=b, rounding=1, seed=13, stream_id=4)
    pa = hb.im2col_packed_t(to_dev(x), 3, 3, 1, gfmt(fd))
    assert hb.device_status() == 0
    cols = oracle.im2col(x, 3, 3, 1)
    q_ref, s_ref = oracle.quantize_indexed(cols, 0, ofmt(fd), oracle.im2col_index(n, hw, hw, c, 3, 3, 1))
    q, s = decode_packed(pa, hb.packed_layout(pa.rows, pa.k, pa.fmt))
    assert np.array_equal(s, s_ref) and np.array_equal(q, q_ref)


IMPLICIT_CASES = [
    # n, h, w, c, filters, kh, pad, weight law: shapes the implicit-GEMM kernel covers
    (4, 32, 32, 64, 64, 3, 1),        # the 64 -> 64 convolution of the ResNet configuration (four images)
    (3, 16, 16, 128, 128, 3, 1),      # the 128 -> 128 one; an odd number of 128-pixel row tiles
    (5, 8, 16, 64, 12, 3, 1),         # few filters; a last super tile that is only partly there
    (2, 16, 16, 128, 200, 5, 2),      # 5 x 5 filter, 200 filters (256-wide tile)
    (1, 4, 128, 64, 96, 1, 0),        # 1 x 1 filter, an image row as long as a row tile
    (7, 4, 64, 64, 132, 3, 1),
]


@pytest.mark.parametrize("n,h,w,c,f,k,pad", IMPLICIT_CASES)
def test_implicit_gemm_convolution_equals_oracle_and_the_gather_path(hb, n, h, w, c, f, k, pad):
    """hbfp_conv_forward reads the taps straight from the packed pixels: same numbers as the oracle's GEMM
    on the im2col matrix in its sequential order, and what gather + GEMM gives."""
    x = wl.draw("half_normal", (n * h * w, c), seed=75).reshape(n, h, w, c)
    x *= np.exp(2 * wl.draw("normal", (n * h * w, 1), seed=76)).reshape(n, h, w, 1).astype(np.float32)
    wt = wl.draw("he_weight", (k * k * c, f), seed=77, fan_in=k * k * c)
    fd = dict(mant_bits=8, block=c, rounding=0, seed=0)
    px = hb.quantize(to_dev(x.reshape(n * h * w, c)), 1, gfmt(fd))
    pw = hb.quantize(to_dev(wt), 0, gfmt(fd, stream_id=1))
    Y = hb.conv_forward(px, pw, n, h, w, c, k, k, pad).cpu().numpy()
    assert hb.device_status() == 0
    assert hb.last_gemm_kernel() == "conv_fwd_kernel"
    cols = oracle.im2col(x, k, k, pad)
    ref = oracle.hbfp_gemm(0, 0, cols, wt, ofmt(fd), ofmt(fd, stream_id=1))
    err = np.abs(Y.astype(np.float64) - ref["c_ref"].astype(np.float64))
    assert (err <= TOL * ref["a_mag"]).all(), float((err / np.maximum(ref["a_mag"], 1e-300)).max())
    assert np.array_equal(Y, ref["c_seq"])            # taps in ascending order, one rounding each
    # the gather + GEMM path computes the same product (it may split K for a small output, so its order of
    # accumulation can differ: the tolerance of the GEMM tests)
    pa = hb.im2col_packed(px, n, h, w, c, k, k, pad)
    Y2 = hb.gemm_q(n * h * w, f, k * k * c, pa, pw).cpu().numpy()
    assert (np.abs(Y.astype(np.float64) - Y2.astype(np.float64)) <= 2 * TOL * ref["a_mag"]).all()


def test_implicit_gemm_convolution_says_what_it_does_not_cover(hb):
    n, h, w, c, f = 1, 9, 7, 24, 8
    x = wl.draw("half_normal", (n * h * w, c), seed=78)
    wt = wl.draw("he_weight", (9 * c, f), seed=79, fan_in=9 * c)
    fd = dict(mant_bits=8, block=c)
    px = hb.quantize(to_dev(x), 1, gfmt(fd))
    pw = hb.quantize(to_dev(wt), 0, gfmt(fd))
    with pytest.raises(hb.HbfpError) as e:
        hb.conv_forward(px, pw, n, h, w, c, 3, 3, 1)
    assert e.value.code == hb.ERR_UNSUPPORTED


@pytest.mark.parametrize("taps,c_in,c_out,t,m,rounding", [(9, 64, 64, 64, 8, 0), (9, 128, 96, 32, 8, 1), (25, 24, 40, 24, 6, 0),
                                                          (1, 64, 130, 64, 12, 1), (4, 576, 560, 32, 8, 0)])
def test_convolution_weights_tiled_on_the_feature_map_dimensions(hb, taps, c_in, c_out, t, m, rounding):
    """hbfp_quantize_conv_weights against the oracle: one exponent per (t input maps x t output maps) tile over
    every filter tap, both views bit-exact."""
    w = wl.draw("he_weight", (taps * c_in, c_out), seed=83, fan_in=taps * c_in)
    w *= np.exp(wl.draw("normal", (taps * c_in, 1), seed=84)).astype(np.float32)
    fd = dict(mant_bits=m, block=t, tile=t, rounding=rounding, seed=9, stream_id=2)
    c0, c1, grid = hb.quantize_conv_weights(to_dev(w), taps, gfmt(fd), want_grid=True)
    assert hb.device_status() == 0
    q0, s0 = oracle.quantize_conv_weights(w, taps, 0, ofmt(fd))
    q1, s1 = oracle.quantize_conv_weights(w, taps, 1, ofmt(fd))
    g0, e0 = decode_packed(c0, hb.packed_layout(c0.rows, c0.k, c0.fmt))
    g1, e1 = decode_packed(c1, hb.packed_layout(c1.rows, c1.k, c1.fmt))
    assert np.array_equal(g0, q0) and np.array_equal(e0, s0)
    assert np.array_equal(g1, q1) and np.array_equal(e1, s1)
    assert np.array_equal(grid.cpu().numpy(), s1[:c_in:t, :])


def test_convolution_with_tiled_weights_end_to_end(hb):
    """Pixels converted once, weights tiled over the feature maps, implicit GEMM: the oracle's GEMM on the
    oracle's operands, bit for bit."""
    n, h, w_, c, f = 2, 32, 32, 64, 64
    x = wl.draw("half_normal", (n * h * w_, c), seed=85).reshape(n, h, w_, c)
    wt = wl.draw("he_weight", (9 * c, f), seed=86, fan_in=9 * c)
    fx = dict(mant_bits=8, block=c)
    fw = dict(mant_bits=8, block=c, tile=c, stream_id=1)
    px = hb.quantize(to_dev(x.reshape(n * h * w_, c)), 1, gfmt(fx))
    c0, c1, _ = hb.quantize_conv_weights(to_dev(wt), 9, gfmt(fw))
    Y = hb.conv_forward(px, c0, n, h, w_, c, 3, 3, 1).cpu().numpy()
    assert hb.device_status() == 0
    qa, sa = oracle.quantize(oracle.im2col(x, 3, 3, 1), 1, ofmt(fx))
    qb, sb = oracle.quantize_conv_weights(wt, 9, 0, ofmt(fw))
    ref = oracle.gemm(qa, sa, qb, sb, c)
    assert np.array_equal(Y, ref["c_seq"])


def test_gathered_operand_under_stochastic_rounding_takes_each_activations_draw(hb):
    """Forward operand under stochastic rounding: the pixels were converted with draws keyed by their index in
    the activation tensor, so the gathered operand is the oracle's indexed conversion of the im2col matrix."""
    n, h, w, c = 2, 8, 8, 32
    x = wl.draw("half_normal", (n * h * w, c), seed=89).reshape(n, h, w, c)
    fd = dict(mant_bits=8, block=c, rounding=1, seed=17, stream_id=6)
    px = hb.quantize(to_dev(x.reshape(n * h * w, c)), 1, gfmt(fd))
    pa = hb.im2col_packed(px, n, h, w, c, 3, 3, 1)
    q_ref, s_ref = oracle.quantize_indexed(oracle.im2col(x, 3, 3, 1), 1, ofmt(fd), oracle.im2col_index(n, h, w, c, 3, 3, 1))
    q, s = decode_packed(pa, hb.packed_layout(pa.rows, pa.k, pa.fmt))
    assert np.array_equal(q, q_ref) and np.array_equal(s, s_ref)


@pytest.mark.parametrize("k,c_in,c_out,t,m,rounding", [(3, 64, 64, 64, 8, 0), (3, 128, 64, 64, 8, 1), (5, 64, 128, 32, 6, 0),
                                                       (1, 128, 256, 128, 12, 1), (3, 32, 96, 32, 12, 0)])
def test_backward_data_filter_operand_is_a_regrouping_of_the_forward_weights(hb, k, c_in, c_out, t, m, rounding):
    """hbfp_conv_dgrad_filters moves bytes and tile exponents only: decoded, the operand is the oracle's view c1
    with taps reversed and rows regrouped by input map."""
    taps = k * k
    w = wl.draw("he_weight", (taps * c_in, c_out), seed=91, fan_in=taps * c_in)
    w *= np.exp(wl.draw("normal", (taps * c_in, 1), seed=92)).astype(np.float32)
    fd = dict(mant_bits=m, block=t, tile=t, rounding=rounding, seed=5, stream_id=2)
    _, c1, _ = hb.quantize_conv_weights(to_dev(w), taps, gfmt(fd))
    d = hb.conv_dgrad_filters(c1, k, k, c_in, c_out)
    assert hb.device_status() == 0
    assert (d.rows, d.k) == (c_in, taps * c_out)
    q1, s1 = oracle.quantize_conv_weights(w, taps, 1, ofmt(fd))
    qd, sd = dgrad_filters_view(q1, s1, taps, c_in)
    gd, ed = decode_packed(d, hb.packed_layout(d.rows, d.k, d.fmt))
    assert np.array_equal(gd, qd) and np.array_equal(ed, sd)


@pytest.mark.parametrize("n,h,w_,c_in,c_out,k,pad", [(2, 32, 32, 64, 64, 3, 1), (3, 16, 16, 128, 128, 3, 1), (2, 16, 16, 128, 64, 3, 1),
                                                     (1, 8, 16, 128, 128, 5, 2), (2, 4, 64, 64, 64, 1, 0), (1, 16, 32, 256, 64, 3, 1)])
def test_backward_data_convolution_on_the_packed_gradient_equals_oracle(hb, n, h, w_, c_in, c_out, k, pad):
    """dX as an implicit GEMM: the packed output gradient (one block per pixel) against the regrouped forward
    weights, padding k - 1 - pad. Expected: the oracle's GEMM on the oracle's quantised gather of dY and the
    oracle's tiled weights regrouped the same way, bit for bit in the sequential order."""
    taps = k * k
    ho, wo = h + 2 * pad - k + 1, w_ + 2 * pad - k + 1
    dy = wl.draw("normal", (n * ho * wo, c_out), seed=93).reshape(n, ho, wo, c_out)
    dy *= np.exp(2 * wl.draw("normal", (n * ho * wo, 1), seed=94)).reshape(n, ho, wo, 1).astype(np.float32) * 1e-3
    wt = wl.draw("he_weight", (taps * c_in, c_out), seed=95, fan_in=taps * c_in)
    fg = dict(mant_bits=8, block=c_out, rounding=1, seed=11, stream_id=3)
    fw = dict(mant_bits=8, block=c_out, tile=c_out, stream_id=1)
    pg = hb.quantize(to_dev(dy.reshape(n * ho * wo, c_out)), 1, gfmt(fg))
    _, c1, _ = hb.quantize_conv_weights(to_dev(wt), taps, gfmt(fw))
    d = hb.conv_dgrad_filters(c1, k, k, c_in, c_out)
    dX = hb.conv_forward(pg, d, n, ho, wo, c_out, k, k, k - 1 - pad).cpu().numpy()
    assert hb.device_status() == 0
    assert hb.last_gemm_kernel() == "conv_fwd_kernel"
    assert dX.shape == (n * h * w_, c_in)
    # the oracle's side: every block of the gathered gradient is the pixel's own block (one conversion per pixel,
    # stochastic draws keyed by the element's index in dY), so gather the canonical arrays of the pixels
    qp, sp = oracle.quantize(dy.reshape(n * ho * wo, c_out), 1, ofmt(fg))
    qa = oracle.im2col(qp.reshape(n, ho, wo, c_out), k, k, k - 1 - pad)
    sa = oracle.im2col(sp.reshape(n, ho, wo, 1), k, k, k - 1 - pad)
    q1, s1 = oracle.quantize_conv_weights(wt, taps, 1, ofmt(fw))
    qb, sb = dgrad_filters_view(q1, s1, taps, c_in)
    ref = oracle.gemm(qa, sa, qb, sb, c_out)
    err = np.abs(dX.astype(np.float64) - ref["c_ref"].astype(np.float64))
    assert (err <= TOL * ref["a_mag"]).all()
    assert np.array_equal(dX, ref["c_seq"])


def test_backward_data_filter_operand_says_what_it_does_not_cover(hb):
    w = wl.draw("he_weight", (9 * 24, 40), seed=96, fan_in=9 * 24)
    fd = dict(mant_bits=8, block=24, tile=24)
    _, c1, _ = hb.quantize_conv_weights(to_dev(w), 9, gfmt(fd))
    with pytest.raises(hb.HbfpError) as e:
        hb.conv_dgrad_filters(c1, 3, 3, 24, 40)
    assert e.value.code == hb.ERR_UNSUPPORTED
