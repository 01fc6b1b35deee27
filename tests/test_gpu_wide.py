"""GPU parity of wide weight storage through the C ABI: 16-bit mantissas and tile exponents bit-exact
(nearest-even and stochastic rounding), the narrow views equal to the top bits of the wide mantissas,
the in-place FP32 update equal to the oracle's, and GEMMs on the derived views equal to the oracle's."""
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


def F(m, t, rounding=0, seed=0, stream_id=0):
    return dict(mant_bits=m, block=t, tile=t, rounding=rounding, seed=seed, stream_id=stream_id)


def check_views(hb, views, qm, sm, t):
    """views (c0, c1) against the canonical narrow arrays qm [d0][d1], sm [d0][ceil(d1/t)]."""
    c0, c1 = views
    q1, s1 = decode_packed(c1, hb.packed_layout(c1.rows, c1.k, c1.fmt))
    assert np.array_equal(q1, qm) and np.array_equal(s1, sm)
    q0, s0 = decode_packed(c0, hb.packed_layout(c0.rows, c0.k, c0.fmt))
    grid = sm[::t, :]                                            # [tiles along d0][tiles along d1]
    assert np.array_equal(q0, qm.T)
    assert np.array_equal(s0, np.repeat(grid.T, t, axis=0)[: qm.shape[1], :])


CASES = [
    ((784, 1024), "he_weight", F(8, 24, 1, seed=1, stream_id=1)),      # MLP layer, the paper's sweet spot: tile 24
    ((1024, 10), "he_weight", F(8, 24)),
    ((1000, 4096 // 4), "he_weight", F(12, 64, 1, seed=7, stream_id=11)),
    ((130, 257), "lognormal", F(4, 128)),
    ((61, 100), "lognormal", F(12, 24, 1, seed=5)),
    ((7, 5), "normal", F(8, 16)),
]


@pytest.mark.parametrize("shape,law,fd", CASES)
def test_wide_quantise_and_narrow_views_match_the_oracle(hb, shape, law, fd):
    kw = {"fan_in": shape[0]} if law == "he_weight" else {}
    w = wl.draw(law, shape, seed=21, **kw)
    t, m = fd["tile"], fd["mant_bits"]
    wide, views = hb.wide_quantize(to_dev(w), gfmt(fd))
    assert hb.device_status() == 0
    q16, s16 = oracle.wide_quantize(w, ofmt(fd))
    assert np.array_equal(wide.mant.cpu().numpy(), q16)
    assert np.array_equal(wide.exps.cpu().numpy(), s16[::t, :])
    qm, sm = oracle.wide_narrow(q16, s16, m)
    check_views(hb, views, qm, sm, t)
    # the read-only entry point writes the same views
    again = hb.wide_narrow(wide, gfmt(fd))
    check_views(hb, again, qm, sm, t)
    # the FP32 value of the wide copy is Eq. 1 written out: mantissa times 2^(tile exponent), exact
    val = hb.wide_dequantize(wide).cpu().numpy()
    assert np.array_equal(val, np.ldexp(q16.astype(np.float64), np.repeat(s16, t, axis=1)[:, : shape[1]].astype(np.int64)).astype(np.float32))
    for a, b in zip(again, views):                               # and the same bytes in every documented position
        lay = hb.packed_layout(a.rows, a.k, a.fmt)
        for pl in range(lay["planes"]):
            lo, hi = pl * lay["plane_stride"], pl * lay["plane_stride"] + a.rows * lay["kst"]
            assert np.array_equal(a.mant[lo:hi].cpu().numpy(), b.mant[lo:hi].cpu().numpy())
    # wide storage alone
    wide2, none = hb.wide_quantize(to_dev(w), gfmt(fd), want_views=False)
    assert none is None and np.array_equal(wide2.mant.cpu().numpy(), q16)


@pytest.mark.parametrize("shape,fd", [((784, 1024), F(8, 24, 1, seed=3, stream_id=4)), ((333, 200), F(12, 64)),
                                      ((130, 257), F(8, 128, 1, seed=9))])
def test_wide_update_matches_the_oracle_over_several_steps(hb, shape, fd):
    w = wl.draw("he_weight", shape, seed=22, fan_in=shape[0])
    t, m = fd["tile"], fd["mant_bits"]
    wide, _ = hb.wide_quantize(to_dev(w), gfmt(fd), want_views=False)
    q, s = oracle.wide_quantize(w, ofmt(fd))
    for step in range(3):
        delta = (wl.draw("grad", shape, seed=30 + step) * (10.0 if step == 1 else 1.0)).astype(np.float32)
        if step == 2:
            delta[:, : shape[1] // 2] = 0                        # part of the matrix does not move
        fstep = dict(fd, seed=fd["seed"] + 100 * step)             # fresh draws every step
        views = hb.wide_update(wide, to_dev(delta), gfmt(fstep))
        assert hb.device_status() == 0
        q, s = oracle.wide_update(q, s, delta, ofmt(fstep))
        assert np.array_equal(wide.mant.cpu().numpy(), q)
        assert np.array_equal(wide.exps.cpu().numpy(), s[::t, :])
        qm, sm = oracle.wide_narrow(q, s, m)
        check_views(hb, views, qm, sm, t)


def test_forward_and_backward_data_on_views_derived_from_wide_storage(hb):
    # Y = X W and dX = dY W^T read the same narrow copy (top 8 bits, which can hold -128)
    batch, fin, fout, t = 128, 784, 1024, 24
    fw = F(8, t, 1, seed=1, stream_id=1)
    fx = dict(mant_bits=8, block=t, rounding=1, seed=1, stream_id=0)
    W = wl.draw("he_weight", (fin, fout), seed=23, fan_in=fin)
    X = wl.draw("half_normal", (batch, fin), seed=24)
    dY = wl.draw("grad", (batch, fout), seed=25)
    wide, (c0, c1) = hb.wide_quantize(to_dev(W), gfmt(fw))
    q16, s16 = oracle.wide_quantize(W, ofmt(fw))
    qm, sm = oracle.wide_narrow(q16, s16, 8)
    assert int(qm.min()) >= -128
    grid = sm[::t, :]
    # forward: contraction over fin; B operand canonical [fout][fin]
    qx, sx = oracle.quantize(X, 1, ofmt(fx))
    sB_rows = np.repeat(grid.T, t, axis=0)[:fout, :]
    ref = oracle.gemm(qx, sx, np.ascontiguousarray(qm.T), np.ascontiguousarray(sB_rows), t)
    Y = hb.gemm_q(batch, fout, fin, to_dev(X), c0, fmtA=gfmt(fx)).cpu().numpy()
    err = np.abs(Y.astype(np.float64) - ref["c_ref"].astype(np.float64))
    assert (err <= 1e-6 * ref["a_mag"]).all()
    # backward-data: contraction over fout; B operand canonical [fin][fout] = the stored orientation
    fdy = dict(fx, stream_id=2)
    qd, sd = oracle.quantize(dY, 1, ofmt(fdy))
    ref = oracle.gemm(qd, sd, qm, sm, t)
    dX = hb.gemm_q(batch, fin, fout, to_dev(dY), c1, fmtA=gfmt(fdy)).cpu().numpy()
    err = np.abs(dX.astype(np.float64) - ref["c_ref"].astype(np.float64))
    assert (err <= 1e-6 * ref["a_mag"]).all()
    assert hb.device_status() == 0


def test_wide_argument_errors(hb):
    import torch
    w = to_dev(wl.draw("normal", (64, 64), seed=1))
    with pytest.raises(hb.HbfpError) as e:                          # tile != block
        hb.wide_quantize(w, hb.Format(mant_bits=8, block=32, tile=16))
    assert e.value.code == hb.ERR_INVALID_ARG
    with pytest.raises(hb.HbfpError) as e:                          # tiles above 128 are not supported here
        hb.wide_quantize(w, hb.Format(mant_bits=8, block=256, tile=256))
    assert e.value.code == hb.ERR_UNSUPPORTED
    wide, _ = hb.wide_quantize(w, hb.Format(mant_bits=8, block=16, tile=16), want_views=False)
    with pytest.raises(ValueError):
        hb.wide_update(wide, torch.zeros((32, 64), device="cuda"), hb.Format(mant_bits=8, block=16, tile=16))


def test_wide_storage_of_an_empty_matrix(hb):
    import torch
    f = hb.Format(mant_bits=8, block=16, tile=16)
    wide, views = hb.wide_quantize(torch.empty((0, 32), device="cuda"), f)
    assert wide.mant.numel() == 0 and hb.device_status() == 0
    hb.wide_update(wide, torch.empty((0, 32), device="cuda"), f, views=views)
    hb.wide_narrow(wide, f, views=views)
    assert hb.device_status() == 0
