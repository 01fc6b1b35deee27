"""The three GEMMs of a training step in use: a dense layer whose forward, backward-data and
backward-weight products run through the library (weights in wide storage, updated in place), checked
product by product against the oracle, and a small classifier on synthetic data trained with it beside
the same model in FP32 (the paper's claim, Sec. 6: HBFP follows the FP32 training curve)."""
import numpy as np
import pytest

import oracle
from tests.helpers import dgrad_filters_view, ofmt

pytestmark = pytest.mark.gpu

TOL = 1e-6


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_1804_01526_b200 import autograd as hbfp_nn, binding
    binding.lib()
    return torch, hbfp_nn, binding


def fmt_dict(f):
    return dict(mant_bits=f.mant_bits, block=f.block, tile=f.tile, rounding=f.rounding, seed=f.seed, stream_id=f.stream_id)


def test_layer_products_match_the_oracle(env):
    torch, hbfp_nn, hb = env
    torch.manual_seed(0)
    batch, fin, fout, t = 96, 200, 136, 24
    layer = hbfp_nn.HbfpLinear(fin, fout, mant_bits=8, tile=t, rounding=1, seed=5, stream_id=10, batch_block=32)
    x = torch.randn(batch, fin, device="cuda").relu().requires_grad_(True)
    y = layer(x)
    dy = torch.randn(batch, fout, device="cuda") * 1e-3
    y.backward(dy)
    assert hb.device_status() == 0
    # the narrow copy the layer multiplied by, from its wide storage
    q16, g16 = layer.wide.mant.cpu().numpy(), layer.wide.exps.cpu().numpy()
    s16 = np.repeat(g16, t, axis=0)[:fin, :]
    qm, sm = oracle.wide_narrow(q16, s16, 8)
    grid = sm[::t, :]
    X, dY = x.detach().cpu().numpy(), dy.cpu().numpy()
    # forward
    qx, sx = oracle.quantize(X, 1, ofmt(fmt_dict(layer.fmt_act(0))))
    ref = oracle.gemm(qx, sx, np.ascontiguousarray(qm.T), np.ascontiguousarray(np.repeat(grid.T, t, axis=0)[:fout, :]), t)
    Y = (y - layer.bias).detach().cpu().numpy()
    assert (np.abs(Y.astype(np.float64) - ref["c_ref"]) <= TOL * ref["a_mag"] + 1e-12).all()
    # backward-data
    qd, sd = oracle.quantize(dY, 1, ofmt(fmt_dict(layer.fmt_act(2))))
    ref = oracle.gemm(qd, sd, qm, sm, t)
    assert (np.abs(x.grad.cpu().numpy().astype(np.float64) - ref["c_ref"]) <= TOL * ref["a_mag"]).all()
    # backward-weight: X^T dY with blocks along the batch axis
    ref = oracle.hbfp_gemm(1, 0, X, dY, ofmt(fmt_dict(layer.fmt_act(0, batch_axis=True))),
                           ofmt(fmt_dict(layer.fmt_act(2, batch_axis=True))))
    assert (np.abs(layer.weight.grad.cpu().numpy().astype(np.float64) - ref["c_ref"]) <= TOL * ref["a_mag"]).all()
    # and the update lands in wide storage as the oracle computes it
    delta = (-0.1 * layer.weight.grad).contiguous()
    layer.apply_update(delta)
    q2, s2 = oracle.wide_update(q16, s16, delta.cpu().numpy(), ofmt(fmt_dict(layer.fmt_weight())))
    assert np.array_equal(layer.wide.mant.cpu().numpy(), q2)
    assert np.array_equal(layer.wide.exps.cpu().numpy(), s2[::t, :])


def test_small_classifier_trains_like_fp32(env):
    torch, hbfp_nn, hb = env
    torch.manual_seed(1)
    n_cls, fin, hid, batch, steps, lr = 10, 64, 128, 128, 80, 0.2
    centers = torch.randn(n_cls, fin, device="cuda") * 1.5
    gen = torch.Generator(device="cuda").manual_seed(2)

    def draw():
        labels = torch.randint(0, n_cls, (batch,), device="cuda", generator=gen)
        return centers[labels] + torch.randn(batch, fin, device="cuda", generator=gen), labels

    l1 = hbfp_nn.HbfpLinear(fin, hid, mant_bits=8, tile=24, rounding=1, seed=3, stream_id=0)
    l2 = hbfp_nn.HbfpLinear(hid, n_cls, mant_bits=8, tile=24, rounding=1, seed=3, stream_id=10)
    # the FP32 twin starts from the same (wide-representable) weights
    w1 = l1.weight.detach().clone().requires_grad_(True)
    w2 = l2.weight.detach().clone().requires_grad_(True)
    b1 = torch.zeros(hid, device="cuda", requires_grad=True)
    b2 = torch.zeros(n_cls, device="cuda", requires_grad=True)
    loss_fn = torch.nn.CrossEntropyLoss()
    hist_h, hist_f = [], []
    for _ in range(steps):
        x, labels = draw()
        loss_h = loss_fn(l2(torch.relu(l1(x))), labels)
        for p in (l1.weight, l1.bias, l2.weight, l2.bias):
            p.grad = None
        loss_h.backward()
        with torch.no_grad():
            for layer in (l1, l2):
                layer.apply_update(-lr * layer.weight.grad)          # FP32 optimiser arithmetic, BFP weight storage
                layer.bias -= lr * layer.bias.grad
        loss_f = loss_fn(torch.relu(x @ w1 + b1) @ w2 + b2, labels)
        for p in (w1, b1, w2, b2):
            p.grad = None
        loss_f.backward()
        with torch.no_grad():
            for p in (w1, b1, w2, b2):
                p -= lr * p.grad
        hist_h.append(float(loss_h.detach()))
        hist_f.append(float(loss_f.detach()))
    assert hb.device_status() == 0
    first, last_h, last_f = np.mean(hist_h[:5]), np.mean(hist_h[-10:]), np.mean(hist_f[-10:])
    assert last_h < 0.5 * first, (first, last_h)                     # it learns
    assert abs(last_h - last_f) <= 0.15 * max(last_f, 0.05), (last_h, last_f)   # and follows the FP32 curve


def test_convolution_layer_products_match_the_oracle_and_fp32(env):
    torch, hbfp_nn, hb = env
    torch.manual_seed(2)
    n, hw, c, f = 2, 16, 64, 64
    layer = hbfp_nn.HbfpConv3x3(c, f, mant_bits=8, pixel_block=64)
    x = torch.randn(n, hw, hw, c, device="cuda").relu().requires_grad_(True)
    y = layer(x)
    dy = torch.randn(n, hw, hw, f, device="cuda") * 1e-2
    y.backward(dy)
    assert hb.device_status() == 0
    t = c
    q16, g16 = layer.wide.mant.cpu().numpy(), layer.wide.exps.cpu().numpy()
    s16 = np.repeat(g16, t, axis=0)[: 9 * c, :]
    qm, sm = oracle.wide_narrow(q16, s16, 8)
    grid = sm[::t, :]
    X, dY = x.detach().cpu().numpy(), dy.cpu().numpy().reshape(n * hw * hw, f)
    cols = oracle.im2col(X, 3, 3, 1)
    fa = dict(mant_bits=8, block=c, rounding=0, seed=0)
    # forward
    qx, sx = oracle.quantize(cols, 1, ofmt(fa))
    ref = oracle.gemm(qx, sx, np.ascontiguousarray(qm.T), np.ascontiguousarray(np.repeat(grid.T, t, axis=0)[:f, :]), t)
    Y = y.detach().cpu().numpy().reshape(n * hw * hw, f)
    assert (np.abs(Y.astype(np.float64) - ref["c_ref"]) <= TOL * ref["a_mag"] + 1e-12).all()
    # backward-weight
    fb = dict(mant_bits=8, block=64, rounding=0, seed=0)
    ref = oracle.hbfp_gemm(1, 0, cols, dY, ofmt(fb), ofmt(fb))
    assert (np.abs(layer.weight.grad.cpu().numpy().astype(np.float64) - ref["c_ref"]) <= TOL * ref["a_mag"]).all()
    # backward-data: the GEMM against the oracle, the scatter against torch's own convolution gradient
    qd, sd = oracle.quantize(dY, 1, ofmt(fa))
    ref = oracle.gemm(qd, sd, qm, sm, t)                         # gradient of the im2col matrix [pixels][9 c]
    dcols = ref["c_ref"].reshape(n, hw, hw, 3, 3, c)
    dxp = np.zeros((n, hw + 2, hw + 2, c))
    for i in range(3):
        for j in range(3):
            dxp[:, i:i + hw, j:j + hw, :] += dcols[:, :, :, i, j, :]
    dx_ref = dxp[:, 1:hw + 1, 1:hw + 1, :]
    assert np.allclose(x.grad.cpu().numpy(), dx_ref, rtol=1e-4, atol=1e-6)
    # ... computed as the convolution of the packed gradient with the regrouped forward weights: bit for bit the
    # oracle's GEMM on the gathered quantised gradient, taps in that operand's order
    qa = oracle.im2col(qd.reshape(n, hw, hw, f), 3, 3, 1)
    sa = oracle.im2col(sd.reshape(n, hw, hw, 1), 3, 3, 1)
    qb, sb = dgrad_filters_view(qm, sm, 9, c)
    ref = oracle.gemm(qa, sa, qb, sb, t)
    assert np.array_equal(x.grad.cpu().numpy().reshape(n * hw * hw, c), ref["c_seq"])
    # and the whole layer stays close to the FP32 convolution it stands for
    w4 = layer.weight.detach().view(3, 3, c, f).permute(3, 2, 0, 1).contiguous()          # [f][c][3][3]
    y32 = torch.nn.functional.conv2d(x.detach().permute(0, 3, 1, 2), w4, padding=1).permute(0, 2, 3, 1)
    rel = (y.detach() - y32).norm() / y32.norm()
    assert float(rel) < 2e-2
