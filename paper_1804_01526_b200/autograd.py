"""A dense layer and a 3 x 3 convolution whose three GEMMs run in block floating point (Sec. 4.1, Sec. 5.1).

The paper simulates HBFP by redefining PyTorch's linear module with ``autograd.Function``: the
forward product ``Y = X W``, the backward-data product ``dX = dY W^T`` and the backward-weight
product ``dW = X^T dY`` take BFP operands, every other operation (bias, activations, loss, the
optimiser's arithmetic) stays FP32. This module is that wrapper over the library's calls; it holds
no arithmetic of its own:

* the weights live in wide storage (16-bit mantissas per tile, ``hbfp_wide_quantize``); the two
  packed narrow views the GEMMs read are the top ``mant_bits`` bits (Sec. 4.2);
* forward and backward-data read those views (``hbfp_gemm_q``), so the backward pass converts no
  weights; activations and gradients are converted by the GEMM call with 1-D blocks along the
  contraction axis; backward-weight is ``hbfp_gemm`` with ``transA = 1``;
* ``apply_update(delta)`` hands the optimiser's FP32 update to ``hbfp_wide_update`` and refreshes the
  views in the same launch.

Stochastic rounding draws are keyed by (seed + step, stream id, element index): a layer takes three
consecutive stream ids (X, W, dY) from ``stream_id``.

``HbfpConv3x3`` does the same for a convolution on channels-last activations, on the two operands the
library builds without an FP32 im2col matrix (``hbfp_im2col_packed``, ``hbfp_im2col_packed_t``).
"""
from __future__ import annotations

import torch

from . import binding as hb


class _HbfpLinearFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, weight, bias, layer):
        ctx.layer = layer
        ctx.save_for_backward(x)
        batch = x.shape[0]
        y = hb.gemm_q(batch, layer.fout, layer.fin, x.contiguous(), layer.views[0], fmtA=layer.fmt_act(0))
        return y + bias if bias is not None else y

    @staticmethod
    def backward(ctx, dy):
        layer = ctx.layer
        (x,) = ctx.saved_tensors
        dy = dy.contiguous()
        batch = x.shape[0]
        dx = dw = db = None
        if ctx.needs_input_grad[0]:
            dx = hb.gemm_q(batch, layer.fin, layer.fout, dy, layer.views[1], fmtA=layer.fmt_act(2))
        if ctx.needs_input_grad[1]:
            # contraction over the batch axis: 1-D blocks down the columns of X and dY
            dw = hb.gemm(1, 0, x.contiguous(), dy, layer.fmt_act(0, batch_axis=True), layer.fmt_act(2, batch_axis=True))
        if ctx.needs_input_grad[2]:
            db = dy.sum(dim=0)
        return dx, dw, db, None


class HbfpLinear(torch.nn.Module):
    """``y = x W + b`` with W ``[fin][fout]`` in wide storage; see the module docstring."""

    def __init__(self, fin: int, fout: int, mant_bits: int = 8, tile: int = 24, rounding: int = 1, seed: int = 0,
                 stream_id: int = 0, batch_block: int = 32, bias: bool = True, device="cuda"):
        super().__init__()
        self.fin, self.fout = fin, fout
        self.mant_bits, self.tile, self.rounding, self.seed, self.stream_id = mant_bits, tile, rounding, seed, stream_id
        self.batch_block = batch_block
        self.steps = 0
        w = torch.randn(fin, fout, device=device) * (2.0 / fin) ** 0.5
        self.weight = torch.nn.Parameter(w)
        self.bias = torch.nn.Parameter(torch.zeros(fout, device=device)) if bias else None
        self.wide, self.views = hb.wide_quantize(self.weight.data, self.fmt_weight())
        self._refresh_fp32_copy()

    # ---- formats
    def fmt_weight(self) -> hb.Format:
        return hb.Format(mant_bits=self.mant_bits, block=self.tile, tile=self.tile, rounding=self.rounding,
                         seed=self.seed + self.steps, stream_id=self.stream_id + 1)

    def fmt_act(self, which: int, batch_axis: bool = False) -> hb.Format:
        """Format of X (which = 0) or dY (which = 2); blocks of ``tile`` along a feature axis, of
        ``batch_block`` along the batch axis (backward-weight)."""
        return hb.Format(mant_bits=self.mant_bits, block=self.batch_block if batch_axis else self.tile,
                         rounding=self.rounding, seed=self.seed + self.steps, stream_id=self.stream_id + which)

    # ---- weights
    def _refresh_fp32_copy(self) -> None:
        """The FP32 tensor autograd sees is the value of the wide copy (hbfp_wide_dequantize)."""
        self.weight.data = hb.wide_dequantize(self.wide)

    def apply_update(self, delta: torch.Tensor) -> None:
        """``W <- Q16(float32(W + delta))`` in wide storage, views refreshed by the same launch."""
        self.steps += 1
        hb.wide_update(self.wide, delta.contiguous(), self.fmt_weight(), views=self.views)
        self._refresh_fp32_copy()

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        return _HbfpLinearFn.apply(x, self.weight, self.bias, self)


class _HbfpConv3x3Fn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, weight, layer):
        n, h, w, c = x.shape
        ctx.layer = layer
        ctx.save_for_backward(x)
        x = x.contiguous()
        px = hb.quantize(x.view(n * h * w, c), 1, layer.fmt_pixels(0))
        try:
            # the implicit GEMM reads the taps straight from the packed pixels
            y = hb.conv_forward(px, layer.views[0], n, h, w, c, 3, 3, 1)
        except hb.HbfpError as e:
            if e.code != hb.ERR_UNSUPPORTED:
                raise
            # shapes it does not cover: gather the packed operand, then the ordinary GEMM (same product)
            pa = hb.im2col_packed(px, n, h, w, c, 3, 3, 1)
            y = hb.gemm_q(n * h * w, layer.fout, 9 * c, pa, layer.views[0])
        return y.view(n, h, w, layer.fout)

    @staticmethod
    def backward(ctx, dy):
        layer = ctx.layer
        (x,) = ctx.saved_tensors
        n, h, w, c = x.shape
        f = layer.fout
        dy2 = dy.contiguous().view(n * h * w, f)
        dx = dw = None
        if ctx.needs_input_grad[0]:
            try:
                # the convolution of the packed output gradient with the forward weights regrouped (taps turned by
                # 180 degrees, feature-map roles swapped) yields dX itself
                pg = hb.quantize(dy2, 1, layer.fmt_pixels(2))
                turned = hb.conv_dgrad_filters(layer.views[1], 3, 3, c, f)
                dx = hb.conv_forward(pg, turned, n, h, w, f, 3, 3, 1).view(n, h, w, c)
            except hb.HbfpError as e:
                if e.code != hb.ERR_UNSUPPORTED:
                    raise
        if ctx.needs_input_grad[0] and dx is None:
            # shapes that route does not cover: gradient of the im2col matrix, then its scatter back onto the
            # pixels (an FP32 operation)
            dcols = hb.gemm_q(n * h * w, 9 * c, f, dy2, layer.views[1], fmtA=layer.fmt_pixels(2)).view(n, h, w, 3, 3, c)
            dxp = torch.zeros((n, h + 2, w + 2, c), device=x.device)
            for i in range(3):
                for j in range(3):
                    dxp[:, i:i + h, j:j + w, :] += dcols[:, :, :, i, j, :]
            dx = dxp[:, 1:h + 1, 1:w + 1, :].contiguous()
        if ctx.needs_input_grad[1]:
            pa_t = hb.im2col_packed_t(x.contiguous(), 3, 3, 1, layer.fmt_batch(0))
            dw = hb.gemm_q(9 * c, f, n * h * w, pa_t, dy2, fmtB=layer.fmt_batch(2))
        return dx, dw, None


class HbfpConv3x3(torch.nn.Module):
    """3 x 3 convolution, stride 1, one pixel of zero padding, channels-last activations ``[n][h][w][c]``,
    as three BFP GEMMs (Sec. 5.1) without an FP32 im2col matrix: the forward operand is gathered from
    activations converted once per pixel, the backward-weight operand is converted straight from the
    activations, backward-data is the same implicit GEMM on the packed output gradient with the regrouped
    forward weights (a GEMM followed by the FP32 scatter onto the pixels where that does not apply). The weights
    ``[9 c][filters]`` (rows ordered (filter row, filter column, channel)) live in wide storage with
    ``c x c`` tiles, so the K-blocks of weights and activations coincide. Nearest-even rounding."""

    def __init__(self, c: int, fout: int, mant_bits: int = 8, pixel_block: int = 64, device="cuda"):
        super().__init__()
        self.c, self.fout, self.mant_bits, self.pixel_block = c, fout, mant_bits, pixel_block
        self.weight = torch.nn.Parameter(torch.randn(9 * c, fout, device=device) * (2.0 / (9 * c)) ** 0.5)
        self.wide, self.views = hb.wide_quantize(self.weight.data, self.fmt_weight())
        self._refresh_fp32_copy()

    def fmt_weight(self) -> hb.Format:
        return hb.Format(mant_bits=self.mant_bits, block=self.c, tile=self.c)

    def fmt_pixels(self, which: int) -> hb.Format:
        """X (blocks of c channels per pixel) or dY (blocks of c filters per pixel)."""
        return hb.Format(mant_bits=self.mant_bits, block=self.c, stream_id=which)

    def fmt_batch(self, which: int) -> hb.Format:
        """Backward-weight: blocks of ``pixel_block`` consecutive output pixels."""
        return hb.Format(mant_bits=self.mant_bits, block=self.pixel_block, stream_id=which)

    def _refresh_fp32_copy(self) -> None:
        self.weight.data = hb.wide_dequantize(self.wide)

    def apply_update(self, delta: torch.Tensor) -> None:
        hb.wide_update(self.wide, delta.contiguous(), self.fmt_weight(), views=self.views)
        self._refresh_fp32_copy()

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        return _HbfpConv3x3Fn.apply(x, self.weight, self)
