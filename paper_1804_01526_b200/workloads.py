"""Seeded synthetic inputs and GEMM shape lists of the benchmark configurations.

This module holds no arithmetic of the method: only value laws (plain numpy draws) and
shapes. Both the CUDA path and the CPU oracle are fed the arrays produced here, so that
neither depends on the other. The shapes stand in for the paper's workloads (Sec. 5.2:
ResNet / WideResNet / DenseNet on CIFAR-100, SVHN, ImageNet and an LSTM on PTB), whose
datasets are not available; the value laws are those the benchmark configurations name.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import numpy as np

# ----------------------------------------------------------------------------- value laws


def _rng(seed: int, salt: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(salt)])


def _std_normal(rng: np.random.Generator, shape) -> np.ndarray:
    """float32 N(0,1), drawn in slabs so that a 1 GiB tensor needs no float64 temporary."""
    out = np.empty(shape, dtype=np.float32)
    flat = out.reshape(-1)
    step = 1 << 24
    for i in range(0, flat.size, step):
        flat[i:i + step] = rng.standard_normal(min(step, flat.size - i), dtype=np.float32)
    return out


def draw(law: str, shape: Tuple[int, int], seed: int, salt: int = 0, **kw) -> np.ndarray:
    """One float32 array of ``shape`` from the named law.

    normal        N(0, std^2)                         kw: std (default 1)
    half_normal   max(0, N(0,1)): ReLU outputs, half of the entries are exactly zero
    he_weight     N(0, 2/fan_in)  (variance)          kw: fan_in
    grad          N(0, 1e-3)      (variance)
    outliers      N(0,1), each entry independently x100 with probability 0.01
    lognormal     +-exp(2 z), z ~ N(0,1), sign fair
    """
    rng = _rng(seed, salt)
    if law == "normal":
        x = _std_normal(rng, shape)
        std = float(kw.get("std", 1.0))
        if std != 1.0:
            x *= np.float32(std)
        return x
    if law == "half_normal":
        x = _std_normal(rng, shape)
        np.maximum(x, 0, out=x)
        return x
    if law == "he_weight":
        x = _std_normal(rng, shape)
        x *= np.float32(np.sqrt(2.0 / float(kw["fan_in"])))
        return x
    if law == "grad":
        x = _std_normal(rng, shape)
        x *= np.float32(np.sqrt(1e-3))
        return x
    if law == "outliers":
        x = _std_normal(rng, shape)
        hit = rng.random(shape, dtype=np.float32) < np.float32(0.01)
        x[hit] *= np.float32(100.0)
        return x
    if law == "lognormal":
        z = _std_normal(rng, shape)
        z *= np.float32(2.0)
        np.exp(z, out=z)
        flat = z.reshape(-1)
        step = 1 << 24
        for i in range(0, flat.size, step):
            neg = rng.integers(0, 2, size=min(step, flat.size - i), dtype=np.uint8).astype(bool)
            seg = flat[i:i + step]
            seg[neg] = -seg[neg]
        return z
    raise ValueError(f"unknown law {law!r}")


# ----------------------------------------------------------------------------- GEMM specs


@dataclass(frozen=True)
class GemmSpec:
    """One GEMM ``C[M][N] = op(A) . op(B)`` of a training step.

    ``a_shape`` / ``b_shape`` are the stored (row-major) shapes: A is ``[M][K]`` or, with
    ``transA``, ``[K][M]``; B is ``[K][N]`` or, with ``transB``, ``[N][K]``. ``a_law`` and
    ``b_law`` are ``(law, kwargs)``. ``a_key`` / ``b_key`` name the logical tensor, so that the
    same tensor (X in forward and backward-weight, W in forward and backward-data) is drawn
    once per configuration. ``fmt_a`` / ``fmt_b`` are plain dicts with the format fields
    (mant_bits, block, tile, rounding, seed, stream_id)."""
    name: str
    transA: int
    transB: int
    M: int
    N: int
    K: int
    a_key: str
    b_key: str
    a_law: Tuple[str, dict]
    b_law: Tuple[str, dict]
    fmt_a: dict = field(default_factory=dict)
    fmt_b: dict = field(default_factory=dict)

    @property
    def a_shape(self):
        return (self.K, self.M) if self.transA else (self.M, self.K)

    @property
    def b_shape(self):
        return (self.N, self.K) if self.transB else (self.K, self.N)

    @property
    def ops(self) -> int:
        return 2 * self.M * self.N * self.K


def _fmt(m, block, tile=0, rounding=0, seed=0, stream_id=0):
    return dict(mant_bits=m, block=block, tile=tile, rounding=rounding, seed=seed,
                stream_id=stream_id)


def _layer_gemms(tag, batch, fin, fout, m, block, w_tile, rounding, seed, x_law, sid0):
    """forward, backward-data and backward-weight GEMMs of one dense layer ``fin -> fout``.

    X is [batch][fin], W is [fin][fout] (stored once, shared by forward and backward-data),
    dY is [batch][fout]. Stream ids: X sid0, W sid0+1, dY sid0+2, whichever GEMM uses them."""
    act = lambda sid: _fmt(m, block, 0, rounding, seed, sid)
    wf = _fmt(m, block, w_tile, rounding, seed, sid0 + 1)
    X = (f"{tag}.X", x_law)
    W = (f"{tag}.W", ("he_weight", {"fan_in": fin}))
    dY = (f"{tag}.dY", ("grad", {}))
    return [
        GemmSpec(f"{tag}.fwd", 0, 0, batch, fout, fin, X[0], W[0], X[1], W[1], act(sid0), wf),
        GemmSpec(f"{tag}.dgrad", 0, 1, batch, fin, fout, dY[0], W[0], dY[1], W[1], act(sid0 + 2), wf),
        GemmSpec(f"{tag}.wgrad", 1, 0, fin, fout, batch, X[0], dY[0], X[1], dY[1], act(sid0), act(sid0 + 2)),
    ]


def config_single_256() -> List[GemmSpec]:
    """Single 256^3 GEMM, N(0,1) inputs from seed 0, 8-bit mantissas, block 32, nearest-even."""
    f = _fmt(8, 32)
    return [GemmSpec("c0.gemm", 0, 0, 256, 256, 256, "c0.A", "c0.B", ("normal", {}), ("normal", {}),
                     f, dict(f, stream_id=1))]


def config_mlp(batch: int = 128) -> List[GemmSpec]:
    """MLP 784-1024-1024-10: 8-bit mantissas, 24x24 weight tiles, activation blocks of 24,
    stochastic rounding with seed 1."""
    out = []
    dims = [784, 1024, 1024, 10]
    for li in range(3):
        out += _layer_gemms(f"c1.l{li}", batch, dims[li], dims[li + 1], 8, 24, 24, 1, 1,
                            ("half_normal", {}), 10 * li)
    return out


def config_resnet_im2col(batch: int = 128) -> List[GemmSpec]:
    """CIFAR-style 3x3 convolutions as im2col GEMMs: 64->64 at 32x32 and 128->128 at 16x16;
    8-bit mantissas, 1-D blocks of 64 along each contraction, nearest-even."""
    out = []
    out += _layer_gemms("c2.conv64", batch * 32 * 32, 64 * 9, 64, 8, 64, 0, 0, 0,
                        ("half_normal", {}), 0)
    out += _layer_gemms("c2.conv128", batch * 16 * 16, 128 * 9, 128, 8, 64, 0, 0, 0,
                        ("half_normal", {}), 10)
    return out


def config_transformer(tokens: int = 4096, hidden: int = 1024) -> List[GemmSpec]:
    """Gate / FFN-up projection hidden->4*hidden and FFN-down 4*hidden->hidden: 12-bit
    mantissas, 64x64 weight tiles, activation blocks of 64, stochastic rounding seed 7."""
    out = []
    out += _layer_gemms("c3.up", tokens, hidden, 4 * hidden, 12, 64, 64, 1, 7, ("outliers", {}), 0)
    out += _layer_gemms("c3.down", tokens, 4 * hidden, hidden, 12, 64, 64, 1, 7, ("outliers", {}), 10)
    return out


def config_sweep(n: int, mant_bits: int = 8, block: int = 128, rounding: int = 0) -> List[GemmSpec]:
    """Square GEMM of the large sweep: log-normal magnitudes (sigma 2), random signs."""
    fa = _fmt(mant_bits, block, 0, rounding, 3, 0)
    fb = _fmt(mant_bits, block, 0, rounding, 3, 1)
    return [GemmSpec(f"c4.n{n}.m{mant_bits}.b{block}.r{rounding}", 0, 0, n, n, n,
                     f"c4.A{n}", f"c4.B{n}", ("lognormal", {}), ("lognormal", {}), fa, fb)]


def materialize(specs: List[GemmSpec], seed: int = 0) -> Dict[str, np.ndarray]:
    """Draw every distinct logical tensor the specs name, once, in stored layout.

    A tensor used with and without a trans flag (X in forward and backward-weight) has one
    stored layout: that of its first use without a trans flag, which is how a framework
    would hold it."""
    shapes: Dict[str, Tuple[Tuple[int, int], Tuple[str, dict]]] = {}
    for sp in specs:
        for key, shape, law, trans in ((sp.a_key, sp.a_shape, sp.a_law, sp.transA),
                                       (sp.b_key, sp.b_shape, sp.b_law, sp.transB)):
            if key in shapes:
                assert shapes[key][0] == shape, (key, shapes[key][0], shape)
            else:
                shapes[key] = (shape, law)
    out = {}
    for salt, (key, (shape, law)) in enumerate(sorted(shapes.items())):
        out[key] = draw(law[0], shape, seed, salt, **law[1])
    return out
