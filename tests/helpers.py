"""Shared test plumbing: format conversion, host<->device movement, packed-buffer decoding.

Holds no arithmetic of the method beyond decoding the documented packed layout."""
import numpy as np

import oracle


def ofmt(d: dict, **kw) -> "oracle.Format":
    return oracle.Format(**{**d, **kw})


def gfmt(d: dict, **kw):
    from paper_1804_01526_b200 import binding as hb
    return hb.Format(**{**d, **kw})


def to_dev(x: np.ndarray):
    import torch
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def decode_packed(p, lay):
    """Decode the raw packed buffers of a ``binding.Packed`` on the host, checking that every
    byte the layout documents as zero is zero. Returns canonical (q int16 [rows][k], s int8 [rows][nkb])."""
    mant = p.mant.cpu().numpy()
    exps = p.exps.cpu().numpy()
    rows, k, b, bp, nkb, kst = (lay[n] for n in ("rows", "k", "b", "bp", "nkb", "kst"))
    planes, ps, rs = lay["planes"], lay["plane_stride"], lay["rs"]
    pl = [mant[i * ps: i * ps + rows * kst].reshape(rows, kst).astype(np.int16) for i in range(planes)]
    full = pl[0] if planes == 1 else pl[0] * 16 + pl[1]
    if planes == 2:
        assert pl[1].min(initial=0) >= 0 and pl[1].max(initial=0) <= 15
    blocks = full[:, : nkb * bp].reshape(rows, nkb, bp)
    assert not blocks[:, :, b:].any(), "block padding must be zero"
    assert not full[:, nkb * bp:].any(), "row tail must be zero"
    q = blocks[:, :, :b].reshape(rows, nkb * b)[:, :k]
    assert not blocks[:, :, :b].reshape(rows, nkb * b)[:, k:].any(), "ragged block tail must be zero"
    e = exps[: nkb * rs].reshape(nkb, rs)
    assert not e[:, rows:].any(), "exponent padding must be zero"
    return q.astype(np.int16), np.ascontiguousarray(e[:, :rows].T)


def dgrad_filters_view(q1: np.ndarray, s1: np.ndarray, taps: int, c_in: int) -> tuple:
    """Regroup a ``[taps * c_in][c_out]`` array (and its per-row block array) into the filter operand of the
    backward-data convolution, ``[c_in][taps * c_out]``: row ci holds, tap by tap, the row (taps - 1 - tap, ci)
    of the input (filters turned by 180 degrees, feature-map roles swapped). Pure index movement."""
    c_out, nb = q1.shape[1], s1.shape[1]
    q = q1.reshape(taps, c_in, c_out)[::-1].transpose(1, 0, 2).reshape(c_in, taps * c_out)
    s = s1.reshape(taps, c_in, nb)[::-1].transpose(1, 0, 2).reshape(c_in, taps * nb)
    return np.ascontiguousarray(q), np.ascontiguousarray(s)
