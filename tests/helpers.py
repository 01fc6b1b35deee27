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
