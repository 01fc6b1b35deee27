"""Pins of the oracle's counter-based random stream (Philox4x32-10, 16-bit draws)."""
import os

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answers():
    # Known-answer vectors published with the generator (see the header of the fixture).
    n = 0
    for line in open(GOLDEN):
        line = line.split("#")[0].split()
        if not line:
            continue
        w = [int(t, 16) for t in line]
        out = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(v) for v in out] == w[6:10]
        n += 1
    assert n >= 3


def test_draw_mapping_uses_every_half_word_once():
    # The 8 elements of one counter group take the 8 distinct 16-bit halves of one call.
    seed, sid = 0x123456789ABCDEF0, 5
    for g in (0, 1, 77, (1 << 33) + 3):
        ctr = [g & 0xFFFFFFFF, g >> 32, sid, 0]
        key = [seed & 0xFFFFFFFF, seed >> 32]
        w = [int(v) for v in oracle.philox4x32_10(ctr, key)]
        halves = []
        for word in w:
            halves += [word & 0xFFFF, word >> 16]
        got = [oracle.sr_draw(seed, sid, 8 * g + i) for i in range(8)]
        assert got == halves


def test_draws_depend_on_seed_stream_and_index():
    base = [oracle.sr_draw(1, 0, L) for L in range(64)]
    assert base != [oracle.sr_draw(2, 0, L) for L in range(64)]
    assert base != [oracle.sr_draw(1, 1, L) for L in range(64)]
    assert base == [oracle.sr_draw(1, 0, L) for L in range(64)]
    assert base != [oracle.sr_draw(1 + (1 << 32), 0, L) for L in range(64)]


def test_draws_are_uniform_chi_square():
    # 2^18 draws into 256 bins of the top byte and 256 bins of the low byte.
    n = 1 << 18
    d = np.array([oracle.sr_draw(42, 3, L) for L in range(n)], dtype=np.int64)
    assert d.min() >= 0 and d.max() < 65536
    for v in (d >> 8, d & 0xFF):
        c = np.bincount(v, minlength=256).astype(np.float64)
        chi2 = ((c - n / 256) ** 2 / (n / 256)).sum()
        # 255 degrees of freedom: mean 255, sd 22.6; 6 sd either side.
        assert 255 - 6 * 22.6 < chi2 < 255 + 6 * 22.6
