"""Pins for the oracle's band layout: the paper's Table 1 lengths, cover and dual-window identities (Sec. 2, Sec. 4)."""
import math
import os

import numpy as np
import pytest

from oracle import nsgt_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden", "table1_band_lengths.txt")


def _table1():
    rows, total = [], None
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        p = line.split()
        if p[0] == "total":
            total = tuple(int(v) for v in p[1:])
        else:
            rows.append(tuple(int(v) for v in p))
    return rows, total


def _ceil_pow2(v):
    return 1 << int(math.ceil(math.log2(v)))


def test_width_rule_reproduces_table1_lengths():
    """One power-of-two length per octave = largest support in the octave rounded up (Sec. 4);
    the support width rule f/Q with Q = 1/(2^(1/b) - 2^(-1/b)) gives every printed M."""
    rows, total = _table1()
    N, fs = 65536, 44100.0
    coeffs = 0
    for _, nb, _, f_top, M, b in rows:
        assert _ceil_pow2(orc.support_width(float(f_top), b, N, fs)) == M
        coeffs += nb * M
    n_pos, m_dc, m_ny, n_tot = total
    assert sum(r[1] for r in rows) == n_pos
    assert coeffs + m_dc + m_ny == n_tot
    # DC sideband: plateau band reaching the first centre bin (43 Hz -> bin 64): 2*64-1 = 127 -> 128
    lay = orc.build_layout(fs, 43.07, 81.5, 8, N, policy=orc.M_POW2)
    assert lay.bands[0].sideband == 1 and lay.bands[0].M == m_dc
    # one length per octave = the largest per-band power of two in it
    assert max(bd.M for bd in lay.bands[1:-1]) == rows[0][4]


CFGS = [
    # fs, fmin, fmax, b, N, window, policy, bands, sum S, sum M, distinct M
    (44100.0, 32.70, 22050.0, 12, 1 << 16, orc.HANN, orc.M_MULT4, 114, 67290, 67504),
    (22050.0, 20.0, 11025.0, 48, 1 << 17, orc.HANN, orc.M_SMOOTH, 439, 131987, 137060),
    (44100.0, 32.70, 22050.0, 48, 1 << 15, orc.HANN, orc.M_SMOOTH, 453, 33141, 35188),
    (256.0, 6.0, 128.0, 6, 256, orc.HANN, orc.M_MULT4, None, None, None),
    (48000.0, 20.0, 20000.0, 96, 1 << 14, orc.BLACKMAN_HARRIS, orc.M_SMOOTH, None, None, None),
]


@pytest.mark.parametrize("cfg", CFGS)
def test_layout_invariants(cfg):
    fs, fmin, fmax, b, N, win, pol, nb, sS, sM = cfg
    lay = orc.build_layout(fs, fmin, fmax, b, N, window=win, policy=pol)
    if nb is not None:
        assert len(lay.bands) == nb
        assert sum(len(x.d) for x in lay.bands) == sS
        assert lay.coeff_count == sM
    assert np.all(lay.a > 0)
    acc = np.zeros(N // 2 + 1)
    starts, ends = [], []
    for bd in lay.bands:
        k = bd.kc + bd.d
        # painless case: the support fits the band's slots without collision
        assert len(bd.d) <= bd.M
        assert len(np.unique(bd.d % bd.M)) == len(bd.d)
        assert np.all(np.diff(bd.d) == 1) and np.all(bd.g > 0) and np.allclose(bd.g, bd.g[::-1])
        assert bd.M % 4 == 0
        ok = (k >= 0) & (k <= N // 2)
        assert np.all(bd.h[~ok] == 0)
        np.add.at(acc, k[ok], bd.h[ok] * bd.g[ok])
        starts.append(max(0, k[0])); ends.append(min(N // 2, k[-1]))
    # sum_lambda h g = 1 at every bin (Sec. 2)
    assert np.allclose(acc, 1.0, atol=1e-13)
    # bands sorted by centre have monotone support starts and ends
    assert all(np.diff(starts) >= 0) and all(np.diff(ends) >= 0)
    assert lay.bands[0].sideband == 1 and lay.bands[-1].sideband == 2
    assert lay.bands[0].kc == 0 and lay.bands[-1].kc == N // 2


def test_length_policies():
    assert orc.band_length(3, orc.M_MULT4) == 4
    assert orc.band_length(1437, orc.M_MULT4) == 1440
    assert orc.band_length(1441, orc.M_SMOOTH) == 1500   # 1444..1496 have a prime factor > 5
    assert orc.band_length(14487, orc.M_SMOOTH) == 14580
    assert orc.band_length(129, orc.M_POW2) == 256
    for S in range(1, 3000, 7):
        m = orc.band_length(S, orc.M_SMOOTH)
        assert m >= S and m % 4 == 0
        r = m
        for p in (2, 3, 5):
            while r % p == 0:
                r //= p
        assert r == 1


def test_window_profiles():
    assert orc.window_profile(orc.HANN, 0.0) == 1.0
    assert abs(orc.window_profile(orc.HANN, 0.5)) < 1e-16
    assert abs(orc.window_profile(orc.HANN, 0.25) - 0.5) < 1e-16
    assert abs(orc.window_profile(orc.BLACKMAN_HARRIS, 0.0) - 1.0) < 1e-15
    assert abs(orc.window_profile(orc.BLACKMAN_HARRIS, 0.5) - 6e-5) < 1e-12   # a0-a1+a2-a3
    # Hann flanks of neighbouring bands are power complementary: w(t)^2 + w(1/2 - t)^2 >= 1/2
    t = np.linspace(0, 0.5, 101)
    s = orc.window_profile(orc.HANN, t) ** 2 + orc.window_profile(orc.HANN, 0.5 - t) ** 2
    assert s.min() >= 0.5 - 1e-12


SECTIONS = [(3, 8), (4, 16), (2, 32)]      # octaves, bands per octave (Sec. 4, first paragraph)


def test_multires_layout_reproduces_table1():
    """The multi-resolution band list with one power-of-two length per octave gives the printed band counts,
    per-octave lengths, sideband lengths and coefficient total of Table 1 (Sec. 4)."""
    rows, total = _table1()
    N, fs = 65536, 44100.0
    c, w, octave = orc.multires_bands(fs, fs / 1024.0, N, SECTIONS)
    lay = orc.build_layout_bands(fs, N, c, w, orc.HANN, orc.M_POW2, octave)
    n_pos, m_dc, m_ny, n_tot = total
    assert len(c) == n_pos and len(lay.bands) == n_pos + 2
    assert lay.bands[0].M == m_dc and lay.bands[-1].M == m_ny and lay.coeff_count == n_tot
    for o, (_, nb, f_lo, f_hi, M, b) in enumerate(rows):
        mine = [bd for bd, oo in zip(lay.bands[1:-1], octave) if oo == o]
        assert len(mine) == nb and all(bd.M == M for bd in mine)
        # the printed centres are the cited layout's (stretched so that the last centre nears Nyquist); this
        # reading stays within one band step of them
        step = 2.0 ** (1.0 / b)
        assert 1 / step < mine[0].centre_hz / f_lo < step and 1 / step < mine[-1].centre_hz / f_hi < step
        # resolution of the octave: neighbouring centres a factor 2^(1/b) apart
        assert np.allclose(np.diff(np.log2([bd.centre_hz for bd in mine])), 1.0 / b)
    # supports nest where the resolution doubles: the cover of a bin need not be a contiguous band range
    acc = np.zeros(N // 2 + 1)
    for bd in lay.bands:
        k = bd.kc + bd.d
        ok = (k >= 0) & (k <= N // 2)
        assert len(bd.d) <= bd.M
        np.add.at(acc, k[ok], bd.h[ok] * bd.g[ok])
    assert np.allclose(acc, 1.0, atol=1e-13)


def test_band_list_builder_matches_constant_q():
    """build_layout is build_layout_bands on the constant-Q list; groups only ever raise M to the group's largest."""
    fs, N = 22050.0, 1 << 13
    c, w = orc.constant_q_bands(fs, 40.0, fs / 2, 12, N)
    a = orc.build_layout(fs, 40.0, fs / 2, 12, N, policy=orc.M_SMOOTH)
    b = orc.build_layout_bands(fs, N, c, w, orc.HANN, orc.M_SMOOTH)
    assert [(x.kc, x.M, len(x.d)) for x in a.bands] == [(x.kc, x.M, len(x.d)) for x in b.bands]
    assert all(np.array_equal(x.g, y.g) and np.array_equal(x.h, y.h) for x, y in zip(a.bands, b.bands))
    # spacing: f_{j+1} / f_j = 2^(1/12); width = f/Q bins with Q = 1/(2^(1/12) - 2^(-1/12)) = f_j / (f_{j+1} - f_{j-1})
    assert np.allclose(np.array(c[1:]) / np.array(c[:-1]), 2 ** (1 / 12))
    assert np.allclose(np.array(w[1:-1]), np.maximum(4.0, (np.array(c[2:]) - np.array(c[:-2])) * N / fs))   # min_win = 4
    assert max(w) > 100
    groups = [j // 12 for j in range(len(c))]
    g = orc.build_layout_bands(fs, N, c, w, orc.HANN, orc.M_SMOOTH, groups)
    for j, (x, y) in enumerate(zip(b.bands[1:-1], g.bands[1:-1])):
        same = [b.bands[1 + i].M for i in range(len(c)) if groups[i] == groups[j]]
        assert y.M == max(same) >= x.M
