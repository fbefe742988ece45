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


# ---- pins for the aggregate weight a_k and the dual windows h (Sec. 2: a_k = sum_lambda M_lambda g^2, h = M g / a)

def _hand_layout():
    """Four bands on N = 16 with unequal lengths, small enough to work out by hand."""
    N = 16
    bands = [
        orc.Band(kc=0, d=np.array([-1, 0, 1]), g=np.array([1.0, 1.0, 1.0]), M=4, sideband=1),
        orc.Band(kc=2, d=np.array([-1, 0, 1]), g=np.array([0.5, 1.0, 0.5]), M=4),
        orc.Band(kc=4, d=np.array([-2, -1, 0, 1, 2]), g=np.array([0.25, 0.5, 1.0, 0.5, 0.25]), M=8),
        orc.Band(kc=8, d=np.array([-2, -1, 0, 1, 2]), g=np.array([0.5, 1.0, 1.0, 1.0, 0.5]), M=8, sideband=2),
    ]
    return orc.finish_layout(orc.Layout(N=N, fs=16.0, bands=bands))


def test_aggregate_weight_and_duals_worked_by_hand():
    """a_k and h of a four-band layout with lengths 4, 4, 8, 8, every value worked out on paper from
    a_k = sum M g^2 (entries on bins 0..N/2 only) and h = M g / a_k.  Dropping or misplacing the factor M changes
    every bin two bands of different length share (1, 2, 3, 6)."""
    lay = _hand_layout()
    # bin:      0    1          2               3          4    5          6                7    8
    want_a = [4.0, 4.0 + 1.0, 4.0 + 8.0 / 16, 1.0 + 2.0, 8.0, 8.0 / 4.0, 8.0 / 16 + 8.0 / 4, 8.0, 8.0]
    assert np.allclose(lay.a, want_a, rtol=0, atol=1e-15)
    want_h = [
        [0.0, 1.0, 0.8],                                   # DC band: the entry on bin -1 has no dual weight
        [0.4, 4.0 / 4.5, 2.0 / 3.0],
        [2.0 / 4.5, 4.0 / 3.0, 1.0, 2.0, 2.0 / 2.5],
        [4.0 / 2.5, 1.0, 1.0, 0.0, 0.0],                    # Nyquist band: entries above N/2 have none
    ]
    for bd, wh in zip(lay.bands, want_h):
        assert np.allclose(bd.h, wh, rtol=0, atol=1e-15)


@pytest.mark.parametrize("kstar", [40, 57, 73, 100])
def test_aggregate_weight_from_analysis_energy(kstar):
    """x_j = cos(2 pi k* j / N) on an interior bin that only regular bands cover: each covering band has
    |c_lambda[n]| = (N/2) g[k* - kc] / M for all n (cosine closed form), so ||c_lambda||^2 = (N^2/4) g^2 / M and
    sum_lambda M^2 ||c_lambda||^2 = (N^2/4) sum_lambda M g^2 = (N^2/4) a_{k*}.  The left side comes from the
    analysis alone (pinned by the time-domain atoms); the right side is the layout's a_k."""
    lay = orc.build_layout(fs=256.0, fmin=6.0, fmax=128.0, bins_per_octave=6, N=256, policy=orc.M_SMOOTH)
    N = lay.N
    covering = [bd for bd in lay.bands if bd.kc + bd.d[0] <= kstar <= bd.kc + bd.d[-1]]
    assert covering and all(bd.sideband == 0 for bd in covering)
    assert len({bd.M for bd in covering}) >= 1
    c = orc.analyse(lay, np.cos(2 * np.pi * kstar * np.arange(N) / N))
    lhs = sum(bd.M ** 2 * np.sum(np.abs(cb) ** 2) for bd, cb in zip(lay.bands, c))
    assert abs(lhs - (N * N / 4.0) * lay.a[kstar]) <= 1e-12 * lhs


def test_dual_is_the_length_weighted_least_squares_inverse():
    """With D = diag(M_lambda) on the coefficients, sum_lambda M^2 T_lambda^H T_lambda = F^H diag(a) F, so the
    synthesis of Sec. 2 with h = M g / a is the weighted least-squares inverse (D T)^+ D of the analysis
    matrix.  Checked column by column on the real matrices of a small layout, for the bands whose support
    touches no sideband's support (the sidebands' entries outside bins 0..N/2 carry no dual weight, which
    is a different, equally exact inverse there).  A dual without the factor M, h = g / sum g^2, is also an
    exact inverse but not this one: it fails here wherever two bands of different length overlap."""
    lay = orc.build_layout(fs=64.0, fmin=6.0, fmax=32.0, bins_per_octave=4, N=64, policy=orc.M_MULT4)
    N, P = lay.N, lay.coeff_count

    def flat(c):
        v = np.concatenate([np.asarray(cb).ravel() for cb in c])
        return np.concatenate([v.real, v.imag])

    def unflat(v):
        z = v[:P] + 1j * v[P:]
        out, o = [], 0
        for bd in lay.bands:
            out.append(z[o:o + bd.M]); o += bd.M
        return out

    T = np.stack([flat(orc.analyse(lay, e)) for e in np.eye(N)], axis=1)            # [2P, N]
    S = np.stack([orc.synthesise(lay, unflat(e)) for e in np.eye(2 * P)], axis=1)   # [N, 2P]
    m = np.concatenate([np.full(bd.M, float(bd.M)) for bd in lay.bands])
    D = np.diag(np.concatenate([m, m]))
    W = np.linalg.pinv(D @ T) @ D
    side_bins = set()
    for bd in lay.bands:
        if bd.sideband:
            side_bins |= set(int(abs(k)) if k <= N // 2 else int(N - k) for k in bd.kc + bd.d)
    checked, lengths, o = 0, set(), 0
    for bd in lay.bands:
        cols = np.r_[o:o + bd.M, P + o:P + o + bd.M]
        o += bd.M
        if bd.sideband or side_bins & set(int(k) for k in bd.kc + bd.d):
            continue
        assert np.allclose(S[:, cols], W[:, cols], rtol=0, atol=1e-13)
        checked += 1
        lengths.add(bd.M)
    assert checked >= 5 and len(lengths) >= 2
