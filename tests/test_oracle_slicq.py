"""Pins for the oracle's sliced form (Sec. 4, slicing paragraph): 50 % overlap, Tukey transition window."""
import numpy as np
import pytest

from oracle import nsgt_oracle as orc


@pytest.mark.parametrize("sl,tr", [(64, 8), (64, 32), (1 << 15, 1 << 13), (256, 2)])
def test_shifted_windows_sum_to_one(sl, tr):
    w = orc.slice_window(sl, tr)
    H = sl // 2
    assert np.allclose(w[:H] + w[H:], 1.0, atol=1e-15)
    assert w[sl // 2] == 1.0 and w[0] == 0.0
    assert np.all((w >= 0) & (w <= 1))
    assert np.allclose(w[1:], w[1:][::-1])          # even about the slice centre


def test_nonzero_count_of_the_streaming_configuration():
    w = orc.slice_window(1 << 15, 1 << 13)
    assert np.count_nonzero(w) == 24575
    assert np.all(w[:4097] == 0) and w[4097] > 0     # sample 0 plus 4096 on the left, 4096 on the right
    assert np.all(w[-4096:] == 0) and w[-4097] > 0


def test_cut_and_overlap_add_is_identity():
    sl, tr, n = 128, 16, 1000
    x = np.random.default_rng(0).standard_normal((2, n))
    sl_x = orc.slicq_cut(x, sl, tr)
    assert sl_x.shape == (2, orc.slicq_num_slices(n, sl), sl)
    assert np.allclose(orc.slicq_overlap_add(sl_x, n), x, atol=1e-14)
    # slice s covers samples [sH - sl/2, sH + sl/2)
    H = sl // 2
    w = orc.slice_window(sl, tr)
    s = 3
    assert np.allclose(sl_x[0, s], x[0, s * H - H: s * H + H] * w)
    assert np.allclose(sl_x[0, 0, :H], 0)            # before the start of the stream


def test_sliced_round_trip():
    """Each slice through T then S, plain overlap-add: reconstructs the stream."""
    sl, tr, n = 512, 64, 2000
    lay = orc.build_layout(fs=8000.0, fmin=200.0, fmax=4000.0, bins_per_octave=12, N=sl, policy=orc.M_SMOOTH)
    x = np.random.default_rng(1).standard_normal(n)
    slices = orc.slicq_cut(x, sl, tr)
    rec = np.stack([orc.synthesise(lay, orc.analyse(lay, s)) for s in slices])
    y = orc.slicq_overlap_add(rec, n)
    assert np.linalg.norm(y - x) <= 1e-10 * np.linalg.norm(x)


def test_latency_is_one_slice():
    # one slice of 65,536 samples at 44.1 kHz (the figure quoted for the principal configuration)
    assert abs(65536 / 44100.0 * 1000.0 - 1486.1) < 0.05


def test_assembled_band_series_places_every_coefficient_once():
    """Re-assembly is a plain overlap-add at hop M/2: an impulse in coefficient m of slice i lands at i M/2 + m and
    nowhere else; constants add to 1 + 1 where two slices overlap; the grand total is kept."""
    lay = orc.build_layout(256.0, 6.0, 128.0, 6, 256, policy=orc.M_MULT4)
    n = 4
    rng = np.random.default_rng(3)
    zero = [[np.zeros(b.M, dtype=np.complex128) for b in lay.bands] for _ in range(n)]
    band, i, m = 5, 2, 3
    zero[i][band][m] = 1.0 + 2.0j
    out = orc.slicq_assemble(lay, zero)
    M = lay.bands[band].M
    assert out[band].shape[-1] == (n + 1) * M // 2
    assert out[band][i * M // 2 + m] == 1.0 + 2.0j and np.count_nonzero(out[band]) == 1
    assert all(np.count_nonzero(o) == 0 for j, o in enumerate(out) if j != band)
    ones = [[np.ones(b.M, dtype=np.complex128) for b in lay.bands] for _ in range(n)]
    for b, o in zip(lay.bands, orc.slicq_assemble(lay, ones)):
        h = b.M // 2
        assert np.all(o[:h] == 1) and np.all(o[h:n * h] == 2) and np.all(o[n * h:] == 1)
    c = [[rng.standard_normal(b.M) + 1j * rng.standard_normal(b.M) for b in lay.bands] for _ in range(n)]
    got = orc.slicq_assemble(lay, c)
    for j in range(len(lay.bands)):
        assert abs(got[j].sum() - sum(c[i][j].sum() for i in range(n))) < 1e-10
