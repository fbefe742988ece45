"""GPU tests of the two-pass path for bands too long for one CTA's shared memory."""
import os

import numpy as np
import pytest

import workloads as wl
from helpers import band_rel_errors, library_plan, oracle_layout, small_workload, snr_db, split_bands
from oracle import nsgt_oracle as orc

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("channels", [1, 4, 12])
def test_two_pass_bands_match_oracle_with_a_lowered_cap(channels):
    """With the per-CTA cap lowered, every band above 600 coefficients takes the two-pass kernels; all four
    transforms are then compared with the oracle in full.  The batch sizes make the launcher pick each of its
    three tile widths (the fewer work items, the narrower the tiles)."""
    w = small_workload("forced_two_pass", N=1 << 14, valid_len=15000, fs=44100.0, fmin=32.70, fmax=22050.0,
                       bins_per_octave=12, m_policy=wl.M_SMOOTH, channels=channels, kind="noise_sines")
    plan = library_plan(w, max_cta_elems=600)
    lay = oracle_layout(w)
    assert max(b.M for b in lay.bands) > 600
    x = wl.make_signal(w)
    y = wl.make_cotangent(w, lay.coeff_count)
    c = plan.analyse(_dev(x), valid_len=w.valid_len)
    errs = band_rel_errors(lay, c.cpu().numpy(), orc.analyse(lay, orc.pad_signal(x, w.N)))
    assert errs.max() <= 1e-5, (int(errs.argmax()), errs.max())
    xr = plan.synthesise(c, valid_len=w.valid_len).cpu().numpy()
    assert snr_db(x, xr).min() >= 120.0
    ybands = split_bands(lay, y.astype(np.complex128))
    got = plan.synthesise(_dev(y), valid_len=w.valid_len).cpu().numpy()
    want = orc.synthesise(lay, ybands)[..., :w.valid_len]
    assert (np.linalg.norm(got - want, axis=-1) / np.linalg.norm(want, axis=-1)).max() <= 1e-5
    got = plan.analyse_adjoint(_dev(y), valid_len=w.valid_len).cpu().numpy()
    want = orc.analyse_adjoint(lay, ybands)[..., :w.valid_len]
    assert (np.linalg.norm(got - want, axis=-1) / np.linalg.norm(want, axis=-1)).max() <= 1e-5
    cb = plan.synthesise_adjoint(_dev(x), valid_len=w.valid_len).cpu().numpy()
    errs = band_rel_errors(lay, cb, orc.synthesise_adjoint(lay, orc.pad_signal(x, w.N)))
    assert errs.max() <= 1e-5
    plan.close()


def test_wide_nyquist_sideband():
    """fmax well below Nyquist makes the Nyquist sideband tens of thousands of coefficients long."""
    w = small_workload("wide_nyquist", N=1 << 18, valid_len=(1 << 18) - 999, fs=48000.0, fmin=20.0, fmax=20000.0,
                       bins_per_octave=24, m_policy=wl.M_SMOOTH, window=wl.WIN_BLACKMAN_HARRIS, channels=2,
                       kind="noise_sines")
    lay = oracle_layout(w)
    assert lay.bands[-1].M > 40000
    plan = library_plan(w)
    x = wl.make_signal(w)
    xd = _dev(x)
    c = plan.analyse(xd, valid_len=w.valid_len)
    cn = c.cpu().numpy()
    X = orc.long_dft(orc.pad_signal(x, w.N))
    rng = np.random.default_rng(3)
    offs = lay.coeff_offsets
    for i in (0, 1, len(lay.bands) // 2, len(lay.bands) - 2, len(lay.bands) - 1):
        bd = lay.bands[i]
        n = np.unique(np.concatenate([[0, bd.M - 1], rng.integers(0, bd.M, 96)]))
        want = orc.analyse_band(lay, X, i, n)
        got = cn[:, offs[i] + n]
        rel = np.linalg.norm(got - want, axis=-1) / np.linalg.norm(want, axis=-1)
        assert rel.max() <= 1e-5, (i, rel)
    xr = plan.synthesise(c, valid_len=w.valid_len)
    assert snr_db(x, xr.cpu().numpy()).min() >= 120.0
    # adjoint identities with every operand from the kernels (covers the sideband fold in the two-pass path)
    y = wl.make_cotangent(w, lay.coeff_count)
    yd = _dev(y)
    Tty = plan.analyse_adjoint(yd, valid_len=w.valid_len).cpu().numpy().astype(np.float64)
    Sy = plan.synthesise(yd, valid_len=w.valid_len).cpu().numpy().astype(np.float64)
    Stx = plan.synthesise_adjoint(xd, valid_len=w.valid_len).cpu().numpy().astype(np.complex128)
    Tx, y64, x64 = cn.astype(np.complex128), y.astype(np.complex128), x.astype(np.float64)
    for ch in range(w.channels):
        lhs, rhs = np.real(np.vdot(Tx[ch], y64[ch])), np.dot(x64[ch], Tty[ch])
        assert abs(lhs - rhs) <= 2e-5 * np.linalg.norm(Tx[ch]) * np.linalg.norm(y64[ch])
        lhs, rhs = np.dot(Sy[ch], x64[ch]), np.real(np.vdot(y64[ch], Stx[ch]))
        assert abs(lhs - rhs) <= 2e-5 * np.linalg.norm(Sy[ch]) * np.linalg.norm(x64[ch])
    plan.close()
