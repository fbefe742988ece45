"""Pins for the oracle's analysis, synthesis and adjoints (Sec. 2, Sec. 3.2).

Each test compares the oracle with something other than itself: brute-force time-domain atoms,
closed forms for a bin-centred cosine, numpy.fft as a library routine on slot-placed spectra,
the perfect-reconstruction identity ST = I, an energy invariant, and the adjoint identity
<Tx, y> = <x, T^dagger y> under the real inner product Re(u^H v)."""
import numpy as np
import pytest

from oracle import nsgt_oracle as orc

SMALL = dict(fs=256.0, fmin=6.0, fmax=128.0, bins_per_octave=6, N=256)


def _small_layout(policy=orc.M_MULT4, window=orc.HANN):
    return orc.build_layout(window=window, policy=policy, **SMALL)


def _rdot(a_list, b_list):
    return sum(float(np.real(np.vdot(a, b))) for a, b in zip(a_list, b_list))


def test_time_domain_atoms_bruteforce():
    """c_lambda[n] = <x, phi_{lambda,n}> with the atom written out in the time domain (N = 256)."""
    lay = _small_layout()
    N = lay.N
    x = np.random.default_rng(1).standard_normal(N)
    c = orc.analyse(lay, x)
    j = np.arange(N)
    for bd, cb in zip(lay.bands, c):
        for n in range(0, bd.M, max(1, bd.M // 5)):
            acc = 0.0 + 0.0j
            for di, gi in zip(bd.d, bd.g):
                # conj(atom)[j] = (1/M) g e^{-2 pi i (kc+d) j / N} e^{+2 pi i d n / M}
                acc += gi * np.exp(2j * np.pi * di * n / bd.M) * np.sum(x * np.exp(-2j * np.pi * (bd.kc + di) * j / N))
            acc /= bd.M
            assert abs(acc - cb[n]) <= 1e-11 * (1 + abs(acc))


@pytest.mark.parametrize("kstar", [9, 40, 100, 127])
def test_cosine_closed_form(kstar):
    """x_j = cos(2 pi k* j / N)  =>  c_lambda[n] = (N/2)(g[k*-kc]/M) exp(2 pi i (k*-kc) n / M) on bands covering k*."""
    lay = _small_layout()
    N = lay.N
    x = np.cos(2 * np.pi * kstar * np.arange(N) / N)
    c = orc.analyse(lay, x)
    hit = 0
    for bd, cb in zip(lay.bands, c):
        want = np.zeros(bd.M, dtype=complex)
        for ks in (kstar, -kstar):           # the cosine also has the bin -k*; only sidebands can see it
            dd = ks - bd.kc
            if bd.sideband == 2:
                dd = (ks % N) - bd.kc
            pos = np.nonzero(bd.d == dd)[0]
            if len(pos):
                hit += 1
                want += (N / 2) * (bd.g[pos[0]] / bd.M) * np.exp(2j * np.pi * dd * np.arange(bd.M) / bd.M)
        assert np.allclose(cb, want, atol=1e-11)
    assert hit >= 1


@pytest.mark.parametrize("policy", [orc.M_MULT4, orc.M_SMOOTH, orc.M_POW2])
def test_library_fft_on_slot_placed_spectrum(policy):
    """c_lambda = ifft(u_lambda) with u_lambda[d mod M] = g X_{kc+d}; synthesis through fft + irfft."""
    lay = _small_layout(policy)
    N = lay.N
    rng = np.random.default_rng(2)
    x = rng.standard_normal((2, N))
    X = np.fft.fft(x)
    c = orc.analyse(lay, x)
    for bd, cb in zip(lay.bands, c):
        u = np.zeros((2, bd.M), dtype=complex)
        u[:, bd.d % bd.M] = bd.g * X[:, (bd.kc + bd.d) % N]
        assert np.allclose(cb, np.fft.ifft(u, axis=-1), atol=1e-12)
    # synthesis of ARBITRARY (not analysed) coefficients
    y = [rng.standard_normal((2, bd.M)) + 1j * rng.standard_normal((2, bd.M)) for bd in lay.bands]
    Xh = np.zeros((2, N // 2 + 1), dtype=complex)
    for bd, yb in zip(lay.bands, y):
        U = np.fft.fft(yb, axis=-1)
        k = bd.kc + bd.d
        ok = (k >= 0) & (k <= N // 2)
        Xh[:, k[ok]] += bd.h[ok] * U[:, (bd.d % bd.M)[ok]]
    assert np.allclose(orc.synthesise(lay, y), np.fft.irfft(Xh, N, axis=-1), atol=1e-12)


def test_single_full_band_is_identity():
    """One band with g = 1 on every bin, M = N, centre 0: the slot map is the identity and c = x."""
    N = 64
    d = np.arange(-N // 2 + 1, N // 2 + 1, dtype=np.int64)
    lay = orc.Layout(N=N, fs=1.0, bands=[orc.Band(kc=0, d=d, g=np.ones(N), M=N)])
    orc.finish_layout(lay)
    x = np.random.default_rng(3).standard_normal(N)
    c = orc.analyse(lay, x)[0]
    assert np.allclose(c, x, atol=1e-12)
    assert np.allclose(orc.synthesise(lay, [c]), x, atol=1e-12)


def test_energy_invariant():
    """sum_lambda M^2 ||c_lambda||^2 = sum over all support entries of M g^2 |X_k|^2 (Parseval per band)."""
    lay = _small_layout()
    N = lay.N
    x = np.random.default_rng(4).standard_normal(N)
    X = np.fft.fft(x)
    c = orc.analyse(lay, x)
    lhs = sum(bd.M ** 2 * np.sum(np.abs(cb) ** 2) for bd, cb in zip(lay.bands, c))
    rhs = sum(bd.M * np.sum(bd.g ** 2 * np.abs(X[(bd.kc + bd.d) % N]) ** 2) for bd in lay.bands)
    assert abs(lhs - rhs) <= 1e-12 * rhs


@pytest.mark.parametrize("args", [
    dict(SMALL, window=orc.HANN, policy=orc.M_MULT4),
    dict(SMALL, window=orc.BLACKMAN_HARRIS, policy=orc.M_SMOOTH),
    dict(fs=22050.0, fmin=20.0, fmax=11025.0, bins_per_octave=48, N=4096, window=orc.HANN, policy=orc.M_SMOOTH),
    dict(fs=44100.0, fmin=32.70, fmax=22050.0, bins_per_octave=12, N=1 << 14, window=orc.HANN, policy=orc.M_MULT4),
])
def test_perfect_reconstruction(args):
    """ST = I on real signals (Sec. 2), round-trip error <= 1e-10 relative."""
    lay = orc.build_layout(**args)
    x = np.random.default_rng(5).standard_normal((2, lay.N))
    xr = orc.synthesise(lay, orc.analyse(lay, x))
    assert np.linalg.norm(xr - x) <= 1e-10 * np.linalg.norm(x)


@pytest.mark.parametrize("N,b", [(256, 6), (1024, 12), (4096, 24)])
def test_adjoint_identities(N, b):
    """<Tx, y> = <x, T'y> and <Sy, xb> = <y, S'xb> under Re(u^H v), to 1e-12 relative (Sec. 3.2)."""
    lay = orc.build_layout(fs=float(N), fmin=6.0 * N / 256, fmax=N / 2.0, bins_per_octave=b, N=N,
                           window=orc.HANN, policy=orc.M_SMOOTH)
    rng = np.random.default_rng(N)
    x = rng.standard_normal(N)
    xb = rng.standard_normal(N)
    y = [rng.standard_normal(bd.M) + 1j * rng.standard_normal(bd.M) for bd in lay.bands]
    Tx = orc.analyse(lay, x)
    Tty = orc.analyse_adjoint(lay, y)
    lhs, rhs = _rdot(Tx, y), float(np.dot(x, Tty))
    assert abs(lhs - rhs) <= 1e-12 * max(abs(lhs), np.linalg.norm(x) * np.linalg.norm(Tty))
    Sy = orc.synthesise(lay, y)
    Stx = orc.synthesise_adjoint(lay, xb)
    lhs, rhs = float(np.dot(Sy, xb)), _rdot(y, Stx)
    assert abs(lhs - rhs) <= 1e-12 * max(abs(lhs), np.linalg.norm(Sy) * np.linalg.norm(xb))


def test_adjoints_equal_transposed_matrices():
    """Tiny case: assemble T and S as real matrices column by column and compare the adjoints with
    their transposes entry by entry (catches a wrong weight at DC/Nyquist that a random dot product
    could hide)."""
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
    Tt = np.stack([orc.analyse_adjoint(lay, unflat(e)) for e in np.eye(2 * P)], axis=1)   # [N, 2P]
    St = np.stack([flat(orc.synthesise_adjoint(lay, e)) for e in np.eye(N)], axis=1)      # [2P, N]
    assert np.allclose(Tt, T.T, atol=1e-12)
    assert np.allclose(St, S.T, atol=1e-12)
    assert np.allclose(S @ T, np.eye(N), atol=1e-12)


def test_sampled_outputs_match_full():
    lay = _small_layout()
    x = np.random.default_rng(6).standard_normal(lay.N)
    X = orc.long_dft(x)
    for i, bd in enumerate(lay.bands):
        n = np.array([0, bd.M - 1, bd.M // 3])
        assert np.allclose(orc.analyse_band(lay, X, i, n), orc.analyse_band(lay, X, i)[n], atol=1e-13)


def test_zero_padding_is_plain_padding():
    lay = _small_layout()
    x = np.random.default_rng(7).standard_normal(200)
    xp = orc.pad_signal(x, lay.N)
    assert xp.shape[-1] == lay.N and np.all(xp[200:] == 0) and np.all(xp[:200] == x)


def _multires_small():
    fs, N = 4096.0, 4096
    c, w, octave = orc.multires_bands(fs, 40.0, N, [(2, 4), (2, 8), (1, 16)])
    return orc.build_layout_bands(fs, N, c, w, orc.HANN, orc.M_POW2, octave)


def _irregular_small():
    """A band list that is not constant-Q: centres on a linear-then-geometric grid, widths reaching the neighbours."""
    fs, N = 2048.0, 2048
    c = list(np.arange(24.0, 200.0, 16.0)) + list(200.0 * 2 ** (np.arange(0, 17) / 8.0))
    c = [f for f in c if f < 820.0]
    w = [2.0 * (c[min(i + 1, len(c) - 1)] - c[max(i - 1, 0)]) * N / fs / (2 if 0 < i < len(c) - 1 else 1) for i in range(len(c))]
    return orc.build_layout_bands(fs, N, c, w, orc.BLACKMAN_HARRIS, orc.M_SMOOTH)


@pytest.mark.parametrize("make", [_multires_small, _irregular_small])
def test_band_list_layouts_reconstruct_and_are_adjoint(make):
    """ST = I and both adjoint identities on layouts built from explicit band lists (nested supports where the
    resolution changes; Sec. 2 needs only a cover with a_k > 0)."""
    lay = make()
    rng = np.random.default_rng(11)
    x = rng.standard_normal(lay.N)
    Tx = orc.analyse(lay, x)
    xr = orc.synthesise(lay, Tx)
    assert np.linalg.norm(xr - x) <= 1e-10 * np.linalg.norm(x)
    y = [rng.standard_normal(bd.M) + 1j * rng.standard_normal(bd.M) for bd in lay.bands]
    xb = rng.standard_normal(lay.N)
    Tty = orc.analyse_adjoint(lay, y)
    lhs, rhs = _rdot(Tx, y), float(np.dot(x, Tty))
    assert abs(lhs - rhs) <= 1e-12 * max(abs(lhs), np.linalg.norm(x) * np.linalg.norm(Tty))
    Sy, Stx = orc.synthesise(lay, y), orc.synthesise_adjoint(lay, xb)
    lhs, rhs = float(np.dot(Sy, xb)), _rdot(y, Stx)
    assert abs(lhs - rhs) <= 1e-12 * max(abs(lhs), np.linalg.norm(Sy) * np.linalg.norm(xb))
    # cosine closed form on a bin where the resolution changes: every covering band sees g[k* - kc]
    kstar = lay.bands[len(lay.bands) // 2].kc + 1
    cx = orc.analyse(lay, np.cos(2 * np.pi * kstar * np.arange(lay.N) / lay.N))
    for bd, cb in zip(lay.bands, cx):
        d = kstar - bd.kc
        n = np.arange(bd.M)
        if bd.sideband == 0 and bd.d[0] <= d <= bd.d[-1]:
            want = (lay.N / 2) * (bd.g[d - bd.d[0]] / bd.M) * np.exp(2j * np.pi * d * n / bd.M)
            assert np.max(np.abs(cb - want)) < 1e-9
        elif bd.sideband == 0:
            assert np.max(np.abs(cb)) < 1e-9
