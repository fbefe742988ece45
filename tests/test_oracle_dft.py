"""Pins for the oracle's long DFT and for the packed-spectrum identities (Eq. dft, pack, untangle, retangle)."""
import numpy as np
import pytest

from oracle import nsgt_oracle as orc


def test_direct_dft_closed_forms():
    n = 48
    # impulse at j0: X_k = exp(-2 pi i k j0 / n)
    j0 = 5
    x = np.zeros(n); x[j0] = 1.0
    k = np.arange(n)
    assert np.allclose(orc.dft_direct(x), np.exp(-2j * np.pi * k * j0 / n), atol=1e-13)
    # bin-centred cosine: X_{k*} = X_{n-k*} = n/2, zero elsewhere
    ks = 7
    X = orc.dft_direct(np.cos(2 * np.pi * ks * np.arange(n) / n))
    want = np.zeros(n); want[ks] = want[n - ks] = n / 2
    assert np.allclose(X, want, atol=1e-12)
    # sign convention: a complex exponential exp(+2 pi i k* j / n) lands on bin +k*
    X = orc.dft_direct(np.exp(2j * np.pi * 3 * np.arange(n) / n))
    assert abs(X[3] - n) < 1e-12 and abs(X[n - 3]) < 1e-12


@pytest.mark.parametrize("n", [2, 8, 64, 512, 2048])
def test_radix2_equals_definition(n):
    rng = np.random.default_rng(n)
    x = rng.standard_normal((3, n)) + 1j * rng.standard_normal((3, n))
    assert np.allclose(orc.fft_radix2(x), orc.dft_direct(x), rtol=0, atol=1e-10 * np.sqrt(n))


@pytest.mark.parametrize("n", [1 << 12, 1 << 17])
def test_radix2_equals_library_fft(n):
    rng = np.random.default_rng(n)
    x = rng.standard_normal(n)
    X = orc.long_dft(x)
    ref = np.fft.fft(x)
    assert np.linalg.norm(X - ref) <= 1e-13 * np.linalg.norm(ref)
    assert np.linalg.norm(orc.long_idft(X).imag) <= 1e-13 * np.linalg.norm(x)
    assert np.linalg.norm(orc.long_idft(X).real - x) <= 1e-13 * np.linalg.norm(x)


def test_non_power_of_two_falls_back_to_definition():
    x = np.random.default_rng(0).standard_normal(60)
    assert np.allclose(orc.long_dft(x), np.fft.fft(x), atol=1e-11)


@pytest.mark.parametrize("N", [16, 256, 4096])
def test_untangle_recovers_every_bin(N):
    """Eq. (untangle): any bin of X = F_N x from two bins of the packed spectrum Z = F_{N/2} P x."""
    x = np.random.default_rng(N).standard_normal(N)
    X = np.fft.fft(x)
    Z = np.fft.fft(orc.pack(x))
    k = np.arange(-N, 2 * N)
    assert np.allclose(orc.untangle(Z, k), X[k % N], atol=1e-11 * np.sqrt(N))


@pytest.mark.parametrize("N", [16, 256, 4096])
def test_retangle_inverts_untangle(N):
    """Eq. (retangle): the packed spectrum from the half spectrum, and P^-1 F^-1 of it is the signal."""
    x = np.random.default_rng(N + 1).standard_normal(N)
    Z = np.fft.fft(orc.pack(x))
    Xh = np.fft.rfft(x)
    Zr = orc.retangle(Xh)
    assert np.allclose(Zr, Z, atol=1e-11 * np.sqrt(N))
    z = np.fft.ifft(Zr)
    assert np.allclose(z.real, x[0::2], atol=1e-12) and np.allclose(z.imag, x[1::2], atol=1e-12)


def test_router_weight_identity():
    """Sec. 4: the second router weight g/2 (1 + i w_k) equals g - alpha with alpha = g/2 (1 - i w_k)."""
    N, g = 1024, 0.37
    k = np.arange(N)
    om = np.exp(-2j * np.pi * k / N)
    alpha = 0.5 * g * (1 - 1j * om)
    assert np.allclose(0.5 * g * (1 + 1j * om), g - alpha, atol=1e-16)
