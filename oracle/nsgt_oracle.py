"""fp64 CPU oracle for the invertible constant-Q (NSGT) transform.

THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, double-precision
restatement of what the transform computes, written from the paper's
definitions (Sec. 2 "The invertible transform", Sec. 3 "Packed routing and
arithmetic structure", Sec. 3.2 "Adjoints for training", and the slicing
paragraph of Sec. 4).  It shares no code with the CUDA library and never
imports it; only tests, the smoke check and the CPU-baseline leg of the
benchmark may call it.

Notation follows the paper except for one clash: here ``N`` is the real signal
length and ``Lp = N/2`` the packed length (the paper's ``L``).

Contents
  build_layout          band centres, supports, windows g, lengths M, aggregate
                        weight a_k and dual windows h (Sec. 2; the layout rules
                        the paper leaves open are listed in the docstring)
  build_layout_bands    the same from any list of band centres and widths
  multires_bands        band list of the multi-resolution layout of Sec. 4
  dft_direct / fft_radix2 / long_dft       F_N of Eq. (dft)
  analyse / analyse_band                    Eq. (analysis) + (band-spectrum),
                                            short inverse DFT evaluated DIRECTLY
  synthesise                                Eq. (synthesis)
  analyse_adjoint / synthesise_adjoint      real adjoints of Sec. 3.2
  pack / untangle / retangle                Eq. (pack), (untangle), (retangle)
  slice_window / slicq_*                    sliced form (Sec. 4, slicing paragraph); slicq_assemble lays the
                                            sliced coefficients of each band on one time axis

Parity status: every function here is pinned by tests/test_oracle_*.py against
closed forms, brute-force sums, library routines or identities the paper
states.  The layout RULES of ``build_layout`` (centre rounding, support
strictness, sideband shape, minimum width) are readings of passages the paper
leaves open; for those the header says "parity unpinned against the paper":
they are pinned only by the invariants (cover, sum h g = 1, ST = I) and by the
bandwidth rule's reproduction of the paper's Table 1 lengths.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

HANN = 0
BLACKMAN_HARRIS = 1

M_MULT4 = 0
M_SMOOTH = 1
M_POW2 = 2

_BH = (0.35875, 0.48829, 0.14128, 0.01168)

# The multiple-of-4 length policy is stated for 2^16-sample signals, whose bands stay below 6,400 coefficients.
# A reading for longer transforms: a band beyond this many coefficients takes the next 5-smooth multiple of 4,
# as under M_SMOOTH (any length >= the support keeps the frame painless).
MAX_RAGGED_LENGTH = 12800


# --------------------------------------------------------------------------
# layout (Sec. 2: windows g, lengths M, aggregate weight a_k, duals h)
# --------------------------------------------------------------------------

def window_profile(kind: int, t):
    """Unit-width window profile w(t), |t| < 1/2, peak 1 at t = 0 (scalar or array)."""
    t = np.asarray(t, dtype=np.float64)
    if kind == HANN:
        return 0.5 + 0.5 * np.cos(2.0 * np.pi * t)
    if kind == BLACKMAN_HARRIS:
        a0, a1, a2, a3 = _BH
        return (a0 + a1 * np.cos(2.0 * np.pi * t) + a2 * np.cos(4.0 * np.pi * t)
                + a3 * np.cos(6.0 * np.pi * t))
    raise ValueError("unknown window")


def _is_5_smooth(m: int) -> bool:
    for p in (2, 3, 5):
        while m % p == 0:
            m //= p
    return m == 1


def band_length(S: int, policy: int) -> int:
    """Coefficient count M of a band whose support has S bins (M >= S: painless case)."""
    if policy == M_MULT4 and 4 * ((S + 3) // 4) <= MAX_RAGGED_LENGTH:
        return 4 * ((S + 3) // 4)
    if policy in (M_MULT4, M_SMOOTH):
        m = 4 * ((S + 3) // 4)
        while not _is_5_smooth(m):
            m += 4
        return m
    if policy == M_POW2:
        m = 4
        while m < S:
            m *= 2
        return m
    raise ValueError("unknown length policy")


@dataclass
class Band:
    kc: int                 # centre bin k_lambda
    d: np.ndarray           # support offsets (int64, increasing), bin = kc + d
    g: np.ndarray           # window values on the support (float64)
    M: int                  # number of coefficients
    sideband: int = 0       # 0 regular, 1 DC, 2 Nyquist
    centre_hz: float = 0.0
    h: Optional[np.ndarray] = None   # dual window on the support (0 outside 0..N/2)


@dataclass
class Layout:
    N: int
    fs: float
    bands: List[Band] = field(default_factory=list)
    a: Optional[np.ndarray] = None   # aggregate weight a_k, k = 0..N/2

    @property
    def coeff_count(self) -> int:
        return sum(b.M for b in self.bands)

    @property
    def coeff_offsets(self) -> List[int]:
        off, out = 0, []
        for b in self.bands:
            out.append(off)
            off += b.M
        return out


def finish_layout(lay: Layout) -> Layout:
    """a_k = sum_lambda M g^2 over entries that land on bins 0..N/2; h = M g / a_k (Sec. 2)."""
    N = lay.N
    a = np.zeros(N // 2 + 1)
    for b in lay.bands:
        k = b.kc + b.d
        ok = (k >= 0) & (k <= N // 2)
        np.add.at(a, k[ok], b.M * b.g[ok] ** 2)
    if not np.all(a > 0):
        raise ValueError("windows do not cover every bin (a_k <= 0 somewhere)")
    for b in lay.bands:
        k = b.kc + b.d
        ok = (k >= 0) & (k <= N // 2)
        h = np.zeros_like(b.g)
        h[ok] = b.M * b.g[ok] / a[k[ok]]
        b.h = h
    lay.a = a
    return lay


def support_width(f: float, bins_per_octave: int, N: int, fs: float, min_win: float = 0.0) -> float:
    """Total support width in bins of a band centred on f: (f/Q) N/fs with Q = 1/(2^(1/b) - 2^(-1/b))."""
    b = int(bins_per_octave)
    Q = 1.0 / (math.pow(2.0, 1.0 / b) - math.pow(2.0, -1.0 / b))
    return max(float(min_win), (f / Q) * N / fs)


def constant_q_bands(fs: float, fmin: float, fmax: float, bins_per_octave: int, N: int, min_win: float = 4.0):
    """Centres f_j = fmin 2^(j/b) kept while f_j <= fmax and f_j (1 + 1/(2Q)) <= fs/2, with their
    support widths in bins (Sec. 2: geometric centres, constant Q)."""
    b = int(bins_per_octave)
    Q = 1.0 / (math.pow(2.0, 1.0 / b) - math.pow(2.0, -1.0 / b))
    centres, widths = [], []
    j = 0
    while True:
        f = fmin * math.pow(2.0, j / b)
        if f > fmax or f * (1.0 + 1.0 / (2.0 * Q)) > fs / 2.0:
            break
        centres.append(f)
        widths.append(support_width(f, b, N, fs, min_win))
        j += 1
    return centres, widths


def multires_bands(fs: float, fmin: float, N: int, sections: Sequence[Sequence[int]], min_win: float = 4.0):
    """Multi-resolution band list (Sec. 4, first paragraph): consecutive sections of (octaves, bins per octave);
    section s starts at fmin 2^(octaves before it) and holds octaves*b centres f_start 2^(j/b), each with the
    width f/Q_b of its own resolution.  Returns centres, widths and the octave index of every band (bands of one
    octave share one coefficient length).  A reading: the paper gives the octave counts and resolutions only."""
    centres, widths, octave = [], [], []
    f_start, o = float(fmin), 0
    for n_oct, b in sections:
        for j in range(int(n_oct) * int(b)):
            f = f_start * math.pow(2.0, j / int(b))
            centres.append(f)
            widths.append(support_width(f, int(b), N, fs, min_win))
            octave.append(o + j // int(b))
        f_start *= math.pow(2.0, int(n_oct))
        o += int(n_oct)
    return centres, widths, octave


def build_layout_bands(fs: float, N: int, centres: Sequence[float], widths: Sequence[float],
                       window: int = HANN, policy: int = M_MULT4, groups: Optional[Sequence[int]] = None) -> Layout:
    """Layout from a list of regular bands (centre in Hz, total support width W in bins), low to high.

    Centre bin = floor(f N/fs + 1/2); support = integer offsets with |d| < W/2 (strict); g[d] = w(d / W).
    M follows `policy` from the support size; bands with the same `groups` value share the largest M of
    their group (one coefficient length per octave, Sec. 4).  The DC and Nyquist sidebands are plateau
    windows: 1 in the middle, falling to 0 at the first / last band's centre bin with the mirror image of
    that band's flank.  Then a_k and h as in Sec. 2."""
    if N % 2:
        raise ValueError("N must be even")
    if len(centres) == 0 or len(centres) != len(widths):
        raise ValueError("need one width per centre and at least one band")
    lay = Layout(N=N, fs=float(fs))
    regular: List[Band] = []
    for f, W in zip(centres, widths):
        kc = int(math.floor(f * N / fs + 0.5))
        hw = int(math.ceil(W / 2.0)) - 1          # largest integer strictly below W/2
        d = np.arange(-hw, hw + 1, dtype=np.int64)
        g = window_profile(window, d / W)
        regular.append(Band(kc=kc, d=d, g=g, M=band_length(len(d), policy), centre_hz=float(f)))
    if groups is not None:
        if len(groups) != len(regular):
            raise ValueError("need one group per band")
        biggest = {}
        for bd, gr in zip(regular, groups):
            biggest[gr] = max(biggest.get(gr, 0), bd.M)
        for bd, gr in zip(regular, groups):
            bd.M = biggest[gr]
    k_first, W_first = regular[0].kc, widths[0]
    k_last, W_last = regular[-1].kc, widths[-1]
    if k_first < 2 or N // 2 - k_last < 2:
        raise ValueError("first/last centre too close to DC/Nyquist")

    def plateau(edge: int, W: float) -> Band:
        dd = np.arange(-(edge - 1), edge, dtype=np.int64)
        t = (edge - np.abs(dd)) / W
        gg = np.where(t >= 0.5, 1.0, window_profile(window, 0.5 - np.minimum(t, 0.5)))
        return Band(kc=0, d=dd, g=gg, M=band_length(len(dd), policy))

    dc = plateau(k_first, W_first)
    dc.sideband, dc.kc, dc.centre_hz = 1, 0, 0.0
    ny = plateau(N // 2 - k_last, W_last)
    ny.sideband, ny.kc, ny.centre_hz = 2, N // 2, fs / 2.0
    lay.bands = [dc] + regular + [ny]
    for bd in regular:
        if bd.kc + bd.d[0] < 1 or bd.kc + bd.d[-1] > N // 2 - 1:
            raise ValueError("a regular band reaches DC or Nyquist")
    return finish_layout(lay)


def build_layout(fs: float, fmin: float, fmax: float, bins_per_octave: int, N: int,
                 window: int = HANN, policy: int = M_MULT4, min_win: float = 4.0) -> Layout:
    """Constant-Q band layout on N/2+1 bins.

    What the paper fixes (Sec. 2, Sec. 4): geometric centres with constant Q,
    centres rounded to Fourier bins, real windows whose supports fit in M slots,
    DC and Nyquist sidebands completing the cover, a_k and h as in Sec. 2.
    Readings where it is silent (parity unpinned against the paper):
      * Q = 1/(2^(1/b) - 2^(-1/b)); total support width W = max(min_win, f/Q * N/fs) bins
        (this width rule reproduces every length of the paper's Table 1);
      * centres f_j = fmin 2^(j/b) kept while f_j <= fmax and f_j (1 + 1/(2Q)) <= fs/2;
      * centre bin = floor(f N/fs + 1/2); support = integer offsets with |d| < W/2 (strict);
        g[d] = w(d / W);
      * sidebands are plateau windows: 1 in the middle, falling to 0 at the neighbouring
        band's centre bin with the mirror image of that band's flank.
    """
    centres, widths = constant_q_bands(fs, fmin, fmax, bins_per_octave, N, min_win)
    if not centres:
        raise ValueError("no band fits between fmin and fmax")
    return build_layout_bands(fs, N, centres, widths, window, policy)


# --------------------------------------------------------------------------
# the long DFT F_N (Eq. dft)
# --------------------------------------------------------------------------

def dft_direct(x: np.ndarray) -> np.ndarray:
    """X_k = sum_j x_j exp(-2 pi i k j / n), the definition, O(n^2).  Last axis."""
    x = np.asarray(x)
    n = x.shape[-1]
    w = np.exp(-2j * np.pi * np.arange(n) / n)
    idx = np.outer(np.arange(n), np.arange(n)) % n
    return x.astype(np.complex128) @ w[idx].T


def fft_radix2(x: np.ndarray) -> np.ndarray:
    """Textbook recursive decimation-in-time radix-2 FFT in fp64 (n a power of two).  Last axis."""
    x = np.asarray(x, dtype=np.complex128)
    n = x.shape[-1]
    if n == 1:
        return x.copy()
    if n % 2:
        raise ValueError("length must be a power of two")
    even = fft_radix2(x[..., 0::2])
    odd = fft_radix2(x[..., 1::2])
    tw = np.exp(-2j * np.pi * np.arange(n // 2) / n)
    odd = odd * tw
    return np.concatenate([even + odd, even - odd], axis=-1)


def long_dft(x: np.ndarray) -> np.ndarray:
    n = np.asarray(x).shape[-1]
    if n & (n - 1) == 0:
        return fft_radix2(x)
    return dft_direct(x)


def long_idft(X: np.ndarray) -> np.ndarray:
    """F_n^{-1} = (1/n) F_n^H (Eq. dft)."""
    X = np.asarray(X, dtype=np.complex128)
    return np.conj(long_dft(np.conj(X))) / X.shape[-1]


# --------------------------------------------------------------------------
# direct short DFT over a band's support entries
# --------------------------------------------------------------------------

def _phase_table(M: int) -> np.ndarray:
    return np.exp(2j * np.pi * np.arange(M) / M)


def _direct_band_sum(values: np.ndarray, d: np.ndarray, n: np.ndarray, M: int, sign: int) -> np.ndarray:
    """out[..., i] = sum_j values[..., j] * exp(sign * 2 pi i d_j n_i / M), evaluated term by term."""
    tab = _phase_table(M)
    if sign < 0:
        tab = np.conj(tab)
    out = np.empty(values.shape[:-1] + (len(n),), dtype=np.complex128)
    step = max(1, (1 << 22) // max(1, len(d)))
    for s in range(0, len(n), step):
        nn = n[s:s + step]
        idx = (d[:, None] * nn[None, :]) % M          # exact integers
        out[..., s:s + len(nn)] = values @ tab[idx]
    return out


def _spectrum_at(X: np.ndarray, k: np.ndarray, N: int) -> np.ndarray:
    return X[..., k % N]


# --------------------------------------------------------------------------
# analysis  c_lambda = F_M^{-1} E_lambda diag(g_lambda) F_N x   (Eq. analysis, band-spectrum)
# --------------------------------------------------------------------------

def analyse_band(lay: Layout, X: np.ndarray, band: int, n: Optional[np.ndarray] = None) -> np.ndarray:
    """Coefficients of one band at output indices n (all if None) from the full spectrum X (length N).

    u[d mod M] = g[d] X_{kc+d};  c[n] = (1/M) sum_d u[d mod M] exp(+2 pi i d n / M).
    """
    b = lay.bands[band]
    if n is None:
        n = np.arange(b.M, dtype=np.int64)
    vals = b.g * _spectrum_at(X, b.kc + b.d, lay.N)
    return _direct_band_sum(vals, b.d, np.asarray(n, dtype=np.int64), b.M, +1) / b.M


def analyse(lay: Layout, x: np.ndarray, bands: Optional[Sequence[int]] = None) -> List[np.ndarray]:
    """T x: list over bands (all, or the listed ones) of arrays [..., M_lambda]."""
    x = np.asarray(x, dtype=np.float64)
    X = long_dft(x)
    idx = range(len(lay.bands)) if bands is None else bands
    return [analyse_band(lay, X, i) for i in idx]


def pad_signal(x: np.ndarray, N: int) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    if x.shape[-1] == N:
        return x
    out = np.zeros(x.shape[:-1] + (N,))
    out[..., :x.shape[-1]] = x
    return out


# --------------------------------------------------------------------------
# synthesis  x^ = F_N^{-1} sum_lambda diag(h_lambda) E_lambda^T F_M c_lambda   (Eq. synthesis)
# --------------------------------------------------------------------------

def synthesise(lay: Layout, c: Sequence[np.ndarray], bands: Optional[Sequence[int]] = None) -> np.ndarray:
    """S c.  With `bands`, c lists only those bands and the others contribute nothing."""
    N = lay.N
    lead = np.asarray(c[0]).shape[:-1]
    Xh = np.zeros(lead + (N // 2 + 1,), dtype=np.complex128)
    which = lay.bands if bands is None else [lay.bands[i] for i in bands]
    for b, cb in zip(which, c):
        cb = np.asarray(cb, dtype=np.complex128)
        k = b.kc + b.d
        ok = (k >= 0) & (k <= N // 2)
        # U[m] = sum_n c[n] exp(-2 pi i m n / M) at the slots m = d mod M of the in-range bins
        U = _direct_band_sum(cb, np.arange(b.M, dtype=np.int64), b.d[ok] % b.M, b.M, -1)
        np.add.at(Xh, (Ellipsis, k[ok]), b.h[ok] * U)
    # made real at DC and Nyquist, negative frequencies by conjugate symmetry
    Xh[..., 0] = Xh[..., 0].real
    Xh[..., N // 2] = Xh[..., N // 2].real
    X = np.empty(lead + (N,), dtype=np.complex128)
    X[..., :N // 2 + 1] = Xh
    X[..., N // 2 + 1:] = np.conj(Xh[..., 1:N // 2][..., ::-1])
    return long_idft(X).real


# --------------------------------------------------------------------------
# real adjoints under <u,v> = Re(u^H v)   (Sec. 3.2)
# --------------------------------------------------------------------------

def analyse_adjoint(lay: Layout, ybar: Sequence[np.ndarray], bands: Optional[Sequence[int]] = None) -> np.ndarray:
    """T^dagger ybar = Re( F_N^H sum_lambda diag(g) E^T (1/M) F_M ybar_lambda ), all support entries.
    With `bands`, ybar lists only those bands and the others contribute nothing."""
    N = lay.N
    lead = np.asarray(ybar[0]).shape[:-1]
    V = np.zeros(lead + (N,), dtype=np.complex128)
    which = lay.bands if bands is None else [lay.bands[i] for i in bands]
    for b, yb in zip(which, ybar):
        yb = np.asarray(yb, dtype=np.complex128)
        U = _direct_band_sum(yb, np.arange(b.M, dtype=np.int64), b.d % b.M, b.M, -1)
        np.add.at(V, (Ellipsis, (b.kc + b.d) % N), b.g * U / b.M)
    # F_N^H V = conj(F_N conj V)
    return np.conj(long_dft(np.conj(V))).real


def synthesise_adjoint(lay: Layout, xbar: np.ndarray, bands: Optional[Sequence[int]] = None,
                       n: Optional[Sequence[np.ndarray]] = None) -> List[np.ndarray]:
    """S^dagger xbar: G_k = (w_k/N) [F_N xbar]_k (w = 2, but 1 and real at k = 0, N/2);
    cbar_lambda = M F_M^{-1} E diag(h) G.  With `bands` only those bands are returned; with `n` (one index
    array per returned band) only those output indices of each."""
    N = lay.N
    xbar = np.asarray(xbar, dtype=np.float64)
    X = long_dft(xbar)
    G = np.zeros(X.shape[:-1] + (N // 2 + 1,), dtype=np.complex128)
    G[..., 1:N // 2] = 2.0 * X[..., 1:N // 2] / N
    G[..., 0] = X[..., 0].real / N
    G[..., N // 2] = X[..., N // 2].real / N
    out = []
    which = lay.bands if bands is None else [lay.bands[i] for i in bands]
    for j, b in enumerate(which):
        k = b.kc + b.d
        ok = (k >= 0) & (k <= N // 2)
        vals = b.h[ok] * G[..., k[ok]]
        nn = np.arange(b.M, dtype=np.int64) if n is None else np.asarray(n[j], dtype=np.int64)
        # M * (1/M) sum_d ... : the two factors cancel
        out.append(_direct_band_sum(vals, b.d[ok], nn, b.M, +1))
    return out


# --------------------------------------------------------------------------
# packed real transform identities (Eq. pack, untangle, retangle)
# --------------------------------------------------------------------------

def pack(x: np.ndarray) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    return x[..., 0::2] + 1j * x[..., 1::2]


def untangle(Z: np.ndarray, k: np.ndarray) -> np.ndarray:
    """X_k from the packed spectrum Z = F_Lp z (any integer k)."""
    Lp = Z.shape[-1]
    N = 2 * Lp
    k = np.asarray(k, dtype=np.int64)
    om = np.exp(-2j * np.pi * (k % N) / N)
    return 0.5 * (1 - 1j * om) * Z[..., k % Lp] + 0.5 * (1 + 1j * om) * np.conj(Z[..., (-k) % Lp])


def retangle(Xh: np.ndarray) -> np.ndarray:
    """Z_q, 0 <= q < Lp, from the half spectrum X_0..X_Lp."""
    Lp = Xh.shape[-1] - 1
    q = np.arange(Lp)
    om_c = np.exp(+2j * np.pi * q / (2 * Lp))       # conj(omega_q)
    return 0.5 * ((1 + 1j * om_c) * Xh[..., q] + (1 - 1j * om_c) * np.conj(Xh[..., Lp - q]))


# --------------------------------------------------------------------------
# sliced form (Sec. 4): slices of sl samples, 50 % overlap, Tukey transition window
# --------------------------------------------------------------------------

def slice_window(sl: int, tr: int) -> np.ndarray:
    """w[i] = omega(i - sl/2): 1 on the middle, raised-cosine flanks of tr samples centred on
    +-H/2 (H = sl/2), 0 outside; shifted copies at hop H sum to one."""
    H = sl // 2
    if not (0 < tr <= H):
        raise ValueError("transition must satisfy 0 < tr <= sl/2")
    t = np.abs(np.arange(sl) - sl // 2).astype(np.float64)
    lo, hi = (H - tr) / 2.0, (H + tr) / 2.0
    w = np.zeros(sl)
    w[t <= lo] = 1.0
    mid = (t > lo) & (t < hi)
    w[mid] = 0.5 * (1.0 + np.cos(np.pi * (t[mid] - lo) / tr))
    return w


def slicq_num_slices(n_samples: int, sl: int) -> int:
    """Slices s = 0.. whose span [sH - sl/2, sH + sl/2) meets the stream [0, n_samples)."""
    H = sl // 2
    return (n_samples + H - 1) // H + 1


def slicq_cut(x: np.ndarray, sl: int, tr: int) -> np.ndarray:
    """[..., n_slices, sl]: windowed slices; slice s covers samples [sH - sl/2, sH + sl/2), zeros outside."""
    x = np.asarray(x, dtype=np.float64)
    n = x.shape[-1]
    H = sl // 2
    ns = slicq_num_slices(n, sl)
    w = slice_window(sl, tr)
    padded = np.zeros(x.shape[:-1] + (H + ns * H + sl,))
    padded[..., H:H + n] = x
    out = np.empty(x.shape[:-1] + (ns, sl))
    for s in range(ns):
        out[..., s, :] = padded[..., s * H: s * H + sl] * w
    return out


def slicq_overlap_add(y: np.ndarray, n_samples: int) -> np.ndarray:
    """Plain overlap-add of per-slice reconstructions [..., n_slices, sl] back to n_samples."""
    ns, sl = y.shape[-2], y.shape[-1]
    H = sl // 2
    acc = np.zeros(y.shape[:-2] + (H + ns * H + sl,))
    for s in range(ns):
        acc[..., s * H: s * H + sl] += y[..., s, :]
    return acc[..., H:H + n_samples]


def slicq_assemble(lay: Layout, coeffs: Sequence[Sequence[np.ndarray]]) -> List[np.ndarray]:
    """Re-assembly of sliced coefficients into one time series per band.

    coeffs[i][band] holds the coefficients [..., M] of the i-th of n consecutive slices.  Slice i + 1 starts
    sl/2 samples after slice i, i.e. M/2 coefficient periods later in a band of M coefficients, so band
    lambda's series of length (n + 1) M/2 is the plain overlap-add out[i M/2 + m] += c_i[m].  (A layout of the
    coefficients on a common time axis; sliced coefficients are not the whole-signal coefficients, Sec. 4.)"""
    n = len(coeffs)
    out = []
    for b, band in enumerate(lay.bands):
        M = band.M
        if M % 2:
            raise ValueError("band lengths must be even")
        first = np.asarray(coeffs[0][b])
        acc = np.zeros(first.shape[:-1] + ((n + 1) * (M // 2),), dtype=np.complex128)
        for i in range(n):
            acc[..., i * (M // 2): i * (M // 2) + M] += np.asarray(coeffs[i][b])
        out.append(acc)
    return out
