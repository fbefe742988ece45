"""Seeded synthetic inputs and the five workload descriptions.

This module only DESCRIBES workloads and DRAWS input signals; it holds none of
the transform's arithmetic (no windows, no band layout, no DFT of the method).
Both the CPU oracle's tests and the CUDA library's tests/benchmark take their
inputs from here so that the two sides see identical data.

All signals are generated in fp64 with numpy's PCG64 and cast to fp32.
numpy.fft is used here only to colour noise (pink spectrum), which is input
generation, not part of the transform under test.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional

import numpy as np

WIN_HANN = 0
WIN_BLACKMAN_HARRIS = 1
M_MULT4 = 0
M_SMOOTH = 1
M_POW2 = 2


@dataclass(frozen=True)
class Workload:
    name: str
    fs: float
    fmin: float
    fmax: float
    bins_per_octave: int
    N: int                 # transform length (power of two)
    valid_len: int         # true samples per channel (rest is implicit zero padding)
    channels: int          # batch x channels, flattened
    window: int
    m_policy: int
    seed: int
    kind: str              # which signal recipe
    min_win: float = 4.0
    # sliced streaming only
    slice_len: int = 0
    transition: int = 0
    stream_len: int = 0
    # band-list layouts: consecutive sections of (octaves, bands per octave) starting at fmin with one coefficient
    # length per octave (the multi-resolution layout), or explicit (centre Hz, width in bins) pairs
    sections: tuple = ()
    bands: tuple = ()


CONFIGS = {
    # single mono signal, white noise + 5 sinusoids
    "config1": Workload("config1", 44100.0, 32.70, 22050.0, 12, 1 << 16, 1 << 16, 1,
                        WIN_HANN, M_MULT4, 1001, "noise_sines"),
    # 16 stereo clips of 10 s: pink noise + two linear chirps
    "config2": Workload("config2", 44100.0, 32.70, 22050.0, 24, 1 << 19, 441000, 32,
                        WIN_HANN, M_SMOOTH, 1002, "pink_chirps"),
    # 64 mono clips of 4 s at 22.05 kHz: white noise (forward + analysis adjoint)
    "config3": Workload("config3", 22050.0, 20.0, 11025.0, 48, 1 << 17, 88200, 64,
                        WIN_HANN, M_SMOOTH, 1003, "white"),
    # one 60 s signal at 48 kHz: AM/FM partials + noise, Blackman-Harris
    "config4": Workload("config4", 48000.0, 20.0, 20000.0, 96, 1 << 22, 2880000, 1,
                        WIN_BLACKMAN_HARRIS, M_SMOOTH, 1004, "amfm_partials"),
    # 5 min stereo stream, slices of 2^15 with transition 2^13
    "config5": Workload("config5", 44100.0, 32.70, 22050.0, 48, 1 << 15, 1 << 15, 2,
                        WIN_HANN, M_SMOOTH, 1005, "pink_notes",
                        slice_len=1 << 15, transition=1 << 13, stream_len=300 * 44100),
    # the paper's principal configuration (its Table 1): one slice of 2^16 samples, 3/4/2 octaves at 8/16/32 bands per
    # octave, one power-of-two length per octave; the batch is swept by the benchmark
    "table1": Workload("table1", 44100.0, 44100.0 / 1024.0, 22050.0, 0, 1 << 16, 1 << 16, 1,
                       WIN_HANN, M_POW2, 1006, "noise_sines", sections=((3, 8), (4, 16), (2, 32))),
}


def scaled(w: Workload, channels: Optional[int] = None, stream_len: Optional[int] = None) -> Workload:
    """Same workload with fewer channels / a shorter stream (for tests the oracle finishes quickly)."""
    kw = {}
    if channels is not None:
        kw["channels"] = channels
    if stream_len is not None:
        kw["stream_len"] = stream_len
    return replace(w, **kw)


def _pink(rng: np.random.Generator, n: int, rms: float) -> np.ndarray:
    white = rng.standard_normal(n)
    spec = np.fft.rfft(white)
    k = np.arange(len(spec), dtype=np.float64)
    k[0] = 1.0
    spec = spec / np.sqrt(k)
    spec[0] = 0.0
    y = np.fft.irfft(spec, n)
    return y * (rms / np.sqrt(np.mean(y * y)))


def make_signal(w: Workload, n_channels: Optional[int] = None, length: Optional[int] = None) -> np.ndarray:
    """[channels, length] float32.  Channel c is drawn from its own stream (seed, c) so that a
    subset of channels is a prefix of the full batch."""
    C = w.channels if n_channels is None else n_channels
    n = (w.stream_len or w.valid_len) if length is None else length
    out = np.empty((C, n), dtype=np.float32)
    t = np.arange(n, dtype=np.float64) / w.fs
    for c in range(C):
        rng = np.random.Generator(np.random.PCG64([w.seed, c]))
        if w.kind == "noise_sines":
            x = 0.1 * rng.standard_normal(n)
            for _ in range(5):
                f = np.exp(rng.uniform(np.log(w.fmin), np.log(0.45 * w.fs)))
                ph = rng.uniform(0.0, 2.0 * np.pi)
                x += 0.2 * np.cos(2.0 * np.pi * f * t + ph)
        elif w.kind == "white":
            x = 0.1 * rng.standard_normal(n)
        elif w.kind == "pink_chirps":
            x = _pink(rng, n, 0.1)
            dur = n / w.fs
            for f0, f1 in ((50.0, 16000.0), (16000.0, 50.0)):
                ph = rng.uniform(0.0, 2.0 * np.pi)
                x += 0.2 * np.cos(2.0 * np.pi * (f0 * t + 0.5 * (f1 - f0) / dur * t * t) + ph)
        elif w.kind == "amfm_partials":
            x = np.zeros(n)
            for _ in range(20):
                fc = np.exp(rng.uniform(np.log(40.0), np.log(16000.0)))
                am_d, am_f = rng.uniform(0.0, 0.5), rng.uniform(0.5, 8.0)
                fm_d, fm_f = rng.uniform(0.0, 0.01), rng.uniform(0.5, 8.0)
                ph = rng.uniform(0.0, 2.0 * np.pi)
                phase = 2.0 * np.pi * fc * t + (fc * fm_d / fm_f) * np.sin(2.0 * np.pi * fm_f * t) + ph
                x += (1.0 / 20.0) * (1.0 + am_d * np.cos(2.0 * np.pi * am_f * t)) * np.cos(phase)
            rms = np.sqrt(np.mean(x * x))
            x += rms * 10.0 ** (-30.0 / 20.0) * rng.standard_normal(n)
        elif w.kind == "pink_notes":
            x = _pink(rng, n, 0.05)
            n_notes = rng.poisson(4.0 * n / w.fs)
            for _ in range(n_notes):
                onset = int(rng.integers(0, n))
                f0 = np.exp(rng.uniform(np.log(55.0), np.log(1760.0)))
                tau = rng.uniform(0.1, 0.8)
                pan = rng.uniform(0.0, 1.0)
                gain = 0.2 * (pan if c % 2 else 1.0 - pan)
                m = min(n - onset, int(6.0 * tau * w.fs))
                tt = np.arange(m) / w.fs
                env = np.exp(-tt / tau)
                for hnum in range(1, 7):
                    if f0 * hnum < 0.45 * w.fs:
                        x[onset:onset + m] += gain / hnum * env * np.sin(2.0 * np.pi * f0 * hnum * tt)
        else:
            raise ValueError(w.kind)
        out[c] = x.astype(np.float32)
    return out


def make_cotangent(w: Workload, coeff_count: int, n_channels: Optional[int] = None) -> np.ndarray:
    """[channels, coeff_count] complex64 with iid N(0,1) real and imaginary parts."""
    C = w.channels if n_channels is None else n_channels
    out = np.empty((C, coeff_count), dtype=np.complex64)
    for c in range(C):
        rng = np.random.Generator(np.random.PCG64([w.seed + 500000, c]))
        out[c] = (rng.standard_normal(coeff_count) + 1j * rng.standard_normal(coeff_count)).astype(np.complex64)
    return out
