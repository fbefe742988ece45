"""Shared helpers of the test-suite: build the library plan and the oracle layout for the same workload."""
import numpy as np

import workloads as wl
from oracle import nsgt_oracle as orc


def oracle_layout(w: wl.Workload):
    if w.sections:
        c, wd, octave = orc.multires_bands(w.fs, w.fmin, w.N, w.sections, w.min_win)
        return orc.build_layout_bands(w.fs, w.N, c, wd, w.window, w.m_policy, octave)
    if w.bands:
        return orc.build_layout_bands(w.fs, w.N, [b[0] for b in w.bands], [b[1] for b in w.bands], w.window, w.m_policy)
    return orc.build_layout(w.fs, w.fmin, w.fmax, w.bins_per_octave, w.N, window=w.window, policy=w.m_policy,
                            min_win=w.min_win)


def library_plan(w: wl.Workload, device=None, **tuning):
    from paper_2609_29119_b200 import Plan, multires_bands
    if w.sections:
        c, wd, octave = multires_bands(w.fs, w.fmin, w.N, w.sections, w.min_win)
        return Plan.from_bands(w.fs, w.N, c, wd, octave, window=w.window, m_policy=w.m_policy, device=device)
    if w.bands:
        return Plan.from_bands(w.fs, w.N, [b[0] for b in w.bands], [b[1] for b in w.bands], None, window=w.window,
                               m_policy=w.m_policy, device=device)
    return Plan(w.fs, w.fmin, w.fmax, w.bins_per_octave, w.N, window=w.window, m_policy=w.m_policy,
                min_win=w.min_win, device=device, **tuning)


def split_bands(lay, flat):
    """[..., coeff_count] -> list of per-band arrays."""
    out, o = [], 0
    for b in lay.bands:
        out.append(flat[..., o:o + b.M])
        o += b.M
    return out


def band_rel_errors(lay, got_flat, want_list):
    """max over signals of ||got - want|| / ||want|| per band."""
    errs = []
    for g, w in zip(split_bands(lay, got_flat), want_list):
        num = np.linalg.norm(g - w, axis=-1)
        den = np.linalg.norm(w, axis=-1)
        errs.append(float(np.max(num / den)))
    return np.array(errs)


def snr_db(x, y):
    x = np.asarray(x, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    return 10.0 * np.log10(np.sum(x * x, axis=-1) / np.sum((x - y) ** 2, axis=-1))


def small_workload(name, **kw):
    base = dict(name=name, fs=256.0, fmin=6.0, fmax=128.0, bins_per_octave=6, N=256, valid_len=256, channels=2,
                window=wl.WIN_HANN, m_policy=wl.M_MULT4, seed=7, kind="white")
    base.update(kw)
    return wl.Workload(**base)
