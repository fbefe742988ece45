"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares, its host-side
plan builder agrees with the oracle's independent layout, and argument errors come back as status codes."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import workloads as wl
from helpers import oracle_layout, library_plan, small_workload
import paper_2609_29119_b200 as cq
from oracle import nsgt_oracle as orc
from paper_2609_29119_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2609_29119_b200.build import build
    build()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "cqt.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b((?:cqt|slicq)_[a-z_]+)\s*\(", hdr))
    assert {"cqt_plan_create", "cqt_analyse", "cqt_synthesise", "cqt_analyse_adjoint", "cqt_synthesise_adjoint",
            "slicq_push", "slicq_pull"} <= declared
    lib = C.CDLL(B.lib_path())
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS), declared ^ set(B.EXPORTS)


CASES = [wl.CONFIGS["config1"], wl.CONFIGS["config3"], wl.CONFIGS["config5"], wl.CONFIGS["config2"],
         small_workload("tiny"), small_workload("tiny_bh", window=wl.WIN_BLACKMAN_HARRIS, m_policy=wl.M_SMOOTH),
         small_workload("pow2", N=4096, fs=8000.0, fmin=100.0, fmax=4000.0, bins_per_octave=24, m_policy=wl.M_POW2)]


@pytest.mark.parametrize("name", ["config1", "config2", "config3", "config4", "config5"])
def test_default_length_policy_plans_every_workload(name):
    """cqt_plan_create's policy (multiple of 4) on all five workloads: every band gets a radix plan (host-only
    plans, so no device is needed), lengths up to 12,800 are exactly 4 ceil(S / 4), longer ones are 5-smooth,
    and the layout agrees with the oracle's."""
    import dataclasses
    w = dataclasses.replace(wl.CONFIGS[name], m_policy=wl.M_MULT4)
    lay = oracle_layout(w)
    plan = library_plan(w, device=-1)
    assert plan.num_bands == len(lay.bands) and plan.coeff_count == lay.coeff_count
    ragged = 0
    for i, bd in enumerate(lay.bands):
        bi = plan.band_info(i)
        assert bi.M == bd.M and bi.M >= bi.support and bi.M % 4 == 0
        if bi.M <= 12800:
            assert bi.M == 4 * ((bi.support + 3) // 4)
            ragged += 1
        else:
            m = bi.M
            for p in (2, 3, 5):
                while m % p == 0:
                    m //= p
            assert m == 1
    assert ragged >= len(lay.bands) - 120
    plan.close()


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_host_plan_matches_oracle_layout(w):
    lay = oracle_layout(w)
    plan = library_plan(w, device=-1)
    assert plan.num_bands == len(lay.bands)
    assert plan.coeff_count == lay.coeff_count
    offs = lay.coeff_offsets
    g, h = plan.tables()
    t = 0
    for i, bd in enumerate(lay.bands):
        bi = plan.band_info(i)
        assert (bi.centre_bin, bi.support, bi.first_offset, bi.M, bi.coeff_offset, bi.is_sideband, bi.table_offset) == \
               (bd.kc, len(bd.d), int(bd.d[0]), bd.M, offs[i], bd.sideband, t)
        assert abs(bi.centre_hz - bd.centre_hz) <= 1e-9 * max(1.0, bd.centre_hz)
        assert np.allclose(g[t:t + len(bd.d)], bd.g, rtol=1e-6, atol=1e-9)
        assert np.allclose(h[t:t + len(bd.d)], bd.h, rtol=1e-6, atol=1e-12)
        t += len(bd.d)
    assert plan.workspace_bytes(3) > 0
    plan.close()


def test_error_codes_without_a_device():
    lib = B.load_library()
    h = C.c_void_p()
    d = B.PlanDesc(44100.0, 32.7, 22050.0, 12, 1000, 0, 0, 4.0, -1)
    assert lib.cqt_plan_create_ex(C.byref(d), C.byref(h)) == -2          # not a power of two
    d.L = 1 << 16
    d.fmin = 0.5
    assert lib.cqt_plan_create_ex(C.byref(d), C.byref(h)) == -3          # first centre below bin 2
    d.fmin = -1.0
    assert lib.cqt_plan_create_ex(C.byref(d), C.byref(h)) == -1
    d.fmin = 32.7
    assert lib.cqt_plan_create_ex(None, C.byref(h)) == -1
    assert lib.cqt_plan_create_ex(C.byref(d), C.byref(h)) == 0
    # a host-only plan cannot transform
    assert lib.cqt_analyse(h, 8, 1 << 16, 1, 1 << 16, 8, 256, 1 << 30, None) == -6
    assert lib.cqt_analyse(h, None, 1 << 16, 1, 1 << 16, 8, 256, 1 << 30, None) == -1
    assert lib.cqt_synthesise(h, 8, 1, (1 << 16) + 1, 8, 1 << 17, 256, 1 << 30, None) == -1   # valid_len > N
    bi = B.BandInfo()
    assert lib.cqt_plan_band_info(h, 10**6, C.byref(bi)) == -1
    assert lib.cqt_plan_destroy(h) == 0
    assert lib.cqt_status_string(-3).decode().startswith("band layout")
    out = C.c_void_p()
    assert lib.slicq_create(None, 2, 8, 4, C.byref(out)) == -1


TABLE1_SECTIONS = [(3, 8), (4, 16), (2, 32)]


def _compare_plan(plan, lay):
    assert plan.num_bands == len(lay.bands) and plan.coeff_count == lay.coeff_count
    g, h = plan.tables()
    offs = lay.coeff_offsets
    t = 0
    for i, bd in enumerate(lay.bands):
        bi = plan.band_info(i)
        assert (bi.centre_bin, bi.support, bi.first_offset, bi.M, bi.coeff_offset, bi.is_sideband, bi.table_offset) == \
               (bd.kc, len(bd.d), int(bd.d[0]), bd.M, offs[i], bd.sideband, t)
        assert np.allclose(g[t:t + len(bd.d)], bd.g, rtol=1e-6, atol=1e-9)
        assert np.allclose(h[t:t + len(bd.d)], bd.h, rtol=1e-6, atol=1e-12)
        t += len(bd.d)


def test_multires_plan_matches_oracle_and_table1():
    """cqt_multires_bands + cqt_plan_create_bands against the oracle's own list and layout; the totals are the
    paper's Table 1 (154 bands, 132,992 coefficients)."""
    fs, N = 44100.0, 65536
    c, w, octave = orc.multires_bands(fs, fs / 1024.0, N, TABLE1_SECTIONS)
    lc, lw, lo = cq.multires_bands(fs, fs / 1024.0, N, TABLE1_SECTIONS)
    assert np.allclose(lc, c, rtol=1e-14) and np.allclose(lw, w, rtol=1e-14) and list(lo) == list(octave)
    lay = orc.build_layout_bands(fs, N, c, w, orc.HANN, orc.M_POW2, octave)
    plan = cq.Plan.from_bands(fs, N, lc, lw, lo, m_policy=cq.M_POW2, device=-1)
    assert plan.num_bands == 154 and plan.coeff_count == 132992
    _compare_plan(plan, lay)
    plan.close()
    # falling resolution: the wide bands of the second section start below the last narrow bands of the first
    fs, N = 8192.0, 8192
    c, w, octave = orc.multires_bands(fs, 100.0, N, [(2, 16), (2, 4)])
    lay = orc.build_layout_bands(fs, N, c, w, orc.HANN, orc.M_POW2, octave)
    plan = cq.Plan.from_bands(fs, N, c, w, octave, m_policy=cq.M_POW2, device=-1)
    _compare_plan(plan, lay)
    starts = [b.kc + b.d[0] for b in lay.bands[1:-1]]
    assert min(np.diff(starts)) < 0          # supports do nest
    plan.close()


def test_irregular_band_list_plan_matches_oracle():
    fs, N = 2048.0, 2048
    c = list(np.arange(24.0, 200.0, 16.0)) + list(200.0 * 2 ** (np.arange(0, 17) / 8.0))
    c = [f for f in c if f < 820.0]
    w = [2.0 * (c[min(i + 1, len(c) - 1)] - c[max(i - 1, 0)]) * N / fs / (2 if 0 < i < len(c) - 1 else 1) for i in range(len(c))]
    lay = orc.build_layout_bands(fs, N, c, w, orc.BLACKMAN_HARRIS, orc.M_SMOOTH)
    plan = cq.Plan.from_bands(fs, N, c, w, None, window=cq.WIN_BLACKMAN_HARRIS, m_policy=cq.M_SMOOTH, device=-1)
    _compare_plan(plan, lay)
    plan.close()


def test_band_list_errors():
    ok = dict(fs=1024.0, L=1024, centre_hz=[40.0, 80.0, 160.0], width_bins=[60.0, 120.0, 240.0], device=-1)
    cq.Plan.from_bands(**ok).close()
    for bad, status in [(dict(centre_hz=[80.0, 40.0, 160.0]), -1),       # descending centres
                        (dict(width_bins=[60.0, 1.0, 240.0]), -1),        # width below 2 bins
                        (dict(L=1000), -2),                               # N not a power of two
                        (dict(centre_hz=[40.0, 80.0, 500.0]), -3),        # last band reaches Nyquist
                        (dict(centre_hz=[1.0, 80.0, 160.0], width_bins=[2.0, 120.0, 240.0]), -3)]:   # first centre below bin 2
        with pytest.raises(cq.CqtError) as e:
            cq.Plan.from_bands(**dict(ok, **bad))
        assert e.value.status == status
    # a narrow band nested deep inside a wide neighbour is a legal frame
    cq.Plan.from_bands(1024.0, 1024, [100.0, 101.0, 200.0], [180.0, 8.0, 200.0], device=-1).close()
