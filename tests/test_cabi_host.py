"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares, its host-side
plan builder agrees with the oracle's independent layout, and argument errors come back as status codes."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import workloads as wl
from helpers import oracle_layout, library_plan, small_workload
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
