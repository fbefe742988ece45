"""GPU test of cqt_analyse_static_ws, the analysis entry point for callers that cannot allocate device
memory (fixed memory budgets, real-time threads): its scratch is a fixed array inside the library.
Collected last on purpose, so a run that stops at the first failure has already run everything else.
Two calls in a row on different inputs must both match cqt_analyse: the shared array keeps the
previous call's contents and nothing may depend on them."""
import ctypes as C

import numpy as np
import pytest

import workloads as wl
from helpers import library_plan, small_workload

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def test_static_workspace_analysis_matches_cqt_analyse_twice():
    from paper_2609_29119_b200 import CqtError
    w = small_workload("static_ws", N=1 << 13, valid_len=8000, fs=22050.0, fmin=100.0, fmax=11025.0,
                       bins_per_octave=24, m_policy=wl.M_SMOOTH, channels=3, kind="noise_sines")
    plan = library_plan(w)
    limit = int(plan.lib.cqt_static_workspace_bytes())
    assert limit == 16 << 20 and plan.workspace_bytes(w.channels) <= limit
    x1 = torch.from_numpy(wl.make_signal(w)).cuda()
    x2 = torch.flip(x1, dims=[1]).contiguous() * 0.5 + 0.25
    out = torch.empty((w.channels, plan.coeff_count), dtype=torch.complex64, device="cuda")
    plan.analyse_static_ws(x1, valid_len=w.valid_len, out=out)   # first call on this device: looks the array up
    torch.cuda.synchronize()
    for x in (x1, x2):
        want = plan.analyse(x, valid_len=w.valid_len)
        torch.cuda.synchronize()
        # the call is made for hosts that cannot allocate: with the output preallocated, the device's free
        # memory is the same before and after it
        free_before, _ = torch.cuda.mem_get_info()
        got = plan.analyse_static_ws(x, valid_len=w.valid_len, out=out)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
        # same kernels, same arguments apart from the scratch pointer: the results are identical bit for bit
        assert torch.equal(torch.view_as_real(got), torch.view_as_real(want))
        a, b = got.cpu().numpy().astype(np.complex128), want.cpu().numpy().astype(np.complex128)
        o = 0
        for bi in plan.bands():
            seg = slice(o, o + bi.M)
            err = np.linalg.norm(a[:, seg] - b[:, seg], axis=-1) / np.linalg.norm(b[:, seg], axis=-1)
            assert err.max() <= 1e-5
            o += bi.M
    # a batch whose scratch exceeds the fixed array is refused before anything is launched
    big = 1
    while plan.workspace_bytes(big) <= limit:
        big *= 2
    xb = torch.zeros((big, w.valid_len), device="cuda")
    with pytest.raises(CqtError) as e:
        plan.analyse_static_ws(xb, valid_len=w.valid_len)
    assert e.value.status == -4
    plan.close()
