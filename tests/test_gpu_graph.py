"""The transform calls can be captured in a CUDA graph (the paper times its round trip under graph replay, Sec. 5):
the plan's helper streams fork from and join the capturing stream, and a replay gives bit-for-bit the eager result."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import workloads as wl
from helpers import library_plan, small_workload, snr_db

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("w", [
    small_workload("graph_n16384", N=1 << 14, valid_len=16000, fs=44100.0, fmin=32.70, fmax=22050.0, bins_per_octave=24,
                   m_policy=wl.M_SMOOTH, channels=4),
    wl.scaled(wl.CONFIGS["table1"], channels=2),
], ids=lambda w: w.name)
def test_round_trip_under_graph_replay_equals_eager(w):
    plan = library_plan(w)
    x1 = torch.from_numpy(wl.make_signal(w)).cuda()
    x2 = torch.flip(x1, dims=[1]).contiguous() * 0.5
    x = x1.clone()
    c = torch.empty((w.channels, plan.coeff_count), dtype=torch.complex64, device="cuda")
    y = torch.empty_like(x)
    ws = plan.workspace(w.channels)

    def step(stream):
        plan.analyse(x, valid_len=w.valid_len, out=c, ws=ws, stream=stream)
        plan.synthesise(c, valid_len=w.valid_len, out=y, ws=ws, stream=stream)

    step(torch.cuda.current_stream())                       # eager, also the warm-up before capture
    torch.cuda.synchronize()
    c_eager, y_eager = c.clone(), y.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    launches = plan.launch_count()
    with torch.cuda.graph(g, stream=side):
        step(torch.cuda.current_stream())
    per_step = plan.launch_count() - launches
    assert per_step >= 8
    torch.cuda.current_stream().wait_stream(side)
    c.zero_(); y.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(torch.view_as_real(c), torch.view_as_real(c_eager)) and torch.equal(y, y_eager)
    # new input in the captured buffers, replay again: equals an eager run on that input
    x.copy_(x2)
    g.replay()
    torch.cuda.synchronize()
    c_g, y_g = c.clone(), y.clone()
    step(torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert torch.equal(torch.view_as_real(c), torch.view_as_real(c_g)) and torch.equal(y, y_g)
    assert snr_db(x2.cpu().numpy(), y_g.cpu().numpy()).min() >= 120.0
    assert plan.launch_count() - launches == 2 * per_step  # replays launch through the graph, not through the plan
    plan.close()
