"""GPU tests of the sliced streaming form against the oracle's offline slicing."""
import numpy as np
import pytest

import workloads as wl
from helpers import band_rel_errors, library_plan, oracle_layout, small_workload, snr_db
from oracle import nsgt_oracle as orc

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

W = small_workload("slices_4096", N=4096, valid_len=4096, fs=22050.0, fmin=100.0, fmax=11025.0, bins_per_octave=12,
                   m_policy=wl.M_SMOOTH, channels=2, kind="pink_notes", slice_len=4096, transition=512,
                   stream_len=5 * 4096 + 123)


def _stream(plan, x, chunks, K=4, pull_every=1):
    from paper_2609_29119_b200 import SliCQ
    sq = SliCQ(plan, x.shape[0], W.transition, K)
    xd = torch.from_numpy(x).cuda()
    n = x.shape[1]
    out = torch.zeros((x.shape[0], n + 2 * W.slice_len), device="cuda")
    got, pos, i = 0, 0, 0
    coeffs = {}
    while pos < n:
        m = min(chunks[i % len(chunks)], n - pos)
        i += 1
        before = sq.push(xd[:, :0])
        done = sq.push(xd[:, pos:pos + m])
        for s in range(before, done):
            if s in (0, 1, 3):
                coeffs[s] = sq.coeffs(s).cpu().numpy()
        pos += m
        if i % pull_every == 0:
            got += sq.pull(out[:, got:])
    sq.flush()
    got += sq.pull(out[:, got:])
    nbytes = sq.device_bytes()
    sq.close()
    return out[:, :got].cpu().numpy(), coeffs, nbytes


def test_streaming_matches_offline_slicing():
    lay = oracle_layout(W)
    plan = library_plan(W)
    x = wl.make_signal(W)
    n = x.shape[1]
    H = W.slice_len // 2
    y, coeffs, _ = _stream(plan, x, [H])
    assert y.shape[1] >= n
    # oracle: cut, per-slice T and S, overlap-add
    slices = orc.slicq_cut(x.astype(np.float64), W.slice_len, W.transition)       # [C, ns, sl]
    for s, c in coeffs.items():
        want = orc.analyse(lay, slices[:, s, :])
        errs = band_rel_errors(lay, c, want)
        assert errs.max() <= 1e-5, (s, errs.max())
    rec = np.stack([orc.synthesise(lay, orc.analyse(lay, slices[:, s, :])) for s in range(slices.shape[1])], axis=1)
    want_y = orc.slicq_overlap_add(rec, n)
    rel = np.linalg.norm(y[:, :n] - want_y, axis=-1) / np.linalg.norm(want_y, axis=-1)
    assert rel.max() <= 1e-5
    assert snr_db(x, y[:, :n]).min() >= 120.0
    plan.close()


def test_chunking_does_not_change_the_result_and_memory_is_bounded():
    plan = library_plan(W)
    x = wl.make_signal(W)
    H = W.slice_len // 2
    y1, _, b1 = _stream(plan, x, [H])
    y2, _, b2 = _stream(plan, x, [1, 7, H - 3, 3 * H + 5, 200], pull_every=2)
    m = min(y1.shape[1], y2.shape[1])
    assert m >= x.shape[1]
    assert np.array_equal(y1[:, :m], y2[:, :m])
    # a stream three times as long uses the same device memory
    x3 = wl.make_signal(W, length=3 * x.shape[1])
    y3, _, b3 = _stream(plan, x3, [2 * H])
    assert b1 == b2 == b3
    assert snr_db(x3, y3[:, :x3.shape[1]]).min() >= 120.0
    plan.close()


def test_push_beyond_the_slots_in_flight_is_refused():
    from paper_2609_29119_b200 import CqtError, SliCQ
    plan = library_plan(W)
    sq = SliCQ(plan, 2, W.transition, 2)
    H = W.slice_len // 2
    x = torch.zeros((2, 4 * H), device="cuda")
    assert sq.push(x[:, :2 * H]) == 2
    with pytest.raises(CqtError) as e:
        sq.push(x[:, :H])
    assert e.value.status == -6
    out = torch.empty((2, 8 * H), device="cuda")
    assert sq.pull(out) == H          # slices 0 and 1 synthesised: block 0 is final
    assert sq.push(x[:, :H]) == 3
    sq.reset()
    assert sq.push(x[:, :H]) == 1
    sq.close()
    plan.close()
