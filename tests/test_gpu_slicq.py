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
# a slice long enough for the two-pass long FFT, where the slice cut is fused into the first pass's load
W16 = small_workload("slices_16384", N=16384, valid_len=16384, fs=44100.0, fmin=60.0, fmax=22050.0, bins_per_octave=12,
                     m_policy=wl.M_SMOOTH, channels=2, kind="pink_notes", slice_len=16384, transition=4096,
                     stream_len=4 * 16384 + 321)
BOTH = pytest.mark.parametrize("w", [W, W16], ids=lambda w: w.name)


def _stream(plan, x, chunks, K=4, pull_every=1, w=W):
    from paper_2609_29119_b200 import SliCQ
    sq = SliCQ(plan, x.shape[0], w.transition, K)
    xd = torch.from_numpy(x).cuda()
    n = x.shape[1]
    out = torch.zeros((x.shape[0], n + 2 * w.slice_len), device="cuda")
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


@BOTH
def test_streaming_matches_offline_slicing(w):
    lay = oracle_layout(w)
    plan = library_plan(w)
    x = wl.make_signal(w)
    n = x.shape[1]
    H = w.slice_len // 2
    y, coeffs, _ = _stream(plan, x, [H], w=w)
    assert y.shape[1] >= n
    # oracle: cut, per-slice T and S, overlap-add
    slices = orc.slicq_cut(x.astype(np.float64), w.slice_len, w.transition)       # [C, ns, sl]
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


@BOTH
def test_chunking_does_not_change_the_result_and_memory_is_bounded(w):
    plan = library_plan(w)
    x = wl.make_signal(w)
    H = w.slice_len // 2
    y1, _, b1 = _stream(plan, x, [H], w=w)
    y2, _, b2 = _stream(plan, x, [1, 7, H - 3, 3 * H + 5, 200], pull_every=2, w=w)
    m = min(y1.shape[1], y2.shape[1])
    assert m >= x.shape[1]
    assert np.array_equal(y1[:, :m], y2[:, :m])
    # a stream three times as long uses the same device memory
    x3 = wl.make_signal(w, length=3 * x.shape[1])
    y3, _, b3 = _stream(plan, x3, [2 * H], w=w)
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


def test_assembled_coefficients_match_oracle():
    """slicq_assemble against the oracle's overlap-add of the oracle's own per-slice coefficients."""
    from paper_2609_29119_b200 import CqtError, SliCQ
    lay, plan = oracle_layout(W), library_plan(W)
    x = wl.make_signal(W)
    H = W.slice_len // 2
    sq = SliCQ(plan, x.shape[0], W.transition, 6)
    xd = torch.from_numpy(x).cuda()
    assert sq.push(xd[:, :5 * H]) == 5
    slices = orc.slicq_cut(x.astype(np.float64), W.slice_len, W.transition)
    for first, n in ((0, 5), (1, 3), (4, 1)):
        got = sq.assemble(first, n).cpu().numpy()
        want = orc.slicq_assemble(lay, [orc.analyse(lay, slices[:, s, :]) for s in range(first, first + n)])
        assert got.shape[1] == (n + 1) * lay.coeff_count // 2
        o = 0
        for b, wb in zip(lay.bands, want):
            g = got[:, o:o + wb.shape[-1]]
            assert np.linalg.norm(g - wb) <= 1e-5 * np.linalg.norm(wb), (first, n, b.kc)
            o += wb.shape[-1]
    with pytest.raises(CqtError) as e:
        sq.assemble(3, 3)             # slice 5 has not been analysed
    assert e.value.status == -6
    sq.close()
    plan.close()


def test_coefficients_edited_between_push_and_pull_are_what_is_synthesised():
    """Processing hook: zero all bands above one index in every slice before pulling; the output is the oracle's
    overlap-add of the slices synthesised from the same edited coefficients."""
    from paper_2609_29119_b200 import SliCQ
    lay, plan = oracle_layout(W), library_plan(W)
    x = wl.make_signal(W)
    n, H = x.shape[1], W.slice_len // 2
    keep = lay.coeff_offsets[len(lay.bands) // 2]        # coefficients of the lower half of the bands
    sq = SliCQ(plan, x.shape[0], W.transition, 4)
    xd = torch.from_numpy(x).cuda()
    out = torch.zeros((x.shape[0], n + 2 * W.slice_len), device="cuda")
    got = pos = done = 0
    while pos < n:
        m = min(H, n - pos)
        now = sq.push(xd[:, pos:pos + m])
        for s in range(done, now):
            sq.coeffs(s)[:, keep:] = 0
        done = now
        pos += m
        got += sq.pull(out[:, got:])
    before = sq.push(xd[:, :0])
    sq.flush()
    for s in range(before, sq.push(xd[:, :0])):
        sq.coeffs(s)[:, keep:] = 0
    got += sq.pull(out[:, got:])
    slices = orc.slicq_cut(x.astype(np.float64), W.slice_len, W.transition)
    rec = []
    for s in range(slices.shape[1]):
        c = orc.analyse(lay, slices[:, s, :])
        c = [cb if i < len(lay.bands) // 2 else np.zeros_like(cb) for i, cb in enumerate(c)]
        rec.append(orc.synthesise(lay, c))
    want = orc.slicq_overlap_add(np.stack(rec, axis=1), n)
    y = out[:, :n].cpu().numpy()
    rel = np.linalg.norm(y - want, axis=-1) / np.linalg.norm(want, axis=-1)
    assert rel.max() <= 1e-5, rel
    assert snr_db(x, y).max() < 30.0          # and it is not the identity any more
    sq.close()
    plan.close()


def test_saved_state_resumes_the_stream_bit_for_bit():
    from paper_2609_29119_b200 import CqtError, SliCQ
    plan = library_plan(W)
    x = wl.make_signal(W)
    n, H = x.shape[1], W.slice_len // 2
    xd = torch.from_numpy(x).cuda()

    def run(sq, lo, hi, out, got):
        pos = lo
        while pos < hi:
            m = min(H + 37, hi - pos)
            sq.push(xd[:, pos:pos + m])
            pos += m
            got += sq.pull(out[:, got:])
        return got
    ref = torch.zeros((x.shape[0], n + 2 * W.slice_len), device="cuda")
    a = SliCQ(plan, x.shape[0], W.transition, 4)
    g = run(a, 0, n, ref, 0)
    a.flush()
    g += a.pull(ref[:, g:])
    cut = 2 * H + 301
    out = torch.zeros_like(ref)
    b = SliCQ(plan, x.shape[0], W.transition, 4)
    gb = run(b, 0, cut, out, 0)
    b.push(xd[:, cut:cut + H])               # leaves an analysed slice waiting: saving is refused
    with pytest.raises(CqtError) as e:
        b.save_state()
    assert e.value.status == -6
    gb += b.pull(out[:, gb:])
    state = b.save_state()
    b.close()
    c = SliCQ(plan, x.shape[0], W.transition, 4)
    c.load_state(state)
    gc = run(c, cut + H, n, out, gb)
    c.flush()
    gc += c.pull(out[:, gc:])
    assert gc == g
    assert torch.equal(out[:, :g], ref[:, :g])
    other = SliCQ(plan, x.shape[0], W.transition, 3)
    with pytest.raises(CqtError) as e:
        other.load_state(state)              # saved by an object with another number of slices in flight
    assert e.value.status == -6
    other.close(); c.close(); a.close()
    plan.close()
