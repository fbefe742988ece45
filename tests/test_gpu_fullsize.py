"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times: outputs the oracle
can compute one by one (sampled coefficient indices per band) plus properties that hold at any size."""
import numpy as np
import pytest

import workloads as wl
from helpers import library_plan, oracle_layout, snr_db, split_bands
from oracle import nsgt_oracle as orc

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _sampled_band_errors(lay, X, coeffs, channels, per_band, seed, band_step=1):
    rng = np.random.default_rng(seed)
    offs = lay.coeff_offsets
    worst = (0.0, -1)
    for i in range(0, len(lay.bands), band_step):
        bd = lay.bands[i]
        n = np.unique(np.concatenate([[0, bd.M - 1], rng.integers(0, bd.M, per_band)]))
        want = orc.analyse_band(lay, X, i, n)
        got = coeffs[np.ix_(channels, offs[i] + n)]
        rel = np.linalg.norm(got - want, axis=-1) / np.linalg.norm(want, axis=-1)
        if rel.max() > worst[0]:
            worst = (float(rel.max()), i)
    return worst


def test_workload2_round_trip_full_batch():
    w = wl.CONFIGS["config2"]
    lay = oracle_layout(w)
    plan = library_plan(w)
    x = wl.make_signal(w)
    xd = torch.from_numpy(x).cuda()
    c = plan.analyse(xd, valid_len=w.valid_len)
    xr = plan.synthesise(c, valid_len=w.valid_len)
    assert snr_db(x, xr.cpu().numpy()).min() >= 120.0
    chans = [0, 17, 31]
    X = orc.long_dft(orc.pad_signal(x[chans], w.N))
    worst, band = _sampled_band_errors(lay, X, c.cpu().numpy(), chans, 48, 2)
    assert worst <= 1e-5, (band, worst)
    plan.close()


def test_workload2_under_the_default_length_policy():
    """Workload 2's layout with the lengths cqt_plan_create picks (multiples of 4: prime factors up to several
    thousand, chirp-z and direct-sum paths up to 12,800 coefficients, 5-smooth beyond): round trip and sampled
    coefficients of every third band on two signals."""
    import dataclasses
    w = dataclasses.replace(wl.scaled(wl.CONFIGS["config2"], channels=2), m_policy=wl.M_MULT4)
    lay = oracle_layout(w)
    plan = library_plan(w)
    x = wl.make_signal(w)
    c = plan.analyse(torch.from_numpy(x).cuda(), valid_len=w.valid_len)
    xr = plan.synthesise(c, valid_len=w.valid_len)
    assert snr_db(x, xr.cpu().numpy()).min() >= 120.0
    X = orc.long_dft(orc.pad_signal(x, w.N))
    worst, band = _sampled_band_errors(lay, X, c.cpu().numpy(), [0, 1], 32, 6, band_step=3)
    assert worst <= 1e-5, (band, worst)
    plan.close()


def test_longest_single_cta_class_synthesis_and_adjoints():
    """Workload 2's bands above 13,500 coefficients (the launch class of one 1024-thread CTA per band and signal,
    up to 216 KB of shared memory): synthesis, T^dagger and S^dagger against the oracle restricted to those bands.
    The other bands' coefficients are zero, so the oracle's direct sums stay affordable."""
    w = wl.scaled(wl.CONFIGS["config2"], channels=2)
    lay = oracle_layout(w)
    plan = library_plan(w)
    infos = plan.bands()
    top = max(bi.launch_class for bi in infos)
    long_bands = [i for i, bi in enumerate(infos) if bi.launch_class == top]
    assert len(long_bands) >= 3 and all(13500 < lay.bands[i].M <= 27000 for i in long_bands)
    rng = np.random.default_rng(41)
    offs = lay.coeff_offsets
    y = np.zeros((w.channels, lay.coeff_count), dtype=np.complex64)
    ysel = []
    for i in long_bands:
        M = lay.bands[i].M
        yb = (rng.standard_normal((w.channels, M)) + 1j * rng.standard_normal((w.channels, M))).astype(np.complex64)
        y[:, offs[i]:offs[i] + M] = yb
        ysel.append(yb.astype(np.complex128))
    yd = torch.from_numpy(y).cuda()
    got = plan.synthesise(yd, valid_len=w.valid_len).cpu().numpy()
    want = orc.synthesise(lay, ysel, bands=long_bands)[..., :w.valid_len]
    assert (np.linalg.norm(got - want, axis=-1) / np.linalg.norm(want, axis=-1)).max() <= 1e-5
    got = plan.analyse_adjoint(yd, valid_len=w.valid_len).cpu().numpy()
    want = orc.analyse_adjoint(lay, ysel, bands=long_bands)[..., :w.valid_len]
    assert (np.linalg.norm(got - want, axis=-1) / np.linalg.norm(want, axis=-1)).max() <= 1e-5
    # S^dagger: all bands on the GPU, the long ones compared at sampled output indices
    x = wl.make_signal(w)
    cb = plan.synthesise_adjoint(torch.from_numpy(x).cuda(), valid_len=w.valid_len).cpu().numpy()
    ns = [np.unique(np.concatenate([[0, lay.bands[i].M - 1], rng.integers(0, lay.bands[i].M, 64)])) for i in long_bands]
    want = orc.synthesise_adjoint(lay, orc.pad_signal(x, w.N), bands=long_bands, n=ns)
    for i, n, wb in zip(long_bands, ns, want):
        g = cb[:, offs[i] + n]
        assert (np.linalg.norm(g - wb, axis=-1) / np.linalg.norm(wb, axis=-1)).max() <= 1e-5, i
    plan.close()


def test_workload3_forward_and_adjoint_full_batch():
    w = wl.CONFIGS["config3"]
    lay = oracle_layout(w)
    plan = library_plan(w)
    x = wl.make_signal(w)
    y = wl.make_cotangent(w, lay.coeff_count)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    c = plan.analyse(xd, valid_len=w.valid_len).cpu().numpy()
    xb = plan.analyse_adjoint(yd, valid_len=w.valid_len).cpu().numpy()
    chans = [0, 63]
    X = orc.long_dft(orc.pad_signal(x[chans], w.N))
    worst, band = _sampled_band_errors(lay, X, c, chans, 48, 3)
    assert worst <= 1e-5, (band, worst)
    # adjoint against the oracle on one channel, and <T x, y> = <x, T' y> on all of them
    want = orc.analyse_adjoint(lay, split_bands(lay, y[5:6].astype(np.complex128)))[..., :w.valid_len]
    assert np.linalg.norm(xb[5:6] - want) <= 1e-5 * np.linalg.norm(want)
    for ch in range(0, w.channels, 7):
        lhs = np.real(np.vdot(c[ch].astype(np.complex128), y[ch].astype(np.complex128)))
        rhs = np.dot(x[ch].astype(np.float64), xb[ch].astype(np.float64))
        assert abs(lhs - rhs) <= 2e-5 * np.linalg.norm(c[ch]) * np.linalg.norm(y[ch])
    plan.close()


def test_workload4_long_signal():
    w = wl.CONFIGS["config4"]
    lay = oracle_layout(w)
    plan = library_plan(w)
    x = wl.make_signal(w)
    xd = torch.from_numpy(x).cuda()
    c = plan.analyse(xd, valid_len=w.valid_len)
    xr = plan.synthesise(c, valid_len=w.valid_len)
    assert snr_db(x, xr.cpu().numpy()).min() >= 120.0
    X = orc.long_dft(orc.pad_signal(x, w.N))
    worst, band = _sampled_band_errors(lay, X, c.cpu().numpy(), [0], 24, 4, band_step=3)
    assert worst <= 1e-5, (band, worst)
    i = len(lay.bands) - 1                       # the 720,000-coefficient Nyquist sideband
    worst, band = _sampled_band_errors(lay, X, c.cpu().numpy(), [0], 24, 5, band_step=i)
    assert worst <= 1e-5, (band, worst)
    plan.close()


def test_workload5_stream_prefix():
    """Ten seconds of the stereo stream, pushed in bulk (8 hops per push): output equals the input to >= 120 dB and
    two slices' coefficients match the oracle."""
    from paper_2609_29119_b200 import SliCQ
    w = wl.scaled(wl.CONFIGS["config5"], stream_len=10 * 44100)
    lay = oracle_layout(w)
    plan = library_plan(w)
    x = wl.make_signal(w)
    n, H = x.shape[1], w.slice_len // 2
    sq = SliCQ(plan, w.channels, w.transition, 16)
    xd = torch.from_numpy(x).cuda()
    out = torch.zeros((w.channels, n + 2 * w.slice_len), device="cuda")
    got, pos, kept = 0, 0, {}
    while pos < n:
        m = min(8 * H, n - pos)
        before = sq.push(xd[:, :0])
        done = sq.push(xd[:, pos:pos + m])
        for s in (2, 9):
            if before <= s < done:
                kept[s] = sq.coeffs(s).cpu().numpy()
        pos += m
        got += sq.pull(out[:, got:])
    sq.flush()
    got += sq.pull(out[:, got:])
    assert got >= n
    assert snr_db(x, out[:, :n].cpu().numpy()).min() >= 120.0
    slices = orc.slicq_cut(x.astype(np.float64), w.slice_len, w.transition)
    for s, cs in kept.items():
        want = orc.analyse(lay, slices[:, s, :])
        o = 0
        for bd, wb in zip(lay.bands, want):
            rel = np.linalg.norm(cs[:, o:o + bd.M] - wb, axis=-1) / np.linalg.norm(wb, axis=-1)
            assert rel.max() <= 1e-5
            o += bd.M
    assert sq.device_bytes() < 64 << 20
    sq.close()
    plan.close()
