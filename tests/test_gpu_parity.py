"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded inputs.

Tolerances (fp32 arithmetic against an fp64 reference): per band ||c_gpu - c_oracle||_2 / ||c_oracle||_2 <= 1e-5;
signals from synthesis / adjoints <= 1e-5 relative L2; round trip SNR >= 120 dB on the true samples."""
import numpy as np
import pytest

import workloads as wl
from helpers import band_rel_errors, library_plan, oracle_layout, small_workload, snr_db, split_bands
from oracle import nsgt_oracle as orc

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 1e-5


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


CASES = [
    small_workload("n256"),
    small_workload("n256_bh_smooth", window=wl.WIN_BLACKMAN_HARRIS, m_policy=wl.M_SMOOTH),
    small_workload("n4096_b48", N=4096, valid_len=4096, fs=22050.0, fmin=200.0, fmax=11025.0, bins_per_octave=48,
                   m_policy=wl.M_SMOOTH, channels=3),
    small_workload("n4096_ragged", N=4096, valid_len=3001, fs=22050.0, fmin=200.0, fmax=11025.0, bins_per_octave=12,
                   m_policy=wl.M_MULT4, channels=3),
    # enough (band, signal) items for the lane-group kernels of the shortest bands (8 lanes per item), on lengths
    # with prime factors above 5 (direct-sum stage) and on 5-smooth ones
    small_workload("n4096_b48_mult4_48ch", N=4096, valid_len=3900, fs=22050.0, fmin=200.0, fmax=11025.0,
                   bins_per_octave=48, m_policy=wl.M_MULT4, channels=48),
    small_workload("n4096_b48_smooth_40ch", N=4096, valid_len=4096, fs=22050.0, fmin=200.0, fmax=11025.0,
                   bins_per_octave=48, m_policy=wl.M_SMOOTH, window=wl.WIN_BLACKMAN_HARRIS, channels=40),
    small_workload("n16384_mult4", N=1 << 14, valid_len=1 << 14, fs=44100.0, fmin=32.70, fmax=22050.0,
                   bins_per_octave=12, m_policy=wl.M_MULT4, channels=2),
    small_workload("slice_2e15", N=1 << 15, valid_len=1 << 15, fs=44100.0, fmin=32.70, fmax=22050.0,
                   bins_per_octave=48, m_policy=wl.M_SMOOTH, channels=2),
    wl.CONFIGS["config1"],
    small_workload("n65536_ragged_pow2", N=1 << 16, valid_len=50001, fs=44100.0, fmin=32.70, fmax=22050.0,
                   bins_per_octave=12, m_policy=wl.M_POW2, channels=3),
    wl.scaled(wl.CONFIGS["config3"], channels=2),
    # band-list plans: the paper's Table 1 layout; falling resolution (nested supports, zero-filled plane bins);
    # an irregular list (linear then geometric centres)
    wl.scaled(wl.CONFIGS["table1"], channels=3),
    small_workload("multires_falling", N=8192, valid_len=8000, fs=8192.0, fmin=100.0, fmax=4096.0, bins_per_octave=0,
                   m_policy=wl.M_POW2, channels=2, sections=((2, 16), (2, 4))),
    small_workload("irregular_bands", N=2048, valid_len=2048, fs=2048.0, fmin=24.0, fmax=1024.0, bins_per_octave=0,
                   window=wl.WIN_BLACKMAN_HARRIS, m_policy=wl.M_SMOOTH, channels=2,
                   bands=tuple((f, wd) for f, wd in zip(
                       [24.0 + 16.0 * i for i in range(11)] + [200.0 * 2 ** (i / 8.0) for i in range(17)],
                       [32.0] * 11 + [200.0 * 2 ** (i / 8.0) * 0.36 for i in range(17)]))),
]


@pytest.fixture(scope="module", params=CASES, ids=lambda w: w.name)
def case(request):
    w = request.param
    lay = oracle_layout(w)
    plan = library_plan(w)
    x = wl.make_signal(w)
    yield w, lay, plan, x
    plan.close()


def test_analysis_matches_oracle_per_band(case):
    w, lay, plan, x = case
    c = plan.analyse(_dev(x), valid_len=w.valid_len).cpu().numpy()
    want = orc.analyse(lay, orc.pad_signal(x, w.N))
    errs = band_rel_errors(lay, c, want)
    assert errs.max() <= TOL, (int(errs.argmax()), errs.max())


def test_synthesis_matches_oracle_on_arbitrary_coefficients(case):
    w, lay, plan, x = case
    y = wl.make_cotangent(w, lay.coeff_count)
    got = plan.synthesise(_dev(y), valid_len=w.valid_len).cpu().numpy()
    want = orc.synthesise(lay, split_bands(lay, y.astype(np.complex128)))[..., :w.valid_len]
    rel = np.linalg.norm(got - want, axis=-1) / np.linalg.norm(want, axis=-1)
    assert rel.max() <= TOL, rel


def test_round_trip_snr(case):
    w, lay, plan, x = case
    xd = _dev(x)
    c = plan.analyse(xd, valid_len=w.valid_len)
    xr = plan.synthesise(c, valid_len=w.valid_len).cpu().numpy()
    if w.valid_len == w.N:
        assert snr_db(x, xr).min() >= 120.0, snr_db(x, xr)
    else:
        # truncating the reconstruction of a zero-padded signal: compare on the true samples
        assert snr_db(x, xr).min() >= 120.0, snr_db(x, xr)


def test_adjoints_match_oracle(case):
    w, lay, plan, x = case
    y = wl.make_cotangent(w, lay.coeff_count)
    got = plan.analyse_adjoint(_dev(y), valid_len=w.valid_len).cpu().numpy()
    want = orc.analyse_adjoint(lay, split_bands(lay, y.astype(np.complex128)))[..., :w.valid_len]
    rel = np.linalg.norm(got - want, axis=-1) / np.linalg.norm(want, axis=-1)
    assert rel.max() <= TOL, rel
    cb = plan.synthesise_adjoint(_dev(x), valid_len=w.valid_len).cpu().numpy()
    want_c = orc.synthesise_adjoint(lay, orc.pad_signal(x, w.N))
    errs = band_rel_errors(lay, cb, want_c)
    assert errs.max() <= TOL, (int(errs.argmax()), errs.max())


def test_adjoint_identity_on_gpu_outputs(case):
    """<T x, y> = <x, T' y> and <S y, xb> = <y, S' xb> with every operand computed by the kernels."""
    w, lay, plan, x = case
    y = wl.make_cotangent(w, lay.coeff_count)
    xd, yd = _dev(x), _dev(y)
    Tx = plan.analyse(xd, valid_len=w.valid_len).cpu().numpy().astype(np.complex128)
    Tty = plan.analyse_adjoint(yd, valid_len=w.valid_len).cpu().numpy().astype(np.float64)
    Sy = plan.synthesise(yd, valid_len=w.valid_len).cpu().numpy().astype(np.float64)
    Stx = plan.synthesise_adjoint(xd, valid_len=w.valid_len).cpu().numpy().astype(np.complex128)
    y64, x64 = y.astype(np.complex128), x.astype(np.float64)
    for ch in range(x.shape[0]):
        lhs, rhs = np.real(np.vdot(Tx[ch], y64[ch])), np.dot(x64[ch], Tty[ch])
        assert abs(lhs - rhs) <= 2e-5 * np.linalg.norm(Tx[ch]) * np.linalg.norm(y64[ch])
        lhs, rhs = np.dot(Sy[ch], x64[ch]), np.real(np.vdot(y64[ch], Stx[ch]))
        assert abs(lhs - rhs) <= 2e-5 * np.linalg.norm(Sy[ch]) * np.linalg.norm(x64[ch])


def test_bitwise_reproducible(case):
    w, lay, plan, x = case
    xd = _dev(x)
    c1 = plan.analyse(xd, valid_len=w.valid_len)
    c2 = plan.analyse(xd, valid_len=w.valid_len)
    assert torch.equal(torch.view_as_real(c1), torch.view_as_real(c2))
    x1 = plan.synthesise(c1, valid_len=w.valid_len)
    x2 = plan.synthesise(c1, valid_len=w.valid_len)
    assert torch.equal(x1, x2)


def test_results_do_not_depend_on_the_batch_size():
    """A signal's coefficients and reconstruction are bitwise the same whether it is transformed alone or in a
    large batch (the launch shapes differ: lanes per item of the shortest bands, threads of the long FFT)."""
    w = small_workload("n4096_b48_mult4_64ch", N=4096, valid_len=4001, fs=22050.0, fmin=200.0, fmax=11025.0,
                       bins_per_octave=48, m_policy=wl.M_MULT4, channels=64)
    plan = library_plan(w)
    xd = _dev(wl.make_signal(w))
    c_all = plan.analyse(xd, valid_len=w.valid_len)
    x_all = plan.synthesise(c_all, valid_len=w.valid_len)
    for rows in (slice(0, 1), slice(61, 64)):
        c = plan.analyse(xd[rows].contiguous(), valid_len=w.valid_len)
        assert torch.equal(torch.view_as_real(c), torch.view_as_real(c_all[rows]))
        assert torch.equal(plan.synthesise(c, valid_len=w.valid_len), x_all[rows])
    plan.close()


def test_row_stride_and_padding_are_respected():
    w = CASES[3]
    plan = library_plan(w)
    x = wl.make_signal(w)
    wide = torch.full((w.channels, w.valid_len + 37), 7.0, device="cuda")
    wide[:, :w.valid_len] = _dev(x)
    c_wide = plan.analyse(wide, valid_len=w.valid_len)
    c_ref = plan.analyse(_dev(x), valid_len=w.valid_len)
    assert torch.equal(torch.view_as_real(c_wide), torch.view_as_real(c_ref))
    out = torch.full((w.channels, w.valid_len + 5), -3.0, device="cuda")
    plan.synthesise(c_ref, valid_len=w.valid_len, out=out)
    assert torch.all(out[:, w.valid_len:] == -3.0)          # nothing written past valid_len
    plan.close()


def test_argument_errors_on_device_plan():
    from paper_2609_29119_b200 import CqtError
    w = CASES[0]
    plan = library_plan(w)
    x = _dev(wl.make_signal(w))
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(CqtError) as e:
        plan.analyse(x, ws=small)
    assert e.value.status == -4
    with pytest.raises(CqtError) as e:
        plan.analyse(x, valid_len=w.N + 2)
    assert e.value.status == -1
    plan.close()


def test_unaligned_rows_and_odd_strides():
    """Signal rows that are not 8-byte aligned (odd element offset, odd stride) take the scalar load/store path."""
    w = CASES[3]
    plan = library_plan(w)
    x = wl.make_signal(w)
    base = torch.zeros(w.channels * (w.valid_len + 8) + 3, device="cuda")
    stride = w.valid_len + 7                                   # odd
    view = base[1:1 + w.channels * stride].view(w.channels, stride)   # starts 4 bytes off an 8-byte boundary
    view[:, :w.valid_len] = _dev(x)
    c_ref = plan.analyse(_dev(x), valid_len=w.valid_len)
    c_un = plan.analyse(view, valid_len=w.valid_len)
    assert torch.equal(torch.view_as_real(c_ref), torch.view_as_real(c_un))
    out = torch.full_like(view, 5.0)
    plan.synthesise(c_ref, valid_len=w.valid_len, out=out)
    ref = plan.synthesise(c_ref, valid_len=w.valid_len)
    assert torch.equal(out[:, :w.valid_len], ref)
    assert torch.all(out[:, w.valid_len:] == 5.0)
    plan.close()


def test_plan_create_default_entry_point_and_tiny_inputs():
    """cqt_plan_create (multiple-of-4 lengths, current device) and the smallest signals: N = 64, valid_len = 1."""
    import ctypes as C
    from paper_2609_29119_b200 import binding as B
    lib = B.load_library()
    h = C.c_void_p()
    assert lib.cqt_plan_create(64.0, 4.0, 32.0, 4, 64, 0, C.byref(h)) == 0
    assert lib.cqt_plan_signal_length(h) == 64 and lib.cqt_plan_device(h) == torch.cuda.current_device()
    nb, cc = lib.cqt_plan_num_bands(h), lib.cqt_plan_coeff_count(h)
    lay = orc.build_layout(64.0, 4.0, 32.0, 4, 64)
    assert (nb, cc) == (len(lay.bands), lay.coeff_count)
    ws = torch.empty(lib.cqt_plan_workspace_bytes(h, 2), dtype=torch.uint8, device="cuda")
    for vl in (64, 1, 63):
        x = torch.randn(2, vl, device="cuda")
        c = torch.empty((2, cc), dtype=torch.complex64, device="cuda")
        y = torch.empty_like(x)
        st = torch.cuda.current_stream().cuda_stream
        assert lib.cqt_analyse(h, x.data_ptr(), vl, 2, vl, c.data_ptr(), ws.data_ptr(), ws.numel(), st) == 0
        assert lib.cqt_synthesise(h, c.data_ptr(), 2, vl, y.data_ptr(), vl, ws.data_ptr(), ws.numel(), st) == 0
        want = orc.analyse(lay, orc.pad_signal(x.cpu().numpy(), 64))
        errs = band_rel_errors(lay, c.cpu().numpy(), want)
        assert errs.max() <= TOL
        assert snr_db(x.cpu().numpy(), y.cpu().numpy()).min() >= 120.0
    assert lib.cqt_plan_destroy(h) == 0


def test_plans_created_later_do_not_disturb_earlier_plans():
    """Kernel attributes (dynamic shared-memory limits) are shared by all plans of the process: a plan with small
    needs created after one with large needs must leave the first usable; both run interleaved on two streams."""
    wa = wl.scaled(wl.CONFIGS["config3"], channels=3)
    wb = small_workload("later_small", N=1 << 13, valid_len=1 << 13, fs=22050.0, fmin=100.0, fmax=11025.0,
                        bins_per_octave=12, m_policy=wl.M_SMOOTH, channels=2)
    pa = library_plan(wa)
    xa = _dev(wl.make_signal(wa))
    ref_a = pa.synthesise(pa.analyse(xa, valid_len=wa.valid_len), valid_len=wa.valid_len).clone()
    pb = library_plan(wb)                      # created after pa has run, with smaller kernels' needs
    pc = library_plan(wl.scaled(wl.CONFIGS["table1"], channels=1))
    xb = _dev(wl.make_signal(wb))
    ref_b = pb.synthesise(pb.analyse(xb, valid_len=wb.valid_len), valid_len=wb.valid_len).clone()
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(5):
        ya = pa.synthesise(pa.analyse(xa, valid_len=wa.valid_len, stream=sa), valid_len=wa.valid_len, stream=sa)
        yb = pb.synthesise(pb.analyse(xb, valid_len=wb.valid_len, stream=sb), valid_len=wb.valid_len, stream=sb)
        torch.cuda.synchronize()
        assert torch.equal(ya, ref_a) and torch.equal(yb, ref_b)
    assert snr_db(wl.make_signal(wa), ref_a.cpu().numpy()).min() >= 120.0
    pa.close(); pb.close(); pc.close()
