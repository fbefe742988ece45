"""Gradients through the differentiable wrappers against gradients assembled from the oracle's adjoints (Sec. 3.2):
for L = 1/2 ||S T x - t||^2 the gradient is T' S' (S T x - t); for a loss on the coefficients it is T' of the cotangent."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import workloads as wl
from helpers import library_plan, oracle_layout, small_workload, snr_db, split_bands
from oracle import nsgt_oracle as orc

pytestmark = pytest.mark.gpu

CASES = [
    small_workload("ad_n4096", N=4096, valid_len=4096, fs=22050.0, fmin=200.0, fmax=11025.0, bins_per_octave=24,
                   m_policy=wl.M_SMOOTH, channels=2),
    small_workload("ad_ragged", N=4096, valid_len=3001, fs=22050.0, fmin=200.0, fmax=11025.0, bins_per_octave=12,
                   m_policy=wl.M_MULT4, channels=2),
    small_workload("ad_multires", N=8192, valid_len=8192, fs=8192.0, fmin=100.0, fmax=4096.0, bins_per_octave=0,
                   m_policy=wl.M_POW2, channels=2, sections=((2, 4), (2, 8), (1, 16))),
]


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_round_trip_loss_gradient_matches_oracle_adjoints(w):
    from paper_2609_29119_b200 import autograd as ad
    lay, plan = oracle_layout(w), library_plan(w)
    x = wl.make_signal(w)
    t = np.random.default_rng(w.seed + 1).standard_normal(x.shape).astype(np.float32)
    xd = torch.from_numpy(x).cuda().requires_grad_(True)
    c = ad.analyse(plan, xd, valid_len=w.valid_len)
    c.retain_grad()
    y = ad.synthesise(plan, c, valid_len=w.valid_len)
    loss = 0.5 * ((y - torch.from_numpy(t).cuda()) ** 2).sum()
    loss.backward()
    # oracle: residual r = S T x - t on the true samples (zero beyond), grad_c = S' r, grad_x = T' grad_c
    x64 = orc.pad_signal(x, w.N)
    r = orc.synthesise(lay, orc.analyse(lay, x64))
    r[..., w.valid_len:] = 0.0
    r[..., :w.valid_len] -= t
    gc = orc.synthesise_adjoint(lay, r)
    gx = orc.analyse_adjoint(lay, gc)[..., :w.valid_len]
    got_x = xd.grad.cpu().numpy()
    got_c = split_bands(lay, c.grad.cpu().numpy())
    assert min(snr_db(gx, got_x)) >= 100.0, snr_db(gx, got_x)     # 1e-5 relative
    for a, b in zip(got_c, gc):
        assert np.linalg.norm(a - b) <= 1e-5 * np.linalg.norm(b)
    plan.close()


def test_coefficient_loss_gradient_and_padding_columns():
    """Loss on the coefficients of a strided, over-wide input: gradient = T'(cotangent) on the true samples, zero beyond."""
    from paper_2609_29119_b200 import autograd as ad
    w = CASES[1]
    lay, plan = oracle_layout(w), library_plan(w)
    x = wl.make_signal(w)
    wide = np.zeros((x.shape[0], w.valid_len + 17), dtype=np.float32)
    wide[:, :w.valid_len] = x
    xd = torch.from_numpy(wide).cuda().requires_grad_(True)
    m = wl.make_cotangent(w, lay.coeff_count)
    c = ad.analyse(plan, xd, valid_len=w.valid_len)
    loss = (c * torch.from_numpy(m).cuda().conj()).real.sum()     # <m, c>: cotangent is m
    loss.backward()
    want = orc.analyse_adjoint(lay, split_bands(lay, m.astype(np.complex128)))[..., :w.valid_len]
    got = xd.grad.cpu().numpy()
    assert np.all(got[:, w.valid_len:] == 0)
    assert min(snr_db(want, got[:, :w.valid_len])) >= 100.0
    plan.close()
