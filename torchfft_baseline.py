"""Same-box comparator: the constant-Q round trip evaluated with torch.fft (cuFFT) calls.

This restates the comparison system of the paper's Sec. 5 ("CQT baseline"): one real FFT of the batch, the bands
gathered and weighted from precomputed index and window tables, equal-length band transforms batched into one
inverse FFT per length, and on the way back one forward FFT per length, dual-window weighting, a scatter-add
into the half spectrum and one real inverse FFT.  Same windows, native coefficient lengths and sidebands as the
library (the tables are read from the library's plan), no zero-padding to a common length.

It is NOT part of the library and nothing in the package imports it: bench.py times it beside the library
(`--workload table1`), and a GPU test checks that both compute the same coefficients.
"""
from __future__ import annotations

import numpy as np


class TorchFftCqt:
    def __init__(self, plan, device):
        import torch
        self.N = plan.N
        self.coeff_count = plan.coeff_count
        g, h = plan.tables()
        half = self.N // 2
        groups = {}
        for bi in plan.bands():
            groups.setdefault(int(bi.M), []).append(bi)
        self.groups = []
        for M, bands in sorted(groups.items()):
            nb = len(bands)
            smax = max(int(b.support) for b in bands)
            src = np.zeros((nb, smax), dtype=np.int64)       # bin index into the half spectrum (mirrored where outside)
            conj = np.zeros((nb, smax), dtype=bool)          # bins outside 0..N/2 are conjugates of their mirror bins
            slot = np.zeros((nb, smax), dtype=np.int64)      # local slot d mod M
            gw = np.zeros((nb, smax), dtype=np.float32)      # analysis weight g / 1 (ifft carries the 1/M)
            hw = np.zeros((nb, smax), dtype=np.float32)      # dual weight, 0 on entries outside 0..N/2
            valid = np.zeros((nb, smax), dtype=bool)
            off = np.zeros(nb, dtype=np.int64)
            for r, b in enumerate(bands):
                S, d0, kc, t = int(b.support), int(b.first_offset), int(b.centre_bin), int(b.table_offset)
                d = d0 + np.arange(S)
                k = kc + d
                km = np.where(k < 0, -k, np.where(k > half, self.N - k, k))
                src[r, :S] = km
                conj[r, :S] = (k < 0) | (k > half)
                slot[r, :S] = d % M
                gw[r, :S] = g[t:t + S]
                hw[r, :S] = h[t:t + S]
                valid[r, :S] = True
                off[r] = int(b.coeff_offset)
            # padding entries: weight 0, routed to slot 0 / bin 0 (they add exact zeros)
            dev = lambda a: torch.from_numpy(a).to(device)
            rows = np.arange(nb)[:, None].repeat(smax, 1)
            self.groups.append(dict(M=M, nb=nb, src=dev(src.ravel()), conj=dev(np.where(conj, -1.0, 1.0).astype(np.float32).ravel()),
                                    flat_slot=dev((rows * M + slot).ravel()), gw=dev(gw.ravel()), hw=dev((hw * valid).ravel()),
                                    out_index=dev((off[:, None] + np.arange(M)[None, :]).ravel())))

    def analyse(self, x):
        """x [B, N] float32 -> c [B, coeff_count] complex64."""
        import torch
        B = x.shape[0]
        X = torch.fft.rfft(x, n=self.N)                                       # [B, N/2+1]
        c = torch.empty((B, self.coeff_count), dtype=torch.complex64, device=x.device)
        for g in self.groups:
            v = X[:, g["src"]]
            v = torch.complex(v.real, v.imag * g["conj"]) * g["gw"]
            u = torch.zeros((B, g["nb"] * g["M"]), dtype=torch.complex64, device=x.device)
            u.index_add_(1, g["flat_slot"], v)                               # slots are distinct per band: a plain placement
            cb = torch.fft.ifft(u.view(B, g["nb"], g["M"]), dim=-1)
            c[:, g["out_index"]] = cb.reshape(B, -1)
        return c

    def synthesise(self, c):
        """c [B, coeff_count] complex64 -> x [B, N] float32."""
        import torch
        B = c.shape[0]
        Xh = torch.zeros((B, self.N // 2 + 1), dtype=torch.complex64, device=c.device)
        for g in self.groups:
            U = torch.fft.fft(c[:, g["out_index"]].view(B, g["nb"], g["M"]), dim=-1).reshape(B, -1)
            v = U[:, g["flat_slot"]] * g["hw"]
            Xh.index_add_(1, g["src"], v)                                     # overlap-add with repeated indices
        Xh[:, 0] = Xh[:, 0].real.to(torch.complex64)
        Xh[:, -1] = Xh[:, -1].real.to(torch.complex64)
        return torch.fft.irfft(Xh, n=self.N)


def _smooth_at_least(n: int) -> int:
    """Smallest length 2^a 3^b 5^c >= n."""
    best = None
    p2 = 1
    while p2 < 2 * n:
        p3 = p2
        while p3 < 2 * n:
            p5 = p3
            while p5 < 2 * n:
                if p5 >= n and (best is None or p5 < best):
                    best = p5
                p5 *= 5
            p3 *= 3
        p2 *= 2
    return best


def cufft_same_shape_times(plan, batch, device, class_limits=(128, 1024, 4096, 13500), iters=20, warmup=5):
    """Calibration: what the vendor FFT needs for transforms of the round trip's sizes alone.

    One `torch.fft.rfft` / `irfft` of the batch at the plan's signal length, and per band-length class ONE batched
    complex transform of (bands in the class x batch) rows at the 5-smooth length nearest above the class's mean
    band length, so that each call moves the element count of the class within a few percent.  No windowing,
    gather, zero fill, overlap-add or ragged lengths: this is a lower bound of what a pipeline assembled from
    library FFTs spends inside the FFT calls, measured with CUDA events on the current stream, three rotating
    inputs (together larger than the L2 at the headline size).  Returns microseconds per call.
    """
    import torch

    def timed(fn):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize(device)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize(device)
        return a.elapsed_time(b) / iters * 1e3

    out = {}
    turn = [0]
    xs = [torch.randn(batch, plan.N, device=device) for _ in range(3)]

    def fwd():
        turn[0] += 1
        return torch.fft.rfft(xs[turn[0] % 3])
    out["rfft"] = timed(fwd)
    Xs = [torch.fft.rfft(x) for x in xs]
    del xs

    def inv():
        turn[0] += 1
        return torch.fft.irfft(Xs[turn[0] % 3], n=plan.N)
    out["irfft"] = timed(inv)
    del Xs
    lengths = [int(b.M) for b in plan.bands()]
    lo = 0
    classes = {}
    for ci, hi in enumerate(list(class_limits) + [max(lengths) + 1]):
        mine = [m for m in lengths if lo < m <= hi]
        lo = hi
        if not mine:
            continue
        M = _smooth_at_least(-(-sum(mine) // len(mine)))
        rows = len(mine) * batch
        cs = [torch.randn(rows, M, dtype=torch.complex64, device=device) for _ in range(3)]
        dst = torch.empty_like(cs[0])

        def c2c():
            turn[0] += 1
            torch.fft.fft(cs[turn[0] % 3], out=dst)
        classes[f"class{ci}"] = {"rows": rows, "length": M, "elements_vs_class": rows * M / (sum(mine) * batch),
                                 "us": timed(c2c)}
        del cs, dst
    out["classes"] = classes
    out["band_ffts_one_direction"] = sum(c["us"] for c in classes.values())
    out["round_trip_fft_calls_only"] = out["rfft"] + out["irfft"] + 2 * out["band_ffts_one_direction"]
    return out
