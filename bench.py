#!/usr/bin/env python3
"""Benchmark of the constant-Q analysis + synthesis round trip on B200.

A step is one pass of the whole hot path over one batch: cqt_analyse then cqt_synthesise of
every signal of the workload (default: 16 stereo clips of 10 s at 44.1 kHz, N = 2^19, 24 bins
per octave).  Prints one JSON line: throughput in true samples per second, the same measured end to end from
pinned host buffers, the step replayed as a CUDA graph, per-kernel durations, the dominant kernel and the whole
step against the measured HBM copy bandwidth and the FP32 peak, SM clocks sampled during the timed region, and
the CPU oracle timed on a bounded sample.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload configN]

--impl reference times the fp64 CPU oracle (the only reference implementation that exists for
this method) on a bounded sample of the same workload on the host cores.
With N > 1 ranks every rank runs an independent replica of the batch (the transform has no
exchange step); `value` is the job's aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import workloads as wl  # noqa: E402

METRIC = "cqt_round_trip_throughput"
UNIT = "Msamples/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


# --------------------------------------------------------------------------- CPU oracle arm
def oracle_sample(w: wl.Workload, budget_macs: float = 1.2e8):
    """Times the oracle on ONE channel of the workload, all of the long DFT and a strided subset of the bands
    (analysis and synthesis by direct per-band DFT), and extrapolates by the share of direct-DFT work sampled."""
    from threadpoolctl import threadpool_limits

    from oracle import nsgt_oracle as orc
    if w.sections:
        cen, wid, octave = orc.multires_bands(w.fs, w.fmin, w.N, w.sections, w.min_win)
        lay = orc.build_layout_bands(w.fs, w.N, cen, wid, w.window, w.m_policy, octave)
    else:
        lay = orc.build_layout(w.fs, w.fmin, w.fmax, w.bins_per_octave, w.N, window=w.window, policy=w.m_policy,
                               min_win=w.min_win)
    x = orc.pad_signal(wl.make_signal(w, n_channels=1)[0].astype(np.float64), w.N)
    work = np.array([float(b.M) * len(b.d) for b in lay.bands])
    # every stride-th band, smallest stride that keeps the sampled work under the budget
    stride = 1
    while work[::stride].sum() > budget_macs and stride < len(lay.bands):
        stride += 1
    sel = list(range(0, len(lay.bands), stride))
    frac = float(work[sel].sum() / work.sum())
    with threadpool_limits(limits=1):
        t0 = time.perf_counter()
        X = orc.long_dft(x)
        t1 = time.perf_counter()
        c = [orc.analyse_band(lay, X, i) for i in sel]
        t2 = time.perf_counter()
        orc.synthesise(lay, c, bands=sel)      # includes the inverse long DFT
        t3 = time.perf_counter()
    # long DFTs are done in full; the band work is scaled up to all bands
    t_long = (t1 - t0) * 2.0
    t_band_an = (t2 - t1) / frac
    t_band_sy = max(0.0, (t3 - t2) - (t1 - t0)) / frac
    est = t_long + t_band_an + t_band_sy
    return {"seconds_measured": t3 - t0, "seconds_full_round_trip_one_channel": est,
            "msamples_per_s": w.valid_len / est / 1e6, "work_fraction": frac, "bands_sampled": len(sel),
            "bands": len(lay.bands)}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # Every step is the same bounded sample; the run as a whole is bounded too: steps stop once the wall-clock
    # budget is spent (at least one warm-up-free timed step), and the line reports the steps actually timed.
    budget_s = 240.0
    t_start = time.perf_counter()
    vals, last, warm_done = [], None, 0
    while len(vals) < args.steps:
        spent = time.perf_counter() - t_start
        per = spent / max(1, warm_done + len(vals))
        if (vals or warm_done) and spent + per > budget_s:
            break
        last = oracle_sample(w, budget_macs=args.cpu_budget_macs)
        if warm_done < args.warmup and spent + 3 * per < budget_s and not vals and warm_done < 1:
            warm_done += 1          # one untimed pass warms numpy's caches; more would only spend the budget
        else:
            vals.append(last)
    est = statistics.mean(v["seconds_full_round_trip_one_channel"] for v in vals)
    value = w.valid_len / est / 1e6
    sample = (f"1 of {w.channels} channels; both long DFTs in full; {last['bands_sampled']} of {last['bands']} bands "
              f"({100 * last['work_fraction']:.2f} % of the direct-DFT work) analysed and synthesised, "
              f"band time scaled to all bands")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": len(vals),
            "warmup": warm_done, "steps_requested": args.steps, "warmup_requested": args.warmup,
            "ms_per_step": est * w.channels * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "channels": w.channels, "valid_len": w.valid_len, "N": w.N,
                       "bins_per_octave": w.bins_per_octave},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------- GPU arm
class ClockSampler:
    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
                 "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
                 "clocks_event_reasons.sw_power_cap")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "20",
                                          "-i", str(self.index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.06)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                p = [v.strip() for v in line.split(",")]
                if len(p) < 7:
                    continue
                try:
                    sm.append(float(p[0])); mx.append(float(p[1]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def max_over_ranks(value: float, device=None) -> float:
    """Largest `value` of any rank (the job's step time is the slowest replica's); identity on one rank."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(samples_per_rank: float, world: int, ms_total: float, steps: int) -> float:
    """Whole-job Msamples/s of `world` independent replicas given the slowest rank's time for `steps` steps."""
    return samples_per_rank * world / (ms_total / steps / 1e3) / 1e6


def kernel_algorithmic_bytes(plan, w, batch):
    """Minimal HBM bytes each kernel is responsible for per launch: signal samples, coefficients and window
    tables; the packed spectrum, the half spectrum and the weighted-bin rows are intermediates (0 bytes)."""
    cls_m = {}
    cls_s = {}
    for bi in plan.bands():
        cls_m[bi.launch_class] = cls_m.get(bi.launch_class, 0) + bi.M
        cls_s[bi.launch_class] = cls_s.get(bi.launch_class, 0) + bi.support
    sig = 4 * w.valid_len * batch
    two_pass = plan.N // 2 > 4096
    out = {"rfft_cols_fwd": sig if two_pass else 0, "rfft_rows_fwd": 0 if two_pass else sig,
           "irfft_cols": sig if two_pass else 0, "irfft_rows": 0 if two_pass else sig}
    for c in cls_m:
        b = 8 * cls_m[c] * batch + 4 * cls_s[c]
        if c < 0:      # bands on the two-pass kernels: pass 2 writes (analysis) / pass 1 reads (synthesis) the coefficients
            out["band2p_rows/analysis"] = b
            out["band2p_cols/synthesis"] = b
        else:
            out[f"bands_from_spectrum/class{c}"] = b
            out[f"bands_to_spectrum/class{c}"] = b
    return out


def path_algorithmic_bytes(plan, w, batch, second_is_adjoint=False):
    """Whole step: signal in, coefficients out, coefficients in, signal out, window tables once per transform."""
    return 2 * 4 * w.valid_len * batch + 2 * 8 * plan.coeff_count * batch + 2 * 4 * plan.table_length


def path_algorithmic_flops(plan, w, batch):
    """Radix-2 operation count of one step (two transforms): per signal 2.5 N log2(N/2) for each packed long FFT,
    5 M log2 M for each band transform, 16 per support entry for the window multiply and the fold / overlap-add."""
    import math
    bands = plan.bands()
    per_signal = 2.0 * (2.5 * w.N * math.log2(w.N / 2.0) + sum(5.0 * b.M * math.log2(b.M) for b in bands)) \
        + 2.0 * 16.0 * sum(b.support for b in bands)
    return per_signal * batch


# FP32 peak of the CUDA cores: 148 SMs x 128 lanes x 2 flop (FMA) x 1.965 GHz
FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


TUNING = {}   # fields of cqt_plan_tuning set with --tune (kernel-family comparisons)


def make_plan(w, device):
    from paper_2609_29119_b200 import Plan, multires_bands
    if w.sections:
        cen, wid, octave = multires_bands(w.fs, w.fmin, w.N, w.sections, w.min_win)
        return Plan.from_bands(w.fs, w.N, cen, wid, octave, window=w.window, m_policy=w.m_policy, device=device)
    return Plan(w.fs, w.fmin, w.fmax, w.bins_per_octave, w.N, window=w.window, m_policy=w.m_policy, min_win=w.min_win, **TUNING,
                device=device)


def capture_graph(fn):
    """Captures fn(stream) (library calls on that stream and the plan's helper streams) into a CUDA graph."""
    import torch
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        fn(torch.cuda.current_stream())
    torch.cuda.current_stream().wait_stream(side)
    return g


def measure_secondary(args, local):
    """The other batched workload of the benchmark set in the same run: 64 clips of 88,200 samples, N = 2^17, 48 bins
    per octave; a step is cqt_analyse followed by cqt_analyse_adjoint on a random complex cotangent.  Same protocol
    as the headline (warm-up, regions of K steps between CUDA events, median region), a quarter second of regions."""
    import torch
    w = wl.CONFIGS["config3"]
    dev = torch.device(f"cuda:{local}")
    plan = make_plan(w, local)
    batch = w.channels
    x = torch.from_numpy(wl.make_signal(w)).to(dev)
    cbar = torch.from_numpy(wl.make_cotangent(w, plan.coeff_count)).to(dev)
    c = torch.empty((batch, plan.coeff_count), dtype=torch.complex64, device=dev)
    xb = torch.empty_like(x)
    ws = plan.workspace(batch)
    stream = torch.cuda.current_stream()

    def step():
        plan.analyse(x, valid_len=w.valid_len, out=c, ws=ws, stream=stream)
        plan.analyse_adjoint(cbar, valid_len=w.valid_len, out=xb, ws=ws, stream=stream)

    K = args.steps
    for _ in range(max(3, args.warmup)):
        step()
    plan.synthesise(c, valid_len=w.valid_len, out=xb, ws=ws, stream=stream)
    torch.cuda.synchronize()
    xd, xrd = x.double(), xb.double()
    snr_min = float((10 * torch.log10((xd * xd).sum(1) / ((xd - xrd) ** 2).sum(1))).min().item())
    regions = []
    while (sum(regions) < 250.0 and len(regions) < 1000) or not regions:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(K):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
        regions.append(e0.elapsed_time(e1))
    ms = statistics.median(regions) / K
    peak, peak_kind = measured_peaks()
    path_bytes = path_algorithmic_bytes(plan, w, batch)
    out = {"workload": w.name, "step": "cqt_analyse + cqt_analyse_adjoint", "channels": batch, "valid_len": w.valid_len,
           "N": w.N, "bins_per_octave": w.bins_per_octave, "bands": plan.num_bands, "ms_per_step": ms,
           "ms_per_step_min": min(regions) / K, "ms_per_step_max": max(regions) / K, "regions": len(regions),
           "value": batch * w.valid_len / (ms * 1e-3) / 1e6, "unit": UNIT, "round_trip_snr_db_min": snr_min,
           "path_alg_bytes": path_bytes, "path_achieved": path_bytes / (ms * 1e-3) / 1e9,
           "path_frac": path_bytes / (ms * 1e-3) / 1e9 / peak, "peak_kind": peak_kind}
    plan.close()
    return out


def run_ours(args, w):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    dev = torch.device(f"cuda:{local}")
    batch = w.channels
    plan = make_plan(w, local)
    x_host = torch.from_numpy(wl.make_signal(w)).pin_memory()
    xr_host = torch.empty_like(x_host).pin_memory()
    x = x_host.to(dev)
    c = torch.empty((batch, plan.coeff_count), dtype=torch.complex64, device=dev)
    xr = torch.empty_like(x)
    ws = plan.workspace(batch)
    stream = torch.cuda.current_stream()

    adjoint_step = (w.name == "config3")     # that workload is forward analysis + its adjoint on a random cotangent
    if adjoint_step:
        cbar = torch.from_numpy(wl.make_cotangent(w, plan.coeff_count)).to(dev)

    def step(st=None):
        st = stream if st is None else st
        plan.analyse(x, valid_len=w.valid_len, out=c, ws=ws, stream=st)
        if adjoint_step:
            plan.analyse_adjoint(cbar, valid_len=w.valid_len, out=xr, ws=ws, stream=st)
        else:
            plan.synthesise(c, valid_len=w.valid_len, out=xr, ws=ws, stream=st)

    # End to end: every step copies its input from pinned host memory and its result back.  Three streams and two
    # sets of device buffers let step i+1's upload and step i-1's download run beside step i's kernels, as a caller
    # streaming batches through the public API would do; every copy of every step is inside the timed region.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    x2 = [x, torch.empty_like(x)]
    xr2 = [xr, torch.empty_like(xr)]
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_done = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]
    e2e_state = {"i": 0}

    def step_e2e():
        i = e2e_state["i"]
        e2e_state["i"] = i + 1
        b = i & 1
        s_in.wait_event(ev_done[b])          # the kernels that last read this input buffer have finished
        with torch.cuda.stream(s_in):
            x2[b].copy_(x_host, non_blocking=True)
            ev_in[b].record(s_in)
        stream.wait_event(ev_in[b])
        stream.wait_event(ev_out[b])         # the download that last read this output buffer has finished
        plan.analyse(x2[b], valid_len=w.valid_len, out=c, ws=ws, stream=stream)
        if adjoint_step:
            plan.analyse_adjoint(cbar, valid_len=w.valid_len, out=xr2[b], ws=ws, stream=stream)
        else:
            plan.synthesise(c, valid_len=w.valid_len, out=xr2[b], ws=ws, stream=stream)
        ev_done[b].record(stream)
        s_out.wait_event(ev_done[b])
        with torch.cuda.stream(s_out):
            xr_host.copy_(xr2[b], non_blocking=True)
            ev_out[b].record(s_out)

    def drain_e2e():
        stream.wait_stream(s_in)
        stream.wait_stream(s_out)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, k, after=None):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for _ in range(k):
            fn()
        if after is not None:
            after()                          # the closing event waits for the copies still in flight
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), dev)

    W, K = max(3, args.warmup), args.steps

    def median_region(fn, seconds, after=None):
        r = [timed(fn, K, after)]
        while sum(r) < seconds * 1e3 and len(r) < 1000:
            r.append(timed(fn, K, after))
        return statistics.median(r)

    for _ in range(W):
        step()
    torch.cuda.synchronize()
    # correctness guard of the timed configuration: fp32 round trip >= 120 dB on every channel
    if adjoint_step:
        plan.synthesise(c, valid_len=w.valid_len, out=xr, ws=ws, stream=stream)
    xd, xrd = x.double(), xr.double()
    snr = 10 * torch.log10((xd * xd).sum(1) / ((xd - xrd) ** 2).sum(1))
    snr_min = float(snr.min().item())

    # The K-step timed region is repeated until at least half a second of device time has passed (a single
    # region of 20 steps is 10 ms: too short for the clock sampler and for a steady figure); the median region
    # gives ms_per_step and value, minimum and maximum are printed beside it.
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = plan.launch_count()
    regions = [timed(step, K)]
    launches = plan.launch_count() - launches0
    while sum(regions) < args.min_seconds * 1e3 and len(regions) < 2000:
        regions.append(timed(step, K))
    clocks = sampler.stop()
    ms = statistics.median(regions)

    # the same step captured once as a CUDA graph and replayed (the paper times its round trip this way, Sec. 5)
    graph = capture_graph(step)
    for _ in range(W):
        graph.replay()
    ms_graph = median_region(graph.replay, 0.3 * args.min_seconds)

    # per-kernel durations: the same K steps with an event after every kernel
    plan.set_timing(True)
    for _ in range(K):
        step()
    per = {}
    for name, t in plan.read_timing(capacity=64 * K + 64):
        a = per.setdefault(name, [0, 0.0])
        a[0] += 1
        a[1] += t
    plan.set_timing(False)

    for _ in range(2):
        step_e2e()
    drain_e2e()
    ms_e2e = median_region(step_e2e, 0.3 * args.min_seconds, after=drain_e2e)

    value = job_throughput(float(batch) * w.valid_len, world, ms, K)
    e2e_value = job_throughput(float(batch) * w.valid_len, world, ms_e2e, K)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    alg = kernel_algorithmic_bytes(plan, w, batch)
    tot_ms = sum(v[1] for v in per.values())
    kernels = {n: {"launches": v[0], "avg_us": 1e3 * v[1] / v[0], "share": v[1] / tot_ms,
                   "alg_bytes": alg.get(n, 0),
                   "alg_gbs": alg.get(n, 0) / (v[1] / v[0] * 1e-3) / 1e9} for n, v in per.items()}
    # dominant kernel: the largest share of device time among the kernels that own algorithmic bytes (the passes
    # that only move intermediates have none to be measured against); the largest share overall is printed too
    largest = max(per, key=lambda n: per[n][1])
    dom = max((n for n in per if alg.get(n, 0) > 0), key=lambda n: per[n][1])
    dom_gbs = kernels[dom]["alg_gbs"]
    path_bytes = path_algorithmic_bytes(plan, w, batch)
    path_gbs = path_bytes / (ms / K * 1e-3) / 1e9
    traffic = traffic_total = None
    prof = os.path.join(ROOT, "profiles", "dram_traffic_workload2.txt")
    if os.path.exists(prof):
        try:
            table = json.load(open(prof)).get(w.name, {})
            traffic = table.get(dom)
            traffic_total = sum(table.values()) if table else None
        except Exception:
            traffic = traffic_total = None
    secondary = None
    if world == 1 and w.name == "config2" and not args.channels and not args.no_secondary:
        secondary = measure_secondary(args, local)
    cufft = None
    if world == 1 and not args.no_cufft_calibration:
        # the vendor FFT alone on the same transform sizes (no windowing, gather or overlap-add): context for the
        # per-kernel times above, never part of `value`
        try:
            from torchfft_baseline import cufft_same_shape_times
            cufft = cufft_same_shape_times(plan, batch, dev)
            cufft["unit"] = "us"
            cufft["step_over_fft_calls_only"] = (ms / K * 1e3) / cufft["round_trip_fft_calls_only"]
        except Exception as e:  # a calibration aid must never take the bench line down
            cufft = {"error": f"{type(e).__name__}: {e}"}
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        s = oracle_sample(w, budget_macs=args.cpu_budget_macs)
        cpu = {"value": s["msamples_per_s"], "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": (f"1 of {w.channels} channels; both long DFTs in full; {s['bands_sampled']} of {s['bands']} bands "
                          f"({100 * s['work_fraction']:.2f} % of the direct-DFT work), band time scaled to all bands; "
                          f"{s['seconds_measured']:.1f} s measured")}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "timed_regions": {"count": len(regions), "steps_each": K, "ms_per_step_median": ms / K,
                          "ms_per_step_min": min(regions) / K, "ms_per_step_max": max(regions) / K,
                          # time x clock: what the median step would take at the maximum SM clock
                          "ms_per_step_at_max_clock": (ms / K * clocks["sm_mhz"] / clocks["sm_max_mhz"])
                          if clocks["sm_mhz"] and clocks["sm_max_mhz"] else None},
        "config": {"workload": w.name, "channels_per_gpu": batch, "valid_len": w.valid_len, "N": w.N,
                   "bins_per_octave": w.bins_per_octave, "bands": plan.num_bands, "coeffs_per_channel": plan.coeff_count,
                   "round_trips_per_s": batch * world / (ms / K / 1e3), "l2": "inputs larger than L2 (no flush)",
                   "multi_gpu": "replicas only", "round_trip_snr_db_min": snr_min,
                   "step": "cqt_analyse + cqt_analyse_adjoint" if adjoint_step else "cqt_analyse + cqt_synthesise"},
        "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"],
                   "samples": clocks["samples"]},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(x_host.numel() * 4),
                "d2h_bytes_per_step": int(xr_host.numel() * 4), "ms_per_step": ms_e2e / K},
        "gpu_launches": int(launches),
        "graph_replay": {"ms_per_step": ms_graph / K, "value": job_throughput(float(batch) * w.valid_len, world, ms_graph, K),
                         "unit": UNIT},
        "roofline": {"bound": "hbm", "kernel": dom, "kernel_share": kernels[dom]["share"],
                     "largest_share_kernel": largest, "largest_share": kernels[largest]["share"], "achieved": dom_gbs, "peak": peak, "unit": "GB/s",
                     "frac": dom_gbs / peak, "traffic": traffic, "traffic_total": traffic_total, "peak_kind": peak_kind,
                     "path_achieved": path_gbs, "path_frac": path_gbs / peak, "path_alg_bytes": path_bytes},
        # the path is issue-bound on the CUDA cores, not bandwidth-bound: the same step against their FP32 peak
        "roofline_alu": {"bound": "alu", "achieved": path_algorithmic_flops(plan, w, batch) / (ms / K * 1e-3) / 1e12,
                         "peak": FP32_PEAK_TFLOPS, "unit": "TFLOP/s", "peak_kind": "148 SMs x 128 lanes x 2 x 1.965 GHz",
                         "frac": path_algorithmic_flops(plan, w, batch) / (ms / K * 1e-3) / 1e12 / FP32_PEAK_TFLOPS,
                         "flops_per_step": path_algorithmic_flops(plan, w, batch)},
        "kernels": kernels,
        "secondary": secondary,
        "cufft_same_shape": cufft,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_stream(args, w):
    """Sliced streaming workload: the whole stereo stream is pushed through one SliCQ object in pushes of
    `hops` half-slices and pulled after every push; reports stream samples per second and slices per second."""
    import torch

    from paper_2609_29119_b200 import SliCQ
    torch.cuda.set_device(0)
    plan = make_plan(w, 0)
    x = torch.from_numpy(wl.make_signal(w)).cuda()
    n, H = x.shape[1], w.slice_len // 2
    out = torch.empty((w.channels, n + 2 * w.slice_len), device="cuda")
    res = {}
    for label, hops in (("bulk_64_hops_per_push", 64), ("one_hop_per_push", 1)):
        sq = SliCQ(plan, w.channels, w.transition, max(2, hops + 1))

        def run_once():
            sq.reset()
            got = pos = 0
            while pos < n:
                m = min(hops * H, n - pos)
                sq.push(x[:, pos:pos + m])
                pos += m
                got += sq.pull(out[:, got:])
            sq.flush()
            got += sq.pull(out[:, got:])
            return got
        run_once()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        got = run_once()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        xd, yd = x.double(), out[:, :n].double()
        snr = float((10 * torch.log10((xd * xd).sum(1) / ((xd - yd) ** 2).sum(1))).min())
        slices = (n + H - 1) // H + 1
        res[label] = {"ms_total": ms, "msamples_per_s": w.channels * n / ms / 1e3, "slices_per_s": slices * w.channels / ms * 1e3,
                      "device_bytes": sq.device_bytes(), "snr_db_min": snr, "frames_out": got}
        sq.close()
    line = {"metric": "slicq_stream_throughput", "value": res["bulk_64_hops_per_push"]["msamples_per_s"], "unit": UNIT,
            "n_gpus": 1, "higher_is_better": True, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "channels": w.channels, "stream_samples": n, "slice_len": w.slice_len,
                       "transition": w.transition, "bins_per_octave": w.bins_per_octave}, "stream": res}
    print(json.dumps(line))


# the paper's Fig. 2(a): A100 round trip under graph replay, ms per batch size (its Table 2 row is the B = 1 entry)
PAPER_A100_MS = {1: 0.116, 2: 0.109, 4: 0.131, 8: 0.185, 16: 0.273, 32: 0.461, 64: 0.844, 128: 1.656}
# its Fig. 2(b): analysis, synthesis, squared loss and backpropagation in eager mode, A100, ms
PAPER_A100_BACKWARD_MS = {1: 1.969, 2: 1.975, 4: 2.003, 8: 2.012, 16: 2.031, 32: 2.474, 64: 4.601, 128: 8.779}


def run_sweep(args, w):
    """Batch sweep of the paper's principal configuration (Sec. 4 layout, Sec. 5 protocol): for every batch size the
    round trip is timed eagerly, under graph replay with everything left in cache (the paper's protocol: median of
    50 replays after 3 warm-ups), and under graph replay with the L2 cache flushed before every replay."""
    import torch
    torch.cuda.set_device(0)
    plan = make_plan(w, 0)
    batches = [args.channels] if args.channels else sorted(PAPER_A100_MS)
    if not args.no_torchfft:
        from torchfft_baseline import TorchFftCqt
        tf = TorchFftCqt(plan, torch.device("cuda:0"))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")     # larger than the 126 MB L2
    stream = torch.cuda.current_stream()
    K = min(args.steps, 50)
    W = max(3, args.warmup)
    sweep = {}
    sampler = ClockSampler(0)
    sampler.start()
    launches0 = plan.launch_count()
    for B in batches:
        wb = wl.scaled(w, channels=B)
        x = torch.from_numpy(wl.make_signal(wb)).cuda()
        c = torch.empty((B, plan.coeff_count), dtype=torch.complex64, device="cuda")
        xr = torch.empty_like(x)
        ws = plan.workspace(B)

        def step(st=None):
            st = stream if st is None else st
            plan.analyse(x, valid_len=w.valid_len, out=c, ws=ws, stream=st)
            plan.synthesise(c, valid_len=w.valid_len, out=xr, ws=ws, stream=st)

        def median_ms(fn, cold):
            ts = []
            for i in range(W + K):
                if cold:
                    flush.fill_(i & 255)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                fn()
                e1.record(stream)
                e1.synchronize()
                if i >= W:
                    ts.append(e0.elapsed_time(e1))
            return statistics.median(ts)
        eager = median_ms(step, False)
        # differentiable step (Sec. 5, second experiment): analysis, synthesis, squared loss, backward, eager
        from paper_2609_29119_b200 import autograd as ad
        xg = x.clone().requires_grad_(True)

        def train_step():
            xg.grad = None
            y = ad.synthesise(plan, ad.analyse(plan, xg))
            ((y - x) ** 2).sum().backward()
        backward = median_ms(train_step, False)
        graph = capture_graph(step)
        hot = median_ms(graph.replay, False)
        cold = median_ms(graph.replay, True)
        # same-box comparator (the paper's "CQT baseline": the operator through torch.fft / cuFFT calls)
        tf_res = {}
        if not args.no_torchfft:
            def tf_step(st=None):
                tf.synthesise(tf.analyse(x))
            tf_y = tf.synthesise(tf.analyse(x))
            xd0, yd0 = x.double(), tf_y.double()
            tf_snr = float((10 * torch.log10((xd0 * xd0).sum(1) / ((xd0 - yd0) ** 2).sum(1))).min())
            tf_eager = median_ms(tf_step, False)
            tf_graph = capture_graph(tf_step)
            tf_hot = median_ms(tf_graph.replay, False)
            del tf_graph
            tf_res = {"torchfft_eager_ms": tf_eager, "torchfft_graph_ms": tf_hot, "torchfft_snr_db_min": tf_snr,
                      "speedup_vs_torchfft_graph": tf_hot / hot, "speedup_vs_torchfft_eager": tf_eager / eager}
        xd, xrd = x.double(), xr.double()
        snr = float((10 * torch.log10((xd * xd).sum(1) / ((xd - xrd) ** 2).sum(1))).min())
        sweep[str(B)] = {"eager_ms": eager, "graph_ms": hot, "graph_l2_flushed_ms": cold, "snr_db_min": snr,
                         "paper_a100_graph_ms": PAPER_A100_MS.get(B),
                         "step_with_backward_eager_ms": backward, "paper_a100_backward_ms": PAPER_A100_BACKWARD_MS.get(B), "workspace_mb_per_signal": plan.workspace_bytes(B) / B / 1e6,
                         "msamples_per_s_l2_flushed": B * w.valid_len / cold / 1e3, **tf_res}
        del graph
    launches = plan.launch_count() - launches0
    clocks = sampler.stop()
    top = str(batches[-1])
    peak, peak_kind = measured_peaks()
    path_bytes = path_algorithmic_bytes(plan, w, batches[-1])
    gbs = path_bytes / (sweep[top]["graph_l2_flushed_ms"] * 1e-3) / 1e9
    paper = PAPER_A100_MS.get(batches[-1])
    value = sweep[top]["msamples_per_s_l2_flushed"]
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W,
            "ms_per_step": sweep[top]["graph_l2_flushed_ms"], "higher_is_better": True, "scaling": "weak",
            # the paper's number for this workload and batch is an A100 measurement: context, not a like-for-like target
            "vs_baseline": (value / (batches[-1] * w.valid_len / paper / 1e3)) if paper else None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "batch": batches[-1], "N": w.N, "sections": [list(s) for s in w.sections],
                       "bands": plan.num_bands, "coeffs_per_channel": plan.coeff_count,
                       "l2": "value: L2 flushed (256 MB written) before every timed replay; graph_ms: caches left warm, as the paper times it",
                       "timing": "median of %d graph replays after %d warm-ups, one CUDA-event pair per replay" % (K, W)},
            "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"],
                       "samples": clocks["samples"]},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "kernel": "whole round trip", "achieved": gbs, "peak": peak, "unit": "GB/s",
                         "frac": gbs / peak, "traffic": None, "peak_kind": peak_kind},
            "sweep": sweep}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config2", choices=sorted(wl.CONFIGS))
    ap.add_argument("--channels", type=int, default=None, help="override the number of signals (profiling on small cases)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--single", action="store_true", help="table1: one batch size through the standard step loop instead of the sweep")
    ap.add_argument("--cpu-budget-macs", type=float, default=1.2e8)
    ap.add_argument("--min-seconds", type=float, default=0.5,
                    help="repeat the timed region of --steps steps until this much device time has passed")
    ap.add_argument("--no-secondary", action="store_true", help="skip the second batched workload (config3)")
    ap.add_argument("--no-cufft-calibration", action="store_true",
                    help="skip timing the vendor FFT alone on the step's transform sizes")
    ap.add_argument("--no-torchfft", action="store_true", help="table1 sweep: skip the torch.fft comparator")
    ap.add_argument("--tune", action="append", default=[], metavar="FIELD=VALUE",
                    help="a field of cqt_plan_tuning (max_cta_elems, two_pass_min); "
                         "the defaults are what the library ships with")
    args = ap.parse_args()
    for kv in args.tune:
        k, v = kv.split("=")
        TUNING[k] = int(v)
    w = wl.CONFIGS[args.workload]
    if args.channels:
        w = wl.scaled(w, channels=args.channels)
    if args.impl == "reference":
        run_reference(args, w)
    elif w.slice_len:
        run_stream(args, w)
    elif w.name == "table1" and not args.single:
        run_sweep(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
