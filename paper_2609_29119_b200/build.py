"""Builds libcqt_b200.so (sm_100a) in-tree with nvcc.  Usage: python -m paper_2609_29119_b200.build [--force]"""
from __future__ import annotations

import concurrent.futures as cf
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libcqt_b200.so")
SOURCES = ["layout.cpp", "api.cu", "band.cu", "band_analysis.cu", "band_synthesis.cu", "band_two_pass.cu", "long_fft.cu", "slicq.cu", "static_ws.cu"]
HEADERS = ["layout.hpp", "plan_types.h", "internal.hpp", "engine.cuh", "band_common.cuh", 
           "static_fft.cuh", "codelets_gen.cuh",
           os.path.join("..", "..", "include", "cqt.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """debug_bounds=True (or CQT_DEBUG_BOUNDS=1 in the environment) compiles the index self-checks in: an
    out-of-range index is recorded for cqt_plan_check and the access skipped (slower; for debugging only)."""
    debug_bounds = debug_bounds or os.environ.get("CQT_DEBUG_BOUNDS") == "1"
    flags_extra = ["-DCQT_DEBUG_BOUNDS"] if debug_bounds else []
    stamp = os.path.join(OBJ, "debug_bounds.stamp")
    os.makedirs(OBJ, exist_ok=True)
    if debug_bounds != os.path.exists(stamp):
        force = True
        if debug_bounds:
            open(stamp, "w").close()
        else:
            os.unlink(stamp)
    # the register codelets are written by a script; the header is not under version control
    gen = os.path.join(CSRC, "gen_codelets.py")
    gen_out = os.path.join(CSRC, "codelets_gen.cuh")
    if force or _stale(gen_out, [gen]):
        res = subprocess.run([sys.executable, gen, gen_out], capture_output=True, text=True)
        if res.returncode:
            sys.stderr.write(res.stdout + res.stderr)
            raise RuntimeError("gen_codelets.py failed")
    hdrs = [os.path.join(CSRC, h) for h in HEADERS]
    nvcc = _nvcc()
    jobs = []
    objs = []
    for s in SOURCES:
        src = os.path.join(CSRC, s)
        obj = os.path.join(OBJ, os.path.splitext(s)[0] + ".o")
        objs.append(obj)
        if force or _stale(obj, [src] + hdrs):
            cmd = [nvcc] + NVCC_FLAGS + flags_extra + (["-Xptxas", "-v"] if verbose else []) + ["-x", "cu", "-c", src, "-o", obj]
            jobs.append(cmd)
    if jobs:
        with cf.ThreadPoolExecutor(max_workers=min(8, len(jobs))) as ex:
            for cmd, res in zip(jobs, ex.map(lambda c: subprocess.run(c, capture_output=True, text=True), jobs)):
                if verbose or res.returncode:
                    sys.stderr.write(" ".join(cmd) + "\n" + res.stdout + res.stderr)
                if res.returncode:
                    raise RuntimeError("nvcc failed for " + cmd[-3])
    if jobs or force or _stale(LIB, objs):
        cmd = [nvcc, "-shared", "-o", LIB] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode:
            sys.stderr.write(res.stdout + res.stderr)
            raise RuntimeError("link failed")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
