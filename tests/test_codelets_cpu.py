"""The register codelets the CUDA kernels are built from, checked on the CPU: the generator's output is plain
arithmetic, so it compiles with g++ (the device qualifiers defined away) and every radix is compared with the
DFT definition X_k = sum_n x_n exp(-2 pi i k n / R) evaluated in double precision, for both signs."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2609_29119_b200", "csrc")

HARNESS = r"""
#include <cmath>
#include <complex>
#include <cstdio>
#include <vector>
#define __device__
#define __forceinline__ inline
#include "codelets_gen.cuh"
template <int R> void check() {
    float re[R], im[R], re2[R], im2[R];
    std::vector<std::complex<double>> x(R);
    for (int i = 0; i < R; ++i) {
        re[i] = re2[i] = (float)std::sin(1.3 * i + 0.2);
        im[i] = im2[i] = (float)std::cos(2.1 * i * i + 0.5);
        x[i] = {re[i], im[i]};
    }
    cqt::Codelet<R>::run(re, im);      // forward
    cqt::Codelet<R>::run(im2, re2);    // inverse: the same routine with the arrays exchanged
    double ef = 0, ei = 0, nrm = 0;
    for (int k = 0; k < R; ++k) {
        std::complex<double> f = 0, b = 0;
        for (int n = 0; n < R; ++n) {
            f += x[n] * std::polar(1.0, -2 * M_PI * k * n / R);
            b += x[n] * std::polar(1.0, +2 * M_PI * k * n / R);
        }
        ef += std::norm(f - std::complex<double>(re[k], im[k]));
        ei += std::norm(b - std::complex<double>(re2[k], im2[k]));
        nrm += std::norm(f);
    }
    std::printf("%d %.3e %.3e\n", R, std::sqrt(ef / nrm), std::sqrt(ei / nrm));
}
int main() { RADIX_CALLS return 0; }
"""


def test_generated_codelets_match_the_dft_definition(tmp_path):
    sys.path.insert(0, CSRC)
    try:
        import gen_codelets
    finally:
        sys.path.pop(0)
    hdr = tmp_path / "codelets_gen.cuh"
    gen_codelets.emit(gen_codelets.RADICES, str(hdr))
    calls = " ".join(f"check<{r}>();" for r in gen_codelets.RADICES)
    src = tmp_path / "check.cpp"
    src.write_text(HARNESS.replace("RADIX_CALLS", calls))
    exe = tmp_path / "check"
    subprocess.run(["g++", "-O1", "-std=c++17", "-I", str(tmp_path), str(src), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split("\n")
    seen = []
    for line in out:
        if not line.strip():
            continue
        r, ef, ei = line.split()
        seen.append(int(r))
        # fp32 arithmetic, at most ~10 operations deep: a few ulp
        assert float(ef) < 1e-6 and float(ei) < 1e-6, line
    assert seen == list(gen_codelets.RADICES)
