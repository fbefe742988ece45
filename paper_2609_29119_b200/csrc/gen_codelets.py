#!/usr/bin/env python3
"""Writes codelets_gen.cuh: straight-line, register-resident forward DFTs of small length R.

`Codelet<R>::run(re, im)` overwrites its arguments with X_k = sum_n x_n exp(-2 pi i k n / R), k in natural
order.  The inverse (sign +) is the same routine called with the two arrays exchanged, which costs nothing
in registers.  Composite lengths are built from hand-derived 2, 3, 4 and 5 point kernels with the
Cooley-Tukey split n = RB*na + nb, k = ka + RA*kb; the intermediate twiddles are literal constants and the
trivial ones (1, -1, +-i, (+-1 +- i)/sqrt 2) are special-cased.  Every value carries its sign symbolically,
so a multiplication by -1 or +-i never costs an instruction: it turns a later addition into a subtraction
or flips the sign of a literal.  The scalar type T is a template parameter; the header supplies
mulc(c, x) = c x and fmac(c, x, acc) = c x + acc for float.

The build (paper_2609_29119_b200/build.py) runs this script; the header is not kept under version control.
Run by hand:  python gen_codelets.py [output path]
"""
import math
import os
import sys
SPLIT = {6: (2, 3), 8: (2, 4), 9: (3, 3), 10: (2, 5), 12: (4, 3), 15: (3, 5), 16: (4, 4),
         20: (4, 5), 25: (5, 5), 27: (3, 9), 32: (4, 8), 18: (2, 9), 24: (8, 3), 30: (2, 15)}

class E:
    def __init__(s): s.lines = []; s.n = 0
    def let(s, expr):
        s.n += 1; nm = f"t{s.n}"; s.lines.append(f"    const T {nm} = {expr};"); return nm

def lit(v): return f"{v:.9e}f"
# a value = (name, sign)
def vadd(e, a, b):
    (an, as_), (bn, bs) = a, b
    if as_ > 0 and bs > 0: return (e.let(f"{an} + {bn}"), 1)
    if as_ > 0 and bs < 0: return (e.let(f"{an} - {bn}"), 1)
    if as_ < 0 and bs > 0: return (e.let(f"{bn} - {an}"), 1)
    return (e.let(f"{an} + {bn}"), -1)
def vneg(a): return (a[0], -a[1])
def vsub(e, a, b): return vadd(e, a, vneg(b))
def vscale(e, c, a): return (e.let(f"mulc({lit(c * a[1])}, {a[0]})"), 1)
def vfma(e, c, x, acc):  # acc + c*x
    if acc[1] > 0: return (e.let(f"fmac({lit(c * x[1])}, {x[0]}, {acc[0]})"), 1)
    return (e.let(f"fmac({lit(-c * x[1])}, {x[0]}, {acc[0]})"), -1)
def add(e, a, b): return (vadd(e, a[0], b[0]), vadd(e, a[1], b[1]))
def sub(e, a, b): return (vsub(e, a[0], b[0]), vsub(e, a[1], b[1]))
def mul_neg_i(a): return (a[1], vneg(a[0]))
def mul_pos_i(a): return (vneg(a[1]), a[0])
def cmul_const(e, a, num, den):
    num %= den
    if num == 0: return a
    if 4 * num == den: return mul_neg_i(a)
    if 2 * num == den: return (vneg(a[0]), vneg(a[1]))
    if 4 * num == 3 * den: return mul_pos_i(a)
    ang = -2.0 * math.pi * num / den
    c, s = math.cos(ang), math.sin(ang)
    if 8 * num % den == 0:
        r = math.sqrt(0.5)
        sc, ss = (1 if c > 0 else -1), (1 if s > 0 else -1)
        # r[(sc x - ss y) + i (ss x + sc y)]
        x, y = a
        p = vadd(e, (x[0], x[1] * sc), (y[0], -y[1] * ss))
        q = vadd(e, (x[0], x[1] * ss), (y[0], y[1] * sc))
        return (vscale(e, r, p), vscale(e, r, q))
    x, y = a
    # re = c x - s y ; im = c y + s x
    t1 = vscale(e, -s, y); re = vfma(e, c, x, t1)
    t2 = vscale(e, s, x); im = vfma(e, c, y, t2)
    return (re, im)
def scale(e, a, v): return (vscale(e, v, a[0]), vscale(e, v, a[1]))
def fma_c(e, acc, v, x): return (vfma(e, v, x[0], acc[0]), vfma(e, v, x[1], acc[1]))
def dft2(e, x): return [add(e, x[0], x[1]), sub(e, x[0], x[1])]
def dft3(e, x):
    s = add(e, x[1], x[2]); d = sub(e, x[1], x[2]); X0 = add(e, x[0], s)
    m1 = fma_c(e, x[0], -0.5, s); k = math.sin(2.0 * math.pi / 3.0)
    m2 = (vscale(e, k, d[1]), vscale(e, -k, d[0]))
    return [X0, add(e, m1, m2), sub(e, m1, m2)]
def dft4(e, x):
    a = add(e, x[0], x[2]); b = sub(e, x[0], x[2]); c = add(e, x[1], x[3]); d = sub(e, x[1], x[3])
    nd = mul_neg_i(d)
    return [add(e, a, c), add(e, b, nd), sub(e, a, c), sub(e, b, nd)]
def dft5(e, x):
    c1, c2 = math.cos(2 * math.pi / 5), math.cos(4 * math.pi / 5)
    s1, s2 = math.sin(2 * math.pi / 5), math.sin(4 * math.pi / 5)
    p1 = add(e, x[1], x[4]); p2 = add(e, x[2], x[3]); d1 = sub(e, x[1], x[4]); d2 = sub(e, x[2], x[3])
    X0 = add(e, add(e, x[0], p1), p2)
    a1 = fma_c(e, fma_c(e, x[0], c1, p1), c2, p2)
    a2 = fma_c(e, fma_c(e, x[0], c2, p1), c1, p2)
    b1 = fma_c(e, scale(e, d1, s1), s2, d2)
    b2 = fma_c(e, scale(e, d1, s2), -s1, d2)
    nb1 = mul_neg_i(b1); nb2 = mul_neg_i(b2)
    return [X0, add(e, a1, nb1), add(e, a2, nb2), sub(e, a2, nb2), sub(e, a1, nb1)]
BASE = {2: dft2, 3: dft3, 4: dft4, 5: dft5}
def dft(e, x):
    R = len(x)
    if R in BASE: return BASE[R](e, x)
    RA, RB = SPLIT[R]
    t = [[None] * RA for _ in range(RB)]
    for nb in range(RB):
        col = dft(e, [x[RB * na + nb] for na in range(RA)])
        for ka in range(RA): t[nb][ka] = cmul_const(e, col[ka], nb * ka, R)
    out = [None] * R
    for ka in range(RA):
        row = dft(e, [t[nb][ka] for nb in range(RB)])
        for kb in range(RB): out[ka + RA * kb] = row[kb]
    return out
def emit(radices, path, ns="cqt"):
    out = ["// GENERATED by gen_codelets.py - do not edit by hand.",
           "// Register-resident forward DFT codelets; the inverse is Codelet<R>::run(im, re).",
           "#pragma once", "", f"namespace {ns} {{", "",
           "__device__ __forceinline__ float mulc(float c, float x) { return c * x; }",
           "__device__ __forceinline__ float fmac(float c, float x, float acc) { return fmaf(c, x, acc); }",
           "__device__ __forceinline__ float neg(float x) { return -x; }", "",
           "template <int R> struct Codelet;", ""]
    for R in radices:
        e = E()
        xin = [((e.let(f"re[{i}]"), 1), (e.let(f"im[{i}]"), 1)) for i in range(R)]
        res = dft(e, xin)
        out.append(f"template <> struct Codelet<{R}> {{")
        out.append(f"  template <class T> static __device__ __forceinline__ void run(T (&re)[{R}], T (&im)[{R}]) {{")
        out.extend(e.lines)
        for k, (a, b) in enumerate(res):
            fa = a[0] if a[1] > 0 else f"neg({a[0]})"
            fb = b[0] if b[1] > 0 else f"neg({b[0]})"
            out.append(f"    re[{k}] = {fa}; im[{k}] = {fb};")
        out.append("  }"); out.append("};"); out.append("")
    out.append(f"}}  // namespace {ns}")
    open(path, "w").write("\n".join(out) + "\n")
RADICES = [2, 3, 4, 5, 6, 8, 9, 10, 12, 15, 16]

if __name__ == "__main__":
    here = os.path.dirname(os.path.abspath(__file__))
    emit(RADICES, sys.argv[1] if len(sys.argv) > 1 else os.path.join(here, "codelets_gen.cuh"))
