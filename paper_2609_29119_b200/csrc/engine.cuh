// Shared-memory mixed-radix FFT engine: in-place decimation in frequency on `ncols`
// interleaved columns.  Element (position p, column c) lives at buf[p * pitch + c].
// Input in natural order, output in mixed-radix digit-reversed order (see FftPlan);
// callers fold that permutation into their global-memory loads and stores.
#pragma once
#include <type_traits>
#include <cuda_runtime.h>
#include <stdint.h>

#include "codelets_gen.cuh"
#include "plan_types.h"

namespace cqt {

// Programmatic dependent launch (sm_90 and later): a kernel launched with the programmatic-serialization attribute may
// start while its predecessor in the stream is still running.  Every kernel of the library lets its successor start
// early (pdl_launch_dependents at its top) and waits for its predecessor (pdl_wait) only after the prologue that reads
// nothing but the plan's tables (band record, radix plan, twiddle tables): launch latency and that prologue overlap
// the predecessor's tail.  Without the attribute both calls do nothing.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

struct BlockSync {
    static __device__ __forceinline__ void sync() { __syncthreads(); }
};
struct WarpSync {
    static __device__ __forceinline__ void sync() { __syncwarp(); }
};
// LANES consecutive lanes of a warp (a power of two below 32) working on one item: the groups of a warp may be in
// different places of the code (items with different radix plans), so each synchronises with its own lane mask
template <int LANES>
struct LaneGroupSync {
    static __device__ __forceinline__ void sync() {
        __syncwarp(((1u << LANES) - 1u) << ((threadIdx.x & 31u) & ~(unsigned)(LANES - 1)));
    }
};

__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
    return make_float2(fmaf(a.x, b.x, -a.y * b.y), fmaf(a.x, b.y, a.y * b.x));
}
__device__ __forceinline__ float2 cconj(float2 a) { return make_float2(a.x, -a.y); }

// floor(n / d) for n * d < 2^32 with magic = ceil(2^32 / d); d == 1 is passed through.
__device__ __forceinline__ uint32_t fastdiv(uint32_t n, uint32_t magic, uint32_t d) {
    return d == 1 ? n : __umulhi(n, magic);
}

// exp(-2 pi i y / M) from the two-level table of a length-M plan.
__device__ __forceinline__ float2 twiddle(const float2 *__restrict__ tw, int logC, uint32_t y) {
    const uint32_t C = 1u << logC;
    const float2 lo = __ldg(tw + (y & (C - 1)));
    const float2 hi = __ldg(tw + C + (y >> logC));
    return cmul(lo, hi);
}

// position of frequency k after the DIF stages
__device__ __forceinline__ uint32_t dif_pos(const FftPlan &fp, uint32_t k) {
    uint32_t pos = 0, rem = k;
#pragma unroll 1
    for (int j = 0; j < fp.nstages; ++j) {
        const uint32_t r = fp.st[j].radix;
        const uint32_t q = __umulhi(rem, fp.st[j].rmagic);
        pos = pos * r + (rem - q * r);
        rem = q;
    }
    return pos;
}

template <int R, int SIGN>
__device__ __forceinline__ void dif_stage(float2 *buf, int pitch, int ncols, uint32_t ncols_magic, int M, int n_cur,
                                          int s, uint32_t smagic, int tmul, const float2 *__restrict__ tw, int logC,
                                          int tid, int nthr) {
    const int total = (M / R) * ncols;
    for (int w = tid; w < total; w += nthr) {
        const uint32_t b = fastdiv(w, ncols_magic, ncols);
        const uint32_t col = w - b * ncols;
        const uint32_t blk = fastdiv(b, smagic, s);
        const uint32_t np = b - blk * s;
        float2 *p = buf + (size_t)(blk * n_cur + np) * pitch + col;
        const int step = s * pitch;
        float re[R], im[R];
#pragma unroll
        for (int q = 0; q < R; ++q) {
            const float2 v = p[q * step];
            re[q] = v.x;
            im[q] = v.y;
        }
        if (SIGN < 0)
            Codelet<R>::run(re, im);
        else
            Codelet<R>::run(im, re);
        if (s > 1) {
            const uint32_t y1 = np * tmul;
#pragma unroll
            for (int q = 1; q < R; ++q) {
                float2 t = twiddle(tw, logC, y1 * q);
                if (SIGN > 0) t.y = -t.y;
                const float2 v = cmul(make_float2(re[q], im[q]), t);
                re[q] = v.x;
                im[q] = v.y;
            }
        }
#pragma unroll
        for (int q = 0; q < R; ++q) p[q * step] = make_float2(re[q], im[q]);
    }
}

// Generic first stage for a radix with no codelet (a large prime factor): every output is a
// direct sum over the p inputs of its butterfly; written to `alt`, then copied back.  `wp` (p entries of
// shared memory) receives the table exp(-+2 pi i x / p) first, so the inner loop is two shared loads and a MAC.
template <int SIGN, class Sync>
__device__ void dif_stage_generic(float2 *buf, float2 *alt, float2 *wp, int pitch, int ncols, int M, int p,
                                  const float2 *__restrict__ tw, int logC, int tid, int nthr) {
    const int s = M / p;
    const int tstep = M / p;  // W_p^x = W_M^{x * M/p}
    for (int x = tid; x < p; x += nthr) {
        float2 t = twiddle(tw, logC, (uint32_t)x * tstep);
        if (SIGN > 0) t.y = -t.y;
        wp[x] = t;
    }
    Sync::sync();
    for (int w = tid; w < M * ncols; w += nthr) {
        const int e = w / ncols, col = w - e * ncols;
        const int kq = e / s, np = e - kq * s;
        float ax = 0.f, ay = 0.f;
        int x = 0;
        const float2 *src = buf + (size_t)np * pitch + col;
        const int step = s * pitch;
        for (int q = 0; q < p; ++q) {
            const float2 t = wp[x];
            const float2 v = src[(size_t)q * step];
            ax = fmaf(v.x, t.x, ax); ax = fmaf(-v.y, t.y, ax);
            ay = fmaf(v.x, t.y, ay); ay = fmaf(v.y, t.x, ay);
            x += kq;
            if (x >= p) x -= p;
        }
        float2 t = twiddle(tw, logC, (uint32_t)np * kq);
        if (SIGN > 0) t.y = -t.y;
        alt[(size_t)e * pitch + col] = cmul(make_float2(ax, ay), t);
    }
    Sync::sync();
    for (int w = tid; w < M * ncols; w += nthr) {
        const int e = w / ncols, col = w - e * ncols;
        buf[(size_t)e * pitch + col] = alt[(size_t)e * pitch + col];
    }
}

// SIGN = -1: forward DFT (exp(-...)), SIGN = +1: unnormalised inverse.
// POW2 restricts the radix switch to powers of two (long-FFT kernels).
// The caller must synchronise before (inputs visible); the routine ends with a sync.
template <int SIGN, class Sync, bool POW2>
__device__ void fft_dif(float2 *buf, float2 *alt, int pitch, int ncols, uint32_t ncols_magic, const FftPlan &fp,
                        const float2 *__restrict__ tw_base, int tid, int nthr) {
    const float2 *tw = tw_base + fp.tw_off;
    const int M = fp.M, logC = fp.logC;
    int n_cur = M, tmul = 1;
#pragma unroll 1
    for (int j = 0; j < fp.nstages; ++j) {
        const int r = fp.st[j].radix, s = fp.st[j].stride;
        const uint32_t sm = fp.st[j].smagic;
#define CQT_STAGE(RR)                                                                                      \
    case RR:                                                                                               \
        dif_stage<RR, SIGN>(buf, pitch, ncols, ncols_magic, M, n_cur, s, sm, tmul, tw, logC, tid, nthr); \
        break;
        if (POW2) {
            switch (r) {
                CQT_STAGE(2) CQT_STAGE(4) CQT_STAGE(8) CQT_STAGE(16)
                default: break;
            }
        } else {
            switch (r) {
                CQT_STAGE(2) CQT_STAGE(3) CQT_STAGE(4) CQT_STAGE(5) CQT_STAGE(6) CQT_STAGE(8) CQT_STAGE(9)
                CQT_STAGE(10) CQT_STAGE(12) CQT_STAGE(15) CQT_STAGE(16)
                default:
                    dif_stage_generic<SIGN, Sync>(buf, alt, alt + (size_t)M * pitch, pitch, ncols, M, r, tw, logC, tid, nthr);
                    break;
            }
        }
#undef CQT_STAGE
        Sync::sync();
        n_cur = s;
        tmul *= r;
    }
}

// ======================================================================================
// Fused engine.  The first stage reads its operands through a caller functor (straight from
// global memory), the last stage hands its results to a caller functor (straight to global
// memory), the stages in between run in shared memory.  Twiddles: one two-level lookup per
// butterfly from a shared-memory copy of the plan's table, the powers w^2 .. w^(R-1) are formed
// in registers by balanced products (depth <= log2 R, so rounding grows with the depth only).
// ======================================================================================

// copies the two-level table of a plan into shared memory (caller synchronises afterwards)
__device__ __forceinline__ void stage_twiddles(float2 *dst, const float2 *__restrict__ tw_base, const FftPlan &fp, int tid,
                                               int nthr) {
    const float2 *src = tw_base + fp.tw_off;
    for (int i = tid; i < fp.tw_count; i += nthr) dst[i] = __ldg(src + i);
}

__device__ __forceinline__ float2 twiddle_s(const float2 *tw, int logC, uint32_t y) {
    const uint32_t C = 1u << logC;
    return cmul(tw[y & (C - 1)], tw[C + (y >> logC)]);
}

// Multiplies re/im[q] by w^q, q = 1 .. R-1, where w = exp(-+2 pi i y1 / M).  The powers w^1, w^2, w^4, w^8
// are looked up (two-level table), the others are products of at most three of those: raising one rounded
// w to the q-th power would multiply its phase error by q, a product of looked-up factors only adds errors.
template <int R, int SIGN>
__device__ __forceinline__ void apply_twiddle_powers(const float2 *tw, int logC, uint32_t y1, float (&re)[R], float (&im)[R]) {
    float wr[R], wi[R];
    wr[0] = 1.f; wi[0] = 0.f;
#pragma unroll
    for (int q = 1; q < R; ++q) {
        if ((q & (q - 1)) == 0) {
            const float2 w = twiddle_s(tw, logC, y1 * q);
            wr[q] = w.x;
            wi[q] = SIGN > 0 ? -w.y : w.y;
        } else {
            const int hb = q >= 16 ? 16 : (q >= 8 ? 8 : (q >= 4 ? 4 : 2)), lo = q - hb;
            wr[q] = fmaf(wr[hb], wr[lo], -wi[hb] * wi[lo]);
            wi[q] = fmaf(wr[hb], wi[lo], wi[hb] * wr[lo]);
        }
    }
#pragma unroll
    for (int q = 1; q < R; ++q) {
        const float x = re[q], y = im[q];
        re[q] = fmaf(x, wr[q], -y * wi[q]);
        im[q] = fmaf(x, wi[q], y * wr[q]);
    }
}

// Same with a full table twf[y] = exp(-2 pi i y / M): one load per power, no products (short power-of-two plans).
template <int R, int SIGN>
__device__ __forceinline__ void apply_twiddle_direct(const float2 *twf, uint32_t y1, float (&re)[R], float (&im)[R]) {
#pragma unroll
    for (int q = 1; q < R; ++q) {
        const float2 w = twf[y1 * q];
        const float wi = SIGN > 0 ? -w.y : w.y;
        const float x = re[q], y = im[q];
        re[q] = fmaf(x, w.x, -y * wi);
        im[q] = fmaf(x, wi, y * w.x);
    }
}

// position of frequency k for a power-of-two plan: digit reversal by shifts
__device__ __forceinline__ uint32_t dif_pos_pow2(const FftPlan &fp, uint32_t k) {
    uint32_t pos = 0, rem = k;
#pragma unroll 1
    for (int j = 0; j < fp.nstages; ++j) {
        const int l = fp.st[j].lg;
        pos = (pos << l) | (rem & ((1u << l) - 1));
        rem >>= l;
    }
    return pos;
}

struct Tile {
    float2 *buf;
    int pitch;             // elements between consecutive positions
    int ncols;             // interleaved columns
    uint32_t ncols_magic;
    int limit;             // elements available at buf (checked in CQT_DEBUG_BOUNDS builds)
    int *dbg;              // debug status words (may be null)
};

// Debug build (-DCQT_DEBUG_BOUNDS): every instrumented access checks its index, records the first
// violation {site, index, limit, block x, block y, thread} in the plan's status words and skips the access.
#ifdef CQT_DEBUG_BOUNDS
__device__ __forceinline__ bool dbg_ok(int *dbg, int site, long long idx, long long limit) {
    if (idx >= 0 && idx < limit) return true;
    if (dbg && atomicCAS(&dbg[0], 0, site) == 0) {
        dbg[1] = (int)idx; dbg[2] = (int)(idx >> 32); dbg[3] = (int)limit; dbg[4] = (int)(limit >> 32);
        dbg[5] = blockIdx.x; dbg[6] = blockIdx.y; dbg[7] = threadIdx.x;
    }
    return false;
}
#define CQT_CHK(dbg, site, idx, limit) cqt::dbg_ok(dbg, site, (long long)(idx), (long long)(limit))
#else
#define CQT_CHK(dbg, site, idx, limit) true
#endif

// first stage: operands from load(pos, col); results to shared memory.
// COLFAST: consecutive threads take consecutive columns, else consecutive butterflies.
template <int R, int SIGN, bool PAD, bool COLFAST, bool DIRECT, class Sync, class Load>
__device__ __forceinline__ void first_stage(const Tile &t, const FftPlan &fp, const float2 *tw, Load load, int tid, int nthr) {
    // plan fields are read once, ahead of the loops: the plan may sit in shared memory beside the data buffer,
    // where the compiler must assume that a data store changes it
    const StageRec sr = fp.st[0];
    const int s = sr.stride;
    const int total = s * t.ncols;
    const int spad = PAD ? s + fp.pad_delta : s;
    const int logC = fp.logC;
    const uint32_t smagic0 = sr.smagic;
    // every thread of the group runs every round: the first round contains the barrier that makes the
    // staged twiddle table visible, placed after the operand loads so both are in flight together
    for (int base = 0; base < total; base += nthr) {
        const int w = base + tid;
        const bool active = w < total;
        uint32_t b = 0, col = 0;
        if (active) {
            if (t.ncols == 1) { b = w; }
            else if (COLFAST) { b = fastdiv(w, t.ncols_magic, t.ncols); col = w - b * t.ncols; }
            else { col = fastdiv(w, smagic0, s); b = w - col * s; }
        }
        float re[R], im[R];
        if (active) {
#pragma unroll
            for (int q = 0; q < R; ++q) {
                const float2 v = load((int)(b + q * s), (int)col);
                re[q] = v.x; im[q] = v.y;
            }
            if (SIGN < 0) Codelet<R>::run(re, im); else Codelet<R>::run(im, re);
        }
        if (base == 0) Sync::sync();
        if (active) {
            if (DIRECT) apply_twiddle_direct<R, SIGN>(tw, b, re, im);
            else apply_twiddle_powers<R, SIGN>(tw, logC, b, re, im);
            float2 *p = t.buf + (b * (uint32_t)t.pitch + col);
            const uint32_t qstep = (uint32_t)spad * (uint32_t)t.pitch;
#pragma unroll
            for (int q = 0; q < R; ++q)
                if (CQT_CHK(t.dbg, 101, b * t.pitch + col + q * qstep, t.limit))
                    p[q * qstep] = make_float2(re[q], im[q]);
        }
    }
}

template <int R, int SIGN, bool PAD, bool DIRECT>
__device__ __forceinline__ void middle_stage(const Tile &t, const FftPlan &fp, const float2 *tw, int j, int n_cur, int tmul,
                                             int tid, int nthr) {
    const StageRec sr = fp.st[j];
    const int s = sr.stride;
    const int total = (fp.M / R) * t.ncols;
    const uint32_t smagic = sr.smagic, k1magic = sr.k1magic;
    const int k1div = sr.k1div, logC = fp.logC;
    const bool padded = PAD && fp.pad_delta != 0;
    // Short strides: blocks of one first-stage chunk sit a multiple of 16 elements apart, so neighbouring threads on
    // neighbouring blocks would all hit the same banks.  Then the first-stage digit k0 runs fastest over the threads
    // instead: chunks are s_0 + 1 elements apart (the pad), which spreads a warp over all banks.
    const bool chunk_fastest = padded && s < 16;
    const uint32_t r0 = fp.st[0].radix, r0magic = fp.st[0].rmagic;
    for (int w = tid; w < total; w += nthr) {
        const uint32_t b = fastdiv(w, t.ncols_magic, t.ncols);
        const uint32_t col = w - b * t.ncols;
        uint32_t blk, np, pad = 0;
        if (chunk_fastest) {
            const uint32_t x = fastdiv(b, r0magic, r0), k0 = b - x * r0;
            const uint32_t rest = fastdiv(x, smagic, s);
            np = x - rest * s;
            blk = k0 * (uint32_t)k1div + rest;
            pad = k0;
        } else {
            blk = fastdiv(b, smagic, s);
            np = b - blk * s;
            if (padded) pad = fastdiv(blk, k1magic, k1div);
        }
        const uint32_t pos = blk * n_cur + np + pad;
        float2 *p = t.buf + (pos * (uint32_t)t.pitch + col);
        const uint32_t step = (uint32_t)s * (uint32_t)t.pitch;
        float re[R], im[R];
        if (!CQT_CHK(t.dbg, 102, pos * t.pitch + col + (R - 1) * step, t.limit)) continue;
#pragma unroll
        for (int q = 0; q < R; ++q) {
            const float2 v = p[q * step];
            re[q] = v.x; im[q] = v.y;
        }
        if (SIGN < 0) Codelet<R>::run(re, im); else Codelet<R>::run(im, re);
        if (DIRECT) { if (s > 1) apply_twiddle_direct<R, SIGN>(tw, np * tmul, re, im); }
        else apply_twiddle_powers<R, SIGN>(tw, logC, np * tmul, re, im);
#pragma unroll
        for (int q = 0; q < R; ++q) p[q * step] = make_float2(re[q], im[q]);
    }
}

// A store functor may split its work in two: pre(k, col), called before the butterfly's operands are read, fetches
// whatever the store needs from global memory (a window value) so that the load's latency hides behind the
// butterfly; operator()(k, col, value, fetched) then finishes.  Plain functors take (k, col, value).
template <class Store>
constexpr bool kStoreHasPre = !std::is_invocable<Store, int, int, float2>::value;

// last stage (stride 1): operands from shared memory, result k of column col to store(k, col, value).
// REV: thread index = low digits of k (consecutive threads store consecutive k), else thread index =
// butterfly position.  COLFAST as above.
template <int R, int SIGN, bool PAD, bool REV, bool COLFAST, class Store>
__device__ __forceinline__ void last_stage(const Tile &t, const FftPlan &fp, Store store, int tid, int nthr) {
    const int nb = fp.M / R;
    const int total = nb * t.ncols;
    const int d = fp.nstages;
    const bool padded = PAD && fp.pad_delta != 0;
    const StageRec sr = fp.st[d - 1];
    const uint32_t k1magic = sr.k1magic;
    const int k1div = sr.k1div;
    for (int w = tid; w < total; w += nthr) {
        uint32_t u, col;
        if (t.ncols == 1) { u = w; col = 0; }
        else if (COLFAST) { u = fastdiv(w, t.ncols_magic, t.ncols); col = w - u * t.ncols; }
        else { col = (uint32_t)w / (uint32_t)nb; u = w - col * nb; }
        uint32_t b, klow;
        if (REV) {           // u = k_0 + r_0 (k_1 + ...)  ->  b = ((k_0 r_1 + k_1) r_2 + ...)
            klow = u;
            uint32_t rem = u;
            // Horner over the digits, most significant first
            b = 0;
#pragma unroll 1
            for (int j = 0; j < d - 1; ++j) {
                const uint32_t r = fp.st[j].radix;
                const uint32_t qd = __umulhi(rem, fp.st[j].rmagic);
                b = b * r + (rem - qd * r);
                rem = qd;
            }
        } else {             // u = b  ->  k_low = k_0 + r_0 (k_1 + r_1 (...)), digits of b least significant first
            b = u; klow = 0;
            uint32_t rem = u;
#pragma unroll 1
            for (int j = d - 2; j >= 0; --j) {
                const uint32_t r = fp.st[j].radix;
                const uint32_t qd = __umulhi(rem, fp.st[j].rmagic);
                klow = klow * r + (rem - qd * r);
                rem = qd;
            }
        }
        uint32_t pos = b * R;
        if (padded) pos += fastdiv(b, k1magic, k1div);
        const float2 *p = t.buf + (pos * (uint32_t)t.pitch + col);
        float re[R], im[R];
        if (!CQT_CHK(t.dbg, 103, pos * t.pitch + col + (R - 1) * t.pitch, t.limit)) continue;
        if constexpr (kStoreHasPre<Store>) {
            decltype(store.pre(0, 0)) fetched[R];
#pragma unroll
            for (int q = 0; q < R; ++q) fetched[q] = store.pre((int)(klow + q * nb), (int)col);
#pragma unroll
            for (int q = 0; q < R; ++q) {
                const float2 v = p[q * (uint32_t)t.pitch];
                re[q] = v.x; im[q] = v.y;
            }
            if (SIGN < 0) Codelet<R>::run(re, im); else Codelet<R>::run(im, re);
#pragma unroll
            for (int q = 0; q < R; ++q) store((int)(klow + q * nb), (int)col, make_float2(re[q], im[q]), fetched[q]);
        } else {
#pragma unroll
            for (int q = 0; q < R; ++q) {
                const float2 v = p[q * (uint32_t)t.pitch];
                re[q] = v.x; im[q] = v.y;
            }
            if (SIGN < 0) Codelet<R>::run(re, im); else Codelet<R>::run(im, re);
#pragma unroll
            for (int q = 0; q < R; ++q) store((int)(klow + q * nb), (int)col, make_float2(re[q], im[q]));
        }
    }
}

// single-stage transform (M = R): no shared memory at all
template <int R, int SIGN, class Load, class Store>
__device__ __forceinline__ void only_stage(const Tile &t, Load load, Store store, int tid, int nthr) {
    for (int col = tid; col < t.ncols; col += nthr) {
        float re[R], im[R];
#pragma unroll
        for (int q = 0; q < R; ++q) {
            const float2 v = load(q, col);
            re[q] = v.x; im[q] = v.y;
        }
        if (SIGN < 0) Codelet<R>::run(re, im); else Codelet<R>::run(im, re);
#pragma unroll
        for (int q = 0; q < R; ++q) {
            if constexpr (kStoreHasPre<Store>) store(q, col, make_float2(re[q], im[q]), store.pre(q, col));
            else store(q, col, make_float2(re[q], im[q]));
        }
    }
}

// One stage of the inverse of the DIF network, run backwards (j = d-1 .. 0): conjugate twiddles first, then the
// inverse butterfly.  Turns digit-reversed spectra back into natural order; the result is L times the inverse DFT
// of what a forward (SIGN = -1) DIF run produced.
template <int R>
__device__ __forceinline__ void dit_stage(const Tile &t, const FftPlan &fp, const float2 *tw, int j, int n_cur, int tmul,
                                          int tid, int nthr) {
    const int s = fp.st[j].stride;
    const int total = (fp.M / R) * t.ncols;
    for (int w = tid; w < total; w += nthr) {
        const uint32_t b = fastdiv(w, t.ncols_magic, t.ncols);
        const uint32_t col = w - b * t.ncols;
        const uint32_t blk = fastdiv(b, fp.st[j].smagic, s);
        const uint32_t np = b - blk * s;
        const uint32_t pos = blk * n_cur + np;
        float2 *p = t.buf + (pos * (uint32_t)t.pitch + col);
        const uint32_t step = (uint32_t)s * (uint32_t)t.pitch;
        float re[R], im[R];
#pragma unroll
        for (int q = 0; q < R; ++q) {
            const float2 v = p[q * step];
            re[q] = v.x; im[q] = v.y;
        }
        if (s > 1) apply_twiddle_powers<R, +1>(tw, fp.logC, np * tmul, re, im);
        Codelet<R>::run(im, re);
#pragma unroll
        for (int q = 0; q < R; ++q) p[q * step] = make_float2(re[q], im[q]);
    }
}

// all stages backwards, in shared memory; power-of-two plans only; ends with a sync
template <class Sync>
__device__ void fft_dit_inverse(const Tile &t, const FftPlan &fp, const float2 *tw, int tid, int nthr) {
    const int d = fp.nstages;
#pragma unroll 1
    for (int j = d - 1; j >= 0; --j) {
        const int n_cur = j == 0 ? fp.M : fp.st[j - 1].stride;
        int tmul = 1;
        for (int i = 0; i < j; ++i) tmul *= fp.st[i].radix;
        switch (fp.st[j].radix) {
            case 2: dit_stage<2>(t, fp, tw, j, n_cur, tmul, tid, nthr); break;
            case 4: dit_stage<4>(t, fp, tw, j, n_cur, tmul, tid, nthr); break;
            case 8: dit_stage<8>(t, fp, tw, j, n_cur, tmul, tid, nthr); break;
            case 16: dit_stage<16>(t, fp, tw, j, n_cur, tmul, tid, nthr); break;
            default: break;
        }
        Sync::sync();
    }
}

#define CQT_RADIX_CASES_ALL(X) X(2) X(3) X(4) X(5) X(6) X(8) X(9) X(10) X(12) X(15) X(16)
#define CQT_RADIX_CASES_POW2(X) X(2) X(4) X(8) X(16)

// Runs the first `nrun` stages of the plan (nrun = nstages: the whole transform with the last stage fused
// into `store`; nrun = nstages - 1... not offered: use fft_fused_keep for "results stay in shared memory").
// MAXR: largest radix the plan may contain (larger cases are not compiled; the plan builder caps the radices of
// short bands, whose kernels need neither the code nor the registers of the big codelets).
// Requires a non-generic plan.  tw = shared-memory copy of the plan's two-level table, written by the
// caller (stage_twiddles) WITHOUT a barrier after it: the first stage synchronises once its operand loads
// are issued.  The routine synchronises between stages, not at the end.
template <int SIGN, class Sync, bool POW2, bool PAD, bool COLFAST_IN, bool REV, bool COLFAST_OUT, bool DIRECT, int MAXR = 16, class Load, class Store>
__device__ __forceinline__ void fft_fused(const Tile &t, const FftPlan &fp, const float2 *tw, Load load, Store store, int tid, int nthr) {
    const int d = fp.nstages;
    if (d == 1) {
        Sync::sync();   // tables staged by the caller become visible to the functors
#define X(RR) case RR: if constexpr (POW2 || RR <= MAXR) only_stage<RR, SIGN>(t, load, store, tid, nthr); break;
        if (POW2) { switch (fp.st[0].radix) { CQT_RADIX_CASES_POW2(X) default: break; } }
        else { switch (fp.st[0].radix) { CQT_RADIX_CASES_ALL(X) default: break; } }
#undef X
        return;
    }
#define X(RR) case RR: if constexpr (POW2 || RR <= MAXR) first_stage<RR, SIGN, PAD, COLFAST_IN, DIRECT, Sync>(t, fp, tw, load, tid, nthr); break;
    if (POW2) { switch (fp.st[0].radix) { CQT_RADIX_CASES_POW2(X) default: break; } }
    else { switch (fp.st[0].radix) { CQT_RADIX_CASES_ALL(X) default: break; } }
#undef X
    Sync::sync();
    int n_cur = fp.st[0].stride, tmul = fp.st[0].radix;
#pragma unroll 1
    for (int j = 1; j < d - 1; ++j) {
#define X(RR) case RR: if constexpr (POW2 || RR <= MAXR) middle_stage<RR, SIGN, PAD, DIRECT>(t, fp, tw, j, n_cur, tmul, tid, nthr); break;
        if (POW2) { switch (fp.st[j].radix) { CQT_RADIX_CASES_POW2(X) default: break; } }
        else { switch (fp.st[j].radix) { CQT_RADIX_CASES_ALL(X) default: break; } }
#undef X
        Sync::sync();
        n_cur = fp.st[j].stride;
        tmul *= fp.st[j].radix;
    }
#define X(RR) case RR: if constexpr (POW2 || RR <= MAXR) last_stage<RR, SIGN, PAD, REV, COLFAST_OUT>(t, fp, store, tid, nthr); break;
    if (POW2) { switch (fp.st[d - 1].radix) { CQT_RADIX_CASES_POW2(X) default: break; } }
    else { switch (fp.st[d - 1].radix) { CQT_RADIX_CASES_ALL(X) default: break; } }
#undef X
}

// Same, but every stage after the first runs in shared memory and the results stay there
// (digit-reversed positions, see dif_pos); ends with a sync.
template <int SIGN, class Sync, bool POW2, bool COLFAST_IN, bool DIRECT, class Load>
__device__ __forceinline__ void fft_fused_keep(const Tile &t, const FftPlan &fp, const float2 *tw, Load load, int tid, int nthr) {
    const int d = fp.nstages;
    if (d == 1) {
        auto keep = [&](int k, int col, float2 v) { t.buf[(size_t)k * t.pitch + col] = v; };
#define X(RR) case RR: only_stage<RR, SIGN>(t, load, keep, tid, nthr); break;
        if (POW2) { switch (fp.st[0].radix) { CQT_RADIX_CASES_POW2(X) default: break; } }
        else { switch (fp.st[0].radix) { CQT_RADIX_CASES_ALL(X) default: break; } }
#undef X
        Sync::sync();
        return;
    }
#define X(RR) case RR: first_stage<RR, SIGN, false, COLFAST_IN, DIRECT, Sync>(t, fp, tw, load, tid, nthr); break;
    if (POW2) { switch (fp.st[0].radix) { CQT_RADIX_CASES_POW2(X) default: break; } }
    else { switch (fp.st[0].radix) { CQT_RADIX_CASES_ALL(X) default: break; } }
#undef X
    Sync::sync();
    int n_cur = fp.st[0].stride, tmul = fp.st[0].radix;
#pragma unroll 1
    for (int j = 1; j < d; ++j) {
#define X(RR) case RR: middle_stage<RR, SIGN, false, DIRECT>(t, fp, tw, j, n_cur, tmul, tid, nthr); break;
        if (POW2) { switch (fp.st[j].radix) { CQT_RADIX_CASES_POW2(X) default: break; } }
        else { switch (fp.st[j].radix) { CQT_RADIX_CASES_ALL(X) default: break; } }
#undef X
        Sync::sync();
        n_cur = fp.st[j].stride;
        tmul *= fp.st[j].radix;
    }
}

}  // namespace cqt
