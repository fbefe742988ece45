// Shared-memory mixed-radix FFT engine: in-place decimation in frequency on `ncols`
// interleaved columns.  Element (position p, column c) lives at buf[p * pitch + c].
// Input in natural order, output in mixed-radix digit-reversed order (see FftPlan);
// callers fold that permutation into their global-memory loads and stores.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "codelets_gen.cuh"
#include "plan_types.h"

namespace cqt {

struct BlockSync {
    static __device__ __forceinline__ void sync() { __syncthreads(); }
};
struct WarpSync {
    static __device__ __forceinline__ void sync() { __syncwarp(); }
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
        const uint32_t r = fp.radix[j];
        const uint32_t q = __umulhi(rem, fp.rmagic[j]);
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
// direct sum over the p inputs of its butterfly; written to `alt`, then copied back.
template <int SIGN, class Sync>
__device__ void dif_stage_generic(float2 *buf, float2 *alt, int pitch, int ncols, int M, int p,
                                  const float2 *__restrict__ tw, int logC, int tid, int nthr) {
    const int s = M / p;
    const int tstep = M / p;  // W_p^x = W_M^{x * M/p}
    for (int w = tid; w < M * ncols; w += nthr) {
        const int e = w / ncols, col = w - e * ncols;
        const int kq = e / s, np = e - kq * s;
        float2 acc = make_float2(0.f, 0.f);
        int x = 0;
        for (int q = 0; q < p; ++q) {
            float2 t = twiddle(tw, logC, (uint32_t)x * tstep);
            if (SIGN > 0) t.y = -t.y;
            const float2 v = buf[(size_t)(q * s + np) * pitch + col];
            acc.x += v.x * t.x - v.y * t.y;
            acc.y += v.x * t.y + v.y * t.x;
            x += kq;
            if (x >= p) x -= p;
        }
        float2 t = twiddle(tw, logC, (uint32_t)np * kq);
        if (SIGN > 0) t.y = -t.y;
        alt[(size_t)e * pitch + col] = cmul(acc, t);
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
        const int r = fp.radix[j], s = fp.stride[j];
        const uint32_t sm = fp.smagic[j];
#define CQT_STAGE(RR)                                                                                      \
    case RR:                                                                                               \
        dif_stage<RR, SIGN>(buf, pitch, ncols, ncols_magic, M, n_cur, s, sm, tmul, tw, logC, tid, nthr); \
        break;
        if (POW2) {
            switch (r) {
                CQT_STAGE(2) CQT_STAGE(4) CQT_STAGE(8) CQT_STAGE(16) CQT_STAGE(32)
                default: break;
            }
        } else {
            switch (r) {
                CQT_STAGE(2) CQT_STAGE(3) CQT_STAGE(4) CQT_STAGE(5) CQT_STAGE(6) CQT_STAGE(8) CQT_STAGE(9)
                CQT_STAGE(10) CQT_STAGE(12) CQT_STAGE(15) CQT_STAGE(16)
                default:
                    dif_stage_generic<SIGN, Sync>(buf, alt, pitch, ncols, M, r, tw, logC, tid, nthr);
                    break;
            }
        }
#undef CQT_STAGE
        Sync::sync();
        n_cur = s;
        tmul *= r;
    }
}

}  // namespace cqt
