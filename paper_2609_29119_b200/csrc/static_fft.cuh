// Three-stage tile transform with every stride, radix and column count known at compile time (the common
// shapes of the long FFT passes: 512 = 8 x 8 x 8 points on 16 or 18 interleaved columns).  Same data flow as the
// run-time planned engine (first stage from a load functor, middle stage in shared memory, last stage to a
// store functor or back to shared memory); with constant strides the index arithmetic folds into immediates.
#pragma once
#include "engine.cuh"

namespace cqt {

template <int R0, int R1, int R2, int NC, int PITCH, int SIGN, bool COLFAST_IN, bool KEEP, class Load, class Store>
__device__ __forceinline__ void tile_fft3(float2 *buf, const float2 *twf, Load load, Store store, int tid, int nthr) {
    constexpr int M = R0 * R1 * R2;
    constexpr int S0 = R1 * R2;
    // ---- stage 0: operands from the functor, butterflies over positions b + q S0
    {
        constexpr int total = S0 * NC;
        for (int base = 0; base < total; base += nthr) {
            const int w = base + tid;
            const bool active = w < total;
            const int b = COLFAST_IN ? w / NC : w % S0;
            const int col = COLFAST_IN ? w % NC : w / S0;
            float re[R0], im[R0];
            if (active) {
#pragma unroll
                for (int q = 0; q < R0; ++q) {
                    const float2 v = load(b + q * S0, col);
                    re[q] = v.x; im[q] = v.y;
                }
                if (SIGN < 0) Codelet<R0>::run(re, im); else Codelet<R0>::run(im, re);
            }
            if (base == 0) __syncthreads();   // staged tables become visible
            if (active) {
                apply_twiddle_direct<R0, SIGN>(twf, (uint32_t)b, re, im);
                float2 *p = buf + b * PITCH + col;
#pragma unroll
                for (int q = 0; q < R0; ++q) p[q * S0 * PITCH] = make_float2(re[q], im[q]);
            }
        }
    }
    __syncthreads();
    // ---- stage 1: sub-transforms of length S0, stride R2
    {
        constexpr int total = (M / R1) * NC;
        for (int w = tid; w < total; w += nthr) {
            const int b = w / NC, col = w % NC;
            const int blk = b / R2, np = b % R2;
            float2 *p = buf + (blk * S0 + np) * PITCH + col;
            float re[R1], im[R1];
#pragma unroll
            for (int q = 0; q < R1; ++q) {
                const float2 v = p[q * R2 * PITCH];
                re[q] = v.x; im[q] = v.y;
            }
            if (SIGN < 0) Codelet<R1>::run(re, im); else Codelet<R1>::run(im, re);
            apply_twiddle_direct<R1, SIGN>(twf, (uint32_t)(np * R0), re, im);
#pragma unroll
            for (int q = 0; q < R1; ++q) p[q * R2 * PITCH] = make_float2(re[q], im[q]);
        }
    }
    __syncthreads();
    // ---- stage 2: stride 1; butterfly b = k0 R1 + k1 holds frequencies k0 + R0 k1 + R0 R1 q
    {
        constexpr int total = (M / R2) * NC;
        for (int w = tid; w < total; w += nthr) {
            const int b = w / NC, col = w % NC;
            float2 *p = buf + (b * R2) * PITCH + col;
            float re[R2], im[R2];
#pragma unroll
            for (int q = 0; q < R2; ++q) {
                const float2 v = p[q * PITCH];
                re[q] = v.x; im[q] = v.y;
            }
            if (SIGN < 0) Codelet<R2>::run(re, im); else Codelet<R2>::run(im, re);
            if (KEEP) {
#pragma unroll
                for (int q = 0; q < R2; ++q) p[q * PITCH] = make_float2(re[q], im[q]);
            } else {
                const int klow = b / R1 + R0 * (b % R1);
#pragma unroll
                for (int q = 0; q < R2; ++q) store(klow + q * (R0 * R1), col, make_float2(re[q], im[q]));
            }
        }
    }
    if (KEEP) __syncthreads();
}

// Two-stage variant: M = R0 * R1.
template <int R0, int R1, int NC, int PITCH, int SIGN, bool COLFAST_IN, bool KEEP, class Load, class Store>
__device__ __forceinline__ void tile_fft2(float2 *buf, const float2 *twf, Load load, Store store, int tid, int nthr) {
    constexpr int M = R0 * R1;
    constexpr int S0 = R1;
    {
        constexpr int total = S0 * NC;
        for (int base = 0; base < total; base += nthr) {
            const int w = base + tid;
            const bool active = w < total;
            const int b = COLFAST_IN ? w / NC : w % S0;
            const int col = COLFAST_IN ? w % NC : w / S0;
            float re[R0], im[R0];
            if (active) {
#pragma unroll
                for (int q = 0; q < R0; ++q) {
                    const float2 v = load(b + q * S0, col);
                    re[q] = v.x; im[q] = v.y;
                }
                if (SIGN < 0) Codelet<R0>::run(re, im); else Codelet<R0>::run(im, re);
            }
            if (base == 0) __syncthreads();   // staged tables become visible
            if (active) {
                apply_twiddle_direct<R0, SIGN>(twf, (uint32_t)b, re, im);
                float2 *p = buf + b * PITCH + col;
#pragma unroll
                for (int q = 0; q < R0; ++q) p[q * S0 * PITCH] = make_float2(re[q], im[q]);
            }
        }
    }
    __syncthreads();
    {
        constexpr int total = (M / R1) * NC;   // butterfly b = k0 holds frequencies k0 + R0 q
        for (int w = tid; w < total; w += nthr) {
            const int b = w / NC, col = w % NC;
            float2 *p = buf + (b * R1) * PITCH + col;
            float re[R1], im[R1];
#pragma unroll
            for (int q = 0; q < R1; ++q) {
                const float2 v = p[q * PITCH];
                re[q] = v.x; im[q] = v.y;
            }
            if (SIGN < 0) Codelet<R1>::run(re, im); else Codelet<R1>::run(im, re);
            if (KEEP) {
#pragma unroll
                for (int q = 0; q < R1; ++q) p[q * PITCH] = make_float2(re[q], im[q]);
            } else {
#pragma unroll
                for (int q = 0; q < R1; ++q) store(b + q * R0, col, make_float2(re[q], im[q]));
            }
        }
    }
    if (KEEP) __syncthreads();
}

// Compile-time shape of a tile transform: R0 = 0 means "use the run-time planned engine", R2 = 1 two stages.
template <int R0_, int R1_, int R2_, int NC_, int PITCH_>
struct Shape {
    static constexpr int R0 = R0_, R1 = R1_, R2 = R2_, NC = NC_, PITCH = PITCH_;
    static constexpr bool is_static = R0_ > 0;
    static __host__ __device__ __forceinline__ bool matches(const FftPlan &fp, int ncols) {
        if constexpr (R0_ == 0) return true;
        else if constexpr (R2_ == 1) return ncols == NC_ && fp.nstages == 2 && fp.st[0].radix == R0_ && fp.st[1].radix == R1_;
        else return ncols == NC_ && fp.nstages == 3 && fp.st[0].radix == R0_ && fp.st[1].radix == R1_ && fp.st[2].radix == R2_;
    }
    // position of frequency k after a KEEP transform
    static __device__ __forceinline__ uint32_t pos(const FftPlan &fp, uint32_t k) {
        if constexpr (R0_ == 0) return dif_pos_pow2(fp, k);
        else if constexpr (R2_ == 1) return (k % R0_) * R1_ + k / R0_;
        else return ((k % R0_) * R1_ + (k / R0_) % R1_) * R2_ + k / (R0_ * R1_);
    }
};

template <class SH, int SIGN, bool COLFAST_IN, bool KEEP, class Load, class Store>
__device__ __forceinline__ void tile_fft_static(float2 *buf, const float2 *twf, Load load, Store store, int tid, int nthr) {
    if constexpr (SH::R2 == 1) tile_fft2<SH::R0, SH::R1, SH::NC, SH::PITCH, SIGN, COLFAST_IN, KEEP>(buf, twf, load, store, tid, nthr);
    else tile_fft3<SH::R0, SH::R1, (SH::R2 > 1 ? SH::R2 : 2), SH::NC, SH::PITCH, SIGN, COLFAST_IN, KEEP>(buf, twf, load, store, tid, nthr);
}

// position of frequency k after tile_fft3 with KEEP: k = k0 + R0 k1 + R0 R1 k2 sits at (k0 R1 + k1) R2 + k2
template <int R0, int R1, int R2>
__device__ __forceinline__ int tile_fft3_pos(int k) {
    return ((k % R0) * R1 + (k / R0) % R1) * R2 + k / (R0 * R1);
}

__device__ __forceinline__ bool plan_is(const FftPlan &fp, int r0, int r1, int r2) {
    return fp.nstages == 3 && fp.st[0].radix == r0 && fp.st[1].radix == r1 && fp.st[2].radix == r2;
}

}  // namespace cqt
