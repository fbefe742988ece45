// Fused band kernels.
//  bands_from_spectrum: analysis form (Eq. analysis / band-spectrum).  One work item = (band, signal):
//      gather the band's bins from the half spectrum, multiply by the window table, place bin
//      kc + d in slot d mod M, zero the other slots, M-point inverse DFT in shared memory,
//      write the coefficients in time order.
//  bands_to_spectrum: synthesis form (Eq. synthesis).  M-point forward DFT of the coefficients in
//      shared memory, multiply the support slots by the dual-window table and write them in bin
//      order to the weighted-bin row of the signal (summed later, in fixed order, by the first pass
//      of the inverse long FFT).
// The same two kernels serve the adjoints with other tables (Sec. "Adjoints for training").
// This header: what the analysis-form and the synthesis-form kernels (one translation unit each) share.
#pragma once
#include "engine.cuh"
#include "internal.hpp"

namespace cqt {

struct BandArgs {
    const BandItem *items;   // per band of the class, in launch order (longest first): record + radix plan
    const FftPlan *ffts;
    const float2 *tw;
    const float *table;
    int n_work;
    int batch;
    int N;
    int max_elems;           // shared-memory elements per item
    int fold;                // synthesis form: add conj of the mirrored slot for sidebands
    const float2 *spec;      // analysis form: half spectrum rows; synthesis form: unused
    long long spec_pitch;
    float2 *coef;            // coefficients (read or written)
    long long coeff_count;
    float2 *Y;               // synthesis form: weighted-bin rows
    long long y_pitch;
    long long table_len;
    int *dbg;
};

// THREADS / MINB: launch bounds of the class (64 registers per thread when THREADS * MINB = 1024 ... 2048)
// LANES: 0 = the whole CTA works on one item; 32, 16, 8 = that many consecutive lanes per item (THREADS / LANES items
// per CTA): the shortest bands have fewer butterflies per stage than a warp has lanes
template <int LANES>
struct Group {
    __device__ static int tid() { return LANES ? (int)(threadIdx.x & (LANES - 1)) : (int)threadIdx.x; }
    __device__ static int nthr() { return LANES ? LANES : (int)blockDim.x; }
    __device__ static int per_cta() { return LANES ? (int)blockDim.x / (LANES ? LANES : 1) : 1; }
    __device__ static int slot() { return LANES ? (int)threadIdx.x / (LANES ? LANES : 1) : 0; }
    __device__ static int item() { return LANES ? (int)blockIdx.x * per_cta() + slot() : (int)blockIdx.x; }
};
template <int LANES>
using GroupSync = typename std::conditional<LANES == 0, BlockSync,
                                            typename std::conditional<LANES == 32, WarpSync, LaneGroupSync<(LANES ? LANES : 1)>>::type>::type;

extern __shared__ float2 smem_band[];

// The work item's band record and radix plan are fetched together, once, into shared memory: their fields are
// read inside the stage loops, where a shared-memory copy costs a short-latency load and the global original a
// cache lookup, and one cooperative load replaces a chain of two dependent ones.
template <class Sync>
__device__ __forceinline__ void fetch_item(const BandItem &g, BandItem &s, int tid, int nthr) {
    constexpr int kWords = (int)(sizeof(BandItem) / sizeof(int));
    for (int i = tid; i < kWords; i += nthr) reinterpret_cast<int *>(&s)[i] = __ldg(reinterpret_cast<const int *>(&g) + i);
    Sync::sync();
}

// Chirp-z (Bluestein) evaluation of an M-point DFT of sign SIGN whose length has a large prime factor:
//   X[k] = c[k] sum_n (x[n] c[n]) conj(c[k-n]),  c[n] = exp(SIGN i pi n^2 / M),
// the convolution through two power-of-two transforms of length L >= 2M - 1 in shared memory: forward DIF
// (natural -> digit-reversed), product with the precomputed filter spectrum (stored in that order, 1/L included),
// the DIF network backwards (digit-reversed -> natural).  load(n) yields x[n]; store(k, ., X[k]).
template <int SIGN, class Sync, class Load, class Store>
__device__ __forceinline__ void chirp_z_transform(float2 *buf, const FftPlan &fp, const FftPlan *ffts, const float2 *tw,
                                                  Load load, Store store, int *dbg, int tid, int nthr) {
    const FftPlan &fl = ffts[fp.blu_fft];
    const int M = fp.M, L = fp.blu_L;
    float2 *twl = buf + L;
    stage_twiddles(twl, tw, fl, tid, nthr);
    const float2 *chirp = tw + fp.blu_chirp_off;   // exp(-i pi n^2 / M)
    const float2 *filt = tw + fp.blu_filter_off;
    const Tile tl{buf, 1, 1, 0u, L, dbg};
    auto loadc = [&](int n, int) -> float2 {
        if (n >= M) return make_float2(0.f, 0.f);
        float2 w = __ldg(chirp + n);
        if (SIGN > 0) w.y = -w.y;
        return cmul(load(n, 0), w);
    };
    fft_fused_keep<-1, Sync, true, false, false>(tl, fl, twl, loadc, tid, nthr);
    for (int p = tid; p < L; p += nthr) {
        float2 f = __ldg(filt + p);
        if (SIGN > 0) f.y = -f.y;
        buf[p] = cmul(buf[p], f);
    }
    Sync::sync();
    fft_dit_inverse<Sync>(tl, fl, twl, tid, nthr);
    for (int k = tid; k < M; k += nthr) {
        float2 w = __ldg(chirp + k);
        if (SIGN > 0) w.y = -w.y;
        store(k, 0, cmul(buf[k], w));
    }
}

// Kernel instantiations: (threads per CTA, CTAs per SM the registers must allow, lanes per item or 0 for the whole CTA, largest radix
// compiled in), each with and without the prime-factor paths (GEN): code a class never runs is left out, which also
// frees registers in the paths it does run.
#define CQT_KERNEL_TABLE(X) \
    X(256, 4, 8, 8) X(256, 4, 32, 8) X(64, 16, 0, 8) X(128, 8, 0, 12) X(256, 4, 0, 12) X(512, 2, 0, 16) X(1024, 1, 0, 16)

}  // namespace cqt
