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
#include "engine.cuh"
#include "internal.hpp"

namespace cqt {

struct BandArgs {
    const BandItem *items;   // per band: record + radix plan
    const FftPlan *ffts;
    const float2 *tw;
    const float *table;
    const int32_t *work;     // band indices of this class, longest first
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
template <bool WARP>
struct Group {
    __device__ static int tid() { return WARP ? (threadIdx.x & 31) : threadIdx.x; }
    __device__ static int nthr() { return WARP ? 32 : blockDim.x; }
    __device__ static int item() { return WARP ? blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5) : blockIdx.x; }
    __device__ static int slot() { return WARP ? (threadIdx.x >> 5) : 0; }
};

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

template <int THREADS, int MINB, bool WARP, int MAXR, bool GEN>
__global__ void __launch_bounds__(THREADS, MINB) bands_from_spectrum_kernel(BandArgs a) {
    using G = Group<WARP>;
    using Sync = typename std::conditional<WARP, WarpSync, BlockSync>::type;
    const int item = G::item();
    if (item >= a.n_work * a.batch) return;   // whole group exits together
    const int tid = G::tid(), nthr = G::nthr();
    __shared__ BandItem item_s[WARP ? 8 : 1];
    BandItem &it = item_s[G::slot()];
    fetch_item<Sync>(a.items[a.work[item / a.batch]], it, tid, nthr);
    const BandRec br = it.br;
    const int ch = item % a.batch;
    const FftPlan &fp = it.fp;
    float2 *buf = smem_band + (size_t)G::slot() * a.max_elems;
    const float2 *X = a.spec + (long long)ch * a.spec_pitch;
    const float *tab = a.table + br.tab_off;
    const int M = br.M, half = a.N >> 1;
    const int last_pos = br.d0 + br.S - 1;   // largest offset (>= 0)
    const int first_neg = M + br.d0;          // slot of the most negative offset
    // slot m holds tab[d] X[kc + d] with d = m (m <= last_pos) or m - M (m >= first_neg), else zero
    auto load = [&](int m, int) -> float2 {
        const bool lo = m <= last_pos;
        if (!lo && m < first_neg) return make_float2(0.f, 0.f);
        const int d = lo ? m : m - M;
        if (!CQT_CHK(a.dbg, 301, br.tab_off + (d - br.d0), a.table_len)) return make_float2(0.f, 0.f);
        const float g = __ldg(tab + (d - br.d0));
        const int k = br.kc + d;
        // bins outside 0..N/2 are the conjugates of their mirror bins
        const bool mirrored = k < 0 || k > half;
        const int km = k < 0 ? -k : (k > half ? a.N - k : k);
        if (!CQT_CHK(a.dbg, 302, km, half + 1)) return make_float2(0.f, 0.f);
        const float2 xv = __ldg(X + km);
        return make_float2(g * xv.x, mirrored ? -(g * xv.y) : g * xv.y);
    };
    float2 *out = a.coef + (long long)ch * a.coeff_count + br.coeff_off;
    // GEN: the class holds lengths with prime factors above 5 (only the multiple-of-4 length policy makes them);
    // the other instantiations leave the chirp-z and direct-sum code out
    if (GEN && fp.generic == 2) {
        auto store_c = [&](int n, int, float2 v) { out[n] = v; };
        chirp_z_transform<+1, Sync>(buf, fp, a.ffts, a.tw, load, store_c, a.dbg, tid, nthr);
        return;
    }
    if (GEN && fp.generic) {
        float2 *alt = buf + M;
        for (int m = tid; m < M; m += nthr) buf[m] = load(m, 0);
        Sync::sync();
        fft_dif<+1, Sync, false>(buf, alt, 1, 1, 0u, fp, a.tw, tid, nthr);
        for (int n = tid; n < M; n += nthr) out[n] = buf[dif_pos(fp, n)];
        return;
    }
    float2 *tws = buf + M + 16;
    if (fp.nstages > 1) stage_twiddles(tws, a.tw, fp, tid, nthr);
    const Tile t{buf, 1, 1, 0u, M + 16, a.dbg};
    auto store = [&](int n, int, float2 v) { if (CQT_CHK(a.dbg, 303, n, M)) out[n] = v; };
    if (br.side == 0) {
        // regular band: every support bin lies in 1..N/2-1; spectrum and table share the support index j = d - d0
        const float2 *Xs = X + (br.kc + br.d0);
        const int shift_neg = M + br.d0;
        auto load_regular = [&](int m, int) -> float2 {
            const bool lo = m <= last_pos;
            if (!lo && m < first_neg) return make_float2(0.f, 0.f);
            const int j = lo ? m - br.d0 : m - shift_neg;
            if (!CQT_CHK(a.dbg, 309, j, br.S)) return make_float2(0.f, 0.f);
            const float g = __ldg(tab + j);
            const float2 xv = __ldg(Xs + j);
            return make_float2(g * xv.x, g * xv.y);
        };
        fft_fused<+1, Sync, false, true, false, true, false, false, MAXR>(t, fp, tws, load_regular, store, tid, nthr);
        return;
    }
    fft_fused<+1, Sync, false, true, false, true, false, false, MAXR>(t, fp, tws, load, store, tid, nthr);
}

// Synthesis store of a regular band (all bins in range; plane row and table share the support index j = d - d0):
// the window value is fetched ahead of the last butterfly, the product is stored after it.
struct RegularStore {
    const float *tab;
    float2 *Ys;
    int last_pos, first_neg, d0, shift_neg;
    struct Fetched { float h; int j; };
    __device__ __forceinline__ Fetched pre(int m, int) const {
        const bool lo = m <= last_pos;
        const bool ok = lo || m >= first_neg;
        const int j = lo ? m - d0 : m - shift_neg;
        Fetched f;
        f.j = ok ? j : -1;
        f.h = ok ? __ldg(tab + j) : 0.f;
        return f;
    }
    __device__ __forceinline__ void operator()(int, int, float2 u, Fetched f) const {
        if (f.j >= 0) Ys[f.j] = make_float2(f.h * u.x, f.h * u.y);
    }
};

template <int THREADS, int MINB, bool WARP, int MAXR, bool GEN>
__global__ void __launch_bounds__(THREADS, MINB) bands_to_spectrum_kernel(BandArgs a) {
    using G = Group<WARP>;
    using Sync = typename std::conditional<WARP, WarpSync, BlockSync>::type;
    const int item = G::item();
    if (item >= a.n_work * a.batch) return;
    const int tid = G::tid(), nthr = G::nthr();
    __shared__ BandItem item_s[WARP ? 8 : 1];
    BandItem &it = item_s[G::slot()];
    fetch_item<Sync>(a.items[a.work[item / a.batch]], it, tid, nthr);
    const BandRec br = it.br;
    const int ch = item % a.batch;
    const FftPlan &fp = it.fp;
    float2 *buf = smem_band + (size_t)G::slot() * a.max_elems;
    const int M = br.M;
    const float2 *in = a.coef + (long long)ch * a.coeff_count + br.coeff_off;
    // adjoint of analysis, sidebands: U[m] + conj U[-m] is the DFT of 2 Re c
    const bool fold = a.fold && br.side != 0;
    auto load = [&](int n, int) -> float2 {
        if (!CQT_CHK(a.dbg, 304, n, M)) return make_float2(0.f, 0.f);
        float2 v = __ldg(in + n);
        if (fold) v = make_float2(2.f * v.x, 0.f);
        return v;
    };
    const float *tab = a.table + br.tab_off;
    float2 *Y = a.Y + (long long)ch * a.y_pitch + br.y_off;
    const int last_pos = br.d0 + br.S - 1, first_neg = M + br.d0;
    // slot m -> offset d -> bin kc + d of the band's plane (only bins 0..N/2 are kept)
    const int half = a.N >> 1;
    auto store = [&](int m, int, float2 u) {
        int d;
        if (m <= last_pos) d = m;
        else if (m >= first_neg) d = m - M;
        else return;
        const int k = br.kc + d;
        if (k < 0 || k > half) return;
        if (!CQT_CHK(a.dbg, 305, br.tab_off + (d - br.d0), a.table_len)) return;
        const float h = __ldg(tab + (d - br.d0));
        if (CQT_CHK(a.dbg, 306, (long long)br.y_off + k, a.y_pitch)) Y[k] = make_float2(h * u.x, h * u.y);
    };
    // GEN: the class holds lengths with prime factors above 5 (only the multiple-of-4 length policy makes them);
    // the other instantiations leave the chirp-z and direct-sum code out
    if (GEN && fp.generic == 2) {
        chirp_z_transform<-1, Sync>(buf, fp, a.ffts, a.tw, load, store, a.dbg, tid, nthr);
        return;
    }
    if (GEN && fp.generic) {
        float2 *alt = buf + M;
        for (int n = tid; n < M; n += nthr) buf[n] = load(n, 0);
        Sync::sync();
        fft_dif<-1, Sync, false>(buf, alt, 1, 1, 0u, fp, a.tw, tid, nthr);
        for (int m = tid; m < M; m += nthr) store(m, 0, buf[dif_pos(fp, m)]);
        return;
    }
    float2 *tws = buf + M + 16;
    if (fp.nstages > 1) stage_twiddles(tws, a.tw, fp, tid, nthr);
    const Tile t{buf, 1, 1, 0u, M + 16, a.dbg};
    if (br.side == 0) {
        // regular band: all bins in range, plane row and table share the support index j = d - d0
        float2 *Ys = Y + (br.kc + br.d0);
        const int shift_neg = M + br.d0;
        const RegularStore store_regular{tab, Ys, last_pos, first_neg, br.d0, shift_neg};
        auto load_regular = [&](int n, int) -> float2 { return __ldg(in + n); };
        fft_fused<-1, Sync, false, true, false, true, false, false, MAXR>(t, fp, tws, load_regular, store_regular, tid, nthr);
        return;
    }
    fft_fused<-1, Sync, false, true, false, true, false, false, MAXR>(t, fp, tws, load, store, tid, nthr);
}

static BandArgs make_args(const cqt_plan &p, const BandClass &c, const float *table, int64_t batch) {
    BandArgs a{};
    a.items = p.d.items;
    a.ffts = p.d.ffts;
    a.tw = p.d.tw;
    a.table = table;
    a.work = c.d_work;
    a.n_work = c.n_bands;
    a.batch = (int)batch;
    a.N = (int)p.N;
    a.max_elems = c.max_elems;
    a.coeff_count = p.lay.coeff_count;
    a.y_pitch = p.y_pitch;
    a.table_len = p.lay.table_len;
    a.dbg = p.d.dbg;
    return a;
}

// kernel instantiations: (threads per CTA, CTAs per SM the registers must allow, one warp per item, largest radix
// compiled in).  The first five are the default classes; the last two serve the class-tuning environment hooks.
#define CQT_KERNEL_TABLE(X) \
    X(256, 4, true, 8) X(64, 16, false, 8) X(256, 4, false, 12) X(512, 2, false, 16) X(1024, 1, false, 16) \
    X(128, 8, false, 16) X(256, 2, false, 16)

template <bool ANALYSIS>
static const void *class_kernel(const BandClass &c) {
#define X(T, B, W, R)                                                                          \
    if (c.threads == T && c.min_blocks == B && (c.items_per_cta > 1) == W && c.max_radix <= R) { \
        if (c.has_generic)                                                                     \
            return ANALYSIS ? (const void *)bands_from_spectrum_kernel<T, B, W, R, true>       \
                            : (const void *)bands_to_spectrum_kernel<T, B, W, R, true>;        \
        return ANALYSIS ? (const void *)bands_from_spectrum_kernel<T, B, W, R, false>          \
                        : (const void *)bands_to_spectrum_kernel<T, B, W, R, false>;           \
    }
    CQT_KERNEL_TABLE(X)
#undef X
    return nullptr;
}

template <bool ANALYSIS>
static cudaError_t launch_class(const cqt_plan &p, int cls, const char *name, BandArgs &a, cudaStream_t st) {
    const BandClass &c = p.cls[cls];
    if (c.n_bands == 0) return cudaSuccess;
    const long long items = (long long)c.n_bands * a.batch;
    const size_t smem = (size_t)c.max_elems * c.items_per_cta * sizeof(float2);
    const long long grid = (items + c.items_per_cta - 1) / c.items_per_cta;
    void *args[] = {&a};
    const void *fn = class_kernel<ANALYSIS>(c);
    if (!fn) return cudaErrorInvalidDeviceFunction;
    cudaError_t e = cudaLaunchKernel(fn, dim3((unsigned)grid), dim3(c.threads), args, smem, st);
    note_launch(p, name, st);
    return e;
}

// The classes of one call are independent (disjoint outputs), and the short-band classes alone leave most SMs
// idle, so they run on two helper streams beside the long-band classes: fork after the caller's stream, join
// back into it.  With event timing on, everything stays on the caller's stream.
struct ForkJoin {
    const cqt_plan &p;
    cudaStream_t st;
    bool used[2] = {false, false};
    bool serial;
    ForkJoin(const cqt_plan &plan, cudaStream_t s) : p(plan), st(s), serial(plan.timing || !plan.aux[0] || !plan.aux[1]) {
        if (!serial) cudaEventRecord(p.ev_fork, st);
    }
    cudaStream_t stream_for(int cls) {
        if (serial || cls == 3 || p.cls[cls].n_bands == 0) return st;
        // the longest bands (one CTA per SM, fewer CTAs than SMs) and the middle class share one helper stream,
        // the two short classes the other; the 4096 < M <= 13,500 class stays on the caller's stream
        const int i = (cls == 2 || cls == 4) ? 0 : 1;
        if (!used[i]) { cudaStreamWaitEvent(p.aux[i], p.ev_fork, 0); used[i] = true; }
        return p.aux[i];
    }
    void join() {
        for (int i = 0; i < 2; ++i)
            if (used[i]) { cudaEventRecord(p.ev_join[i], p.aux[i]); cudaStreamWaitEvent(st, p.ev_join[i], 0); }
    }
};

cudaError_t launch_bands_from_spectrum(const cqt_plan &p, const float *table, const float2 *X, float2 *c,
                                       int64_t batch, cudaStream_t st) {
    ForkJoin fj(p, st);
    static const char *names[kNumClasses] = {"bands_from_spectrum/class0", "bands_from_spectrum/class1",
                                              "bands_from_spectrum/class2", "bands_from_spectrum/class3",
                                              "bands_from_spectrum/class4"};
    for (int i = kNumClasses - 1; i >= 0; --i) {   // longest bands first
        BandArgs a = make_args(p, p.cls[i], table, batch);
        a.spec = X;
        a.spec_pitch = p.lf.x_pitch;
        a.coef = c;
        cudaError_t e = launch_class<true>(p, i, names[i], a, fj.stream_for(i));
        if (e != cudaSuccess) { fj.join(); return e; }
    }
    fj.join();
    return cudaSuccess;
}

// Zero-fill of the bins between a band's support and its widened range (layouts with nested supports).
__global__ void __launch_bounds__(128) zero_fill_kernel(float2 *Y, long long y_pitch, const int2 *seg) {
    const int2 sg = seg[blockIdx.x];
    float2 *y = Y + (long long)blockIdx.y * y_pitch + sg.x;
    for (int i = threadIdx.x; i < sg.y; i += blockDim.x) y[i] = make_float2(0.f, 0.f);
}

cudaError_t launch_bands_to_spectrum(const cqt_plan &p, const float *table, bool fold_sidebands, const float2 *c,
                                     float2 *Y, int64_t batch, cudaStream_t st) {
    if (p.n_zero_seg > 0) {
        zero_fill_kernel<<<dim3((unsigned)p.n_zero_seg, (unsigned)batch), 128, 0, st>>>(Y, p.y_pitch, p.d.zero_seg);
        note_launch(p, "zero_fill", st);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    ForkJoin fj(p, st);
    static const char *names[kNumClasses] = {"bands_to_spectrum/class0", "bands_to_spectrum/class1",
                                              "bands_to_spectrum/class2", "bands_to_spectrum/class3",
                                              "bands_to_spectrum/class4"};
    for (int i = kNumClasses - 1; i >= 0; --i) {
        BandArgs a = make_args(p, p.cls[i], table, batch);
        a.coef = const_cast<float2 *>(c);
        a.Y = Y;
        a.fold = fold_sidebands ? 1 : 0;
        cudaError_t e = launch_class<false>(p, i, names[i], a, fj.stream_for(i));
        if (e != cudaSuccess) { fj.join(); return e; }
    }
    fj.join();
    return cudaSuccess;
}

cudaError_t configure_band_kernels(const cqt_plan &p) {
    for (int i = 0; i < kNumClasses; ++i) {
        const size_t s = (size_t)p.cls[i].max_elems * p.cls[i].items_per_cta * sizeof(float2);
        if (s <= 48 * 1024) continue;
        if (!class_kernel<true>(p.cls[i])) return cudaErrorInvalidDeviceFunction;
        cudaError_t e = cudaFuncSetAttribute(class_kernel<true>(p.cls[i]), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(class_kernel<false>(p.cls[i]), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace cqt
