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
    const BandRec *bands;
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
};

template <bool WARP>
struct Group {
    __device__ static int tid() { return WARP ? (threadIdx.x & 31) : threadIdx.x; }
    __device__ static int nthr() { return WARP ? 32 : blockDim.x; }
    __device__ static int item() { return WARP ? blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5) : blockIdx.x; }
    __device__ static int slot() { return WARP ? (threadIdx.x >> 5) : 0; }
};

extern __shared__ float2 smem_band[];

template <bool WARP>
__global__ void __launch_bounds__(WARP ? 256 : 512) bands_from_spectrum_kernel(BandArgs a) {
    using G = Group<WARP>;
    using Sync = typename std::conditional<WARP, WarpSync, BlockSync>::type;
    const int item = G::item();
    if (item >= a.n_work * a.batch) return;   // whole group exits together
    const int tid = G::tid(), nthr = G::nthr();
    const BandRec br = a.bands[a.work[item / a.batch]];
    const int ch = item % a.batch;
    const FftPlan &fp = a.ffts[br.fft];
    float2 *buf = smem_band + (size_t)G::slot() * a.max_elems;
    float2 *alt = buf + br.M;
    const float2 *X = a.spec + (long long)ch * a.spec_pitch;
    const float *tab = a.table + br.tab_off;
    const int M = br.M, half = a.N >> 1;
    const int last_pos = br.d0 + br.S - 1;   // largest offset (>= 0)
    const int first_neg = M + br.d0;          // slot of the most negative offset
    for (int m = tid; m < M; m += nthr) {
        int d;
        bool in = true;
        if (m <= last_pos) d = m;
        else if (m >= first_neg) d = m - M;
        else { in = false; d = 0; }
        float2 v = make_float2(0.f, 0.f);
        if (in) {
            const float g = __ldg(tab + (d - br.d0));
            int k = br.kc + d;
            float2 xv;
            if (k < 0) xv = cconj(__ldg(X + (-k)));
            else if (k > half) xv = cconj(__ldg(X + (a.N - k)));
            else xv = __ldg(X + k);
            v = make_float2(g * xv.x, g * xv.y);
        }
        buf[m] = v;
    }
    Sync::sync();
    fft_dif<+1, Sync, false>(buf, alt, 1, 1, 0u, fp, a.tw, tid, nthr);
    float2 *out = a.coef + (long long)ch * a.coeff_count + br.coeff_off;
    for (int n = tid; n < M; n += nthr) out[n] = buf[dif_pos(fp, n)];
}

template <bool WARP>
__global__ void __launch_bounds__(WARP ? 256 : 512) bands_to_spectrum_kernel(BandArgs a) {
    using G = Group<WARP>;
    using Sync = typename std::conditional<WARP, WarpSync, BlockSync>::type;
    const int item = G::item();
    if (item >= a.n_work * a.batch) return;
    const int tid = G::tid(), nthr = G::nthr();
    const BandRec br = a.bands[a.work[item / a.batch]];
    const int ch = item % a.batch;
    const FftPlan &fp = a.ffts[br.fft];
    float2 *buf = smem_band + (size_t)G::slot() * a.max_elems;
    float2 *alt = buf + br.M;
    const int M = br.M;
    const float2 *in = a.coef + (long long)ch * a.coeff_count + br.coeff_off;
    // adjoint of analysis, sidebands: U[m] + conj U[-m] is the DFT of 2 Re c
    const bool fold = a.fold && br.side != 0;
    for (int n = tid; n < M; n += nthr) {
        float2 v = __ldg(in + n);
        if (fold) v = make_float2(2.f * v.x, 0.f);
        buf[n] = v;
    }
    Sync::sync();
    fft_dif<-1, Sync, false>(buf, alt, 1, 1, 0u, fp, a.tw, tid, nthr);
    const float *tab = a.table + br.tab_off;
    float2 *Y = a.Y + (long long)ch * a.y_pitch + br.y_off;
    for (int i = tid; i < br.n_in; i += nthr) {
        const int j = br.j_lo + i;
        const int d = br.d0 + j;
        const int m = d < 0 ? d + M : d;
        const float2 u = buf[dif_pos(fp, m)];
        const float h = __ldg(tab + j);
        Y[i] = make_float2(h * u.x, h * u.y);
    }
}

static BandArgs make_args(const cqt_plan &p, const BandClass &c, const float *table, int64_t batch) {
    BandArgs a{};
    a.bands = p.d.bands;
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
    return a;
}

template <class K>
static cudaError_t launch_class(const cqt_plan &p, const char *name, K warp_kernel, K block_kernel, const BandClass &c,
                                BandArgs &a, cudaStream_t st) {
    if (c.n_bands == 0) return cudaSuccess;
    const long long items = (long long)c.n_bands * a.batch;
    const size_t smem = (size_t)c.max_elems * c.items_per_cta * sizeof(float2);
    const long long grid = (items + c.items_per_cta - 1) / c.items_per_cta;
    if (c.items_per_cta > 1)
        warp_kernel<<<(unsigned)grid, c.threads, smem, st>>>(a);
    else
        block_kernel<<<(unsigned)grid, c.threads, smem, st>>>(a);
    note_launch(p, name, st);
    return cudaGetLastError();
}

cudaError_t launch_bands_from_spectrum(const cqt_plan &p, const float *table, const float2 *X, float2 *c,
                                       int64_t batch, cudaStream_t st) {
    for (int i = kNumClasses - 1; i >= 0; --i) {   // longest bands first
        BandArgs a = make_args(p, p.cls[i], table, batch);
        a.spec = X;
        a.spec_pitch = p.lf.x_pitch;
        a.coef = c;
        static const char *names[kNumClasses] = {"bands_from_spectrum/class0", "bands_from_spectrum/class1",
                                                  "bands_from_spectrum/class2", "bands_from_spectrum/class3"};
        cudaError_t e = launch_class(p, names[i], bands_from_spectrum_kernel<true>, bands_from_spectrum_kernel<false>, p.cls[i], a, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_bands_to_spectrum(const cqt_plan &p, const float *table, bool fold_sidebands, const float2 *c,
                                     float2 *Y, int64_t batch, cudaStream_t st) {
    for (int i = kNumClasses - 1; i >= 0; --i) {
        BandArgs a = make_args(p, p.cls[i], table, batch);
        a.coef = const_cast<float2 *>(c);
        a.Y = Y;
        a.fold = fold_sidebands ? 1 : 0;
        static const char *names[kNumClasses] = {"bands_to_spectrum/class0", "bands_to_spectrum/class1",
                                                  "bands_to_spectrum/class2", "bands_to_spectrum/class3"};
        cudaError_t e = launch_class(p, names[i], bands_to_spectrum_kernel<true>, bands_to_spectrum_kernel<false>, p.cls[i], a, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t configure_band_kernels(const cqt_plan &p) {
    size_t need = 0;
    for (int i = 0; i < kNumClasses; ++i) {
        const size_t s = (size_t)p.cls[i].max_elems * p.cls[i].items_per_cta * sizeof(float2);
        if (s > need) need = s;
    }
    if (need <= 48 * 1024) return cudaSuccess;
    cudaError_t e;
    e = cudaFuncSetAttribute(bands_from_spectrum_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(bands_to_spectrum_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
    return e;
}

}  // namespace cqt
