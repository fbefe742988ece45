// Two-pass band transforms: M = A * B, pass 1 transforms columns (first index), multiplies by the inter-pass
// twiddle and writes an L2-resident scratch row, pass 2 transforms rows.  Used for bands above a length
// threshold: every CTA then works on a small tile (16 columns), so many CTAs share an SM and the latency of
// the global loads is hidden, at the price of one extra trip of the band through L2.  The band's gather /
// window / slot map is fused into the loads of pass 1 (analysis form); the dual-window multiply and the
// bin-ordered store into the stores of pass 2 (synthesis form).
//   analysis form:   m = m1*B + m2, n = n1 + A*n2
//      c[n1 + A n2] = sum_m2 e^{+2 pi i m2 n2 / B} [ e^{+2 pi i m2 n1 / M} sum_m1 e^{+2 pi i m1 n1 / A} u[m1 B + m2] ]
//   synthesis form:  n = n1*B + n2, m = m1 + A*m2, same structure with the opposite sign.
// Both sub-transforms run on the fused engine with full twiddle tables of length A and B in shared memory.
#include <algorithm>
#include <cstdlib>

#include "engine.cuh"
#include "internal.hpp"

namespace cqt {

extern __shared__ float2 smem_tp[];


struct TwoPassArgs {
    const TwoPassRec *recs;
    const BandRec *bands;
    const FftPlan *ffts;
    const float2 *tw;
    const float *table;
    int batch;
    int ch_per_cta;          // signals one CTA works through (tables and records are read once)
    int groups;              // ceil(batch / ch_per_cta)
    int N;
    int fold;                // synthesis form, adjoint: sideband input is replaced by 2 Re c
    const float2 *spec;      // analysis form: half-spectrum rows
    long long spec_pitch;
    float2 *coef;
    long long coeff_count;
    float2 *Y;
    long long y_pitch;
    float2 *scratch;         // [batch][scratch_pitch]
    long long scratch_pitch;
    int *dbg;
};

__device__ __forceinline__ float2 slot_value(const BandRec &br, const float *__restrict__ tab,
                                             const float2 *__restrict__ X, int N, int m) {
    const int last_pos = br.d0 + br.S - 1, first_neg = br.M + br.d0;
    int d;
    if (m <= last_pos) d = m;
    else if (m >= first_neg) d = m - br.M;
    else return make_float2(0.f, 0.f);
    const float g = __ldg(tab + (d - br.d0));
    const int k = br.kc + d;
    float2 xv;
    if (k < 0) xv = cconj(__ldg(X + (-k)));
    else if (k > (N >> 1)) xv = cconj(__ldg(X + (N - k)));
    else xv = __ldg(X + k);
    return make_float2(g * xv.x, g * xv.y);
}

__device__ __forceinline__ void copy_table(float2 *dst, const float2 *__restrict__ src, int n, int tid, int nthr) {
    for (int i = tid; i < n; i += nthr) dst[i] = __ldg(src + i);
}

// pass 1: TW adjacent columns (second index), A-point transform over the first index, inter-pass twiddle
template <int THREADS, int MINB, bool ANALYSIS, int TW>
__global__ void __launch_bounds__(THREADS, MINB) band2p_cols_kernel(TwoPassArgs a) {
    pdl_launch_dependents();
    const int tid = threadIdx.x, nthr = blockDim.x;
    const TwoPassRec rec = a.recs[blockIdx.y / a.groups];
    const int ch0 = (blockIdx.y % a.groups) * a.ch_per_cta, ch1 = min(a.batch, ch0 + a.ch_per_cta);
    const int c0 = blockIdx.x * TW;
    if (c0 >= rec.B) return;
    const int ncols = min(TW, rec.B - c0);
    const BandRec br = a.bands[rec.band];
    const FftPlan &fp = a.ffts[rec.fft_A];
    float2 *buf = smem_tp;
    float2 *twf = buf + (size_t)rec.A * TW;
    float2 *wm = twf + rec.A;
    copy_table(twf, a.tw + fp.tw_full_off, rec.A, tid, nthr);
    copy_table(wm, a.tw + rec.tw_m, rec.n_m, tid, nthr);
    const float *tab = a.table + br.tab_off;
    const bool fold = !ANALYSIS && a.fold && br.side != 0;
    const Tile t{buf, TW, TW, 0x80000000u / (TW / 2), rec.A * TW, a.dbg};
    pdl_wait();   // tables and records belong to the plan; the loop touches the predecessor's output
    for (int ch = ch0; ch < ch1; ++ch) {
    const float2 *X = ANALYSIS ? a.spec + (long long)ch * a.spec_pitch : nullptr;
    const float2 *cin = ANALYSIS ? nullptr : a.coef + (long long)ch * a.coeff_count + br.coeff_off;
    float2 *T = a.scratch + (long long)ch * a.scratch_pitch + rec.scratch_off;
    auto load = [&](int r, int c) -> float2 {
        if (c >= ncols) return make_float2(0.f, 0.f);
        const int idx = r * rec.B + c0 + c;
        if (ANALYSIS) return slot_value(br, tab, X, a.N, idx);
        float2 v = __ldg(cin + idx);
        if (fold) v = make_float2(2.f * v.x, 0.f);
        return v;
    };
    auto store = [&](int r, int c, float2 v) {
        if (c >= ncols) return;
        float2 w = twiddle_s(wm, rec.log_m_c, (uint32_t)(c0 + c) * (uint32_t)r);
        if (ANALYSIS) w.y = -w.y;
        if (CQT_CHK(a.dbg, 401, (long long)r * rec.B + c0 + c, br.M)) T[(long long)r * rec.B + c0 + c] = cmul(v, w);
    };
    fft_fused<ANALYSIS ? +1 : -1, BlockSync, false, false, true, false, true, true>(t, fp, twf, load, store, tid, nthr);
    __syncthreads();   // the next signal's first stage overwrites the tile
    }
}

// pass 2: TW adjacent rows (first output index), B-point transform over the second index
template <int THREADS, int MINB, bool ANALYSIS, int TW>
__global__ void __launch_bounds__(THREADS, MINB) band2p_rows_kernel(TwoPassArgs a) {
    pdl_launch_dependents();
    const int tid = threadIdx.x, nthr = blockDim.x;
    const TwoPassRec rec = a.recs[blockIdx.y / a.groups];
    const int ch0 = (blockIdx.y % a.groups) * a.ch_per_cta, ch1 = min(a.batch, ch0 + a.ch_per_cta);
    const int r0 = blockIdx.x * TW;
    if (r0 >= rec.A) return;
    const int nrows = min(TW, rec.A - r0);
    const BandRec br = a.bands[rec.band];
    const FftPlan &fp = a.ffts[rec.fft_B];
    float2 *buf = smem_tp;
    constexpr int pitch = TW + 1;
    float2 *twf = buf + (size_t)rec.B * pitch;
    copy_table(twf, a.tw + fp.tw_full_off, rec.B, tid, nthr);
    const Tile t{buf, pitch, TW, 0x80000000u / (TW / 2), rec.B * pitch, a.dbg};
    pdl_wait();   // tables and records belong to the plan; the loop touches the predecessor's output
    for (int ch = ch0; ch < ch1; ++ch) {
    const float2 *T = a.scratch + (long long)ch * a.scratch_pitch + rec.scratch_off;
    auto load = [&](int p, int r) -> float2 {
        if (r >= nrows) return make_float2(0.f, 0.f);
        const long long i = (long long)(r0 + r) * rec.B + p;
        return CQT_CHK(a.dbg, 402, i, br.M) ? __ldg(T + i) : make_float2(0.f, 0.f);
    };
    if (ANALYSIS) {
        float2 *out = a.coef + (long long)ch * a.coeff_count + br.coeff_off;
        auto store = [&](int q, int r, float2 v) {
            const long long n = (long long)(r0 + r) + (long long)rec.A * q;
            if (r < nrows && CQT_CHK(a.dbg, 403, n, br.M)) out[n] = v;
        };
        fft_fused<+1, BlockSync, false, false, false, false, true, true>(t, fp, twf, load, store, tid, nthr);
    } else {
        const float *tab = a.table + br.tab_off;
        float2 *Y = a.Y + (long long)ch * a.y_pitch + br.y_off;
        const int M = br.M, last_pos = br.d0 + br.S - 1, first_neg = M + br.d0, half = a.N >> 1;
        auto store = [&](int q, int r, float2 u) {
            if (r >= nrows) return;
            const long long m = (long long)(r0 + r) + (long long)rec.A * q;
            int d;
            if (m <= last_pos) d = (int)m;
            else if (m >= first_neg) d = (int)(m - M);
            else return;
            const int k = br.kc + d;
            if (k < 0 || k > half) return;
            const float h = __ldg(tab + (d - br.d0));
            if (CQT_CHK(a.dbg, 404, (long long)br.y_off + k, a.y_pitch)) Y[k] = make_float2(h * u.x, h * u.y);
        };
        fft_fused<-1, BlockSync, false, false, false, false, true, true>(t, fp, twf, load, store, tid, nthr);
    }
    __syncthreads();   // the next signal's first stage overwrites the tile
    }
}

// group 0: both factors <= 256 (small tiles, 128 threads at the full width, many CTAs per SM); group 1: the rest.
// wi: index into kTwoPassWidths
template <bool ANALYSIS>
static const void *cols_kernel(int g, int wi) {
    if (g == 1) {
        if (wi == 0) return (const void *)band2p_cols_kernel<512, 2, ANALYSIS, 16>;
        if (wi == 1) return (const void *)band2p_cols_kernel<512, 2, ANALYSIS, 8>;
        return (const void *)band2p_cols_kernel<512, 2, ANALYSIS, 4>;
    }
    if (wi == 0) return (const void *)band2p_cols_kernel<128, 8, ANALYSIS, 16>;
    if (wi == 1) return (const void *)band2p_cols_kernel<128, 8, ANALYSIS, 8>;
    return (const void *)band2p_cols_kernel<128, 8, ANALYSIS, 4>;
}
template <bool ANALYSIS>
static const void *rows_kernel(int g, int wi) {
    if (g == 1) {
        if (wi == 0) return (const void *)band2p_rows_kernel<512, 2, ANALYSIS, 16>;
        if (wi == 1) return (const void *)band2p_rows_kernel<512, 2, ANALYSIS, 8>;
        return (const void *)band2p_rows_kernel<512, 2, ANALYSIS, 4>;
    }
    if (wi == 0) return (const void *)band2p_rows_kernel<128, 8, ANALYSIS, 16>;
    if (wi == 1) return (const void *)band2p_rows_kernel<128, 8, ANALYSIS, 8>;
    return (const void *)band2p_rows_kernel<128, 8, ANALYSIS, 4>;
}

template <bool ANALYSIS>
static cudaError_t run_group(const cqt_plan &p, int g, const float *table, bool fold, const float2 *X, float2 *coef,
                             float2 *Y, float2 *scratch, int64_t batch, cudaStream_t st) {
    const TwoPassGroup &grp = p.two_pass[g];
    if (grp.bands.empty()) return cudaSuccess;
    TwoPassArgs a{};
    a.recs = grp.d_recs;
    a.bands = p.d.bands;
    a.ffts = p.d.ffts;
    a.tw = p.d.tw;
    a.table = table;
    a.batch = (int)batch;
    a.N = (int)p.N;
    a.fold = fold ? 1 : 0;
    a.spec = X; a.spec_pitch = p.lf.x_pitch;
    a.coef = coef; a.coeff_count = p.lay.coeff_count;
    a.Y = Y; a.y_pitch = p.y_pitch;
    a.scratch = scratch; a.scratch_pitch = p.two_pass_pitch;
    a.dbg = p.d.dbg;
    // tile width: the widest whose grid still has a CTA for every SM (a single long signal has one huge band and a
    // batch of one: 16-wide tiles would leave two thirds of the SMs without work), else the narrowest
    int wi = 0;
    while (wi < 2 && (long long)std::min(grp.max_tiles_cols[wi], grp.max_tiles_rows[wi]) * (long long)grp.bands.size() * batch < p.sm_count) ++wi;
    // narrow tiles mean few CTAs: each keeps the full thread count, so that a thread has one or two butterflies per
    // stage and the chain of dependent instructions per warp stays short
    const int threads = g == 0 ? 128 : 512;
    // signals per CTA: as many as keep at least ~6 CTAs per resident slot
    const long long slots = (long long)p.sm_count * (g == 0 ? 8 : 2);
    const long long tiles = (long long)std::min(grp.max_tiles_cols[wi], grp.max_tiles_rows[wi]) * (long long)grp.bands.size();
    int cpc = 1;
    while (cpc < 8 && tiles * ((batch + 2 * cpc - 1) / (2 * cpc)) >= 6 * slots) cpc *= 2;
    a.ch_per_cta = cpc;
    a.groups = (int)((batch + cpc - 1) / cpc);
    void *args[] = {&a};
    dim3 g1((unsigned)grp.max_tiles_cols[wi], (unsigned)(grp.bands.size() * a.groups));
    cudaError_t e = launch_kernel(cols_kernel<ANALYSIS>(g, wi), g1, dim3(threads), args, grp.smem_cols[wi], st);
    note_launch(p, ANALYSIS ? (g ? "band2p_cols/analysis/large" : "band2p_cols/analysis") : (g ? "band2p_cols/synthesis/large" : "band2p_cols/synthesis"), st);
    if (e != cudaSuccess) return e;
    dim3 g2((unsigned)grp.max_tiles_rows[wi], (unsigned)(grp.bands.size() * a.groups));
    e = launch_kernel(rows_kernel<ANALYSIS>(g, wi), g2, dim3(threads), args, grp.smem_rows[wi], st);
    note_launch(p, ANALYSIS ? (g ? "band2p_rows/analysis/large" : "band2p_rows/analysis") : (g ? "band2p_rows/synthesis/large" : "band2p_rows/synthesis"), st);
    return e;
}

cudaError_t launch_two_pass_from_spectrum(const cqt_plan &p, const float *table, const float2 *X, float2 *c,
                                          float2 *scratch, int64_t batch, cudaStream_t st) {
    for (int g = 1; g >= 0; --g) {
        cudaError_t e = run_group<true>(p, g, table, false, X, c, nullptr, scratch, batch, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_two_pass_to_spectrum(const cqt_plan &p, const float *table, bool fold, const float2 *c, float2 *Y,
                                        float2 *scratch, int64_t batch, cudaStream_t st) {
    for (int g = 1; g >= 0; --g) {
        cudaError_t e = run_group<false>(p, g, table, fold, nullptr, const_cast<float2 *>(c), Y, scratch, batch, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

size_t two_pass_smem_cols(const TwoPassBand &b, int width) { return ((size_t)b.A * width + b.A + b.n_m) * sizeof(float2); }
size_t two_pass_smem_rows(const TwoPassBand &b, int width) { return ((size_t)b.B * (width + 1) + b.B) * sizeof(float2); }

cudaError_t configure_two_pass_kernels(const cqt_plan &p) {
    cudaError_t e = cudaSuccess;
    auto set = [&](const void *f, size_t s) {
        if (e == cudaSuccess) e = allow_dynamic_smem(f, s, p);
    };
    for (int g = 0; g < 2; ++g) {
        if (p.two_pass[g].bands.empty()) continue;
        for (int wi = 0; wi < 3; ++wi) {
            set(cols_kernel<true>(g, wi), p.two_pass[g].smem_cols[wi]);
            set(cols_kernel<false>(g, wi), p.two_pass[g].smem_cols[wi]);
            set(rows_kernel<true>(g, wi), p.two_pass[g].smem_rows[wi]);
            set(rows_kernel<false>(g, wi), p.two_pass[g].smem_rows[wi]);
        }
    }
    return e;
}

}  // namespace cqt
