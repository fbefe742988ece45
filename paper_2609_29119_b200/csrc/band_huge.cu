// Bands whose length M exceeds what one CTA can hold in shared memory (for example a wide Nyquist
// sideband): the M-point transform is split M = A * B and run as two passes through an L2-resident
// scratch row, with the band's gather / window / slot map fused into the first pass (analysis form)
// or the dual-window multiply and bin-ordered store fused into the second (synthesis form).
//   analysis form:   m = m1*B + m2, n = n1 + A*n2
//      c[n1 + A n2] = sum_m2 e^{+2 pi i m2 n2 / B} [ e^{+2 pi i m2 n1 / M} sum_m1 e^{+2 pi i m1 n1 / A} u[m1 B + m2] ]
//   synthesis form:  n = n1*B + n2, m = m1 + A*m2, same structure with the opposite sign.
#include "engine.cuh"
#include "internal.hpp"

namespace cqt {

extern __shared__ float2 smem_huge[];

struct HugeArgs {
    BandRec br;
    const FftPlan *ffts;
    const float2 *tw;
    int fft_A, fft_B, A, B, TW;
    int tw_m, log_m_c;       // two-level table of W_M
    const float *table;
    int N;
    int fold;                // synthesis form, adjoint: sideband input is replaced by 2 Re c
    const float2 *spec;      // analysis form: half-spectrum rows
    long long spec_pitch;
    float2 *coef;
    long long coeff_count;
    float2 *Y;
    long long y_pitch;
    float2 *scratch;         // [batch][M]
    long long scratch_pitch;
    uint32_t tw_magic;
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

// pass 1: TW adjacent columns (second index), A-point transform over the first index, inter-pass twiddle
template <bool ANALYSIS>
__global__ void __launch_bounds__(512) huge_cols_kernel(HugeArgs a) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int c0 = blockIdx.x * a.TW;
    const int ncols = min(a.TW, a.B - c0);
    const int ch = blockIdx.y;
    const FftPlan &fp = a.ffts[a.fft_A];
    float2 *buf = smem_huge;
    const int pitch = a.TW;
    const float *tab = a.table + a.br.tab_off;
    const float2 *X = ANALYSIS ? a.spec + (long long)ch * a.spec_pitch : nullptr;
    const float2 *cin = ANALYSIS ? nullptr : a.coef + (long long)ch * a.coeff_count + a.br.coeff_off;
    const bool fold = !ANALYSIS && a.fold && a.br.side != 0;
    for (int e = tid; e < a.A * a.TW; e += nthr) {
        const int r = e / a.TW, c = e - r * a.TW;
        float2 v = make_float2(0.f, 0.f);
        if (c < ncols) {
            const int idx = r * a.B + c0 + c;
            if (ANALYSIS) v = slot_value(a.br, tab, X, a.N, idx);
            else {
                v = __ldg(cin + idx);
                if (fold) v = make_float2(2.f * v.x, 0.f);
            }
        }
        buf[r * pitch + c] = v;
    }
    __syncthreads();
    fft_dif<ANALYSIS ? +1 : -1, BlockSync, false>(buf, nullptr, pitch, a.TW, a.tw_magic, fp, a.tw, tid, nthr);
    float2 *T = a.scratch + (long long)ch * a.scratch_pitch;
    const float2 *wm = a.tw + a.tw_m;
    for (int e = tid; e < a.A * a.TW; e += nthr) {
        const int r = e / a.TW, c = e - r * a.TW;
        if (c >= ncols) continue;
        const float2 v = buf[dif_pos(fp, r) * pitch + c];
        float2 w = twiddle(wm, a.log_m_c, (uint32_t)(c0 + c) * (uint32_t)r);
        if (ANALYSIS) w.y = -w.y;
        T[(long long)r * a.B + c0 + c] = cmul(v, w);
    }
}

// pass 2: TW adjacent rows (first output index), B-point transform over the second index
template <bool ANALYSIS>
__global__ void __launch_bounds__(512) huge_rows_kernel(HugeArgs a) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int r0 = blockIdx.x * a.TW;
    const int nrows = min(a.TW, a.A - r0);
    const int ch = blockIdx.y;
    const FftPlan &fp = a.ffts[a.fft_B];
    float2 *buf = smem_huge;
    const int pitch = a.TW + 1;
    const float2 *T = a.scratch + (long long)ch * a.scratch_pitch;
    for (int e = tid; e < a.TW * a.B; e += nthr) {
        const int r = e / a.B, p = e - r * a.B;
        buf[(size_t)p * pitch + r] = r < nrows ? __ldg(T + (long long)(r0 + r) * a.B + p) : make_float2(0.f, 0.f);
    }
    __syncthreads();
    fft_dif<ANALYSIS ? +1 : -1, BlockSync, false>(buf, nullptr, pitch, a.TW, a.tw_magic, fp, a.tw, tid, nthr);
    if (ANALYSIS) {
        float2 *out = a.coef + (long long)ch * a.coeff_count + a.br.coeff_off;
        for (int e = tid; e < a.TW * a.B; e += nthr) {
            const int q = e / a.TW, r = e - q * a.TW;
            if (r < nrows) out[(long long)(r0 + r) + (long long)a.A * q] = buf[(size_t)dif_pos(fp, q) * pitch + r];
        }
    } else {
        const float *tab = a.table + a.br.tab_off;
        float2 *Y = a.Y + (long long)ch * a.y_pitch + a.br.y_off;
        const int M = a.br.M, last_pos = a.br.d0 + a.br.S - 1, first_neg = M + a.br.d0;
        for (int e = tid; e < a.TW * a.B; e += nthr) {
            const int q = e / a.TW, r = e - q * a.TW;
            if (r >= nrows) continue;
            const long long m = (long long)(r0 + r) + (long long)a.A * q;
            int d;
            if (m <= last_pos) d = (int)m;
            else if (m >= first_neg) d = (int)(m - M);
            else continue;
            const int k = a.br.kc + d;
            if (k < 0 || k > (a.N >> 1)) continue;
            const float2 u = buf[(size_t)dif_pos(fp, q) * pitch + r];
            const float h = __ldg(tab + (d - a.br.d0));
            Y[k] = make_float2(h * u.x, h * u.y);
        }
    }
}

static uint32_t magic_of(uint32_t d) { return d <= 1 ? 0u : (uint32_t)(((1ull << 32) + d - 1) / d); }

template <bool ANALYSIS>
static cudaError_t run_huge(const cqt_plan &p, const HugeBand &hb, const float *table, bool fold, const float2 *X,
                            float2 *coef, float2 *Y, float2 *scratch, int64_t batch, cudaStream_t st) {
    HugeArgs a{};
    a.br = p.bands[hb.band];
    a.ffts = p.d.ffts;
    a.tw = p.d.tw;
    a.fft_A = hb.fft_A; a.fft_B = hb.fft_B; a.A = hb.A; a.B = hb.B; a.TW = hb.TW;
    a.tw_m = hb.tw_m; a.log_m_c = hb.log_m_c;
    a.table = table;
    a.N = (int)p.N;
    a.fold = fold ? 1 : 0;
    a.spec = X; a.spec_pitch = p.lf.x_pitch;
    a.coef = coef; a.coeff_count = p.lay.coeff_count;
    a.Y = Y; a.y_pitch = p.y_pitch;
    a.scratch = scratch + hb.scratch_off; a.scratch_pitch = p.huge_pitch;
    a.tw_magic = magic_of(hb.TW);
    dim3 g1((unsigned)((hb.B + hb.TW - 1) / hb.TW), (unsigned)batch), g2((unsigned)((hb.A + hb.TW - 1) / hb.TW), (unsigned)batch);
    const size_t s1 = (size_t)hb.A * hb.TW * 8, s2 = (size_t)hb.B * (hb.TW + 1) * 8;
    huge_cols_kernel<ANALYSIS><<<g1, 512, s1, st>>>(a);
    note_launch(p, ANALYSIS ? "huge_band_cols/analysis" : "huge_band_cols/synthesis", st);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    huge_rows_kernel<ANALYSIS><<<g2, 512, s2, st>>>(a);
    note_launch(p, ANALYSIS ? "huge_band_rows/analysis" : "huge_band_rows/synthesis", st);
    return cudaGetLastError();
}

cudaError_t launch_huge_from_spectrum(const cqt_plan &p, const float *table, const float2 *X, float2 *c, float2 *scratch,
                                      int64_t batch, cudaStream_t st) {
    for (const HugeBand &hb : p.huge) {
        cudaError_t e = run_huge<true>(p, hb, table, false, X, c, nullptr, scratch, batch, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_huge_to_spectrum(const cqt_plan &p, const float *table, bool fold, const float2 *c, float2 *Y,
                                    float2 *scratch, int64_t batch, cudaStream_t st) {
    for (const HugeBand &hb : p.huge) {
        cudaError_t e = run_huge<false>(p, hb, table, fold, nullptr, const_cast<float2 *>(c), Y, scratch, batch, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t configure_huge_kernels(const cqt_plan &p) {
    size_t need = 0;
    for (const HugeBand &hb : p.huge)
        need = std::max(need, std::max((size_t)hb.A * hb.TW * 8, (size_t)hb.B * (hb.TW + 1) * 8));
    if (need <= 48 * 1024) return cudaSuccess;
    cudaError_t e = cudaSuccess;
    auto set = [&](const void *f) { if (e == cudaSuccess) e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need); };
    set((const void *)huge_cols_kernel<true>);
    set((const void *)huge_cols_kernel<false>);
    set((const void *)huge_rows_kernel<true>);
    set((const void *)huge_rows_kernel<false>);
    return e;
}

}  // namespace cqt
