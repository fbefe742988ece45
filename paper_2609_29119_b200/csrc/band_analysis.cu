// Analysis-form band kernels (see band_common.cuh).
#include "band_common.cuh"

namespace cqt {

template <int THREADS, int MINB, int LANES, int MAXR, bool GEN>
__global__ void __launch_bounds__(THREADS, MINB) bands_from_spectrum_kernel(BandArgs a) {
    pdl_launch_dependents();
    using G = Group<LANES>;
    using Sync = GroupSync<LANES>;
    const int item = G::item();
    if (item >= a.n_work * a.batch) return;   // whole group exits together
    const int tid = G::tid(), nthr = G::nthr();
    __shared__ BandItem item_s[LANES ? THREADS / (LANES ? LANES : 1) : 1];
    BandItem &it = item_s[G::slot()];
    fetch_item<Sync>(a.items[item / a.batch], it, tid, nthr);   // records in launch order of the class
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
    if (GEN && fp.generic) pdl_wait();
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
    pdl_wait();   // record, plan and twiddle table belong to the plan; what follows touches the predecessor's output
    const Tile t{buf, 1, 1, 0u, M + 16, a.dbg};
    // coefficients are written once and not read again by this call: streaming stores keep the L2 for the spectrum
    auto store = [&](int n, int, float2 v) { if (CQT_CHK(a.dbg, 303, n, M)) __stcs(out + n, v); };
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

const void *band_analysis_kernel(const BandClass &c, int lanes) {
#define X(T, B, W, R)                                                                          \
    if (c.threads == T && c.min_blocks == B && lanes == W && c.max_radix <= R)  \
        return c.has_generic ? (const void *)bands_from_spectrum_kernel<T, B, W, R, true> : (const void *)bands_from_spectrum_kernel<T, B, W, R, false>;
    CQT_KERNEL_TABLE(X)
#undef X
    return nullptr;
}

}  // namespace cqt
