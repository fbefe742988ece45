// Synthesis-form band kernels (see band_common.cuh).
#include "band_common.cuh"

namespace cqt {

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

template <int THREADS, int MINB, int LANES, int MAXR, bool GEN>
__global__ void __launch_bounds__(THREADS, MINB) bands_to_spectrum_kernel(BandArgs a) {
    pdl_launch_dependents();
    using G = Group<LANES>;
    using Sync = GroupSync<LANES>;
    const int item = G::item();
    if (item >= a.n_work * a.batch) return;
    const int tid = G::tid(), nthr = G::nthr();
    __shared__ BandItem item_s[LANES ? THREADS / (LANES ? LANES : 1) : 1];
    BandItem &it = item_s[G::slot()];
    fetch_item<Sync>(a.items[item / a.batch], it, tid, nthr);   // records in launch order of the class
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
        float2 v = __ldcs(in + n);
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
    if (GEN && fp.generic) pdl_wait();
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
    pdl_wait();   // record, plan and twiddle table belong to the plan; what follows touches the predecessor's output
    const Tile t{buf, 1, 1, 0u, M + 16, a.dbg};
    if (br.side == 0) {
        // regular band: all bins in range, plane row and table share the support index j = d - d0
        float2 *Ys = Y + (br.kc + br.d0);
        const int shift_neg = M + br.d0;
        const RegularStore store_regular{tab, Ys, last_pos, first_neg, br.d0, shift_neg};
        // coefficients are read once: streaming loads keep the L2 for the weighted-bin planes
        auto load_regular = [&](int n, int) -> float2 { return __ldcs(in + n); };
        fft_fused<-1, Sync, false, true, false, true, false, false, MAXR>(t, fp, tws, load_regular, store_regular, tid, nthr);
        return;
    }
    fft_fused<-1, Sync, false, true, false, true, false, false, MAXR>(t, fp, tws, load, store, tid, nthr);
}

const void *band_synthesis_kernel(const BandClass &c, int lanes) {
#define X(T, B, W, R)                                                                          \
    if (c.threads == T && c.min_blocks == B && lanes == W && c.max_radix <= R)  \
        return c.has_generic ? (const void *)bands_to_spectrum_kernel<T, B, W, R, true> : (const void *)bands_to_spectrum_kernel<T, B, W, R, false>;
    CQT_KERNEL_TABLE(X)
#undef X
    return nullptr;
}

}  // namespace cqt
