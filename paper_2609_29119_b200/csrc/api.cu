// Plan construction and the C ABI of the transform calls (see include/cqt.h).
#include <algorithm>
#include <cmath>
#include <complex>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <new>

#include "../../include/cqt.h"
#include "internal.hpp"

using namespace cqt;

namespace {

const double kPi = 3.14159265358979323846;

uint32_t magic_of(uint32_t d) { return d <= 1 ? 0u : (uint32_t)(((1ull << 32) + d - 1) / d); }

// two-level table of exp(-2 pi i y / n), 0 <= y < n, appended to tw; returns offset and log2 C
int append_twiddles(std::vector<float2> &tw, int64_t n, int &logC) {
    logC = 0;
    while ((1ll << (2 * logC)) < n) ++logC;
    const int64_t C = 1ll << logC;
    const int64_t nhi = (n + C - 1) / C;
    const int off = (int)tw.size();
    for (int64_t j = 0; j < C; ++j) {
        const double ang = -2.0 * kPi * (double)(j % n) / (double)n;
        tw.push_back(make_float2((float)std::cos(ang), (float)std::sin(ang)));
    }
    for (int64_t i = 0; i < nhi; ++i) {
        const double ang = -2.0 * kPi * (double)((i * C) % n) / (double)n;
        tw.push_back(make_float2((float)std::cos(ang), (float)std::sin(ang)));
    }
    return off;
}

const int kBandRadices[] = {16, 15, 12, 10, 9, 8, 6, 5, 4, 3, 2};
const int kPow2Radices[] = {16, 8, 4, 2};

// fewest stages, then smallest largest radix; no radix above `cap`
bool best_split(int64_t m, const int *radices, int nr, int cap, std::map<int64_t, std::vector<int>> &memo, std::vector<int> &out) {
    if (m == 1) { out.clear(); return true; }
    auto it = memo.find(m);
    if (it != memo.end()) { out = it->second; return !out.empty(); }
    std::vector<int> best;
    for (int i = 0; i < nr; ++i) {
        const int r = radices[i];
        if (m % r || r > cap) continue;
        std::vector<int> sub;
        if (!best_split(m / r, radices, nr, cap, memo, sub)) continue;
        sub.push_back(r);
        std::sort(sub.begin(), sub.end(), [](int a, int b) { return a > b; });
        if (best.empty() || sub.size() < best.size() || (sub.size() == best.size() && sub[0] < best[0])) best = sub;
    }
    memo[m] = best;
    out = best;
    return !best.empty();
}

// returns false if M cannot be planned
bool make_fft_plan(int64_t M, bool pow2, std::vector<float2> &tw, FftPlan &fp, bool want_full = false, int radix_cap = 16) {
    std::memset(&fp, 0, sizeof(fp));
    fp.M = (int32_t)M;
    int64_t smooth = M, rest = 1;
    if (!pow2) {
        smooth = 1;
        int64_t m = M;
        for (int p : {2, 3, 5})
            while (m % p == 0) { m /= p; smooth *= p; }
        rest = m;
        if (rest > 4096) return false;
    }
    std::map<int64_t, std::vector<int>> memo;
    std::vector<int> radices;
    if (!best_split(smooth, pow2 ? kPow2Radices : kBandRadices, pow2 ? 4 : 11, radix_cap, memo, radices)) return false;
    if (rest > 1) { radices.insert(radices.begin(), (int)rest); fp.generic = 1; }
    if (radices.empty()) radices.push_back(1);
    if ((int)radices.size() > kMaxStages) return false;
    fp.nstages = (int32_t)radices.size();
    int64_t n_cur = M;
    for (int j = 0; j < fp.nstages; ++j) {
        fp.st[j].radix = radices[j];
        fp.st[j].stride = (int32_t)(n_cur / radices[j]);
        fp.st[j].rmagic = magic_of((uint32_t)radices[j]);
        fp.st[j].smagic = magic_of((uint32_t)fp.st[j].stride);
        const int64_t kd = j == 0 ? 1 : fp.st[0].stride / n_cur;
        fp.st[j].k1div = (int32_t)kd;
        fp.st[j].k1magic = magic_of((uint32_t)kd);
        n_cur /= radices[j];
    }
    int logC;
    fp.tw_off = append_twiddles(tw, M, logC);
    fp.logC = logC;
    fp.tw_count = (int32_t)((1ll << logC) + (M + (1ll << logC) - 1) / (1ll << logC));
    fp.pad_delta = (fp.nstages > 1 && (fp.st[0].stride % 2 == 0)) ? 1 : 0;
    fp.tw_full_off = -1;
    if (pow2 || want_full) {
        fp.tw_full_off = (int32_t)tw.size();
        for (int64_t y = 0; y < M; ++y) {
            const double ang = -2.0 * kPi * (double)y / (double)M;
            tw.push_back(make_float2((float)std::cos(ang), (float)std::sin(ang)));
        }
        for (int j = 0; j < fp.nstages && pow2; ++j) {
            int l = 0;
            while ((1 << l) < fp.st[j].radix) ++l;
            fp.st[j].lg = l;
        }
    }
    return true;
}

// host-side helpers for the chirp-z tables
void host_fft_pow2(std::vector<std::complex<double>> &v) {   // in-place radix-2, forward sign
    const size_t n = v.size();
    for (size_t i = 1, j = 0; i < n; ++i) {
        size_t bit = n >> 1;
        for (; j & bit; bit >>= 1) j ^= bit;
        j ^= bit;
        if (i < j) std::swap(v[i], v[j]);
    }
    for (size_t len = 2; len <= n; len <<= 1) {
        const double ang = -2.0 * kPi / (double)len;
        for (size_t i = 0; i < n; i += len)
            for (size_t k = 0; k < len / 2; ++k) {
                const std::complex<double> w = std::polar(1.0, ang * (double)k);
                const std::complex<double> u = v[i + k], t = v[i + k + len / 2] * w;
                v[i + k] = u + t;
                v[i + k + len / 2] = u - t;
            }
    }
}

int64_t host_dif_pos(const FftPlan &fp, int64_t k) {
    int64_t pos = 0, rem = k;
    for (int j = 0; j < fp.nstages; ++j) { pos = pos * fp.st[j].radix + rem % fp.st[j].radix; rem /= fp.st[j].radix; }
    return pos;
}

// chirp exp(-i pi n^2 / M) and the filter spectrum DFT_L(conj chirp, wrapped) / L in the DIF output order of `fl`
void make_chirp_tables(int64_t M, const FftPlan &fl, std::vector<float2> &tw, FftPlan &fp) {
    const int64_t L = fl.M;
    fp.blu_L = (int32_t)L;
    fp.blu_chirp_off = (int32_t)tw.size();
    std::vector<std::complex<double>> b(L, 0.0);
    for (int64_t n = 0; n < M; ++n) {
        const double ang = -kPi * (double)((n * n) % (2 * M)) / (double)M;
        tw.push_back(make_float2((float)std::cos(ang), (float)std::sin(ang)));
        const std::complex<double> c = std::polar(1.0, -ang);   // conj chirp
        b[n] = c;
        if (n) b[L - n] = c;
    }
    host_fft_pow2(b);
    fp.blu_filter_off = (int32_t)tw.size();
    std::vector<float2> perm(L);
    for (int64_t k = 0; k < L; ++k) {
        const std::complex<double> v = b[k] / (double)L;
        perm[host_dif_pos(fl, k)] = make_float2((float)v.real(), (float)v.imag());
    }
    tw.insert(tw.end(), perm.begin(), perm.end());
}

template <class T>
cudaError_t upload(T *&dst, const std::vector<T> &src) {
    dst = nullptr;
    if (src.empty()) return cudaSuccess;
    cudaError_t e = cudaMalloc((void **)&dst, src.size() * sizeof(T));
    if (e != cudaSuccess) return e;
    return cudaMemcpy(dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice);
}

void free_device(cqt_plan *p) {
    if (p->device < 0) return;
    int cur = 0;
    cudaGetDevice(&cur);
    cudaSetDevice(p->device);
    cudaFree(p->d.bands); cudaFree(p->d.ffts); cudaFree(p->d.tw);
    cudaFree(p->d.tab_analysis); cudaFree(p->d.tab_synthesis);
    cudaFree(p->d.tab_analysis_adj); cudaFree(p->d.tab_synthesis_adj);
    cudaFree(p->d.cover); cudaFree(p->d.dbg); cudaFree(p->d.zero_seg);
    for (auto &c : p->cls) cudaFree(c.d_items);
    for (auto &g : p->two_pass) cudaFree(g.d_recs);
    for (cudaEvent_t e : p->ev) cudaEventDestroy(e);
    for (int i = 0; i < cqt_plan::kHelpers; ++i) {
        if (p->aux[i]) cudaStreamDestroy(p->aux[i]);
        if (p->ev_join[i]) cudaEventDestroy(p->ev_join[i]);
    }
    if (p->ev_fork) cudaEventDestroy(p->ev_fork);
    cudaSetDevice(cur);
}

bool is_pow2(int64_t v) { return v > 0 && (v & (v - 1)) == 0; }

}  // namespace

extern "C" {

const char *cqt_status_string(cqt_status s) {
    switch (s) {
        case CQT_OK: return "ok";
        case CQT_ERR_INVALID_ARG: return "invalid argument";
        case CQT_ERR_UNSUPPORTED: return "unsupported size or layout";
        case CQT_ERR_BAD_LAYOUT: return "band layout is not a painless frame";
        case CQT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case CQT_ERR_CUDA: return "CUDA error";
        case CQT_ERR_STATE: return "call not valid in this state";
        case CQT_ERR_DEVICE_CHECK: return "device-side check failed";
    }
    return "unknown status";
}

cqt_status cqt_plan_create(double fs, double fmin, double fmax, int bins_per_octave, int64_t L, cqt_window window,
                           cqt_plan **out) {
    cqt_plan_desc d;
    d.fs = fs; d.fmin = fmin; d.fmax = fmax; d.bins_per_octave = bins_per_octave; d.L = L;
    d.window = (int)window; d.m_policy = CQT_M_MULT4; d.min_win = 4.0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return CQT_ERR_CUDA;
    d.device = dev;
    return cqt_plan_create_ex(&d, out);
}

static cqt_status finish_plan(cqt_plan *p, int64_t N, int device, const cqt_plan_tuning &tune, cqt_plan **out);

static bool length_supported(int64_t N) { return is_pow2(N) && N >= 64 && N <= (1ll << 22); }

cqt_status cqt_plan_create_ex(const cqt_plan_desc *desc, cqt_plan **out) {
    return cqt_plan_create_tuned(desc, nullptr, out);
}

cqt_status cqt_plan_create_tuned(const cqt_plan_desc *desc, const cqt_plan_tuning *tuning, cqt_plan **out) {
    if (!desc || !out) return CQT_ERR_INVALID_ARG;
    cqt_plan_tuning tune{};
    if (tuning) tune = *tuning;
    if (tune.max_cta_elems < 0 || tune.two_pass_min < 0) return CQT_ERR_INVALID_ARG;
    const int64_t N = desc->L;
    if (N < 0) return CQT_ERR_INVALID_ARG;
    if (!length_supported(N)) return CQT_ERR_UNSUPPORTED;
    cqt_plan *p = new (std::nothrow) cqt_plan();
    if (!p) return CQT_ERR_CUDA;
    LayoutDesc ld{desc->fs, desc->fmin, desc->fmax, desc->bins_per_octave, N, desc->window, desc->m_policy,
                  desc->min_win > 0 ? desc->min_win : 4.0};
    std::string why;
    int rc = build_layout(ld, p->lay, why);
    if (rc != 0) { delete p; return (cqt_status)rc; }
    return finish_plan(p, N, desc->device, tune, out);
}

cqt_status cqt_plan_create_bands(const cqt_band_list_desc *desc, cqt_plan **out) {
    if (!desc || !out || !desc->centre_hz || !desc->width_bins || desc->n_bands < 1 || desc->L < 0) return CQT_ERR_INVALID_ARG;
    const int64_t N = desc->L;
    if (!length_supported(N)) return CQT_ERR_UNSUPPORTED;
    if (desc->n_bands > 100000) return CQT_ERR_UNSUPPORTED;
    std::vector<BandSpec> specs((size_t)desc->n_bands);
    for (int64_t i = 0; i < desc->n_bands; ++i)
        specs[i] = BandSpec{desc->centre_hz[i], desc->width_bins[i], desc->group ? desc->group[i] : -1};
    cqt_plan *p = new (std::nothrow) cqt_plan();
    if (!p) return CQT_ERR_CUDA;
    LayoutDesc ld{desc->fs, 0.0, 0.0, 0, N, desc->window, desc->m_policy, 4.0};
    std::string why;
    int rc = build_layout_bands(ld, specs, p->lay, why);
    if (rc != 0) { delete p; return (cqt_status)rc; }
    return finish_plan(p, N, desc->device, cqt_plan_tuning{}, out);
}

cqt_status cqt_multires_bands(double fs, double fmin, int64_t L, const int *octaves, const int *bins_per_octave,
                              int n_sections, double min_win, int64_t capacity, double *centre_hz, double *width_bins,
                              int32_t *group, int64_t *n_bands) {
    if (!n_bands || capacity < 0) return CQT_ERR_INVALID_ARG;
    std::vector<BandSpec> specs;
    std::string why;
    int rc = multires_bands(fs, fmin, L, octaves, bins_per_octave, n_sections, min_win > 0 ? min_win : 4.0, specs, why);
    if (rc != 0) return (cqt_status)rc;
    *n_bands = (int64_t)specs.size();
    for (int64_t i = 0; i < std::min<int64_t>(capacity, (int64_t)specs.size()); ++i) {
        if (centre_hz) centre_hz[i] = specs[i].f;
        if (width_bins) width_bins[i] = specs[i].W;
        if (group) group[i] = specs[i].group;
    }
    return CQT_OK;
}

static cqt_status finish_plan(cqt_plan *p, int64_t N, int device, const cqt_plan_tuning &tune, cqt_plan **out) {
    p->N = N;
    p->device = device;
    const HostLayout &L = p->lay;
    p->g32.resize(L.table_len);
    p->h32.resize(L.table_len);
    for (int64_t i = 0; i < L.table_len; ++i) { p->g32[i] = (float)L.g[i]; p->h32[i] = (float)L.h[i]; }
    p->y_planes = 1;
    for (int64_t k = 0; k <= N / 2; ++k) p->y_planes = std::max(p->y_planes, (int)L.cover_n[k]);
    p->y_plane = (N / 2 + 1 + 7) / 8 * 8;
    p->y_pitch = p->y_plane * p->y_planes;

    // ---- transform-length plans and twiddles
    std::vector<float2> tw;
    std::map<int64_t, int> fft_of;
    enum { kPlanBand = 0, kPlanPow2 = 1, kPlanFull = 2 };
    auto plan_for = [&](int64_t M, int kind, int cap) -> int {
        const int64_t key = M + ((int64_t)kind << 40) + ((int64_t)cap << 44);
        auto it = fft_of.find(key);
        if (it != fft_of.end()) return it->second;
        FftPlan fp;
        if (!make_fft_plan(M, kind == kPlanPow2, tw, fp, kind == kPlanFull, cap)) return fft_of[key] = -1;
        p->ffts.push_back(fp);
        return fft_of[key] = (int)p->ffts.size() - 1;
    };
    LongFft &lf = p->lf;
    lf.Lp = N / 2;
    if (lf.Lp <= 4096) { lf.A = 1; lf.B = lf.Lp; }   // one CTA per signal: data and full twiddle table in shared memory
    else {
        int lg = 0;
        while ((1ll << lg) < lf.Lp) ++lg;
        lf.B = std::min<int64_t>(1024, 1ll << ((lg + 1) / 2));
        lf.A = lf.Lp / lf.B;
    }
    lf.fft_B = plan_for(lf.B, kPlanPow2, 16);
    lf.fft_A = lf.A > 1 ? plan_for(lf.A, kPlanPow2, 16) : lf.fft_B;
    lf.tw_lp = append_twiddles(tw, lf.Lp, lf.log_lp_c);
    lf.n_lp = (int)tw.size() - lf.tw_lp;
    lf.tw_n = append_twiddles(tw, N, lf.log_n_c);
    lf.n_n = (int)tw.size() - lf.tw_n;
    // tile widths chosen so that two CTAs of the row kernels (three of the column kernels) share an SM
    lf.tw_rows = lf.A == 1 ? 1 : (int)std::min<int64_t>(lf.B <= 512 ? 8 : 4, lf.A / 2);
    lf.tw_cols = lf.A == 1 ? 1 : (int)std::min<int64_t>(lf.A <= 512 ? 16 : 8, lf.B);
    lf.x_pitch = (lf.Lp + 1 + 7) / 8 * 8;

    // ---- band records
    p->bands.resize(L.bands.size());
    for (size_t i = 0; i < L.bands.size(); ++i) {
        const HostBand &hb = L.bands[i];
        BandRec &br = p->bands[i];
        br.kc = (int32_t)hb.kc; br.d0 = (int32_t)hb.d0; br.S = (int32_t)hb.S; br.M = (int32_t)hb.M;
        br.tab_off = (int32_t)hb.tab_off; br.coeff_off = (int32_t)hb.coeff_off;
        br.y_off = (int32_t)((int64_t)(i % p->y_planes) * p->y_plane);
        br.side = hb.side;
        br.fft = -1;
    }
    // ---- launch classes by band length
    // class 0: 8 lanes per item, 32 items per CTA; the others one CTA per item, sized so that several CTAs
    // share an SM (64 registers per thread) except for the longest bands, which fill its shared memory
    const int limits[kNumClasses] = {128, 1024, 4096, 13500, 1 << 30};
    {
        const int threads[kNumClasses] = {256, 64, 256, 512, 1024};
        const int minb[kNumClasses] = {4, 16, 4, 2, 1};
        for (int c = 0; c < kNumClasses; ++c) {
            p->cls[c].threads = threads[c];
            p->cls[c].min_blocks = minb[c];
            p->cls[c].lanes_few = c == 0 ? 32 : 0;
            p->cls[c].lanes_many = c == 0 ? 8 : 0;
            p->cls[c].max_radix = c <= 1 ? 8 : (c == 2 ? 12 : 16);
        }
    }
    std::vector<int> order(L.bands.size());
    for (size_t i = 0; i < order.size(); ++i) order[i] = (int)i;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return L.bands[a].M > L.bands[b].M; });
    int64_t smem_cap_elems = (227 * 1024) / 8;
    // test hook: a smaller cap sends shorter bands through the two-pass (huge band) kernels
    if (tune.max_cta_elems >= 64 && tune.max_cta_elems < smem_cap_elems) smem_cap_elems = tune.max_cta_elems;
    // bands above this length take the two-pass kernels (small tiles, many CTAs per SM)
    const int64_t two_pass_min = tune.two_pass_min > 0 ? std::max<int64_t>(64, tune.two_pass_min) : (1ll << 40);
    // M = A * B with plannable factors: fewest stages, then the most balanced split; 0 if there is none
    const int tp_radix_cap = 16;
    auto split_two_pass = [&](int64_t M) -> int64_t {
        int64_t bestA = 0;
        int best_cost = 1 << 30;
        for (int64_t a = 2; a * a <= M; ++a) {
            if (M % a || M / a > 1600) continue;
            FftPlan t1, t2;
            std::vector<float2> scratch_tw;
            if (!make_fft_plan(a, false, scratch_tw, t1, false, tp_radix_cap) || t1.generic) continue;
            if (!make_fft_plan(M / a, false, scratch_tw, t2, false, tp_radix_cap) || t2.generic) continue;
            const int cost = t1.nstages + t2.nstages;
            if (cost <= best_cost) { best_cost = cost; bestA = a; }
        }
        return bestA;
    };
    for (int i : order) {
        const int64_t M = L.bands[i].M;
        int c = 0;
        while (M > limits[c]) ++c;
        bool single = M <= two_pass_min;
        int64_t A2 = 0;
        if (!single) { A2 = split_two_pass(M); single = A2 == 0; }
        if (single) {
            // short bands: fewer registers, more CTAs per SM
            p->bands[i].fft = plan_for(M, kPlanBand, p->cls[c].max_radix);
            if (p->bands[i].fft < 0) { delete p; return CQT_ERR_UNSUPPORTED; }
            // a length with a large prime factor is evaluated as a chirp-z transform (two power-of-two transforms
            // of length L >= 2M - 1 in shared memory) instead of direct sums
            if (p->ffts[p->bands[i].fft].generic == 1 && p->ffts[p->bands[i].fft].st[0].radix >= 32 && M <= 8192) {
                int64_t Lz = 64;
                while (Lz < 2 * M - 1) Lz *= 2;
                const int fl = plan_for(Lz, kPlanPow2, 16);
                FftPlan &bfz = p->ffts[p->bands[i].fft];
                make_chirp_tables(M, p->ffts[fl], tw, bfz);
                bfz.blu_fft = fl;
                bfz.generic = 2;
            }
            // shared memory per item: padded buffer + two-level twiddle table (two buffers for generic radices,
            // the length-L buffer and that plan's table for chirp-z)
            const FftPlan &bf = p->ffts[p->bands[i].fft];
            const int64_t elems = bf.generic == 2 ? bf.blu_L + p->ffts[bf.blu_fft].tw_count
                                                  : (bf.generic ? 2 * M + bf.st[0].radix : M + 16 + bf.tw_count);
            if (elems > smem_cap_elems) {   // the cap is per work item; the classes with several items per CTA are far below it
                A2 = split_two_pass(M);
                if (!A2) { delete p; return CQT_ERR_UNSUPPORTED; }
                single = false;
            } else {
                p->cls[c].work.push_back(i);
                p->cls[c].max_elems = (int)std::max<int64_t>(p->cls[c].max_elems, elems);
                p->cls[c].n_bands++;
                if (bf.generic) p->cls[c].has_generic = true;
            }
        }
        if (!single) {
            TwoPassBand tb{};
            tb.band = i;
            tb.A = (int32_t)A2;
            tb.B = (int32_t)(M / A2);
            tb.fft_A = plan_for(tb.A, kPlanFull, tp_radix_cap);
            tb.fft_B = plan_for(tb.B, kPlanFull, tp_radix_cap);
            int lc = 0;
            tb.tw_m = append_twiddles(tw, M, lc);
            tb.log_m_c = lc;
            tb.n_m = (int32_t)tw.size() - tb.tw_m;
            tb.scratch_off = p->two_pass_pitch;
            p->two_pass_pitch += (M + 7) / 8 * 8;
            TwoPassGroup &g = p->two_pass[(tb.A <= 256 && tb.B <= 256) ? 0 : 1];
            g.bands.push_back(tb);
            for (int wi = 0; wi < 3; ++wi) {
                const int tw_tile = kTwoPassWidths[wi];
                g.max_tiles_cols[wi] = std::max(g.max_tiles_cols[wi], (tb.B + tw_tile - 1) / tw_tile);
                g.max_tiles_rows[wi] = std::max(g.max_tiles_rows[wi], (tb.A + tw_tile - 1) / tw_tile);
                g.smem_cols[wi] = std::max(g.smem_cols[wi], two_pass_smem_cols(tb, tw_tile));
                g.smem_rows[wi] = std::max(g.smem_rows[wi], two_pass_smem_rows(tb, tw_tile));
            }
        }
    }
    // a middle class whose longest band has at most one butterfly per thread at half the threads runs narrower CTAs
    if (p->cls[2].n_bands && L.bands[(size_t)p->cls[2].work[0]].M <= 2304) { p->cls[2].threads = 128; p->cls[2].min_blocks = 8; }
    // estimates for the per-call assignment of classes to streams (band.cu): total work, and the time one CTA
    // needs for the longest item (microseconds per element by class, from measured kernel times)
    {
        const double us_per_elem[kNumClasses] = {0.04, 0.015, 0.004, 0.0016, 0.0016};
        // classes holding lengths with a prime factor above 5 (direct sums, chirp-z with two longer transforms)
        const double generic_factor[kNumClasses] = {1.3, 1.3, 2.0, 3.5, 3.5};
        for (int c = 0; c < kNumClasses; ++c) {
            BandClass &bc = p->cls[c];
            int64_t longest = 0;
            for (int32_t b : bc.work) {
                const int64_t M = p->bands[(size_t)b].M;
                bc.stage_work += (double)M * (p->ffts[(size_t)p->bands[(size_t)b].fft].nstages + 1);
                longest = std::max(longest, M);
            }
            bc.latency_us = bc.n_bands ? (5.0 + us_per_elem[c] * (double)longest) * (bc.has_generic ? generic_factor[c] : 1.0) : 0.0;
        }
    }
    if (p->device < 0) { *out = p; return CQT_OK; }

    // ---- device tables
    int cur = 0;
    if (cudaGetDevice(&cur) != cudaSuccess || cudaSetDevice(p->device) != cudaSuccess) { p->device = -1; delete p; return CQT_ERR_CUDA; }
    std::vector<float> tA(L.table_len), tS(L.table_len), tTA(L.table_len), tSA(L.table_len);
    for (size_t i = 0; i < L.bands.size(); ++i) {
        const HostBand &hb = L.bands[i];
        for (int64_t j = 0; j < hb.S; ++j) {
            const int64_t k = hb.kc + hb.d0 + j;
            const double g = L.g[hb.tab_off + j], h = L.h[hb.tab_off + j];
            const double wk = (k == 0 || k == N / 2) ? 1.0 : 2.0;
            tA[hb.tab_off + j] = (float)(g / (double)hb.M);
            tS[hb.tab_off + j] = (float)h;
            tTA[hb.tab_off + j] = (float)((double)N * g / (2.0 * (double)hb.M));
            tSA[hb.tab_off + j] = (float)(h * wk / (double)N);
        }
    }
    std::vector<int32_t> cover(N / 2 + 1);
    for (int64_t k = 0; k <= N / 2; ++k) cover[k] = ((L.cover_lo[k] % p->y_planes) << 8) | L.cover_n[k];
    cudaError_t e = cudaSuccess;
    auto chk = [&](cudaError_t r) { if (e == cudaSuccess) e = r; };
    chk(upload(p->d.bands, p->bands));
    chk(upload(p->d.ffts, p->ffts));
    chk(upload(p->d.tw, tw));
    chk(upload(p->d.tab_analysis, tA));
    chk(upload(p->d.tab_synthesis, tS));
    chk(upload(p->d.tab_analysis_adj, tTA));
    chk(upload(p->d.tab_synthesis_adj, tSA));
    chk(upload(p->d.cover, cover));
    // nested supports: the bins of a band's widened range outside its support hold zeros in the band's plane
    std::vector<int2> zero_seg;
    for (size_t i = 0; i < L.bands.size(); ++i) {
        const HostBand &hb = L.bands[i];
        const int64_t s = hb.kc + hb.d0, en = s + hb.S - 1;
        if (hb.zl > 0) zero_seg.push_back(make_int2((int)(p->bands[i].y_off + s - hb.zl), (int)hb.zl));
        if (hb.zr > 0) zero_seg.push_back(make_int2((int)(p->bands[i].y_off + en + 1), (int)hb.zr));
    }
    p->n_zero_seg = (int)zero_seg.size();
    if (p->n_zero_seg) chk(upload(p->d.zero_seg, zero_seg));
    chk(upload(p->d.dbg, std::vector<int>(8, 0)));
    for (auto &c : p->cls) {
        // record and radix plan of every band of the class, in launch order: what a work item fetches first
        std::vector<BandItem> items(c.work.size());
        for (size_t i = 0; i < items.size(); ++i) {
            const int b = c.work[i];
            items[i].br = p->bands[(size_t)b];
            items[i].fp = p->ffts[(size_t)p->bands[(size_t)b].fft];
        }
        chk(upload(c.d_items, items));
    }
    cudaDeviceProp prop;
    chk(cudaGetDeviceProperties(&prop, p->device));
    p->sm_count = prop.multiProcessorCount;
    p->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
    // the helper streams carry the shorter classes: at the highest priority their CTAs are placed ahead of the
    // long class on the caller's stream, whatever order the launches (or the nodes of a captured graph) arrive in
    int prio_least = 0, prio_greatest = 0;
    chk(cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest));
    for (int i = 0; i < cqt_plan::kHelpers && e == cudaSuccess; ++i) {
        chk(cudaStreamCreateWithPriority(&p->aux[i], cudaStreamNonBlocking, prio_greatest));
        chk(cudaEventCreateWithFlags(&p->ev_join[i], cudaEventDisableTiming));
    }
    chk(cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming));
    if (e == cudaSuccess) chk(configure_band_kernels(*p));
    if (e == cudaSuccess) chk(configure_long_fft_kernels(*p));
    for (auto &g : p->two_pass) chk(upload(g.d_recs, g.bands));
    if (e == cudaSuccess) chk(configure_two_pass_kernels(*p));
    cudaSetDevice(cur);
    if (e != cudaSuccess) { cqt_plan_destroy(p); return CQT_ERR_CUDA; }
    *out = p;
    return CQT_OK;
}

cqt_status cqt_plan_destroy(cqt_plan *p) {
    if (!p) return CQT_OK;
    free_device(p);
    delete p;
    return CQT_OK;
}

int64_t cqt_plan_num_bands(const cqt_plan *p) { return p ? (int64_t)p->lay.bands.size() : -1; }
int64_t cqt_plan_coeff_count(const cqt_plan *p) { return p ? p->lay.coeff_count : -1; }
int64_t cqt_plan_signal_length(const cqt_plan *p) { return p ? p->N : -1; }
int64_t cqt_plan_table_length(const cqt_plan *p) { return p ? p->lay.table_len : -1; }
int cqt_plan_device(const cqt_plan *p) { return p ? p->device : -1; }

cqt_status cqt_plan_band_info(const cqt_plan *p, int64_t band, cqt_band_info *out) {
    if (!p || !out || band < 0 || band >= (int64_t)p->lay.bands.size()) return CQT_ERR_INVALID_ARG;
    const HostBand &hb = p->lay.bands[band];
    out->centre_hz = hb.centre_hz; out->centre_bin = hb.kc; out->support = hb.S; out->first_offset = hb.d0;
    out->M = hb.M; out->coeff_offset = hb.coeff_off; out->table_offset = hb.tab_off; out->is_sideband = hb.side;
    out->launch_class = -1;   // two-pass bands belong to no single-CTA class
    for (int c = 0; c < kNumClasses; ++c)
        for (int32_t b : p->cls[c].work)
            if (b == band) out->launch_class = c;
    return CQT_OK;
}

size_t cqt_plan_workspace_bytes(const cqt_plan *p, int64_t batch) {
    if (!p || batch <= 0) return 0;
    const int64_t t = p->lf.A > 1 ? p->lf.Lp : 0;
    const int64_t per = t + std::max<int64_t>(p->lf.x_pitch, p->y_pitch) + p->two_pass_pitch;
    return (size_t)(256 + batch * per * (int64_t)sizeof(float2));
}

cqt_status cqt_plan_tables(const cqt_plan *p, const float **g_host, const float **h_host) {
    if (!p) return CQT_ERR_INVALID_ARG;
    if (g_host) *g_host = p->g32.data();
    if (h_host) *h_host = p->h32.data();
    return CQT_OK;
}

cqt_status cqt_plan_check(const cqt_plan *p) {
    if (!p) return CQT_ERR_INVALID_ARG;
    if (p->device < 0 || !p->d.dbg) return CQT_OK;
    int w[8];
    if (cudaMemcpy(w, p->d.dbg, sizeof(w), cudaMemcpyDeviceToHost) != cudaSuccess) return CQT_ERR_CUDA;
    if (w[0] == 0) return CQT_OK;
    std::fprintf(stderr, "cqt debug check: site %d index %lld limit %lld block (%d,%d) thread %d\n", w[0],
                 ((long long)w[2] << 32) | (unsigned)w[1], ((long long)w[4] << 32) | (unsigned)w[3], w[5], w[6], w[7]);
    return CQT_ERR_DEVICE_CHECK;
}

}  // extern "C"

namespace cqt {

void note_launch(const cqt_plan &p, const char *name, cudaStream_t st) {
    if (name) ++p.launches;
    if (!p.timing) return;
    if (p.ev_used == p.ev.size()) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return;
        p.ev.push_back(e);
        p.ev_name.push_back(nullptr);
    }
    p.ev_name[p.ev_used] = name;
    cudaEventRecord(p.ev[p.ev_used], st);
    ++p.ev_used;
}

}  // namespace cqt

extern "C" {

int64_t cqt_plan_launch_count(const cqt_plan *p) { return p ? p->launches : -1; }

cqt_status cqt_plan_set_timing(const cqt_plan *p, int enable) {
    if (!p) return CQT_ERR_INVALID_ARG;
    p->timing = enable != 0;
    p->ev_used = 0;
    return CQT_OK;
}

cqt_status cqt_plan_read_timing(const cqt_plan *p, const char **names, float *ms, int64_t capacity, int64_t *count) {
    if (!p || !count || capacity < 0 || (capacity > 0 && (!names || !ms))) return CQT_ERR_INVALID_ARG;
    int64_t n = 0;
    for (size_t i = 1; i < p->ev_used; ++i) {
        if (!p->ev_name[i]) continue;   // start-of-call marker
        if (n < capacity) {
            if (cudaEventSynchronize(p->ev[i]) != cudaSuccess) return CQT_ERR_CUDA;
            if (cudaEventElapsedTime(&ms[n], p->ev[i - 1], p->ev[i]) != cudaSuccess) return CQT_ERR_CUDA;
            names[n] = p->ev_name[i];
        }
        ++n;
    }
    *count = n;
    p->ev_used = 0;
    return CQT_OK;
}

}  // extern "C"

namespace {

struct Call {
    const cqt_plan *p;
    float2 *T, *second, *huge;   // workspace regions
    cudaStream_t st;
    int prev_dev;
};

cqt_status begin_call(const cqt_plan *p, const void *sig, int64_t stride, int64_t batch, int64_t valid_len,
                      const void *coef, void *ws, size_t ws_bytes, void *stream, Call &c) {
    if (!p || !sig || !coef) return CQT_ERR_INVALID_ARG;
    if (batch <= 0 || batch > 65535 || valid_len <= 0 || valid_len > p->N || stride < valid_len) return CQT_ERR_INVALID_ARG;
    if (p->device < 0) return CQT_ERR_STATE;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) || ws_bytes < cqt_plan_workspace_bytes(p, batch)) return CQT_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(coef) & 7) || (reinterpret_cast<uintptr_t>(sig) & 3)) return CQT_ERR_INVALID_ARG;
    c.p = p;
    c.T = reinterpret_cast<float2 *>(ws);
    c.second = c.T + (p->lf.A > 1 ? batch * p->lf.Lp : 0);
    c.huge = c.second + batch * std::max<int64_t>(p->lf.x_pitch, p->y_pitch);
    c.st = reinterpret_cast<cudaStream_t>(stream);
    if (cudaGetDevice(&c.prev_dev) != cudaSuccess) return CQT_ERR_CUDA;
    if (c.prev_dev != p->device && cudaSetDevice(p->device) != cudaSuccess) return CQT_ERR_CUDA;
    note_launch(*p, nullptr, c.st);
    return CQT_OK;
}

cqt_status end_call(const Call &c, cudaError_t e) {
    if (c.prev_dev != c.p->device) cudaSetDevice(c.prev_dev);
    return e == cudaSuccess ? CQT_OK : CQT_ERR_CUDA;
}

cqt_status run_analysis_form(const cqt_plan *p, const float *table, const float *x, int64_t x_stride, int64_t batch,
                             int64_t valid_len, cqt_c64 *c, void *ws, size_t ws_bytes, void *stream,
                             const cqt::SliceSource *src = nullptr) {
    Call k;
    cqt_status s = begin_call(p, x, x_stride, batch, valid_len, c, ws, ws_bytes, stream, k);
    if (s != CQT_OK) return s;
    cudaError_t e = launch_rfft_forward(*p, x, x_stride, batch, valid_len, k.T, k.second, k.st, src);
    if (e == cudaSuccess) e = launch_bands_from_spectrum(*p, table, k.second, reinterpret_cast<float2 *>(c), k.huge, batch, k.st);
    return end_call(k, e);
}

cqt_status run_synthesis_form(const cqt_plan *p, const float *table, bool fold, const cqt_c64 *c, int64_t batch,
                              int64_t valid_len, float *x, int64_t x_stride, void *ws, size_t ws_bytes, void *stream) {
    Call k;
    cqt_status s = begin_call(p, x, x_stride, batch, valid_len, c, ws, ws_bytes, stream, k);
    if (s != CQT_OK) return s;
    cudaError_t e = launch_bands_to_spectrum(*p, table, fold, reinterpret_cast<const float2 *>(c), k.second, k.huge, batch, k.st);
    if (e == cudaSuccess) e = launch_rfft_inverse(*p, k.second, k.T, x, x_stride, batch, valid_len, k.st);
    return end_call(k, e);
}

}  // namespace

namespace cqt {

// Analysis of slices cut from a stream's ring buffer (slicq.cu): cqt_analyse with the slice cut fused into the load of
// the long FFT's first pass.  batch = slices x channels rows of the plan's full length.
cqt_status analyse_slices(const cqt_plan *p, const SliceSource &src, int64_t batch, cqt_c64 *c, void *ws, size_t ws_bytes,
                          void *stream) {
    if (!p || !src.ring || !src.win || !can_fuse_slice_cut(*p)) return CQT_ERR_INVALID_ARG;
    return run_analysis_form(p, p->d.tab_analysis, src.ring, p->N, batch, p->N, c, ws, ws_bytes, stream, &src);
}

}  // namespace cqt

extern "C" {

cqt_status cqt_analyse(const cqt_plan *p, const float *x, int64_t x_stride, int64_t batch, int64_t valid_len,
                       cqt_c64 *c, void *ws, size_t ws_bytes, void *stream) {
    return run_analysis_form(p, p ? p->d.tab_analysis : nullptr, x, x_stride, batch, valid_len, c, ws, ws_bytes, stream);
}

cqt_status cqt_synthesise(const cqt_plan *p, const cqt_c64 *c, int64_t batch, int64_t valid_len, float *x,
                          int64_t x_stride, void *ws, size_t ws_bytes, void *stream) {
    return run_synthesis_form(p, p ? p->d.tab_synthesis : nullptr, false, c, batch, valid_len, x, x_stride, ws, ws_bytes, stream);
}

cqt_status cqt_analyse_adjoint(const cqt_plan *p, const cqt_c64 *c_bar, int64_t batch, int64_t valid_len, float *x_bar,
                               int64_t x_stride, void *ws, size_t ws_bytes, void *stream) {
    return run_synthesis_form(p, p ? p->d.tab_analysis_adj : nullptr, true, c_bar, batch, valid_len, x_bar, x_stride, ws, ws_bytes, stream);
}

cqt_status cqt_synthesise_adjoint(const cqt_plan *p, const float *x_bar, int64_t x_stride, int64_t batch,
                                  int64_t valid_len, cqt_c64 *c_bar, void *ws, size_t ws_bytes, void *stream) {
    return run_analysis_form(p, p ? p->d.tab_synthesis_adj : nullptr, x_bar, x_stride, batch, valid_len, c_bar, ws, ws_bytes, stream);
}

}  // extern "C"
