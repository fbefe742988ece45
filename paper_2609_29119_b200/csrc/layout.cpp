#include "layout.hpp"

#include <algorithm>
#include <cmath>
#include <map>

namespace cqt {

static const double kPi = 3.14159265358979323846;

static double window_profile(int kind, double t) {
    if (kind == 0) return 0.5 + 0.5 * std::cos(2.0 * kPi * t);
    const double a0 = 0.35875, a1 = 0.48829, a2 = 0.14128, a3 = 0.01168;  // 4-term Blackman-Harris
    return a0 + a1 * std::cos(2.0 * kPi * t) + a2 * std::cos(4.0 * kPi * t) + a3 * std::cos(6.0 * kPi * t);
}

static bool five_smooth(int64_t m) {
    for (int p : {2, 3, 5})
        while (m % p == 0) m /= p;
    return m == 1;
}

int64_t band_length(int64_t S, int policy) {
    int64_t m = 4 * ((S + 3) / 4);
    // Beyond kMaxRaggedLength coefficients a band no longer fits one CTA's shared memory together with the second
    // buffer a length with a large prime factor needs, and the two-pass kernels take smooth factors only: longer
    // bands get a 5-smooth length under the multiple-of-4 policy too.
    if (policy == 0 && m <= kMaxRaggedLength) return m;
    if (policy == 0 || policy == 1) {
        while (!five_smooth(m)) m += 4;
        return m;
    }
    m = 4;
    while (m < S) m *= 2;
    return m;
}

static double q_factor(int b) { return 1.0 / (std::pow(2.0, 1.0 / b) - std::pow(2.0, -1.0 / b)); }

int constant_q_bands(const LayoutDesc &d, std::vector<BandSpec> &out, std::string &why) {
    if (!(d.fs > 0) || !(d.fmin > 0) || !(d.fmax >= d.fmin) || d.fmax > d.fs / 2 * (1 + 1e-12) ||
        d.bins_per_octave < 1 || d.N < 4 || !(d.min_win >= 2.0)) {
        why = "invalid plan descriptor";
        return -1;
    }
    const int b = d.bins_per_octave;
    const double Q = q_factor(b);
    out.clear();
    for (int j = 0;; ++j) {
        const double f = d.fmin * std::pow(2.0, (double)j / b);
        if (f > d.fmax || f * (1.0 + 1.0 / (2.0 * Q)) > d.fs / 2.0) break;
        double W = (f / Q) * (double)d.N / d.fs;
        if (W < d.min_win) W = d.min_win;
        out.push_back(BandSpec{f, W, -1});
        if (j > 100000) { why = "too many bands"; return -2; }
    }
    if (out.empty()) { why = "no band fits between fmin and fmax"; return -3; }
    return 0;
}

int multires_bands(double fs, double fmin, int64_t N, const int *octaves, const int *bins_per_octave, int n_sections,
                   double min_win, std::vector<BandSpec> &out, std::string &why) {
    if (!(fs > 0) || !(fmin > 0) || N < 4 || n_sections < 1 || !octaves || !bins_per_octave || !(min_win >= 2.0)) {
        why = "invalid section list";
        return -1;
    }
    out.clear();
    double f_start = fmin;
    int oct0 = 0;
    for (int s = 0; s < n_sections; ++s) {
        const int b = bins_per_octave[s], no = octaves[s];
        if (b < 1 || no < 1 || (int64_t)b * no > 100000) { why = "invalid section"; return -1; }
        const double Q = q_factor(b);
        for (int j = 0; j < no * b; ++j) {
            const double f = f_start * std::pow(2.0, (double)j / b);
            double W = (f / Q) * (double)N / fs;
            if (W < min_win) W = min_win;
            out.push_back(BandSpec{f, W, oct0 + j / b});
        }
        f_start *= std::pow(2.0, (double)no);
        oct0 += no;
    }
    return 0;
}

int build_layout(const LayoutDesc &d, HostLayout &L, std::string &why) {
    std::vector<BandSpec> specs;
    const int rc = constant_q_bands(d, specs, why);
    if (rc != 0) return rc;
    return build_layout_bands(d, specs, L, why);
}

int build_layout_bands(const LayoutDesc &d, const std::vector<BandSpec> &specs, HostLayout &L, std::string &why) {
    const int64_t N = d.N;
    if (!(d.fs > 0) || N < 4 || (N & 1) || d.window < 0 || d.window > 1 || d.m_policy < 0 || d.m_policy > 2 ||
        specs.empty() || specs.size() > 100000) {
        why = "invalid plan descriptor";
        return -1;
    }
    L = HostLayout();
    L.desc = d;

    struct Reg { double f, W; int64_t kc, hw, M, s, e; int32_t group; };
    std::vector<Reg> reg;
    for (const BandSpec &sp : specs) {
        if (!(sp.f > 0) || !(sp.W >= 2.0) || !(sp.f <= d.fs / 2)) { why = "band centre or width out of range"; return -1; }
        Reg r;
        r.f = sp.f;
        r.W = sp.W;
        r.kc = (int64_t)std::floor(sp.f * (double)N / d.fs + 0.5);
        r.hw = (int64_t)std::ceil(sp.W / 2.0) - 1;  // largest integer strictly below W/2
        r.M = band_length(2 * r.hw + 1, d.m_policy);
        r.group = sp.group;
        if (!reg.empty() && r.kc < reg.back().kc) { why = "band centres must ascend"; return -1; }
        reg.push_back(r);
    }
    const int64_t k_first = reg.front().kc, k_last = reg.back().kc;
    if (k_first < 2 || N / 2 - k_last < 2) { why = "first or last centre within 2 bins of DC / Nyquist"; return -3; }
    for (const Reg &r : reg)
        if (r.kc - r.hw < 1 || r.kc + r.hw > N / 2 - 1) { why = "a regular band reaches DC or Nyquist"; return -3; }
    // bands of one group share the largest length of the group (one length per octave, Sec. 4)
    {
        std::map<int32_t, int64_t> biggest;
        for (const Reg &r : reg)
            if (r.group >= 0) biggest[r.group] = std::max(biggest[r.group], r.M);
        for (Reg &r : reg)
            if (r.group >= 0) r.M = biggest[r.group];
    }
    // Where supports nest (a wide band next to narrower ones) the bands covering a bin need not be consecutive.
    // Each band therefore gets a widened range [s, e] >= its support whose starts and ends are both monotone in
    // the band index; synthesis writes zeros on the extra bins, and the bands whose widened range holds a bin form
    // one contiguous index range.
    for (size_t i = 0; i < reg.size(); ++i) {
        reg[i].s = reg[i].kc - reg[i].hw;
        reg[i].e = reg[i].kc + reg[i].hw;
        if (i > 0) reg[i].e = std::max(reg[i].e, reg[i - 1].e);
    }
    for (size_t i = reg.size() - 1; i-- > 0;) reg[i].s = std::min(reg[i].s, reg[i + 1].s);

    auto push_band = [&](double f, int64_t kc, int64_t d0, int64_t S, int side, int64_t M) {
        HostBand hb;
        hb.centre_hz = f; hb.kc = kc; hb.d0 = d0; hb.S = S; hb.side = side;
        hb.M = M; hb.zl = 0; hb.zr = 0;
        hb.tab_off = L.table_len; hb.coeff_off = L.coeff_count;
        int64_t lo = 0, n = 0;
        bool first = true;
        for (int64_t j = 0; j < S; ++j) {
            const int64_t k = kc + d0 + j;
            if (k >= 0 && k <= N / 2) { if (first) { lo = j; first = false; } ++n; }
        }
        hb.j_lo = lo; hb.n_in = n;
        L.table_len += S; L.coeff_count += hb.M;
        L.bands.push_back(hb);
    };
    auto plateau = [&](int64_t edge, double W, std::vector<double> &g) {
        for (int64_t dd = -(edge - 1); dd <= edge - 1; ++dd) {
            const double t = (double)(edge - (dd < 0 ? -dd : dd)) / W;
            g.push_back(t >= 0.5 ? 1.0 : window_profile(d.window, 0.5 - t));
        }
    };
    // DC sideband, regular bands low to high, Nyquist sideband
    push_band(0.0, 0, -(k_first - 1), 2 * k_first - 1, 1, band_length(2 * k_first - 1, d.m_policy));
    plateau(k_first, reg.front().W, L.g);
    for (const Reg &r : reg) {
        push_band(r.f, r.kc, -r.hw, 2 * r.hw + 1, 0, r.M);
        L.bands.back().zl = (r.kc - r.hw) - r.s;
        L.bands.back().zr = r.e - (r.kc + r.hw);
        for (int64_t dd = -r.hw; dd <= r.hw; ++dd) L.g.push_back(window_profile(d.window, (double)dd / r.W));
    }
    const int64_t e = N / 2 - k_last;
    push_band(d.fs / 2.0, N / 2, -(e - 1), 2 * e - 1, 2, band_length(2 * e - 1, d.m_policy));
    plateau(e, reg.back().W, L.g);

    // aggregate weight and duals (Sec. 2): a_k = sum M g^2, h = M g / a_k on bins 0..N/2
    L.a.assign(N / 2 + 1, 0.0);
    for (const HostBand &hb : L.bands)
        for (int64_t j = hb.j_lo; j < hb.j_lo + hb.n_in; ++j) {
            const double gv = L.g[hb.tab_off + j];
            L.a[hb.kc + hb.d0 + j] += (double)hb.M * gv * gv;
        }
    for (int64_t k = 0; k <= N / 2; ++k)
        if (!(L.a[k] > 0)) { why = "windows do not cover every bin"; return -3; }
    L.h.assign(L.table_len, 0.0);
    for (const HostBand &hb : L.bands) {
        if (hb.S > hb.M) { why = "support exceeds band length"; return -3; }
        for (int64_t j = hb.j_lo; j < hb.j_lo + hb.n_in; ++j)
            L.h[hb.tab_off + j] = (double)hb.M * L.g[hb.tab_off + j] / L.a[hb.kc + hb.d0 + j];
    }
    // per-bin cover ranges over the widened in-range supports; their starts and ends must be monotone
    L.cover_lo.assign(N / 2 + 1, -1);
    L.cover_n.assign(N / 2 + 1, 0);
    int64_t prev_s = -1, prev_e = -1;
    for (size_t i = 0; i < L.bands.size(); ++i) {
        const HostBand &hb = L.bands[i];
        const int64_t s = hb.kc + hb.d0 + hb.j_lo - hb.zl, en = s + hb.zl + hb.n_in - 1 + hb.zr;
        if (s < prev_s || en < prev_e) { why = "band supports are not monotone"; return -3; }
        prev_s = s; prev_e = en;
        for (int64_t k = s; k <= en; ++k) {
            if (L.cover_lo[k] < 0) L.cover_lo[k] = (int32_t)i;
            if (L.cover_lo[k] + L.cover_n[k] != (int32_t)i) { why = "cover of a bin is not a contiguous band range"; return -3; }
            ++L.cover_n[k];
            if (L.cover_n[k] > 255) { why = "more than 255 bands cover one bin"; return -3; }
        }
    }
    return 0;
}

}  // namespace cqt
