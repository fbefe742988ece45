// Host-side band layout of the constant-Q NSGT (Sec. 2 and Sec. 4 of the paper): centres,
// supports, windows g, lengths M, aggregate weight a_k and dual windows h.  Pure C++, no CUDA.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

namespace cqt {

// Longest band the multiple-of-4 policy leaves ragged (see band_length): 2 M + M / 4 complex values must fit the
// 227 KB of one CTA.
constexpr int64_t kMaxRaggedLength = 12800;

struct LayoutDesc {
    double fs, fmin, fmax;
    int bins_per_octave;
    int64_t N;
    int window;    // 0 Hann, 1 Blackman-Harris
    int m_policy;  // 0 multiple of 4, 1 5-smooth multiple of 4, 2 power of two
    double min_win;
};

// One regular band of an explicit band list.
struct BandSpec {
    double f;       // centre, Hz
    double W;       // total support width in bins (real valued)
    int32_t group;  // bands with the same group >= 0 share the largest M of the group; -1: own length
};

struct HostBand {
    double centre_hz;
    int64_t kc;       // centre bin
    int64_t d0;       // first support offset
    int64_t S;        // support size (offsets d0 .. d0 + S - 1)
    int64_t M;
    int64_t tab_off;  // into g / h
    int64_t coeff_off;
    int side;         // 0 regular, 1 DC, 2 Nyquist
    int64_t j_lo;     // first support index with 0 <= kc + d <= N/2
    int64_t n_in;     // number of such entries
    int64_t zl, zr;   // bins below / above the support that synthesis zero-fills in this band's plane (nested supports)
};

struct HostLayout {
    LayoutDesc desc;
    std::vector<HostBand> bands;
    std::vector<double> g, h;   // fp64 tables, sum of S entries
    std::vector<double> a;      // N/2 + 1
    int64_t coeff_count = 0;
    int64_t table_len = 0;
    std::vector<int32_t> cover_lo;  // per bin 0..N/2: first covering band
    std::vector<int32_t> cover_n;   // per bin: number of covering bands
};

// Returns 0 on success, else a cqt_status error code (-1 invalid, -2 unsupported, -3 bad layout).
int build_layout(const LayoutDesc &d, HostLayout &out, std::string &why);
// The same from an explicit list of regular bands, low to high (fmin, fmax, bins_per_octave, min_win of d unused).
int build_layout_bands(const LayoutDesc &d, const std::vector<BandSpec> &bands, HostLayout &out, std::string &why);
// Band lists: constant-Q (fmin 2^(j/b)), and consecutive sections of (octaves, bins per octave) (Sec. 4).
int constant_q_bands(const LayoutDesc &d, std::vector<BandSpec> &out, std::string &why);
int multires_bands(double fs, double fmin, int64_t N, const int *octaves, const int *bins_per_octave, int n_sections,
                   double min_win, std::vector<BandSpec> &out, std::string &why);

int64_t band_length(int64_t S, int policy);

}  // namespace cqt
