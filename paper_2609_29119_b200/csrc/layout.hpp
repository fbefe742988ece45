// Host-side band layout of the constant-Q NSGT (Sec. 2 and Sec. 4 of the paper): centres,
// supports, windows g, lengths M, aggregate weight a_k and dual windows h.  Pure C++, no CUDA.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

namespace cqt {

struct LayoutDesc {
    double fs, fmin, fmax;
    int bins_per_octave;
    int64_t N;
    int window;    // 0 Hann, 1 Blackman-Harris
    int m_policy;  // 0 multiple of 4, 1 5-smooth multiple of 4, 2 power of two
    double min_win;
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

int64_t band_length(int64_t S, int policy);

}  // namespace cqt
