// Structures shared by the host plan builder and the kernels (plain data, no CUDA types).
#pragma once
#include <stdint.h>

namespace cqt {

constexpr int kMaxStages = 8;

// In-place decimation-in-frequency plan of one transform length M = r_1 r_2 ... r_d.
// Stage j works on sub-transforms of length n_j = M / (r_1 .. r_{j-1}) with butterfly stride
// s_j = n_j / r_j.  Frequency k = k_1 + r_1 (k_2 + r_2 (...)) ends at position
// ((k_1 r_2 + k_2) r_3 + ...) (mixed-radix digit reversal).
// Twiddles exp(-2 pi i y / M) are the product of two table entries:
//   tw[tw_off + (y & (C-1))] * tw[tw_off + C + (y >> logC)],  C = 1 << logC.
// Constants of one DIF stage.  radix and rmagic come first: the digit loops of the fused last stage read just those.
struct alignas(16) StageRec {
    int32_t radix;      // r_j
    uint32_t rmagic;    // ceil(2^32 / r_j)
    int32_t stride;     // s_j
    uint32_t smagic;    // ceil(2^32 / s_j)
    int32_t k1div;      // s_0 / n_j: butterfly blocks of stage j per first-stage output digit
    uint32_t k1magic;
    int32_t lg;         // log2 r_j for power-of-two plans
    int32_t pad_;
};

struct FftPlan {
    int32_t M;
    int32_t nstages;
    int32_t logC;
    int32_t tw_off;                 // into the plan's twiddle array (float2 elements)
    int32_t generic;                // 1: stage 0 is a generic (direct-sum) radix; 2: chirp-z (Bluestein) transform, see blu_*
    int32_t tw_count;               // entries of the two-level table (C + ceil(M / C))
    int32_t pad_delta;              // 1 if single-column buffers skip one element per s_0 positions (bank spread)
    int32_t tw_full_off;            // power-of-two plans: offset of the full table exp(-2 pi i y / M), y < M; else -1
    StageRec st[kMaxStages];        // per-stage constants, one 32-byte record each (two 16-byte loads in the kernels)
    // chirp-z evaluation of a length with a large prime factor: two power-of-two transforms of length blu_L
    int32_t blu_L;                  // power of two >= 2 M - 1
    int32_t blu_fft;                // FftPlan index of the length-blu_L plan
    int32_t blu_chirp_off;          // exp(-i pi n^2 / M), n < M, in the twiddle array
    int32_t blu_filter_off;         // DFT of the conjugate chirp / blu_L, in the digit-reversed order of that plan
};

// One band of the layout as the kernels see it.
struct BandRec {
    int32_t kc;         // centre bin
    int32_t d0;         // first (most negative) support offset
    int32_t S;          // support size
    int32_t M;          // coefficients
    int32_t tab_off;    // into the window tables (S entries, offset order)
    int32_t coeff_off;  // into one signal's coefficient row
    int32_t y_off;      // offset of the band's plane in one signal's weighted-bin scratch (entries indexed by bin)
    int32_t side;       // 0 regular, 1 DC, 2 Nyquist
    int32_t fft;        // index of the FftPlan for M (-1 for bands on the two-pass kernels)
    int32_t pad_[3];    // 48 bytes: the plan that follows a record in a BandItem stays 16-byte aligned
};

// A band record together with the radix plan of its length: what one work item of the band kernels needs,
// fetched in one cooperative load.
struct BandItem {
    BandRec br;
    FftPlan fp;
};

// A band transformed in two passes (M = A * B) through a scratch row.
struct TwoPassRec {
    int32_t band;
    int32_t A, B;
    int32_t fft_A, fft_B;        // FftPlan indices (plans with full twiddle tables)
    int32_t tw_m, log_m_c, n_m;  // two-level table of W_M
    int64_t scratch_off;         // into one signal's two-pass scratch row
};

// Per-bin cover: bands cover_lo .. cover_lo + cover_n - 1 contain the bin (contiguous because
// support starts and ends are monotone in the band index).
struct BinCover {
    int32_t lo_n;       // (cover_lo << 8) | cover_n
};

}  // namespace cqt
