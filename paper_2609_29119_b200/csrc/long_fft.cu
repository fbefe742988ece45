// Packed real FFT of length N through a complex FFT of length Lp = N/2 = A * B (Eq. pack), with
// the conjugate-symmetric fold (Eq. untangle) in the epilogue of the last forward pass; on the way back the
// prologue of the first inverse pass sums, per bin and in fixed band order, the weighted bins of the bands
// covering it and applies the inverse fold (Eq. retangle).
//
// Index split:  sample index j = j1 * B + j2,  bin index k = k1 + A * k2  (j1,k1 < A; j2,k2 < B).
//   forward  pass C ("columns"): for TWc adjacent j2, A-point DFT over j1, times W_Lp^{j2 k1},
//                                written to T[k1][j2].  First stage on registers straight from the
//                                signal (packing on load), last stage straight to T.
//            pass R ("rows"):    for a set of rows k1, B-point DFT over j2 gives Z[k1 + A k2];
//                                a CTA owns TWr rows and their mirror images A - k1 so both operands
//                                of Eq. untangle are in its shared memory (see row_of); writes the half
//                                spectrum X[0 .. Lp].
//   inverse  pass R':            a CTA owns the same rows as in forward pass R; per bin pair (q, Lp - q) it forms
//                                X^_q = sum over covering bands once and Z_q, Z_{Lp-q} by Eq. retangle in shared
//                                memory, then the inverse B-point DFT over q2, times conj W_Lp^{j2 q1}, written
//                                transposed to Tinv[j2][q1].
//            pass C':            inverse A-point DFT over q1, scaled, unpacked to x[2j], x[2j+1].
// When Lp is small (A == 1) the row kernels read / write the signal directly and passes C, C' vanish.
//
// Weighted-bin scratch: P planes of Lp+1 bins per signal; band b writes plane b mod P, where P is the
// largest number of bands covering one bin, so two bands of one plane never share a bin and the sum
// over the bands covering bin k reads planes (lo + i) mod P, i < n, at index k: coalesced, no atomics.
#include <algorithm>

#include "engine.cuh"
#include "internal.hpp"
#include "static_fft.cuh"

namespace cqt {

extern __shared__ float2 smem_long[];

struct LongArgs {
    const FftPlan *ffts;
    const float2 *tw;
    int fft_A, fft_B;
    int A, B, Lp;
    int tw_lp, log_lp_c, n_lp;   // two-level table of W_Lp and its entry count
    int tw_n, log_n_c, n_n;      // two-level table of W_N
    int tw_cols, tw_rows;
    int valid_len;
    int aligned;           // signal rows allow float2 access
    long long x_stride;
    const float *x_in;
    float *x_out;
    float2 *T;
    long long t_pitch;
    float2 *X;             // half spectrum rows (forward)
    long long x_pitch;
    // inverse: overlap-add + retangle in the prologue of the row pass
    int log_b, log_own;    // log2 B, log2 (2 TWr)
    const float2 *Y;
    long long y_pitch;     // per signal
    long long y_plane;     // per plane
    int planes;
    const int32_t *cover;
    float scale;
    uint32_t cols_magic, rows_magic;
    int *dbg;
    // sliced source (forward column pass of the streaming form): row r is slice r / channels of channel r % channels,
    // its sample i is slice_win[i] * ring[channel][(slice_first + (r / channels) * hop + i) mod ring_len], zero
    // before the start of the stream
    const float *ring;
    const float *slice_win;
    long long ring_len, slice_first, hop;
    int channels;
};

__device__ __forceinline__ float2 load_packed(const float *row, int j, int valid_len, int aligned) {
    const int i = 2 * j;
    if (i + 1 < valid_len) {
        if (aligned) return __ldcs(reinterpret_cast<const float2 *>(row + i));   // read once: streaming
        return make_float2(__ldcs(row + i), __ldcs(row + i + 1));
    }
    if (i < valid_len) return make_float2(__ldcs(row + i), 0.f);
    return make_float2(0.f, 0.f);
}

__device__ __forceinline__ void store_packed(float *row, int j, float2 v, int valid_len, int aligned) {
    const int i = 2 * j;
    if (i + 1 < valid_len) {
        if (aligned) __stcs(reinterpret_cast<float2 *>(row + i), v);
        else { __stcs(row + i, v.x); __stcs(row + i + 1, v.y); }
    } else if (i < valid_len) {
        __stcs(row + i, v.x);
    }
}

// copies the full twiddle table of a power-of-two plan into shared memory
__device__ __forceinline__ void stage_full(float2 *dst, const float2 *__restrict__ tw_base, const FftPlan &fp, int tid, int nthr) {
    const float2 *src = tw_base + fp.tw_full_off;
    for (int i = tid; i < fp.M; i += nthr) dst[i] = __ldg(src + i);
}

__device__ __forceinline__ void stage_table(float2 *dst, const float2 *__restrict__ src, int n, int tid, int nthr) {
    for (int i = tid; i < n; i += nthr) dst[i] = __ldg(src + i);
}

// Every pass exists once as a template over a compile-time Shape (radices, columns, pitch) and is instantiated
// for the common shapes plus the run-time planned fallback.
using DynShape = Shape<0, 0, 0, 0, 0>;
using Sh_16_16_8_8_9 = Shape<16, 16, 8, 8, 9>;
using Sh_8_8_8_16_16 = Shape<8, 8, 8, 16, 16>;
using Sh_16_16_1_16_16 = Shape<16, 16, 1, 16, 16>;
using Sh_16_8_1_16_16 = Shape<16, 8, 1, 16, 16>;
using Sh_16_8_8_8_8 = Shape<16, 8, 8, 8, 8>;
using Sh_16_16_8_8_8 = Shape<16, 16, 8, 8, 8>;
using Sh_8_8_8_16_17 = Shape<8, 8, 8, 16, 17>;
using Sh_16_16_1_16_17 = Shape<16, 16, 1, 16, 17>;
using Sh_16_8_1_16_17 = Shape<16, 8, 1, 16, 17>;
using Sh_16_8_8_8_9 = Shape<16, 8, 8, 8, 9>;

// The host picks the instantiation that matches the plan (pick_kernel below): a kernel holds the code of one shape only.
// ---------------------------------------------------------------- forward, pass C
// SLICED: the rows are slices cut from a ring buffer of the stream and multiplied by the slice window on load
// (the slice cut of the sliced transform, fused into this pass: no staged copy of the windowed slices)
template <class SH, bool SLICED>
__device__ __forceinline__ void cols_fwd_body(const LongArgs &a, const FftPlan &fp, float2 *buf, const float2 *tws,
                                              const float2 *wl, int j2_0, int ch, int tid, int nthr) {
    const int TW = a.tw_cols;
    float2 *T = a.T + (long long)ch * a.t_pitch;
    auto store = [&](int k1, int c, float2 v) {
        const float2 w = twiddle_s(wl, a.log_lp_c, (uint32_t)(j2_0 + c) * (uint32_t)k1);
        if (CQT_CHK(a.dbg, 201, k1 * a.B + j2_0 + c, a.Lp)) T[k1 * a.B + j2_0 + c] = cmul(v, w);
    };
    auto run = [&](auto load) {
        if constexpr (SH::is_static) {
            tile_fft_static<SH, -1, true, false>(buf, tws, load, store, tid, nthr);
        } else {
            const Tile t{buf, TW, TW, a.cols_magic, a.A * TW, a.dbg};
            fft_fused<-1, BlockSync, true, false, true, false, true, true>(t, fp, tws, load, store, tid, nthr);
        }
    };
    if constexpr (SLICED) {
        const int s_rel = ch / a.channels, chan = ch - s_rel * a.channels;
        const long long first = a.slice_first + (long long)s_rel * a.hop;   // stream index of the slice's sample 0
        const float *ring = a.ring + (long long)chan * a.ring_len;
        // position of sample 0 in the ring; the slice is no longer than the ring, so one conditional subtraction wraps
        const int R = (int)a.ring_len;
        const int base = (int)(((first % a.ring_len) + a.ring_len) % a.ring_len);
        const int lead = first < 0 ? (int)(-first) : 0;                      // samples before the start of the stream
        const float *win = a.slice_win;
        auto sample = [&](int i) -> float {
            if (i < lead) return 0.f;
            int p = base + i;
            if (p >= R) p -= R;
            if (!CQT_CHK(a.dbg, 212, p, R)) return 0.f;
            return __ldg(win + i) * __ldg(ring + p);
        };
        run([&](int j1, int c) -> float2 {
            const int i = 2 * (j1 * a.B + j2_0 + c);
            return make_float2(sample(i), sample(i + 1));
        });
    } else {
        const float *row = a.x_in + (long long)ch * a.x_stride;
        run([&](int j1, int c) -> float2 { return load_packed(row, j1 * a.B + j2_0 + c, a.valid_len, a.aligned); });
    }
}

template <class SH, bool SLICED = false>
__global__ void __launch_bounds__(512, 2) rfft_cols_fwd_kernel(LongArgs a) {
    pdl_launch_dependents();
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int TW = a.tw_cols;
    const int j2_0 = blockIdx.x * TW;
    const int ch = blockIdx.y;
    const FftPlan &fp = a.ffts[a.fft_A];
    float2 *buf = smem_long;
    float2 *tws = buf + (size_t)a.A * TW;
    float2 *wl = tws + fp.M;
    stage_full(tws, a.tw, fp, tid, nthr);
    stage_table(wl, a.tw + a.tw_lp, a.n_lp, tid, nthr);
    pdl_wait();   // the tables above belong to the plan; what follows reads the predecessor's output
    cols_fwd_body<SH, SLICED>(a, fp, buf, tws, wl, j2_0, ch, tid, nthr);
}

// Rows of CTA t of the forward row kernel, column r of its tile: r < TW is row TW t + 1 + r, r >= TW its mirror
// A - (TW t + 1 + (r - TW)).  Eq. untangle pairs row k1 with row A - k1, so both operands of every output are in
// the tile.  The last tile's row A/2 is its own mirror; the column that would repeat it holds row 0, which pairs
// with itself too: every row sits in exactly one tile and nothing is transformed twice.
__device__ __forceinline__ int row_of(int t, int r, int TW, int A) {
    const int k1 = r < TW ? TW * t + 1 + r : A - (TW * t + 1 + (r - TW));
    return (r >= TW && 2 * k1 == A) ? 0 : k1;
}

// ---------------------------------------------------------------- forward, pass R (+ untangle)
template <class SH>
__device__ __forceinline__ void rows_fwd_body(const LongArgs &a, const FftPlan &fp, float2 *buf, const float2 *tws,
                                              const float2 *wn, int t, int ch, int tid, int nthr) {
    const int A = a.A, B = a.B, TW = a.tw_rows;
    const bool direct = (A == 1);
    const int ncols = direct ? 1 : 2 * TW;
    const int pitch = SH::is_static ? SH::PITCH : (direct ? 1 : ncols + 1);   // odd: conflict-free transposing accesses
    if (direct) {
        const float *row = a.x_in + (long long)ch * a.x_stride;
        const Tile tile{buf, pitch, ncols, a.rows_magic, B * pitch, a.dbg};
        auto load = [&](int j, int) -> float2 { return load_packed(row, j, a.valid_len, a.aligned); };
        fft_fused_keep<-1, BlockSync, true, false, true>(tile, fp, tws, load, tid, nthr);
    } else {
        const float2 *T = a.T + (long long)ch * a.t_pitch;
        auto load = [&](int j2, int r) -> float2 {
            const int i = row_of(t, r, TW, A) * B + j2;
            return CQT_CHK(a.dbg, 202, i, a.Lp) ? __ldg(T + i) : make_float2(0.f, 0.f);
        };
        if constexpr (SH::is_static) {
            auto nostore = [](int, int, float2) {};
            tile_fft_static<SH, -1, false, true>(buf, tws, load, nostore, tid, nthr);
        } else {
            const Tile tile{buf, pitch, ncols, a.rows_magic, B * pitch, a.dbg};
            fft_fused_keep<-1, BlockSync, true, false, true>(tile, fp, tws, load, tid, nthr);
        }
    }
    float2 *X = a.X + (long long)ch * a.x_pitch;
    // epilogue: each thread keeps one row (column r) and walks k2; for rows other than k1 = 0 the partner
    // Z_{Lp-k} sits in the mirror row's column at k2' = B-1-k2, whose position is the digit-wise complement B-1-pos(k2);
    // row 0 pairs with itself at k2' = (B - k2) mod B, row A/2 with itself at B-1-k2
    const int nown = direct ? 1 : 2 * TW;
    const int r = direct ? 0 : (tid & (nown - 1));
    const int kstart = direct ? tid : (tid >> a.log_own), kstep = direct ? nthr : (nthr >> a.log_own);
    const int k1 = direct ? 0 : row_of(t, r, TW, A);
    const int rp = (direct || k1 == 0 || 2 * k1 == A) ? r : (r < TW ? r + TW : r - TW);
    for (int k2 = kstart; k2 < B; k2 += kstep) {
        const uint32_t pos = SH::pos(fp, (uint32_t)k2);
        uint32_t posp;
        const int rpp = rp;
        if (k1 == 0) posp = k2 == 0 ? 0u : SH::pos(fp, (uint32_t)(B - k2));
        else posp = (uint32_t)(B - 1) - pos;
        const int k = k1 + A * k2;
        if (!CQT_CHK(a.dbg, 203, k, a.Lp) || !CQT_CHK(a.dbg, 204, (size_t)posp * pitch + rpp, B * pitch) ||
            !CQT_CHK(a.dbg, 209, (size_t)pos * pitch + r, B * pitch))
            continue;
        const float2 z = buf[pos * (uint32_t)pitch + r];
        const float2 zp = buf[posp * (uint32_t)pitch + rpp];
        // X_k = 1/2 (1 - i w) Z_k + 1/2 (1 + i w) conj Z_{Lp-k},  w = exp(-2 pi i k / N)
        const float2 w = twiddle_s(wn, a.log_n_c, (uint32_t)k);
        const float2 ev = make_float2(0.5f * (z.x + zp.x), 0.5f * (z.y - zp.y));   // (Z + conj Zp)/2
        const float2 od = make_float2(0.5f * (z.x - zp.x), 0.5f * (z.y + zp.y));   // (Z - conj Zp)/2
        // -i w od = (w.y od.x + w.x od.y) + i (w.y od.y - w.x od.x)
        const float2 xk = make_float2(ev.x + (w.y * od.x + w.x * od.y), ev.y + (w.y * od.y - w.x * od.x));
        X[k] = xk;
        if (k == 0) X[a.Lp] = make_float2(z.x - z.y, 0.f);
    }
}

template <class SH>
__global__ void __launch_bounds__(512, 2) rfft_rows_fwd_kernel(LongArgs a) {
    pdl_launch_dependents();
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int ch = blockIdx.y, t = blockIdx.x;
    const bool direct = (a.A == 1);
    const int ncols = direct ? 1 : 2 * a.tw_rows;
    const int pitch = direct ? 1 : ncols + 1;
    const FftPlan &fp = a.ffts[a.fft_B];
    float2 *buf = smem_long;
    float2 *tws = buf + (size_t)a.B * pitch;
    float2 *wn = tws + fp.M;
    stage_full(tws, a.tw, fp, tid, nthr);
    stage_table(wn, a.tw + a.tw_n, a.n_n, tid, nthr);
    pdl_wait();   // the tables above belong to the plan; what follows reads the predecessor's output
    rows_fwd_body<SH>(a, fp, buf, tws, wn, t, ch, tid, nthr);
}

// ---------------------------------------------------------------- inverse: overlap-add + retangle
// sum over the bands covering bin k, in band order
// Sum over the bands covering bin k, in band order.  The cover word is (plane of the first covering band << 8) | number
// of covering bands; band i of the range sits in plane (first + i) mod planes.  The first kUnroll plane values are loaded
// unconditionally-predicated before any is used, so that their latencies overlap; absent terms add +0.
constexpr int kGatherUnroll = 3;
struct GatherLoads {
    float2 v[kGatherUnroll];
    int n, off, plane_len, wrap;
};
__device__ __forceinline__ GatherLoads gather_issue(const LongArgs &a, const float2 *__restrict__ Y, int k, int32_t cv) {
    GatherLoads g;
    g.n = cv & 255;
    g.plane_len = (int)a.y_plane;
    g.wrap = a.planes * g.plane_len;
    g.off = (cv >> 8) * g.plane_len + k;
    if (!CQT_CHK(a.dbg, 206, g.n, a.planes + 1)) g.n = 0;
#pragma unroll
    for (int i = 0; i < kGatherUnroll; ++i) {
        g.v[i] = i < g.n ? __ldg(Y + g.off) : make_float2(0.f, 0.f);
        g.off += g.plane_len;
        if (g.off >= g.wrap) g.off -= g.wrap;
    }
    return g;
}
__device__ __forceinline__ float2 gather_finish(const float2 *__restrict__ Y, GatherLoads &g) {
    float2 acc = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < kGatherUnroll; ++i) { acc.x += g.v[i].x; acc.y += g.v[i].y; }
    for (int i = kGatherUnroll; i < g.n; ++i) {
        const float2 v = __ldg(Y + g.off);
        acc.x += v.x;
        acc.y += v.y;
        g.off += g.plane_len;
        if (g.off >= g.wrap) g.off -= g.wrap;
    }
    return acc;
}

// One pair (q, m = Lp - q) of packed bins: both half-spectrum bins are summed once (bands in fixed order) and both
// packed bins follow from the same two values (Eq. retangle with w_{Lp-q} = -conj w_q):
//   Z_q      = s [ (X_q + conj X_m) + i conj(w) (X_q - conj X_m) ]
//   Z_{Lp-q} = s [ (X_m + conj X_q) - i w (X_m - conj X_q) ],   w = exp(-2 pi i q / N), s = 1/(2 Lp)
// wn: two-level table of W_N (shared memory).
__device__ __forceinline__ void retangle_finish(const LongArgs &a, const float2 *__restrict__ Y, const float2 *wn, int q,
                                                GatherLoads &gq, GatherLoads &gm, float2 &zq, float2 &zm) {
    float2 xq = gather_finish(Y, gq);
    float2 xm = gather_finish(Y, gm);
    if (q == 0) { xq.y = 0.f; xm.y = 0.f; }   // bins 0 and N/2 are made real
    const float2 w = twiddle_s(wn, a.log_n_c, (uint32_t)q);
    {
        const float2 ev = make_float2(xq.x + xm.x, xq.y - xm.y);   // X_q + conj X_m
        const float2 od = make_float2(xq.x - xm.x, xq.y + xm.y);   // X_q - conj X_m
        const float2 rot = cmul(make_float2(w.y, w.x), od);        // i conj(w) = (w.y, w.x)
        zq = make_float2(a.scale * (ev.x + rot.x), a.scale * (ev.y + rot.y));
    }
    {
        const float2 ev = make_float2(xm.x + xq.x, xm.y - xq.y);   // X_m + conj X_q
        const float2 od = make_float2(xm.x - xq.x, xm.y + xq.y);   // X_m - conj X_q
        const float2 rot = cmul(make_float2(w.y, -w.x), od);       // -i w = (w.y, -w.x)
        zm = make_float2(a.scale * (ev.x + rot.x), a.scale * (ev.y + rot.y));
    }
}
__device__ __forceinline__ void retangle_pair(const LongArgs &a, const float2 *__restrict__ Y, const float2 *wn, int q, int m,
                                              float2 &zq, float2 &zm) {
    const int32_t cvq = __ldg(a.cover + q), cvm = __ldg(a.cover + m);
    GatherLoads gq = gather_issue(a, Y, q, cvq), gm = gather_issue(a, Y, m, cvm);
    retangle_finish(a, Y, wn, q, gq, gm, zq, zm);
}

// ---------------------------------------------------------------- inverse, pass R' (overlap-add + retangle + B-point pass)
// The tile holds TW rows q1 and their mirror rows A - q1 (the same rows as the forward row pass, see row_of), so
// the two packed bins of every pair (q, Lp - q) lie in one tile: the prologue sums each half-spectrum bin once and
// writes both packed bins to shared memory, then the B-point inverse pass runs in place.
template <class SH>
__device__ __forceinline__ void rows_inv_body(const LongArgs &a, const FftPlan &fp, float2 *buf, const float2 *tws,
                                              const float2 *wl, const float2 *wn, int t, int ch, int tid, int nthr) {
    const int A = a.A, B = a.B, TW = a.tw_rows, Lp = a.Lp;
    const bool direct = (A == 1);
    const int ncols = direct ? 1 : 2 * TW;
    const int pitch = SH::is_static ? SH::PITCH : (direct ? 1 : ncols + 1);
    const float2 *Y = a.Y + (long long)ch * a.y_pitch;
    __syncthreads();   // the table of W_N is staged
    if (direct) {
        for (int q = tid; q <= (Lp >> 1); q += nthr) {
            const int m = Lp - q;
            float2 zq, zm;
            retangle_pair(a, Y, wn, q, m, zq, zm);
            buf[q] = zq;
            if (q != 0 && m != q) buf[m] = zm;
        }
    } else {
        // Four pairs per thread and round: all cover words are fetched first, then the plane values of two pairs
        // at a time, so that the dependent loads of one pair overlap those of the others.
        const int log_tw = 31 - __clz(TW);
        constexpr int kPairs = 4;
        for (int base = 0; base < TW * B; base += kPairs * nthr) {
            int q[kPairs], r[kPairs], q2[kPairs];
            int32_t cq[kPairs], cm[kPairs];
            bool ok[kPairs], self[kPairs];
#pragma unroll
            for (int u = 0; u < kPairs; ++u) {
                const int idx = base + u * nthr + tid;
                r[u] = idx & (TW - 1);
                q2[u] = idx >> log_tw;
                const int k1 = TW * t + 1 + r[u];
                self[u] = 2 * k1 == A;           // row A/2 is its own mirror: the pairs (q2, B-1-q2) of one column
                ok[u] = idx < TW * B && !(self[u] && q2[u] >= (B >> 1));
                q[u] = ok[u] ? k1 + A * q2[u] : 1;
                if (!CQT_CHK(a.dbg, 210, Lp - q[u], Lp) || !CQT_CHK(a.dbg, 211, q[u], Lp)) { ok[u] = false; q[u] = 1; }
                cq[u] = __ldg(a.cover + q[u]);
                cm[u] = __ldg(a.cover + (Lp - q[u]));
            }
#pragma unroll
            for (int u = 0; u < kPairs; u += 2) {
                GatherLoads g0q = gather_issue(a, Y, q[u], cq[u]), g0m = gather_issue(a, Y, Lp - q[u], cm[u]);
                GatherLoads g1q = gather_issue(a, Y, q[u + 1], cq[u + 1]), g1m = gather_issue(a, Y, Lp - q[u + 1], cm[u + 1]);
                float2 zq, zm;
                retangle_finish(a, Y, wn, q[u], g0q, g0m, zq, zm);
                if (ok[u]) {
                    buf[q2[u] * pitch + r[u]] = zq;
                    buf[(B - 1 - q2[u]) * pitch + (self[u] ? r[u] : r[u] + TW)] = zm;
                }
                retangle_finish(a, Y, wn, q[u + 1], g1q, g1m, zq, zm);
                if (ok[u + 1]) {
                    buf[q2[u + 1] * pitch + r[u + 1]] = zq;
                    buf[(B - 1 - q2[u + 1]) * pitch + (self[u + 1] ? r[u + 1] : r[u + 1] + TW)] = zm;
                }
            }
        }
        if (2 * TW * (t + 1) == A) {
            // the last tile's spare column holds row 0, which pairs with itself: bins A q2 and A (B - q2)
            const int rz = 2 * TW - 1;
            for (int q2 = tid; q2 <= (B >> 1); q2 += nthr) {
                const int q = A * q2, m = Lp - q;
                float2 zq, zm;
                retangle_pair(a, Y, wn, q, m, zq, zm);
                buf[q2 * pitch + rz] = zq;
                if (q2 != 0 && m != q) buf[(B - q2) * pitch + rz] = zm;
            }
        }
    }
    __syncthreads();
    auto load = [&](int q2, int r) -> float2 { return buf[q2 * pitch + r]; };
    if constexpr (SH::is_static) {
        auto nostore = [](int, int, float2) {};
        tile_fft_static<SH, +1, true, true>(buf, tws, load, nostore, tid, nthr);
    } else {
        const Tile tile{buf, pitch, ncols, a.rows_magic, B * pitch, a.dbg};
        fft_fused_keep<+1, BlockSync, true, true, true>(tile, fp, tws, load, tid, nthr);
    }
    if (direct) {
        float *row = a.x_out + (long long)ch * a.x_stride;
        for (int j = tid; j < B; j += nthr) store_packed(row, j, buf[SH::pos(fp, (uint32_t)j)], a.valid_len, a.aligned);
    } else {
        float2 *T = a.T + (long long)ch * a.t_pitch;
        // The inverse keeps its intermediate transposed, Tinv[j2][q1]: consecutive threads take consecutive columns r, so
        // the shared-memory reads (odd pitch) are conflict-free and the 8-byte stores of a warp fall in runs of TW rows;
        // reading the digit-reversed positions of consecutive j2 instead would hit one bank 16 times.
        for (int e = tid; e < ncols * B; e += nthr) {
            const int j2 = e >> a.log_own, r = e - (j2 << a.log_own);
            const int q1 = row_of(t, r, TW, A);
            const float2 v = buf[SH::pos(fp, (uint32_t)j2) * (uint32_t)pitch + r];
            const float2 w = cconj(twiddle_s(wl, a.log_lp_c, (uint32_t)j2 * (uint32_t)q1));
            if (CQT_CHK(a.dbg, 207, j2 * A + q1, a.Lp)) T[j2 * A + q1] = cmul(v, w);
        }
    }
}

template <class SH>
__global__ void __launch_bounds__(512, 2) irfft_rows_kernel(LongArgs a) {
    pdl_launch_dependents();
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int ch = blockIdx.y, t = blockIdx.x;
    const bool direct = (a.A == 1);
    const int ncols = direct ? 1 : 2 * a.tw_rows;
    const int pitch = direct ? 1 : ncols + 1;
    const FftPlan &fp = a.ffts[a.fft_B];
    float2 *buf = smem_long;
    float2 *tws = buf + (size_t)a.B * pitch;
    float2 *wn = tws + fp.M;
    float2 *wl = wn + a.n_n;
    stage_full(tws, a.tw, fp, tid, nthr);
    stage_table(wn, a.tw + a.tw_n, a.n_n, tid, nthr);
    if (!direct) stage_table(wl, a.tw + a.tw_lp, a.n_lp, tid, nthr);
    pdl_wait();   // the tables above belong to the plan; what follows reads the predecessor's output
    rows_inv_body<SH>(a, fp, buf, tws, wl, wn, t, ch, tid, nthr);
}

// ---------------------------------------------------------------- inverse, pass C' (+ unpack)
template <class SH>
__device__ __forceinline__ void cols_inv_body(const LongArgs &a, const FftPlan &fp, float2 *buf, const float2 *tws,
                                              int j2_0, int ch, int tid, int nthr) {
    const int TW = a.tw_cols;
    const float2 *T = a.T + (long long)ch * a.t_pitch;
    float *row = a.x_out + (long long)ch * a.x_stride;
    // Tinv[j2][q1]: a column of the tile is a contiguous run of A values, so consecutive threads take consecutive q1
    auto load = [&](int q1, int c) -> float2 {
        const int i = (j2_0 + c) * a.A + q1;
        return CQT_CHK(a.dbg, 208, i, a.Lp) ? __ldg(T + i) : make_float2(0.f, 0.f);
    };
    auto store = [&](int j1, int c, float2 v) { store_packed(row, j1 * a.B + j2_0 + c, v, a.valid_len, a.aligned); };
    if constexpr (SH::is_static) {
        tile_fft_static<SH, +1, false, false>(buf, tws, load, store, tid, nthr);
    } else {
        const Tile t{buf, TW | 1, TW, a.cols_magic, a.A * (TW | 1), a.dbg};
        fft_fused<+1, BlockSync, true, false, false, false, true, true>(t, fp, tws, load, store, tid, nthr);
    }
}

template <class SH>
__global__ void __launch_bounds__(512, 2) irfft_cols_kernel(LongArgs a) {
    pdl_launch_dependents();
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int TW = a.tw_cols;
    const int j2_0 = blockIdx.x * TW;
    const int ch = blockIdx.y;
    const FftPlan &fp = a.ffts[a.fft_A];
    float2 *buf = smem_long;
    float2 *tws = buf + (size_t)a.A * (TW | 1);
    stage_full(tws, a.tw, fp, tid, nthr);
    pdl_wait();   // the tables above belong to the plan; what follows reads the predecessor's output
    cols_inv_body<SH>(a, fp, buf, tws, j2_0, ch, tid, nthr);
}

// ---------------------------------------------------------------- host side
static uint32_t magic_of(uint32_t d) { return d <= 1 ? 0u : (uint32_t)(((1ull << 32) + d - 1) / d); }

static LongArgs base_args(const cqt_plan &p, int64_t valid_len, int64_t x_stride, const void *xptr) {
    LongArgs a{};
    a.ffts = p.d.ffts;
    a.tw = p.d.tw;
    a.fft_A = p.lf.fft_A;
    a.fft_B = p.lf.fft_B;
    a.A = (int)p.lf.A;
    a.B = (int)p.lf.B;
    a.Lp = (int)p.lf.Lp;
    a.tw_lp = p.lf.tw_lp;
    a.log_lp_c = p.lf.log_lp_c;
    a.n_lp = p.lf.n_lp;
    a.tw_n = p.lf.tw_n;
    a.log_n_c = p.lf.log_n_c;
    a.n_n = p.lf.n_n;
    a.tw_cols = p.lf.tw_cols;
    a.tw_rows = p.lf.tw_rows;
    a.valid_len = (int)valid_len;
    a.x_stride = x_stride;
    a.aligned = ((reinterpret_cast<uintptr_t>(xptr) & 7) == 0 && (x_stride & 1) == 0) ? 1 : 0;
    a.t_pitch = p.lf.Lp;
    a.x_pitch = p.lf.x_pitch;
    a.y_pitch = p.y_pitch;
    a.y_plane = p.y_plane;
    a.planes = p.y_planes;
    a.cover = p.d.cover;
    a.cols_magic = magic_of(a.tw_cols);
    a.dbg = p.d.dbg;
    a.log_b = 0;
    while ((1ll << a.log_b) < p.lf.B) ++a.log_b;
    a.log_own = 0;
    while ((1 << a.log_own) < 2 * p.lf.tw_rows) ++a.log_own;
    return a;
}

static size_t plan_tw(const cqt_plan &p, int fft) { return (size_t)p.ffts[fft].M; }

static size_t rows_fwd_smem(const cqt_plan &p) {
    const LongFft &lf = p.lf;
    const size_t data = lf.A == 1 ? (size_t)lf.B : (size_t)lf.B * (2 * lf.tw_rows + 1);
    return (data + plan_tw(p, lf.fft_B) + lf.n_n) * 8;
}
static size_t rows_inv_smem(const cqt_plan &p) {
    const LongFft &lf = p.lf;
    const size_t data = lf.A == 1 ? (size_t)lf.B : (size_t)lf.B * (2 * lf.tw_rows + 1);
    return (data + plan_tw(p, lf.fft_B) + lf.n_n + (lf.A == 1 ? 0 : lf.n_lp)) * 8;
}
static size_t cols_smem(const cqt_plan &p) {
    const LongFft &lf = p.lf;
    return ((size_t)lf.A * (lf.tw_cols | 1) + plan_tw(p, lf.fft_A) + lf.n_lp) * 8;   // odd pitch in the inverse pass
}


// first shape of the list that matches the plan, else the run-time planned instantiation
template <template <class> class K, class... SHs>
struct PickKernel;
template <template <class> class K>
struct PickKernel<K> {
    static const void *get(const FftPlan &, int) { return (const void *)K<DynShape>::fn; }
};
template <template <class> class K, class SH, class... Rest>
struct PickKernel<K, SH, Rest...> {
    static const void *get(const FftPlan &fp, int ncols) {
        return SH::matches(fp, ncols) ? (const void *)K<SH>::fn : PickKernel<K, Rest...>::get(fp, ncols);
    }
};
template <class SH> struct ColsFwdK { static constexpr auto fn = rfft_cols_fwd_kernel<SH, false>; };
template <class SH> struct ColsFwdSlicedK { static constexpr auto fn = rfft_cols_fwd_kernel<SH, true>; };
template <class SH> struct RowsFwdK { static constexpr auto fn = rfft_rows_fwd_kernel<SH>; };
template <class SH> struct RowsInvK { static constexpr auto fn = irfft_rows_kernel<SH>; };
template <class SH> struct ColsInvK { static constexpr auto fn = irfft_cols_kernel<SH>; };

static const void *cols_fwd_fn(const cqt_plan &p) {
    return PickKernel<ColsFwdK, Sh_8_8_8_16_16, Sh_16_16_1_16_16, Sh_16_8_1_16_16, Sh_16_8_8_8_8, Sh_16_16_8_8_8>::get(
        p.ffts[p.lf.fft_A], p.lf.tw_cols);
}
// the slice lengths in use give 16 x 8 or 16 x 16 or 8 x 8 x 8 tiles; other plans take the run-time planned instantiation
static const void *cols_fwd_sliced_fn(const cqt_plan &p) {
    return PickKernel<ColsFwdSlicedK, Sh_8_8_8_16_16, Sh_16_16_1_16_16, Sh_16_8_1_16_16>::get(p.ffts[p.lf.fft_A], p.lf.tw_cols);
}
static const void *rows_fwd_fn(const cqt_plan &p) {
    const int ncols = p.lf.A == 1 ? 1 : 2 * p.lf.tw_rows;
    return PickKernel<RowsFwdK, Sh_8_8_8_16_17, Sh_16_16_1_16_17, Sh_16_8_1_16_17, Sh_16_8_8_8_9>::get(p.ffts[p.lf.fft_B], ncols);
}
static const void *rows_inv_fn(const cqt_plan &p) {
    const int ncols = p.lf.A == 1 ? 1 : 2 * p.lf.tw_rows;
    return PickKernel<RowsInvK, Sh_8_8_8_16_17, Sh_16_16_1_16_17, Sh_16_8_1_16_17, Sh_16_8_8_8_9>::get(p.ffts[p.lf.fft_B], ncols);
}
static const void *cols_inv_fn(const cqt_plan &p) {
    return PickKernel<ColsInvK, Sh_8_8_8_16_17, Sh_16_16_1_16_17, Sh_16_8_1_16_17, Sh_16_8_8_8_9, Sh_16_16_8_8_9>::get(
        p.ffts[p.lf.fft_A], p.lf.tw_cols);
}
static cudaError_t launch_long(const void *fn, dim3 grid, int threads, size_t smem, LongArgs &a, cudaStream_t st) {
    void *args[] = {&a};
    return launch_kernel(fn, grid, dim3((unsigned)threads), args, smem, st);
}

// one thread per butterfly of the stage with the most butterflies (the smallest radix of the plan), up to 512
static int threads_for(size_t elements, const FftPlan &fp) {
    int rmin = 16;
    for (int j = 0; j < fp.nstages; ++j) rmin = std::min(rmin, (int)fp.st[j].radix);
    const size_t butterflies = elements / (size_t)std::max(rmin, 2);
    int t = 64;
    while (t < 512 && (size_t)t < butterflies) t *= 2;
    return t;
}

cudaError_t launch_rfft_forward(const cqt_plan &p, const float *x, int64_t x_stride, int64_t batch, int64_t valid_len,
                                float2 *T, float2 *X, cudaStream_t st, const SliceSource *src) {
    LongArgs a = base_args(p, valid_len, x_stride, x);
    a.x_in = x;
    a.T = T;
    a.X = X;
    const LongFft &lf = p.lf;
    if (src) {
        if (lf.A == 1 || src->channels <= 0 || src->ring_len < p.N) return cudaErrorInvalidValue;
        a.ring = src->ring; a.slice_win = src->win;
        a.ring_len = src->ring_len; a.slice_first = src->first; a.hop = src->hop; a.channels = src->channels;
    }
    if (lf.A > 1) {
        dim3 grid((unsigned)(lf.B / lf.tw_cols), (unsigned)batch);
        launch_long(src ? cols_fwd_sliced_fn(p) : cols_fwd_fn(p), grid, threads_for((size_t)lf.A * lf.tw_cols, p.ffts[lf.fft_A]), cols_smem(p), a, st);
        note_launch(p, "rfft_cols_fwd", st);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        a.rows_magic = magic_of(2 * lf.tw_rows);
        dim3 grid2((unsigned)(lf.A / (2 * lf.tw_rows)), (unsigned)batch);
        launch_long(rows_fwd_fn(p), grid2, threads_for((size_t)lf.B * (2 * lf.tw_rows), p.ffts[lf.fft_B]), rows_fwd_smem(p), a, st);
    } else {
        a.rows_magic = 0;
        dim3 grid2(1, (unsigned)batch);
        launch_long(rows_fwd_fn(p), grid2, threads_for((size_t)lf.B, p.ffts[lf.fft_B]), rows_fwd_smem(p), a, st);
    }
    note_launch(p, "rfft_rows_fwd", st);
    return cudaGetLastError();
}

cudaError_t launch_rfft_inverse(const cqt_plan &p, const float2 *Y, float2 *T, float *x, int64_t x_stride,
                                int64_t batch, int64_t valid_len, cudaStream_t st) {
    LongArgs a = base_args(p, valid_len, x_stride, x);
    a.x_out = x;
    a.T = T;
    a.Y = Y;
    a.scale = (float)(0.5 / (double)p.lf.Lp);
    const LongFft &lf = p.lf;
    if (lf.A > 1) {
        a.rows_magic = magic_of(2 * lf.tw_rows);
        dim3 grid((unsigned)(lf.A / (2 * lf.tw_rows)), (unsigned)batch);
        // the overlap-add prologue is a latency chain per thread: with fewer CTAs than SMs it takes every thread it can get
        const bool few = (long long)grid.x * grid.y < (long long)p.sm_count;
        const int thr = few ? 512 : threads_for((size_t)lf.B * (2 * lf.tw_rows), p.ffts[lf.fft_B]);
        launch_long(rows_inv_fn(p), grid, thr, rows_inv_smem(p), a, st);
        note_launch(p, "irfft_rows", st);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        dim3 grid2((unsigned)(lf.B / lf.tw_cols), (unsigned)batch);
        launch_long(cols_inv_fn(p), grid2, threads_for((size_t)lf.A * lf.tw_cols, p.ffts[lf.fft_A]), cols_smem(p), a, st);
        note_launch(p, "irfft_cols", st);
    } else {
        a.rows_magic = 0;
        dim3 grid(1, (unsigned)batch);
        launch_long(rows_inv_fn(p), grid, threads_for((size_t)lf.B, p.ffts[lf.fft_B]), rows_inv_smem(p), a, st);
        note_launch(p, "irfft_rows", st);
    }
    return cudaGetLastError();
}

cudaError_t configure_long_fft_kernels(const cqt_plan &p) {
    cudaError_t e;
    e = allow_dynamic_smem(rows_fwd_fn(p), rows_fwd_smem(p), p);
    if (e != cudaSuccess) return e;
    e = allow_dynamic_smem(rows_inv_fn(p), rows_inv_smem(p), p);
    if (e != cudaSuccess) return e;
    if (p.lf.A > 1) {
        e = allow_dynamic_smem(cols_fwd_fn(p), cols_smem(p), p);
        if (e != cudaSuccess) return e;
        e = allow_dynamic_smem(cols_fwd_sliced_fn(p), cols_smem(p), p);
        if (e != cudaSuccess) return e;
        e = allow_dynamic_smem(cols_inv_fn(p), cols_smem(p), p);
    }
    return e;
}

}  // namespace cqt
