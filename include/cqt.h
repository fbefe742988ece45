/*
 * cqt.h - C ABI of the B200 (sm_100a) invertible constant-Q transform library.
 *
 * The library computes the nonstationary-Gabor constant-Q transform of real
 * signals, its exact inverse, the real adjoints of both, and the sliced
 * streaming form, with hand-written CUDA kernels.  Citations name the passage
 * of the paper "Exact Factorisation and Fast Computation of Invertible
 * Constant-Q Transforms" that defines each operation.
 *
 * Conventions
 *   N         real signal length of a plan (the argument L of cqt_plan_create;
 *             a power of two, 64 <= N <= 2^22).  The paper's packed length L is N/2.
 *   batch     number of independent signals (batch x channels, flattened).
 *   x rows    fp32, row r at x + r * x_stride (elements), valid_len <= N samples per
 *             row; samples valid_len..N-1 are implicit zeros and are never read
 *             (analysis) or written (synthesis).
 *   c         complex64, interleaved (re, im); [batch][coeff_count]; band b of signal r
 *             at c + r * coeff_count + band_info(b).coeff_offset, M_b entries in time
 *             order.  Bands are ordered DC sideband, regular bands low to high,
 *             Nyquist sideband.
 *   pointers  x, c and ws are DEVICE pointers owned by the caller unless a comment
 *             says "host".  Plans own their host and device tables.
 *   ws        scratch of at least cqt_plan_workspace_bytes(plan, batch) bytes,
 *             256-byte aligned; contents are undefined after a call.  Calls that run
 *             concurrently on different streams need different workspaces.
 *   stream    a cudaStream_t passed as void*; all transform calls are asynchronous
 *             on it and never synchronise the device.  A plan owns five helper streams
 *             that fork from and join the caller's stream inside every call (the calls
 *             can be captured in a CUDA graph).
 *   threads   calls on ONE plan (or one cqt_slicq) must come from one host thread at a
 *             time: its helper streams, events and launch counters are shared state.
 *             Different plans may be used from different threads, and one thread may
 *             issue calls on one plan to several streams (with distinct workspaces).
 *   errors    every function returns a cqt_status; argument errors are detected on
 *             the host before any launch; nothing throws, aborts or traps.
 *             There is no CPU fallback: without a usable CUDA device the transform
 *             calls fail with CQT_ERR_CUDA or CQT_ERR_STATE.
 */
#ifndef CQT_B200_H
#define CQT_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CQT_OK = 0,
    CQT_ERR_INVALID_ARG = -1,  /* null pointer, negative size, valid_len > N, stride < valid_len ... */
    CQT_ERR_UNSUPPORTED = -2,  /* N not a power of two in range, a band too long for the kernels */
    CQT_ERR_BAD_LAYOUT = -3,   /* windows do not cover every bin, first centre below bin 2, support > M */
    CQT_ERR_WORKSPACE = -4,    /* ws null, misaligned or smaller than cqt_plan_workspace_bytes */
    CQT_ERR_CUDA = -5,         /* a CUDA runtime call or launch failed */
    CQT_ERR_STATE = -6,        /* host-only plan used for a transform; slicq call out of order */
    CQT_ERR_DEVICE_CHECK = -7  /* reserved: a device-side self check reported a violation */
} cqt_status;

typedef struct { float re, im; } cqt_c64; /* layout-compatible with torch.complex64 */

typedef enum { CQT_WIN_HANN = 0, CQT_WIN_BLACKMAN_HARRIS = 1 } cqt_window;

/* how the coefficient count M of a band follows from its support S (number of nonzero window bins) */
typedef enum {
    CQT_M_MULT4 = 0,  /* 4 * ceil(S / 4); a band beyond 12,800 coefficients takes the CQT_M_SMOOTH length */
    CQT_M_SMOOTH = 1, /* smallest multiple of 4 of the form 2^a 3^b 5^c that is >= S */
    CQT_M_POW2 = 2    /* smallest power of two >= max(S, 4) */
} cqt_m_policy;

typedef struct {
    double fs;            /* sample rate, Hz */
    double fmin;          /* lowest band centre, Hz */
    double fmax;          /* no centre above this, Hz (<= fs/2) */
    int bins_per_octave;  /* b; Q = 1 / (2^(1/b) - 2^(-1/b)) */
    int64_t L;            /* N, real samples per transform */
    int window;           /* cqt_window */
    int m_policy;         /* cqt_m_policy */
    double min_win;       /* minimum support width in bins (default 4); lowers Q of the lowest bands */
    int device;           /* CUDA device ordinal; -1 builds a host-only plan (queries and tables only) */
} cqt_plan_desc;

/*
 * A plan from an explicit list of regular bands, low to high (any painless non-stationary Gabor layout, Sec. 2;
 * the multi-resolution layout of Sec. 4 is one, see cqt_multires_bands).  Band i has centre centre_hz[i],
 * rounded to the bin floor(f L/fs + 1/2), and a window of total width width_bins[i] bins (real valued, >= 2)
 * sampled symmetrically about that bin at the integer offsets |d| < W/2.  M_i follows m_policy from the
 * support size; bands with the same group[i] >= 0 share the largest M of their group ("one coefficient length
 * per octave", Sec. 4); group == NULL or group[i] < 0: the band's own length.  The DC and Nyquist sidebands are
 * added as in cqt_plan_create.  The arrays are host memory, read during the call only.
 */
typedef struct {
    double fs;                /* sample rate, Hz */
    int64_t L;                /* N, real samples per transform */
    int window;               /* cqt_window */
    int m_policy;             /* cqt_m_policy */
    int device;               /* CUDA device ordinal; -1 builds a host-only plan */
    int64_t n_bands;          /* regular bands (>= 1) */
    const double *centre_hz;  /* [n_bands], centre bins must not descend */
    const double *width_bins; /* [n_bands] */
    const int32_t *group;     /* [n_bands] or NULL */
} cqt_band_list_desc;

typedef struct {
    double centre_hz;
    int64_t centre_bin;   /* k_lambda */
    int64_t support;      /* S_lambda, bins kc + first_offset ... kc + first_offset + S - 1 */
    int64_t first_offset; /* most negative support offset d */
    int64_t M;            /* coefficients */
    int64_t coeff_offset; /* into one signal's coefficient row */
    int64_t table_offset; /* into the g / h tables returned by cqt_plan_tables */
    int is_sideband;      /* 0 regular, 1 DC, 2 Nyquist */
    int launch_class;     /* which of the band kernels' length classes (0 = shortest) runs this band; -1: two-pass kernels */
} cqt_band_info;

typedef struct cqt_plan cqt_plan;
typedef struct cqt_slicq cqt_slicq;

/*
 * Plan construction (host work, then one upload of the tables).
 * Builds the band layout of Sec. 2 / Sec. 4: geometric centres fmin * 2^(j/b) rounded to
 * Fourier bins, real spectral windows g_lambda whose total width is f/Q bins of the N-point
 * spectrum, per-band lengths M_lambda >= support (painless case), DC and Nyquist sidebands
 * that complete the cover, the aggregate weight a_k = sum M g^2 and the dual windows
 * h = M g / a_k (Sec. 2).  Also factors every M_lambda into butterfly radices and groups
 * bands into launch classes.
 * cqt_plan_create uses CQT_M_MULT4, min_win = 4 and the current device.
 * Errors: INVALID_ARG, UNSUPPORTED, BAD_LAYOUT, CUDA.  *out is set only on CQT_OK.
 */
cqt_status cqt_plan_create(double fs, double fmin, double fmax, int bins_per_octave, int64_t L,
                           cqt_window window, cqt_plan **out);
cqt_status cqt_plan_create_ex(const cqt_plan_desc *desc, cqt_plan **out);
/*
 * The same with the few choices of the plan builder that are not part of the transform's definition: every
 * setting computes the same coefficients up to fp32 rounding, only the kernels that run differ.  A zero field
 * (or tuning == NULL) means the default.  Used by the tests to reach every kernel family on small inputs and
 * by the benchmark to compare them.
 */
typedef struct {
    int64_t max_cta_elems; /* complex elements of shared memory one CTA may use for a band (>= 64): bands needing more
                              take the two-pass kernels, which by default only bands beyond 227 KB do */
    int64_t two_pass_min;  /* bands with more coefficients than this take the two-pass kernels */
} cqt_plan_tuning;
cqt_status cqt_plan_create_tuned(const cqt_plan_desc *desc, const cqt_plan_tuning *tuning, cqt_plan **out);
/* Errors as above. */
cqt_status cqt_plan_create_bands(const cqt_band_list_desc *desc, cqt_plan **out);
/*
 * Band list of the multi-resolution layout (Sec. 4, first paragraph): n_sections consecutive sections of
 * octaves[s] octaves at bins_per_octave[s] bands per octave.  Section s starts at fmin * 2^(octaves before it) and
 * holds centres f_start * 2^(j/b), each with the width (f/Q_b) L/fs bins (at least min_win; <= 0 means 4) of its own
 * resolution; group[i] is the octave index counted from fmin.  Host arrays of `capacity` entries (any may be
 * NULL); *n_bands receives the number of bands whether or not they fit.  Pure host arithmetic.
 */
cqt_status cqt_multires_bands(double fs, double fmin, int64_t L, const int *octaves, const int *bins_per_octave,
                              int n_sections, double min_win, int64_t capacity, double *centre_hz, double *width_bins,
                              int32_t *group, int64_t *n_bands);
cqt_status cqt_plan_destroy(cqt_plan *plan);

/* Host-side queries; no device access. */
int64_t cqt_plan_num_bands(const cqt_plan *plan);
int64_t cqt_plan_coeff_count(const cqt_plan *plan);   /* sum of M_lambda: complex values per signal */
int64_t cqt_plan_signal_length(const cqt_plan *plan); /* N */
int64_t cqt_plan_table_length(const cqt_plan *plan);  /* sum of S_lambda: entries of the g / h tables */
int cqt_plan_device(const cqt_plan *plan);            /* CUDA device ordinal of the plan, -1 if host-only */
cqt_status cqt_plan_band_info(const cqt_plan *plan, int64_t band, cqt_band_info *out);
size_t cqt_plan_workspace_bytes(const cqt_plan *plan, int64_t batch);
/* Host copies of the fp32 window tables g and h (length cqt_plan_table_length), owned by the plan. */
cqt_status cqt_plan_tables(const cqt_plan *plan, const float **g_host, const float **h_host);
/* Reserved for device-side self checks; returns CQT_OK in release builds. May synchronise. */
cqt_status cqt_plan_check(const cqt_plan *plan);

/*
 * Benchmark aids (the paper has no counterpart).  cqt_plan_launch_count: kernels launched through this
 * plan since it was created.  cqt_plan_set_timing(plan, 1): every later transform call records a CUDA
 * event on its stream before its first kernel and after each kernel; cqt_plan_read_timing waits for those
 * events, returns for each kernel launched since the last read its name (static strings) and its
 * duration in milliseconds (at most `capacity` entries are written; *count receives the total), and clears
 * the record.  Not thread safe; leave timing off in production calls.
 */
int64_t cqt_plan_launch_count(const cqt_plan *plan);
cqt_status cqt_plan_set_timing(const cqt_plan *plan, int enable);
cqt_status cqt_plan_read_timing(const cqt_plan *plan, const char **names, float *ms, int64_t capacity, int64_t *count);

/*
 * Analysis T (Eq. analysis, band-spectrum, packed-analysis):
 *   c_lambda = F_M^{-1} E_lambda diag(g_lambda) F_N x   for every band, every row.
 * Computed as one packed real FFT of length N/2 (Eq. pack) whose last pass applies the
 * conjugate-symmetric fold (Eq. untangle), then one fused kernel per band that gathers the
 * band's bins, multiplies by g, places bin kc + d in slot d mod M and runs the M-point
 * inverse DFT (including 1/M) in shared memory.
 */
cqt_status cqt_analyse(const cqt_plan *plan, const float *x, int64_t x_stride, int64_t batch,
                       int64_t valid_len, cqt_c64 *c, void *ws, size_t ws_bytes, void *stream);

/*
 * Analysis without any allocation by anyone (the paper has no counterpart; this is a deployment aid).
 * For callers that must not call cudaMalloc: processes running inside a device-memory budget that
 * was fixed when they started (audio engines with a real-time thread, plug-in hosts, sandboxes),
 * or code that runs where the allocator is off limits.  Same result as cqt_analyse, but the scratch
 * comes from a fixed array of CQT_STATIC_WS_BYTES (16 MiB) inside the library image instead of a
 * caller buffer; every GPU that loads the library holds that array until the process exits.
 *   - batch is limited by cqt_plan_workspace_bytes(plan, batch) <= cqt_static_workspace_bytes();
 *     larger requests return CQT_ERR_WORKSPACE and launch nothing.
 *   - The first call on each device looks up the array's device address (once per device, with that
 *     device current); make that first call before any stream capture begins.
 *   - All calls share the one array and it keeps whatever the last call left in it; every call
 *     overwrites what it reads, nothing needs clearing.  Two calls that overlap on the GPU (different
 *     streams, or different plans) race on it: serialise them.
 *   - Calls no cudaMalloc / cudaFree and no allocating library routine, provided event timing
 *     (cqt_plan_set_timing) is off for the plan.
 */
#define CQT_STATIC_WS_BYTES (16u << 20)
size_t cqt_static_workspace_bytes(void);
cqt_status cqt_analyse_static_ws(const cqt_plan *plan, const float *x, int64_t x_stride, int64_t batch,
                                 int64_t valid_len, cqt_c64 *c, void *stream);

/*
 * Synthesis S (Eq. synthesis, packed-synthesis):
 *   x^ = F_N^{-1} sum_lambda diag(h_lambda) E_lambda^T F_M c_lambda, imaginary parts at DC and
 *   Nyquist dropped, negative frequencies by conjugate symmetry.  S T = I on real signals.
 * Per band: M-point DFT in shared memory, dual-window multiply, weighted bins written in bin
 * order to scratch; the first pass of the packed inverse FFT sums, per bin and in fixed band
 * order (no atomics, bitwise reproducible), the bands that cover it and applies Eq. retangle.
 */
cqt_status cqt_synthesise(const cqt_plan *plan, const cqt_c64 *c, int64_t batch, int64_t valid_len,
                          float *x, int64_t x_stride, void *ws, size_t ws_bytes, void *stream);

/*
 * Real adjoints under <u, v> = Re(u^H v) (Sec. "Adjoints for training", Eq. analysis-adjoint,
 * synthesis-adjoint).  cqt_analyse_adjoint maps a coefficient cotangent to a signal cotangent
 * (x_bar = T^dagger c_bar, the backward of cqt_analyse); cqt_synthesise_adjoint maps a signal
 * cotangent to a coefficient cotangent (c_bar = S^dagger x_bar, the backward of
 * cqt_synthesise).  T^dagger has the form of synthesis with g / M in place of h and both
 * signs of each sideband bin folded; S^dagger has the form of analysis with M h w_k / N in
 * place of g (w_k = 2, but 1 at DC and Nyquist).  Nothing from the forward pass is needed.
 */
cqt_status cqt_analyse_adjoint(const cqt_plan *plan, const cqt_c64 *c_bar, int64_t batch, int64_t valid_len,
                               float *x_bar, int64_t x_stride, void *ws, size_t ws_bytes, void *stream);
cqt_status cqt_synthesise_adjoint(const cqt_plan *plan, const float *x_bar, int64_t x_stride, int64_t batch,
                                  int64_t valid_len, cqt_c64 *c_bar, void *ws, size_t ws_bytes, void *stream);

/*
 * Sliced streaming form (Sec. 4, slicing paragraph): slices of sl = N samples of slice_plan,
 * hop sl/2, multiplied by a Tukey window whose raised-cosine flanks are `transition` samples
 * long (0 < transition <= sl/2) so that shifted windows sum to one; every slice is analysed
 * and synthesised on its own and the reconstructions are overlap-added.  Slice s covers stream
 * samples [s sl/2 - sl/2, s sl/2 + sl/2) with zeros before the start of the stream.
 *
 * The object owns all its device memory (input ring, per-slice coefficient slots, output
 * accumulator, transform workspace), bounded by max_slices_in_flight and independent of the
 * stream's duration; slicq_device_bytes reports it.
 *
 *   slicq_push   appends n frames per channel (x: device, [channels][n], row stride x_stride) and
 *                analyses every slice they complete; *slices_completed (host, may be null) receives
 *                the number of slices analysed so far.  At most max_slices_in_flight analysed
 *                slices may await slicq_pull; pushing more returns CQT_ERR_STATE and consumes nothing.
 *   slicq_coeffs device pointer to slice `slice_index`'s coefficients [channels][coeff_count],
 *                valid (and editable in place) until the slice is pulled.
 *   slicq_pull   synthesises every analysed slice not yet pulled, overlap-adds (older slice
 *                first) and writes up to n_max finished frames per channel to y (device,
 *                [channels][n_max], row stride y_stride); *n_written (host) receives the count.  Frame n
 *                is finished once slice floor(n / (sl/2)) + 1 has been synthesised: one slice of latency.
 *   slicq_flush  pushes zeros (between sl/2 and sl per channel) up to the next multiple of sl/2 plus sl/2, so
 *                that every frame pushed so far becomes final and can be pulled.
 *   Push, pull and flush of one object must be issued on the same stream (they share staging buffers).
 *   slicq_reset  drops all state and restarts at slice 0; waits for the stream of the object's latest push, pull or
 *                flush (no other stream of the device is synchronised).
 *   Every slicq call runs on the plan's device and restores the caller's current device.
 */
cqt_status slicq_create(const cqt_plan *slice_plan, int channels, int64_t transition,
                        int64_t max_slices_in_flight, cqt_slicq **out);
cqt_status slicq_push(cqt_slicq *s, const float *x, int64_t x_stride, int64_t n, void *stream,
                      int64_t *slices_completed);
cqt_status slicq_coeffs(cqt_slicq *s, int64_t slice_index, cqt_c64 **c);
cqt_status slicq_pull(cqt_slicq *s, float *y, int64_t y_stride, int64_t n_max, void *stream, int64_t *n_written);
cqt_status slicq_flush(cqt_slicq *s, void *stream);
cqt_status slicq_reset(cqt_slicq *s);
cqt_status slicq_destroy(cqt_slicq *s);
size_t slicq_device_bytes(const cqt_slicq *s);

/*
 * Extras of the sliced form (the paper gives the slicing only; these make it usable for spectral processing).
 *
 * Processing between analysis and synthesis: the coefficients of an analysed slice (slicq_coeffs) may be edited
 * in place, by kernels on the object's stream, until slicq_pull synthesises them.
 *
 * slicq_assemble lays the coefficients of n_slices consecutive analysed, not yet pulled slices
 * first_slice .. first_slice + n_slices - 1 on one time axis per band: slice i + 1 starts sl/2 samples, i.e.
 * M/2 coefficient periods of a band with M coefficients, after slice i, so band lambda's series has
 * (n_slices + 1) M/2 entries, series[i M/2 + m] = sum over slices of c_i[m] (at most two terms, older slice
 * first).  out (device): [channels][out_stride] complex64, band lambda's series starting at
 * (n_slices + 1) * coeff_offset_lambda / 2; slicq_assembled_length = (n_slices + 1) * coeff_count / 2 entries per
 * channel.  Entry t of a band's series belongs to stream time (first_slice - 1) sl/2 + t sl/M samples.  Sliced
 * coefficients are not the coefficients of the whole signal (Sec. 4).  Errors: INVALID_ARG, STATE (a slice of the
 * range is not held), CUDA.
 *
 * slicq_save_state / slicq_load_state copy the stream state (counters, input ring, overlap-add accumulator) to /
 * from a host buffer of slicq_state_bytes, so that a stream can be suspended and resumed, also by another object
 * created with the same plan shape, channels, transition and slices in flight (else CQT_ERR_STATE).  Saving needs
 * every analysed slice to have been pulled (else CQT_ERR_STATE).  Both synchronise `stream`.
 */
int64_t slicq_assembled_length(const cqt_slicq *s, int64_t n_slices);
cqt_status slicq_assemble(cqt_slicq *s, int64_t first_slice, int64_t n_slices, cqt_c64 *out, int64_t out_stride,
                          void *stream);
size_t slicq_state_bytes(const cqt_slicq *s);
cqt_status slicq_save_state(cqt_slicq *s, void *host_buf, size_t bytes, void *stream);
cqt_status slicq_load_state(cqt_slicq *s, const void *host_buf, size_t bytes, void *stream);

const char *cqt_status_string(cqt_status status);

#ifdef __cplusplus
}
#endif
#endif /* CQT_B200_H */
