// Internal interfaces between the plan builder, the kernel launchers and the C ABI.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>
#include <string>
#include <vector>

#include "layout.hpp"
#include "plan_types.h"

namespace cqt {

constexpr int kNumClasses = 5;
// Launch shape of one band-length class.
struct BandClass {
    int threads = 0;         // threads per CTA
    int min_blocks = 1;      // CTAs per SM the kernel instantiation is compiled for (register budget)
    int lanes_few = 0, lanes_many = 0;   // > 0: several (band, signal) items per CTA, that many lanes each, in a call
                                         // with few / many items; 0: one item per CTA
    int max_radix = 16;      // largest butterfly radix in the class's plans
    bool has_generic = false; // some band of the class has a prime factor above 5 (direct-sum stage or chirp-z)
    int max_elems = 0;       // shared-memory elements (float2) per item
    int n_bands = 0;         // bands in the class
    double stage_work = 0.0; // element-stages of the class's transforms per signal (stream assignment)
    double latency_us = 0.0; // estimated run time of the class's longest work item alone
    BandItem *d_items = nullptr;   // records + radix plans of the class's bands, longest first
    std::vector<int32_t> work;
};

struct LongFft {
    int64_t Lp = 0, A = 1, B = 0;
    int fft_A = -1, fft_B = -1;   // FftPlan indices
    int tw_lp = 0, tw_n = 0;      // two-level tables of W_Lp and W_N inside the twiddle array
    int log_lp_c = 0, log_n_c = 0;
    int n_lp = 0, n_n = 0;        // entry counts of those tables
    int tw_rows = 1;              // rows per mirrored half handled by one CTA of the row kernels (forward and inverse)
    int tw_cols = 1;              // columns per CTA of the column kernels
    int64_t x_pitch = 0;          // elements per signal of the half-spectrum buffer (Lp + 1 rounded up)
};

using TwoPassBand = TwoPassRec;

struct TwoPassGroup {
    std::vector<TwoPassBand> bands;
    TwoPassRec *d_recs = nullptr;
    // per tile width (kTwoPassWidths): CTAs along the tiled index and shared memory of the two passes
    int max_tiles_cols[3] = {0, 0, 0}, max_tiles_rows[3] = {0, 0, 0};
    size_t smem_cols[3] = {0, 0, 0}, smem_rows[3] = {0, 0, 0};
};

struct DevicePlan {
    BandRec *bands = nullptr;
    FftPlan *ffts = nullptr;
    float2 *tw = nullptr;
    float *tab_analysis = nullptr;     // g / M
    float *tab_synthesis = nullptr;    // h
    float *tab_analysis_adj = nullptr; // N g / (2 M)
    float *tab_synthesis_adj = nullptr;// h w_k / N
    int32_t *cover = nullptr;          // per bin: (plane of the first covering band << 8) | number of covering bands
    int *dbg = nullptr;                // 8 status words of the debug-bounds build
    int2 *zero_seg = nullptr;          // (offset into one signal's weighted-bin scratch, length): bins synthesis zero-fills
};

}  // namespace cqt

struct cqt_plan {
    cqt::HostLayout lay;
    std::vector<float> g32, h32;
    std::vector<cqt::FftPlan> ffts;
    std::vector<cqt::BandRec> bands;
    int device = -1;
    int64_t N = 0;
    int64_t y_pitch = 0;               // weighted-bin scratch elements per signal (y_planes * y_plane)
    int64_t y_plane = 0;               // elements per plane (N/2 + 1 rounded up)
    int y_planes = 1;                  // largest number of bands covering one bin
    int n_zero_seg = 0;                // zero-fill segments (layouts with nested supports only)
    cqt::LongFft lf;
    cqt::BandClass cls[cqt::kNumClasses];
    cqt::TwoPassGroup two_pass[2];     // [0]: both factors <= 256, [1]: larger factors
    int64_t two_pass_pitch = 0;        // scratch elements per signal for the two-pass bands
    cqt::DevicePlan d;
    int max_smem_optin = 0;
    int sm_count = 0;
    // helper streams on which the short-band classes run beside the long-band classes of the same call
    static constexpr int kHelpers = 5;   // one per band class beside the caller's stream, one for the two-pass bands
    cudaStream_t aux[kHelpers] = {};
    cudaEvent_t ev_fork = nullptr, ev_join[kHelpers] = {};
    // launch counter and optional per-kernel event timing (benchmark aid; not thread safe)
    mutable int64_t launches = 0;
    mutable bool timing = false;
    mutable std::vector<cudaEvent_t> ev;
    mutable std::vector<const char *> ev_name;
    mutable size_t ev_used = 0;
};

namespace cqt {

// table selectors of the band kernels
enum { TAB_ANALYSIS = 0, TAB_SYNTHESIS = 1, TAB_ANALYSIS_ADJ = 2, TAB_SYNTHESIS_ADJ = 3 };

// api.cu: called after every kernel launch (and once at the start of a call with name == nullptr)
void note_launch(const cqt_plan &p, const char *name, cudaStream_t st);

// long_fft.cu
// Input of the forward long FFT taken from a ring buffer of a stream instead of signal rows (sliced transform, slice
// cut fused into the load): row r = slice r / channels of channel r % channels; sample i of that slice is
// win[i] * ring[channel * ring_len + (first + (r / channels) * hop + i) mod ring_len], zero before the stream's start.
struct SliceSource {
    const float *ring;
    const float *win;
    long long ring_len, first, hop;
    int channels;
};
// src != nullptr needs a plan whose long FFT runs in two passes (can_fuse_slice_cut)
cudaError_t launch_rfft_forward(const cqt_plan &p, const float *x, int64_t x_stride, int64_t batch, int64_t valid_len,
                                float2 *T, float2 *X, cudaStream_t st, const SliceSource *src = nullptr);
inline bool can_fuse_slice_cut(const cqt_plan &p) { return p.lf.A > 1; }
cudaError_t launch_rfft_inverse(const cqt_plan &p, const float2 *Y, float2 *T, float *x, int64_t x_stride,
                                int64_t batch, int64_t valid_len, cudaStream_t st);
// The dynamic shared-memory limit is a property of the kernel function, shared by every plan of the process: it is
// raised to the device maximum, not to one plan's need (a later plan needing less would otherwise lower it under an
// earlier plan, whose launches would then fail).
inline cudaError_t allow_dynamic_smem(const void *fn, size_t need, const cqt_plan &p) {
    cudaFuncAttributes fa;
    cudaError_t e = cudaFuncGetAttributes(&fa, fn);
    if (e != cudaSuccess) return e;
    const long long most = (long long)p.max_smem_optin - (long long)fa.sharedSizeBytes;   // static + dynamic share the limit
    if ((long long)need > most) return cudaErrorInvalidValue;
    return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most);
}

cudaError_t configure_long_fft_kernels(const cqt_plan &p);

// Launch with the programmatic-serialization attribute (see pdl_wait in engine.cuh).
inline cudaError_t launch_kernel(const void *fn, dim3 grid, dim3 block, void **args, size_t smem, cudaStream_t st) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelExC(&cfg, fn, args);
}

// The same for a kernel called with its arguments (replaces kernel<<<grid, block, smem, st>>>(args...)).
template <class... KArgs, class... Args>
inline cudaError_t launch_kernel_args(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// band.cu
// every band of the plan: the single-CTA classes and, beside them on a stream of their own, the two-pass bands
// (scratch: their rows in the workspace)
cudaError_t launch_bands_from_spectrum(const cqt_plan &p, const float *table, const float2 *X, float2 *c,
                                       float2 *scratch, int64_t batch, cudaStream_t st);
cudaError_t launch_bands_to_spectrum(const cqt_plan &p, const float *table, bool fold_sidebands, const float2 *c,
                                     float2 *Y, float2 *scratch, int64_t batch, cudaStream_t st);
cudaError_t configure_band_kernels(const cqt_plan &p);

// band_two_pass.cu
cudaError_t launch_two_pass_from_spectrum(const cqt_plan &p, const float *table, const float2 *X, float2 *c,
                                          float2 *scratch, int64_t batch, cudaStream_t st);
cudaError_t launch_two_pass_to_spectrum(const cqt_plan &p, const float *table, bool fold, const float2 *c, float2 *Y,
                                        float2 *scratch, int64_t batch, cudaStream_t st);
cudaError_t configure_two_pass_kernels(const cqt_plan &p);
// tile widths (columns of pass 1 / rows of pass 2 per CTA) the kernels are compiled for, widest first
constexpr int kTwoPassWidths[3] = {16, 8, 4};
size_t two_pass_smem_cols(const TwoPassBand &b, int width);
size_t two_pass_smem_rows(const TwoPassBand &b, int width);

}  // namespace cqt
