// Host side of the fused band kernels: per-class launches on the caller's stream and the plan's helper streams.
#include <algorithm>

#include "band_common.cuh"

namespace cqt {

static BandArgs make_args(const cqt_plan &p, const BandClass &c, const float *table, int64_t batch) {
    BandArgs a{};
    a.items = c.d_items;
    a.ffts = p.d.ffts;
    a.tw = p.d.tw;
    a.table = table;
    a.n_work = c.n_bands;
    a.batch = (int)batch;
    a.N = (int)p.N;
    a.max_elems = c.max_elems;
    a.coeff_count = p.lay.coeff_count;
    a.y_pitch = p.y_pitch;
    a.table_len = p.lay.table_len;
    a.dbg = p.d.dbg;
    return a;
}

const void *band_analysis_kernel(const BandClass &c, int lanes);    // band_analysis.cu
const void *band_synthesis_kernel(const BandClass &c, int lanes);   // band_synthesis.cu

template <bool ANALYSIS>
static const void *class_kernel(const BandClass &c, int lanes) {
    return ANALYSIS ? band_analysis_kernel(c, lanes) : band_synthesis_kernel(c, lanes);
}

// Lanes per work item of the class of the shortest bands (0: the class gives every item a whole CTA).  A band of at
// most 128 coefficients has at most 16 radix-8 butterflies per stage, so 8 lanes per item keep the lanes busy: fewer
// warps for the same work, which leaves the SMs to the long-band classes running beside it.  A whole warp per item
// has the shorter critical path, which is what counts in a call with few items (a single signal, one streaming hop).
static int lanes_for(const cqt_plan &p, const BandClass &c, long long items) {
    return items >= 8ll * p.sm_count ? c.lanes_many : c.lanes_few;
}

template <bool ANALYSIS>
static cudaError_t launch_class(const cqt_plan &p, int cls, const char *name, BandArgs &a, cudaStream_t st) {
    const BandClass &c = p.cls[cls];
    if (c.n_bands == 0) return cudaSuccess;
    const long long items = (long long)c.n_bands * a.batch;
    const int lanes = lanes_for(p, c, items);
    const int per_cta = lanes ? c.threads / lanes : 1;
    const size_t smem = (size_t)c.max_elems * per_cta * sizeof(float2);
    const long long grid = (items + per_cta - 1) / per_cta;
    void *args[] = {&a};
    const void *fn = class_kernel<ANALYSIS>(c, lanes);
    if (!fn) return cudaErrorInvalidDeviceFunction;
    cudaError_t e = launch_kernel(fn, dim3((unsigned)grid), dim3(c.threads), args, smem, st);
    note_launch(p, name, st);
    return e;
}

// The classes of one call are independent (disjoint outputs), and most of them alone leave SMs idle, so they run
// side by side on the caller's stream and the plan's helper streams (one stream per class when all five classes
// have bands): fork after the caller's stream, join back into it.
// Per call, each class's run time is estimated as the larger of the time of its longest work item and its work
// at this batch size over the machine's throughput; the classes go, longest first, to the stream with the least
// time so far (the longest one therefore stays on the caller's stream).  With event timing on, everything stays
// on the caller's stream.
struct ForkJoin {
    const cqt_plan &p;
    cudaStream_t st;
    bool used[cqt_plan::kHelpers] = {};
    bool serial;
    int slot[kNumClasses] = {0, 0, 0, 0, 0};
    ForkJoin(const cqt_plan &plan, cudaStream_t s, int64_t batch)
        : p(plan), st(s), serial(plan.timing || !plan.aux[cqt_plan::kHelpers - 1]) {
        if (serial) return;
        constexpr double kElementStagesPerUs = 6.7e5;   // the 4096 < M <= 13,500 class at 32 signals
        double est[kNumClasses], load[cqt_plan::kHelpers] = {};   // the last helper is kept for the two-pass bands
        int order[kNumClasses];
        for (int c = 0; c < kNumClasses; ++c) {
            order[c] = c;
            est[c] = p.cls[c].n_bands ? std::max(p.cls[c].latency_us, p.cls[c].stage_work * (double)batch / kElementStagesPerUs) : 0.0;
        }
        std::stable_sort(order, order + kNumClasses, [&](int a, int b) { return est[a] > est[b]; });
        for (int i = 0; i < kNumClasses; ++i) {
            const int c = order[i];
            if (!p.cls[c].n_bands) continue;
            int best = 0;
            for (int j = 1; j < cqt_plan::kHelpers; ++j)
                if (load[j] < load[best]) best = j;
            slot[c] = best;
            load[best] += est[c];
        }
        cudaEventRecord(p.ev_fork, st);
    }
    cudaStream_t stream_for(int cls) {
        if (serial || slot[cls] == 0 || p.cls[cls].n_bands == 0) return st;
        const int i = slot[cls] - 1;
        if (!used[i]) { cudaStreamWaitEvent(p.aux[i], p.ev_fork, 0); used[i] = true; }
        return p.aux[i];
    }
    cudaStream_t two_pass_stream() {
        if (serial) return st;
        const int i = cqt_plan::kHelpers - 1;
        if (!used[i]) { cudaStreamWaitEvent(p.aux[i], p.ev_fork, 0); used[i] = true; }
        return p.aux[i];
    }
    void join() {
        for (int i = 0; i < cqt_plan::kHelpers; ++i)
            if (used[i]) { cudaEventRecord(p.ev_join[i], p.aux[i]); cudaStreamWaitEvent(st, p.ev_join[i], 0); }
    }
};

cudaError_t launch_bands_from_spectrum(const cqt_plan &p, const float *table, const float2 *X, float2 *c,
                                       float2 *scratch, int64_t batch, cudaStream_t st) {
    ForkJoin fj(p, st, batch);
    if (!p.two_pass[0].bands.empty() || !p.two_pass[1].bands.empty()) {
        cudaError_t e = launch_two_pass_from_spectrum(p, table, X, c, scratch, batch, fj.two_pass_stream());
        if (e != cudaSuccess) { fj.join(); return e; }
    }
    static const char *names[kNumClasses] = {"bands_from_spectrum/class0", "bands_from_spectrum/class1",
                                              "bands_from_spectrum/class2", "bands_from_spectrum/class3",
                                              "bands_from_spectrum/class4"};
    for (int i = kNumClasses - 1; i >= 0; --i) {   // longest bands first
        BandArgs a = make_args(p, p.cls[i], table, batch);
        a.spec = X;
        a.spec_pitch = p.lf.x_pitch;
        a.coef = c;
        cudaError_t e = launch_class<true>(p, i, names[i], a, fj.stream_for(i));
        if (e != cudaSuccess) { fj.join(); return e; }
    }
    fj.join();
    return cudaSuccess;
}

// Zero-fill of the bins between a band's support and its widened range (layouts with nested supports).
__global__ void __launch_bounds__(128) zero_fill_kernel(float2 *Y, long long y_pitch, const int2 *seg) {
    const int2 sg = seg[blockIdx.x];
    float2 *y = Y + (long long)blockIdx.y * y_pitch + sg.x;
    for (int i = threadIdx.x; i < sg.y; i += blockDim.x) y[i] = make_float2(0.f, 0.f);
}

cudaError_t launch_bands_to_spectrum(const cqt_plan &p, const float *table, bool fold_sidebands, const float2 *c,
                                     float2 *Y, float2 *scratch, int64_t batch, cudaStream_t st) {
    if (p.n_zero_seg > 0) {
        zero_fill_kernel<<<dim3((unsigned)p.n_zero_seg, (unsigned)batch), 128, 0, st>>>(Y, p.y_pitch, p.d.zero_seg);
        note_launch(p, "zero_fill", st);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    ForkJoin fj(p, st, batch);
    if (!p.two_pass[0].bands.empty() || !p.two_pass[1].bands.empty()) {
        cudaError_t e = launch_two_pass_to_spectrum(p, table, fold_sidebands, c, Y, scratch, batch, fj.two_pass_stream());
        if (e != cudaSuccess) { fj.join(); return e; }
    }
    static const char *names[kNumClasses] = {"bands_to_spectrum/class0", "bands_to_spectrum/class1",
                                              "bands_to_spectrum/class2", "bands_to_spectrum/class3",
                                              "bands_to_spectrum/class4"};
    for (int i = kNumClasses - 1; i >= 0; --i) {
        BandArgs a = make_args(p, p.cls[i], table, batch);
        a.coef = const_cast<float2 *>(c);
        a.Y = Y;
        a.fold = fold_sidebands ? 1 : 0;
        cudaError_t e = launch_class<false>(p, i, names[i], a, fj.stream_for(i));
        if (e != cudaSuccess) { fj.join(); return e; }
    }
    fj.join();
    return cudaSuccess;
}

cudaError_t configure_band_kernels(const cqt_plan &p) {
    for (int i = 0; i < kNumClasses; ++i) {
        if (p.cls[i].n_bands == 0) continue;
        for (int lanes : {p.cls[i].lanes_few, p.cls[i].lanes_many}) {
            const size_t s = (size_t)p.cls[i].max_elems * (lanes ? p.cls[i].threads / lanes : 1) * sizeof(float2);
            if (!class_kernel<true>(p.cls[i], lanes)) return cudaErrorInvalidDeviceFunction;
            cudaError_t e = allow_dynamic_smem(class_kernel<true>(p.cls[i], lanes), s, p);
            if (e != cudaSuccess) return e;
            e = allow_dynamic_smem(class_kernel<false>(p.cls[i], lanes), s, p);
            if (e != cudaSuccess) return e;
        }
    }
    return cudaSuccess;
}

}  // namespace cqt
