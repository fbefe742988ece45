// Sliced streaming form (Sec. 4, slicing paragraph): slices of sl samples with hop sl/2 and a
// Tukey transition window, each analysed and synthesised independently, reconstructions
// overlap-added in slice order.  All bookkeeping is host-side integer arithmetic; device work is
// enqueued on the caller's stream and never synchronised here.
#include <cstring>
#include <algorithm>
#include <cmath>
#include <new>
#include <vector>

#include "../../include/cqt.h"
#include "engine.cuh"
#include "internal.hpp"

namespace cqt {
// api.cu: cqt_analyse on slices cut from a ring buffer, the cut fused into the load of the long FFT's first pass
cqt_status analyse_slices(const cqt_plan *p, const SliceSource &src, int64_t batch, cqt_c64 *c, void *ws, size_t ws_bytes,
                          void *stream);
}  // namespace cqt

struct cqt_slicq {
    const cqt_plan *plan = nullptr;
    int C = 0;
    int64_t sl = 0, H = 0, tr = 0, K = 0;
    int64_t ring_in = 0, ring_out = 0;   // samples per channel
    float *d_win = nullptr;              // [sl]
    float *d_in = nullptr;               // [C][ring_in], stream sample n at n mod ring_in
    float *d_stage = nullptr;            // [K*C][sl] windowed slices / reconstructed slices
    cqt_c64 *d_coef = nullptr;           // [K][C][coeff_count]
    float *d_out = nullptr;              // [C][ring_out], output sample n at n mod ring_out
    void *d_ws = nullptr;
    int *d_band_off = nullptr;           // [bands + 1] coefficient offsets of the bands, last = coeff_count
    size_t ws_bytes = 0, total_bytes = 0;
    int64_t n_in = 0;        // frames pushed
    int64_t next_slice = 0;  // first slice not yet analysed
    int64_t next_synth = 0;  // first slice not yet synthesised
    int64_t n_out = 0;       // frames pulled
    cudaStream_t last_stream = nullptr;   // stream of the latest push / pull / flush (slicq_reset waits for it)
    bool used = false;
};

namespace {

// The object's kernels and copies run on the plan's device whatever device the caller has current.
struct OnPlanDevice {
    int prev = -1, dev = -1;
    bool ok = true;
    explicit OnPlanDevice(const cqt_slicq *s) {
        dev = s->plan->device;
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~OnPlanDevice() {
        if (prev >= 0 && prev != dev) cudaSetDevice(prev);
    }
};

__global__ void slicq_ingest_kernel(const float *x, long long x_stride, float *ring, long long R, long long pos, long long n, int zero) {
    cqt::pdl_launch_dependents();
    cqt::pdl_wait();
    const int c = blockIdx.y;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        ring[c * R + (pos + i) % R] = zero ? 0.f : x[c * x_stride + i];
}

// stage[(s - s0) * C + c][i] = w[i] * stream[c][s H - H + i]  (zero before the start of the stream)
__global__ void slicq_cut_kernel(const float *ring, long long R, const float *w, float *stage, long long sl, long long H,
                                 long long s0, int C) {
    cqt::pdl_launch_dependents();
    cqt::pdl_wait();
    const long long s = s0 + blockIdx.y / C;
    const int c = blockIdx.y % C;
    float *dst = stage + (long long)blockIdx.y * sl;
    const long long first = s * H - H;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < sl; i += (long long)gridDim.x * blockDim.x) {
        const long long n = first + i;
        dst[i] = n < 0 ? 0.f : w[i] * ring[c * R + n % R];
    }
}

// Overlap-add of reconstructed slices s0 .. s1 into the output ring, older slice first:
// block b = [bH, (b+1)H) = second half of slice b (or what the ring already holds when b < s0)
//                         + first half of slice b + 1 (when b + 1 <= s1).
__global__ void slicq_ola_kernel(const float *stage, float *ring, long long R, long long sl, long long H, long long s0,
                                 long long s1, int C) {
    cqt::pdl_launch_dependents();
    cqt::pdl_wait();
    const int c = blockIdx.y;
    const long long lo = (s0 - 1) * H, hi = (s1 + 1) * H;
    for (long long n = lo + blockIdx.x * (long long)blockDim.x + threadIdx.x; n < hi; n += (long long)gridDim.x * blockDim.x) {
        if (n < 0) continue;
        const long long b = n / H, r = n - b * H;
        float v = b >= s0 ? stage[((b - s0) * C + c) * sl + H + r] : ring[c * R + n % R];
        if (b + 1 <= s1) v += stage[((b + 1 - s0) * C + c) * sl + r];
        ring[c * R + n % R] = v;
    }
}

__global__ void slicq_emit_kernel(const float *ring, long long R, long long pos, float *y, long long y_stride, long long n) {
    cqt::pdl_launch_dependents();
    cqt::pdl_wait();
    const int c = blockIdx.y;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        y[c * y_stride + i] = ring[c * R + (pos + i) % R];
}

// Re-assembly: band series of length (n + 1) M/2 per band, out[c][(n + 1) off/2 + t] = c_{i}[t - i M/2] + c_{i-1}[t - (i-1) M/2]
// with i = floor(t / (M/2)) (terms whose slice index is outside 0..n-1 are absent), older slice first.
// One thread per output; the band of an output follows from a binary search over the coefficient offsets.
__global__ void slicq_assemble_kernel(const cqt_c64 *coef, long long cc, long long K, long long slot0, int C, long long n,
                                      const int *band_off, int n_bands, cqt_c64 *out, long long out_stride) {
    const int c = blockIdx.y;
    const long long total = (n + 1) * (cc / 2);
    for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        // band b: (n + 1) off_b / 2 <= e < (n + 1) off_{b+1} / 2
        int lo = 0, hi = n_bands - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if ((n + 1) * (long long)(band_off[mid] / 2) <= e) lo = mid; else hi = mid - 1;
        }
        const long long off = band_off[lo], M = band_off[lo + 1] - off, h = M / 2;
        const long long t = e - (n + 1) * (off / 2);
        const long long i = t / h, m = t - i * h;
        float re = 0.f, im = 0.f;
        if (i >= 1) {   // second half of the older slice i - 1
            const cqt_c64 v = coef[(((slot0 + i - 1) % K) * C + c) * cc + off + h + m];
            re = v.re; im = v.im;
        }
        if (i < n) {    // first half of slice i
            const cqt_c64 v = coef[(((slot0 + i) % K) * C + c) * cc + off + m];
            re += v.re; im += v.im;
        }
        out[c * out_stride + e] = cqt_c64{re, im};
    }
}

unsigned blocks_for(long long n) { return (unsigned)std::min<long long>(1024, std::max<long long>(1, (n + 255) / 256)); }

cqt_status analyse_ready(cqt_slicq *s, cudaStream_t st) {
    const int64_t ready = s->n_in / s->H;   // slices 0 .. ready - 1 are complete: (s + 1) H <= n_in
    while (s->next_slice < ready) {
        // slices whose coefficient slots are consecutive in memory
        const int64_t slot = s->next_slice % s->K;
        const int64_t cnt = std::min<int64_t>(ready - s->next_slice, s->K - slot);
        cqt_c64 *coef = s->d_coef + slot * s->C * cqt_plan_coeff_count(s->plan);
        cqt_status r;
        if (cqt::can_fuse_slice_cut(*s->plan) && s->ring_in >= s->sl) {
            // the slice cut (window x ring samples) happens in the load of the long FFT's first pass
            const cqt::SliceSource src{s->d_in, s->d_win, s->ring_in, s->next_slice * s->H - s->H, s->H, s->C};
            r = cqt::analyse_slices(s->plan, src, cnt * s->C, coef, s->d_ws, s->ws_bytes, st);
        } else {
            // short slices (one-pass long FFT): a kernel of its own writes the windowed slices to a staging buffer
            dim3 grid(blocks_for(s->sl), (unsigned)(cnt * s->C));
            if (cqt::launch_kernel_args(slicq_cut_kernel, grid, dim3(256), 0, st, s->d_in, s->ring_in, s->d_win, s->d_stage, s->sl,
                                        s->H, s->next_slice, s->C) != cudaSuccess)
                return CQT_ERR_CUDA;
            r = cqt_analyse(s->plan, s->d_stage, s->sl, cnt * s->C, s->sl, coef, s->d_ws, s->ws_bytes, st);
        }
        if (r != CQT_OK) return r;
        s->next_slice += cnt;
    }
    return CQT_OK;
}

cqt_status push_impl(cqt_slicq *s, const float *x, int64_t x_stride, int64_t n, int zero, cudaStream_t st) {
    // slices this push completes must fit the free coefficient slots
    const int64_t will_be_ready = (s->n_in + n) / s->H;
    if (will_be_ready - s->next_synth > s->K) return CQT_ERR_STATE;
    int64_t done = 0;
    while (done < n) {
        // the ring must keep every sample from (next_slice - 1) H on
        const int64_t oldest = std::max<int64_t>(0, (s->next_slice - 1) * s->H);
        const int64_t room = s->ring_in - (s->n_in - oldest);
        const int64_t m = std::min<int64_t>(n - done, room);
        if (m <= 0) return CQT_ERR_STATE;
        dim3 grid(blocks_for(m), (unsigned)s->C);
        if (cqt::launch_kernel_args(slicq_ingest_kernel, grid, dim3(256), 0, st, zero ? (const float *)nullptr : x + done, x_stride, s->d_in,
                               s->ring_in, s->n_in, m, zero) != cudaSuccess)
            return CQT_ERR_CUDA;
        s->n_in += m;
        done += m;
        cqt_status r = analyse_ready(s, st);
        if (r != CQT_OK) return r;
    }
    return CQT_OK;
}

}  // namespace

extern "C" {

cqt_status slicq_create(const cqt_plan *plan, int channels, int64_t transition, int64_t max_slices_in_flight,
                        cqt_slicq **out) {
    if (!plan || !out || channels < 1 || max_slices_in_flight < 1) return CQT_ERR_INVALID_ARG;
    if (plan->device < 0) return CQT_ERR_STATE;
    const int64_t sl = plan->N, H = sl / 2;
    if (transition <= 0 || transition > H) return CQT_ERR_INVALID_ARG;
    if (max_slices_in_flight * channels > 65535) return CQT_ERR_INVALID_ARG;
    cqt_slicq *s = new (std::nothrow) cqt_slicq();
    if (!s) return CQT_ERR_CUDA;
    s->plan = plan; s->C = channels; s->sl = sl; s->H = H; s->tr = transition; s->K = max_slices_in_flight;
    s->ring_in = (s->K + 2) * H;
    s->ring_out = (s->K + 2) * H;
    // Tukey slice window: 1 in the middle, raised-cosine flanks of `transition` samples centred on +-H/2
    std::vector<float> w(sl);
    const double lo = (H - transition) / 2.0, hi = (H + transition) / 2.0;
    for (int64_t i = 0; i < sl; ++i) {
        const double t = std::fabs((double)(i - sl / 2));
        double v = 0.0;
        if (t <= lo) v = 1.0;
        else if (t < hi) v = 0.5 * (1.0 + std::cos(3.14159265358979323846 * (t - lo) / (double)transition));
        w[i] = (float)v;
    }
    int cur = 0;
    cudaGetDevice(&cur);
    if (cudaSetDevice(plan->device) != cudaSuccess) { delete s; return CQT_ERR_CUDA; }
    const int64_t cc = cqt_plan_coeff_count(plan);
    s->ws_bytes = cqt_plan_workspace_bytes(plan, s->K * channels);
    const size_t b_win = sl * sizeof(float), b_in = (size_t)channels * s->ring_in * sizeof(float),
                 b_stage = (size_t)s->K * channels * sl * sizeof(float), b_coef = (size_t)s->K * channels * cc * sizeof(cqt_c64),
                 b_out = (size_t)channels * s->ring_out * sizeof(float);
    cudaError_t e = cudaSuccess;
    auto chk = [&](cudaError_t r) { if (e == cudaSuccess) e = r; };
    chk(cudaMalloc((void **)&s->d_win, b_win));
    chk(cudaMalloc((void **)&s->d_in, b_in));
    chk(cudaMalloc((void **)&s->d_stage, b_stage));
    chk(cudaMalloc((void **)&s->d_coef, b_coef));
    chk(cudaMalloc((void **)&s->d_out, b_out));
    chk(cudaMalloc(&s->d_ws, s->ws_bytes));
    {
        const int64_t nb = cqt_plan_num_bands(plan);
        std::vector<int> off((size_t)nb + 1);
        for (int64_t b = 0; b < nb; ++b) off[(size_t)b] = (int)plan->lay.bands[(size_t)b].coeff_off;
        off[(size_t)nb] = (int)cc;
        chk(cudaMalloc((void **)&s->d_band_off, off.size() * sizeof(int)));
        if (e == cudaSuccess) chk(cudaMemcpy(s->d_band_off, off.data(), off.size() * sizeof(int), cudaMemcpyHostToDevice));
    }
    if (e == cudaSuccess) chk(cudaMemcpy(s->d_win, w.data(), b_win, cudaMemcpyHostToDevice));
    if (e == cudaSuccess) chk(cudaMemset(s->d_out, 0, b_out));
    s->total_bytes = b_win + b_in + b_stage + b_coef + b_out + s->ws_bytes;
    cudaSetDevice(cur);
    if (e != cudaSuccess) { slicq_destroy(s); return CQT_ERR_CUDA; }
    *out = s;
    return CQT_OK;
}

cqt_status slicq_push(cqt_slicq *s, const float *x, int64_t x_stride, int64_t n, void *stream, int64_t *slices_completed) {
    if (!s || n < 0 || (n > 0 && (!x || x_stride < n))) return CQT_ERR_INVALID_ARG;
    OnPlanDevice guard(s);
    if (!guard.ok) return CQT_ERR_CUDA;
    if (n > 0) { s->last_stream = reinterpret_cast<cudaStream_t>(stream); s->used = true; }
    cqt_status r = n > 0 ? push_impl(s, x, x_stride, n, 0, reinterpret_cast<cudaStream_t>(stream)) : CQT_OK;
    if (slices_completed) *slices_completed = s->next_slice;
    return r;
}

cqt_status slicq_flush(cqt_slicq *s, void *stream) {
    if (!s) return CQT_ERR_INVALID_ARG;
    OnPlanDevice guard(s);
    if (!guard.ok) return CQT_ERR_CUDA;
    s->last_stream = reinterpret_cast<cudaStream_t>(stream);
    s->used = true;
    // enough zeros that every frame pushed so far becomes final: n_in -> (ceil(n_in / H) + 1) H
    const int64_t target = ((s->n_in + s->H - 1) / s->H + 1) * s->H;
    return push_impl(s, nullptr, 0, target - s->n_in, 1, reinterpret_cast<cudaStream_t>(stream));
}

cqt_status slicq_coeffs(cqt_slicq *s, int64_t slice_index, cqt_c64 **c) {
    if (!s || !c) return CQT_ERR_INVALID_ARG;
    if (slice_index < s->next_synth || slice_index >= s->next_slice) return CQT_ERR_STATE;
    *c = s->d_coef + (slice_index % s->K) * s->C * cqt_plan_coeff_count(s->plan);
    return CQT_OK;
}

cqt_status slicq_pull(cqt_slicq *s, float *y, int64_t y_stride, int64_t n_max, void *stream, int64_t *n_written) {
    if (!s || n_max < 0 || (n_max > 0 && (!y || y_stride < n_max)) || !n_written) return CQT_ERR_INVALID_ARG;
    OnPlanDevice guard(s);
    if (!guard.ok) return CQT_ERR_CUDA;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    s->last_stream = st;
    s->used = true;
    int64_t written = 0;
    for (;;) {
        // synthesise as many pending slices as the output ring has room for
        while (s->next_synth < s->next_slice) {
            // the ring holds frames n_out .. next_synth * H - 1; every slice adds H frames
            const int64_t room_slices = (s->ring_out - (s->next_synth * s->H - s->n_out)) / s->H;
            const int64_t slot = s->next_synth % s->K;
            const int64_t cnt = std::min<int64_t>({s->next_slice - s->next_synth, s->K - slot, room_slices});
            if (cnt <= 0) break;
            cqt_status r = cqt_synthesise(s->plan, s->d_coef + slot * s->C * cqt_plan_coeff_count(s->plan), cnt * s->C, s->sl,
                                          s->d_stage, s->sl, s->d_ws, s->ws_bytes, st);
            if (r != CQT_OK) return r;
            dim3 grid(blocks_for((cnt + 1) * s->H), (unsigned)s->C);
            if (cqt::launch_kernel_args(slicq_ola_kernel, grid, dim3(256), 0, st, s->d_stage, s->d_out, s->ring_out, s->sl, s->H,
                                   s->next_synth, s->next_synth + cnt - 1, s->C) != cudaSuccess)
                return CQT_ERR_CUDA;
            s->next_synth += cnt;
        }
        // frames below (next_synth - 1) H are final
        const int64_t final_to = std::max<int64_t>(0, (s->next_synth - 1) * s->H);
        const int64_t m = std::min<int64_t>(n_max - written, final_to - s->n_out);
        if (m > 0) {
            dim3 grid(blocks_for(m), (unsigned)s->C);
            if (cqt::launch_kernel_args(slicq_emit_kernel, grid, dim3(256), 0, st, s->d_out, s->ring_out, s->n_out, y + written, y_stride,
                                   m) != cudaSuccess)
                return CQT_ERR_CUDA;
            s->n_out += m;
            written += m;
        }
        if (m <= 0 || written >= n_max || s->next_synth >= s->next_slice) break;
    }
    *n_written = written;
    return CQT_OK;
}

cqt_status slicq_reset(cqt_slicq *s) {
    if (!s) return CQT_ERR_INVALID_ARG;
    OnPlanDevice guard(s);
    if (!guard.ok) return CQT_ERR_CUDA;
    // only the stream this object last worked on is waited for, and cleared on: other streams of the device run on
    cudaError_t e = s->used ? cudaStreamSynchronize(s->last_stream) : cudaSuccess;
    if (e == cudaSuccess) e = cudaMemsetAsync(s->d_out, 0, (size_t)s->C * s->ring_out * sizeof(float), s->last_stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s->last_stream);
    s->n_in = s->next_slice = s->next_synth = s->n_out = 0;
    return e == cudaSuccess ? CQT_OK : CQT_ERR_CUDA;
}

cqt_status slicq_destroy(cqt_slicq *s) {
    if (!s) return CQT_OK;
    int cur = 0;
    cudaGetDevice(&cur);
    cudaSetDevice(s->plan->device);
    cudaFree(s->d_win); cudaFree(s->d_in); cudaFree(s->d_stage); cudaFree(s->d_coef); cudaFree(s->d_out); cudaFree(s->d_ws); cudaFree(s->d_band_off);
    cudaSetDevice(cur);
    delete s;
    return CQT_OK;
}

size_t slicq_device_bytes(const cqt_slicq *s) { return s ? s->total_bytes : 0; }

int64_t slicq_assembled_length(const cqt_slicq *s, int64_t n_slices) {
    if (!s || n_slices < 1) return 0;
    return (n_slices + 1) * (cqt_plan_coeff_count(s->plan) / 2);
}

cqt_status slicq_assemble(cqt_slicq *s, int64_t first_slice, int64_t n_slices, cqt_c64 *out, int64_t out_stride, void *stream) {
    if (!s || !out || n_slices < 1 || first_slice < 0) return CQT_ERR_INVALID_ARG;
    if (out_stride < slicq_assembled_length(s, n_slices)) return CQT_ERR_INVALID_ARG;
    if (first_slice < s->next_synth || first_slice + n_slices > s->next_slice) return CQT_ERR_STATE;
    OnPlanDevice guard(s);
    if (!guard.ok) return CQT_ERR_CUDA;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int64_t cc = cqt_plan_coeff_count(s->plan);
    dim3 grid(blocks_for((n_slices + 1) * (cc / 2)), (unsigned)s->C);
    slicq_assemble_kernel<<<grid, 256, 0, st>>>(s->d_coef, cc, s->K, first_slice % s->K, s->C, n_slices, s->d_band_off,
                                                (int)cqt_plan_num_bands(s->plan), out, out_stride);
    return cudaGetLastError() == cudaSuccess ? CQT_OK : CQT_ERR_CUDA;
}

// Saved state: header, then the input ring and the output ring ([C][ring] floats each).
struct SlicqStateHeader {
    uint32_t magic, version;
    int32_t channels;
    int32_t pad_;
    int64_t sl, tr, K, ring_in, ring_out, coeff_count;
    int64_t n_in, next_slice, next_synth, n_out;
};
static const uint32_t kStateMagic = 0x51436c53u;   // "SlCQ"

size_t slicq_state_bytes(const cqt_slicq *s) {
    if (!s) return 0;
    return sizeof(SlicqStateHeader) + (size_t)s->C * (size_t)(s->ring_in + s->ring_out) * sizeof(float);
}

cqt_status slicq_save_state(cqt_slicq *s, void *host_buf, size_t bytes, void *stream) {
    if (!s || !host_buf) return CQT_ERR_INVALID_ARG;
    if (bytes < slicq_state_bytes(s)) return CQT_ERR_WORKSPACE;
    if (s->next_synth != s->next_slice) return CQT_ERR_STATE;    // analysed slices await slicq_pull
    OnPlanDevice guard(s);
    if (!guard.ok) return CQT_ERR_CUDA;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    SlicqStateHeader h{kStateMagic, 1u, s->C, 0, s->sl, s->tr, s->K, s->ring_in, s->ring_out, cqt_plan_coeff_count(s->plan),
                       s->n_in, s->next_slice, s->next_synth, s->n_out};
    char *p = static_cast<char *>(host_buf);
    std::memcpy(p, &h, sizeof h);
    const size_t b_in = (size_t)s->C * s->ring_in * sizeof(float), b_out = (size_t)s->C * s->ring_out * sizeof(float);
    cudaError_t e = cudaMemcpyAsync(p + sizeof h, s->d_in, b_in, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(p + sizeof h + b_in, s->d_out, b_out, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    return e == cudaSuccess ? CQT_OK : CQT_ERR_CUDA;
}

cqt_status slicq_load_state(cqt_slicq *s, const void *host_buf, size_t bytes, void *stream) {
    if (!s || !host_buf) return CQT_ERR_INVALID_ARG;
    if (bytes < sizeof(SlicqStateHeader)) return CQT_ERR_INVALID_ARG;
    SlicqStateHeader h;
    std::memcpy(&h, host_buf, sizeof h);
    if (h.magic != kStateMagic || h.version != 1u) return CQT_ERR_INVALID_ARG;
    if (h.channels != s->C || h.sl != s->sl || h.tr != s->tr || h.K != s->K || h.ring_in != s->ring_in ||
        h.ring_out != s->ring_out || h.coeff_count != cqt_plan_coeff_count(s->plan))
        return CQT_ERR_STATE;                                     // saved by an object of another shape
    if (bytes < slicq_state_bytes(s)) return CQT_ERR_INVALID_ARG;
    if (h.next_synth != h.next_slice || h.n_in < 0 || h.n_out < 0 || h.n_out > h.n_in) return CQT_ERR_INVALID_ARG;
    OnPlanDevice guard(s);
    if (!guard.ok) return CQT_ERR_CUDA;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    s->last_stream = st;
    s->used = true;
    const char *p = static_cast<const char *>(host_buf);
    const size_t b_in = (size_t)s->C * s->ring_in * sizeof(float), b_out = (size_t)s->C * s->ring_out * sizeof(float);
    cudaError_t e = cudaMemcpyAsync(s->d_in, p + sizeof h, b_in, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(s->d_out, p + sizeof h + b_in, b_out, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);          // the host buffer may be pageable and reused
    if (e != cudaSuccess) return CQT_ERR_CUDA;
    s->n_in = h.n_in; s->next_slice = h.next_slice; s->next_synth = h.next_synth; s->n_out = h.n_out;
    return CQT_OK;
}

}  // extern "C"
