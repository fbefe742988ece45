// cqt_analyse_static_ws: the analysis transform for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at all: code running under a memory budget that
// was fixed at start-up (real-time audio engines, plug-in sandboxes), or code between two points where
// the allocator must not be touched.  cqt_analyse needs scratch for the packed spectrum and the half
// spectrum and normally takes it from the caller.  This variant takes it from a fixed array that is part
// of the library image, so the caller passes only the signal and the coefficient buffer.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/cqt.h"

namespace {

constexpr size_t kStaticWorkspaceBytes = CQT_STATIC_WS_BYTES;
constexpr int kMaxDevices = 64;

// Lives in every GPU that loads the library, from load to exit.
static __device__ __align__(256) unsigned char g_static_ws[kStaticWorkspaceBytes];

std::mutex g_mu;
void *g_ws_ptr[kMaxDevices] = {};   // device address of g_static_ws on each device, filled on first use

// The array's name is only a host-side handle; kernels need its device address, which differs per
// device and must be looked up with that device current.
cqt_status static_ws_for_current_device(void **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CQT_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_ws_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || !p) return CQT_ERR_CUDA;
        g_ws_ptr[dev] = p;
    }
    *out = g_ws_ptr[dev];
    return CQT_OK;
}

}  // namespace

extern "C" {

size_t cqt_static_workspace_bytes(void) { return kStaticWorkspaceBytes; }

cqt_status cqt_analyse_static_ws(const cqt_plan *plan, const float *x, int64_t x_stride, int64_t batch,
                                 int64_t valid_len, cqt_c64 *c, void *stream) {
    if (!plan || batch <= 0) return CQT_ERR_INVALID_ARG;
    const size_t need = cqt_plan_workspace_bytes(plan, batch);
    if (need == 0) return CQT_ERR_INVALID_ARG;
    if (need > kStaticWorkspaceBytes) return CQT_ERR_WORKSPACE;   // beyond the fixed maximum
    const int dev = cqt_plan_device(plan);
    if (dev < 0) return CQT_ERR_STATE;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return CQT_ERR_CUDA;
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) return CQT_ERR_CUDA;
    void *ws = nullptr;
    cqt_status s = static_ws_for_current_device(&ws);
    if (s == CQT_OK) s = cqt_analyse(plan, x, x_stride, batch, valid_len, c, ws, kStaticWorkspaceBytes, stream);
    if (prev != dev) cudaSetDevice(prev);
    return s;
}

}  // extern "C"
