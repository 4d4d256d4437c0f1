// psd_confidence_static: psd_confidence for callers that cannot provide scratch memory.
//
// Some users of this library cannot allocate device memory where they need a confidence pass: a
// serving process that handed all free HBM to its own pool at start-up, or a plug-in called back
// from inside another runtime where cudaMalloc (and the device-wide synchronisation it implies) is
// off limits.  For them the per-split partial triples live in a fixed array that is part of the
// library image: every GPU that loads this part of the library carries PSD_STATIC_SCRATCH_BYTES of
// it until the process exits.  With CUDA's default lazy loading the driver reserves the array when
// the module is first needed on a device, which can be as late as the first call here: such callers
// make one call per device at start-up, before they give the remaining memory away.
#include <mutex>
#include "psd_internal.cuh"

namespace {

// Scratch shared by every call on a device.  The name below is only a host-side handle in host code;
// the device address is looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[PSD_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up on the first call per device).
int scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PSD_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return PSD_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return PSD_OK;
}

}  // namespace

extern "C" int psd_confidence_static(const void* hidden_bf16, const void* w_lm_bf16,
                                     int32_t n_rows, int32_t H, int32_t V,
                                     int32_t* out_token, float* out_conf, float* out_lse,
                                     int32_t* status_dev, void* cuda_stream) {
    if (!hidden_bf16 || !w_lm_bf16 || !out_token || !out_conf) return PSD_ERR_NULL;
    const size_t need = psd_workspace_bytes(n_rows, H, V);
    if (need == 0) return PSD_ERR_SHAPE;
    if (need > (size_t)PSD_STATIC_SCRATCH_BYTES) return PSD_ERR_WORKSPACE;   // problem too large for the fixed scratch
    if ((reinterpret_cast<uintptr_t>(hidden_bf16) & 15) || (reinterpret_cast<uintptr_t>(w_lm_bf16) & 15) ||
        (reinterpret_cast<uintptr_t>(out_token) & 3) || (reinterpret_cast<uintptr_t>(out_conf) & 3) ||
        (reinterpret_cast<uintptr_t>(out_lse) & 3) || (reinterpret_cast<uintptr_t>(status_dev) & 3))
        return PSD_ERR_ALIGN;
    void* scratch = nullptr;
    if (int e = scratch_for_current_device(&scratch)) return e;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    // Nothing in the scratch has to start at zero: the fused kernel writes every (row, split) triple
    // that the combine pass reads, so whatever an earlier call left behind is overwritten first.
    psd::Partials part = psd::carve_partials(scratch, n_rows, V);
    psd::SplitPlan plan;
    if (int rc = psd::launch_confidence(hidden_bf16, w_lm_bf16, n_rows, H, V, part, status_dev, st, &plan)) return rc;
    return psd::launch_combine(part, plan, n_rows, out_token, out_conf, out_lse, st, nullptr, nullptr, 0, status_dev);
}
