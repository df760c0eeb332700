// dyn_eval_select_static: the fused evaluate+select call for callers that cannot allocate device
// memory.  Its scratch is a fixed array in the library image instead of a caller workspace.
#define DYN_TU_ID 7
#include "dyn_internal.cuh"

#include <mutex>

namespace {

// The scratch itself.  One copy exists on every device that loads this library, until exit.
static __device__ __align__(256) unsigned char g_static_scratch[DYN_STATIC_WS_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void *g_scratch_addr[kMaxDevices] = {};      // device address of g_static_scratch, per device ordinal

// In host code the name g_static_scratch is only a handle for the runtime, not a device address, so
// the address a kernel can use has to be asked for: once per device, with that device current.
int scratch_address(void **out) {
    int dev = -1;
    DYN_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return DYN_EUNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        DYN_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p || (reinterpret_cast<uintptr_t>(p) & 255u) != 0) return DYN_EWORKSPACE;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return DYN_OK;
}

}  // namespace

extern "C" int dyn_eval_select_static(const dyn_profile *profile, const dyn_space *space, const float *d_load,
                                      int64_t S, int64_t W, const dyn_select_out *out, void *stream) {
    if (!profile || !space) return DYN_EINVAL;
    const size_t need = dyn_workspace_bytes(profile, space, S, W);
    if (need == 0) return DYN_EINVAL;
    if (need > size_t(DYN_STATIC_WS_BYTES)) return DYN_EUNSUPPORTED;     // larger than the built-in scratch
    void *scratch = nullptr;
    const int rc = scratch_address(&scratch);
    if (rc != DYN_OK) return rc;
    // Nothing in the scratch has to start at zero: the resolve kernel rewrites the tables and the
    // totals kernels rewrite the partial sums before anything reads them.
    return dyn_eval_select(profile, space, d_load, S, W, out, scratch, size_t(DYN_STATIC_WS_BYTES), stream);
}
