// core_project_static: the projection for callers that must not allocate device memory.
//
// core_project keeps the per-CTA partial sums of the projection in a workspace that its
// context obtains with cudaMalloc.  Some callers cannot do that: code that runs while the
// application's memory pool owns all device memory, or inside a region where cudaMalloc's
// implicit device synchronisation is not acceptable (a latency-critical loop, a library hook
// that must not touch the allocator).  For them the partial sums live in the fixed array below,
// which is part of the library image: every GPU onto which this module has been loaded holds these
// 4 MiB until the process exits.  With CUDA's default lazy module loading that happens at the first
// cudaGetSymbolAddress below (first call of the entry point on that device), with eager loading when
// the library is loaded.
//
// The array's name is a device symbol.  In host code it is only a handle, not a device
// address, so the address the kernels receive is looked up once per device with
// cudaGetSymbolAddress while that device is current.
#include "core.h"

#include <mutex>

#include "core_internal.h"

using namespace core;

namespace {

constexpr size_t kStaticScratchFloats = CORE_STATIC_SCRATCH_FLOATS;   // 4 MiB of partial sums
constexpr int kMaxDevices = 64;

static __device__ __align__(256) float g_project_scratch[kStaticScratchFloats];

std::mutex g_setup_mutex;
float *g_scratch_addr[kMaxDevices];                                // device address per device, once known

// Device address of the scratch array on the current device (looked up on first use).
int scratch_for_current_device(float **out, int *device_out, int *last_cuda) {
    int device = -1;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) {
        *last_cuda = (int)e;
        return CORE_ECUDA;
    }
    if (device < 0 || device >= kMaxDevices) return CORE_EINVAL;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[device]) {
        float *ptr = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_project_scratch);
        if (e != cudaSuccess || !ptr) {
            cudaGetLastError();
            *last_cuda = (int)e;
            return CORE_ECUDA;
        }
        g_scratch_addr[device] = ptr;
    }
    *out = g_scratch_addr[device];
    *device_out = device;
    return CORE_OK;
}

// Is p device memory of `device`?  (Managed memory is accepted: it is reachable from every device.)
bool on_device_memory(const void *p, int device) {
    cudaPointerAttributes attr{};
    if (cudaPointerGetAttributes(&attr, p) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    if (attr.type == cudaMemoryTypeManaged) return true;
    return attr.type == cudaMemoryTypeDevice && attr.device == device;
}

}  // namespace

extern "C" {

int core_project_static(uint64_t seed, uint32_t t, int64_t d, int32_t m, const void *G_dev, int dtype, int32_t n,
                        int64_t ldg, float *P_dev, void *cuda_stream, int *cuda_error_out) {
    int last_cuda = 0;
    if (cuda_error_out) *cuda_error_out = 0;
    if (!G_dev || !P_dev || d < 1 || m < 1 || n < 1 || ldg < d || (dtype != CORE_F32 && dtype != CORE_BF16))
        return CORE_EINVAL;
    // one machine group, and at least one CTA column of partial sums must fit
    if (n > kMaxGroup || (size_t)n * (size_t)m > kStaticScratchFloats) return CORE_ELIMIT;

    float *scratch = nullptr;
    int device = -1;
    int rc = scratch_for_current_device(&scratch, &device, &last_cuda);
    if (rc != CORE_OK) {
        if (cuda_error_out) *cuda_error_out = last_cuda;
        return rc;
    }
    // the scratch address belongs to the current device: so must the caller's buffers
    if (!on_device_memory(G_dev, device) || !on_device_memory(P_dev, device)) return CORE_EINVAL;
    int sm_count = 0;
    cudaError_t e = cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) {
        if (cuda_error_out) *cuda_error_out = (int)e;
        return CORE_ECUDA;
    }
    ProjectPlan plan = make_project_plan(n, m, d, dtype, sm_count);
    // fewer CTA columns if the usual number would overflow the array (slower, same result up to
    // the order of the final additions)
    const size_t per_column = (size_t)n * (size_t)m;
    const size_t max_columns = kStaticScratchFloats / per_column;
    if ((size_t)plan.grid_x > max_columns) plan.grid_x = (int)max_columns;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const RoundKeys keys = expand_keys(seed);
    // every (column, machine, vector) entry below grid_x * n * m is overwritten by the kernel
    // before the second kernel reads it: nothing in the array has to start at zero
    e = launch_project(plan, keys, t, G_dev, dtype, n, ldg, d, m, 0, scratch, stream);
    if (e == cudaSuccess) e = launch_finish_project(scratch, plan.grid_x, n, m, P_dev, false, stream);
    if (e != cudaSuccess) {
        if (cuda_error_out) *cuda_error_out = (int)e;
        return CORE_ECUDA;
    }
    return CORE_OK;
}

}  // extern "C"
