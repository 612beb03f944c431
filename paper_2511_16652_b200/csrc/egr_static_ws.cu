// Perturbed linear forward for callers that cannot allocate device memory.
//
// Some hosts of this library have no way to obtain a workspace: code running under a memory budget that is
// fixed before the library is loaded, plug-ins that receive only their input and output buffers from the
// framework that owns the allocator, or sections of a program where cudaMalloc is forbidden because it
// synchronises the device.  For them the scratch of egr_perturbed_linear (status words, the counter the side warps claim
// rows from, per-band ready counters and the skinny product s = X B_p, R*r floats) lives in one file-scope device array of fixed size.  The array is part of
// the loaded module: every GPU that loads the library holds those bytes until the process exits.
#include <cmath>
#include <mutex>

#include "egr_device.cuh"
#include "egr_internal.h"

namespace {

// status block + per-band ready counters (one int per 128 rows, at most 2048 of them) + s
constexpr size_t kStaticScratchBytes = egr::kWsHeader + 8192 + EGR_STATIC_MAX_S_FLOATS * sizeof(float);

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void *g_scratch_ptr[kMaxDevices] = {};      // device address of g_static_scratch, per device ordinal
std::mutex g_scratch_mutex;                 // host threads may make their first call on a device at the same time

// In host code `g_static_scratch` is only a handle for the runtime, not a device address: the address a kernel
// can use has to be asked for, once per device, with that device current.
int static_scratch(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return EGR_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return EGR_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return EGR_OK;
}

}  // namespace

extern "C" int egr_perturbed_linear_static(const egr_layer *L, const void *X, const void *W, float sigma, void *Y,
                                           void *stream)
{
    // the argument rules of the regular entry point come first, so that a layer that is both invalid and too large is
    // reported as invalid
    const int bad = egr::perturbed_linear_check(L, X, W, nullptr, Y);
    if (bad != EGR_OK) return bad;
    const unsigned long long s_floats =
        (unsigned long long)L->n_members * (unsigned long long)L->rows_per_member * (unsigned long long)L->rank;
    if (s_floats > EGR_STATIC_MAX_S_FLOATS) return EGR_ERR_CAPACITY;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev <= 0) return EGR_ERR_CUDA;
    void *scratch = nullptr;
    const int rc = static_scratch(&scratch);
    if (rc != EGR_OK) return rc;
    // Same validation, same kernels; only the origin of the scratch differs.  The status words at the start
    // of the array are cleared by the call itself; s is overwritten for every row before it is read.
    return egr_perturbed_linear(L, X, W, sigma, Y, scratch, kStaticScratchBytes, stream);
}

extern "C" int egr_static_status(void *stream)
{
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev <= 0) return EGR_ERR_CUDA;
    void *scratch = nullptr;
    const int rc = static_scratch(&scratch);
    if (rc != EGR_OK) return rc;
    return egr_workspace_status(scratch, stream);
}
