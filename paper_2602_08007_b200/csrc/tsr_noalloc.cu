// tsr_project_core_static: the core projection C = U^T G V for one matrix block with no device
// memory taken from anybody -- no context, no caller workspace, no cudaMalloc.  The m x r
// intermediate T = G V lives in a fixed array that is part of the library image.
#include <mutex>

#include "tsr_internal.h"

namespace {

// Scratch for T = G V (m x r FP32).  Every GPU that loads the library holds these 4 MiB until
// the process exits.  All calls share it.
__device__ __align__(256) float g_static_t[TSR_STATIC_SCRATCH_FLOATS];

constexpr int kMaxDevices = 64;
float *g_scratch_ptr[kMaxDevices];   // device address of g_static_t on each device, once resolved
std::mutex g_setup_mutex;

// In host code the name g_static_t is only a handle for the symbol, not a device address; the
// address a kernel can use has to be asked for, with the device in question current.
cudaError_t scratch_for_current_device(float **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        float *p = nullptr;
        e = cudaGetSymbolAddress((void **)&p, g_static_t);
        if (e != cudaSuccess) return e;
        if (!p) return cudaErrorInvalidSymbol;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" tsr_status tsr_project_core_static(const void *G, int32_t g_dtype, int64_t m, int64_t n, int64_t ldg,
                                              const float *U, const float *V, int32_t r, float *C, void *stream)
{
    if (!G || !U || !V || !C) return TSR_ERR_INVALID_ARG;
    if (g_dtype != TSR_F32 && g_dtype != TSR_BF16) return TSR_ERR_UNSUPPORTED;
    if (m <= 0 || n <= 0 || r <= 0 || ldg < n || r > m || r > n || m > 0x3fffffff || n > 0x3fffffff) return TSR_ERR_SHAPE;
    if (m * (int64_t)r > (int64_t)TSR_STATIC_SCRATCH_FLOATS) return TSR_ERR_WORKSPACE;   // T does not fit the fixed array
    float *T = nullptr;
    if (scratch_for_current_device(&T) != cudaSuccess) return TSR_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    // T = G V is written in full before it is read, so nothing in the shared array needs clearing.
    if (tsr::simt_gemm((int)m, r, (int)n, G, g_dtype, ldg, 1, V, r, 1, T, r, tsr::SIMT_STORE, 0.f, 0.f, st) != cudaSuccess)
        return TSR_ERR_CUDA;
    // C = U^T T
    if (tsr::simt_gemm(r, r, (int)m, U, TSR_F32, 1, r, T, r, 1, C, r, tsr::SIMT_STORE, 0.f, 0.f, st) != cudaSuccess)
        return TSR_ERR_CUDA;
    return TSR_OK;
}
