// Programmatic dependent launch: the kernels of one optimizer step run back to back on one stream, each reading
// what its predecessor wrote.  A kernel launched with launch_dependent() may become resident while the kernel before
// it is still running (on SMs that kernel has already left, or never used), so its prologue -- barrier set-up,
// tensor-memory allocation, the first look at its tile table -- overlaps the predecessor's tail.  Before it touches
// anything a predecessor wrote, EVERY CTA calls pdl_wait(), which returns once all prerequisite grids have completed
// and their writes are visible (without the launch attribute it returns at once).  A kernel lets its successor in
// with pdl_trigger(); a kernel that never calls it does so implicitly when it completes.
#pragma once
#include <cuda_runtime.h>

namespace tsr {

__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Launches kern with programmatic stream serialization allowed (and, when cluster_z > 1, as clusters of that many
// CTAs along z).  Only for kernels whose every CTA calls pdl_wait() before its first dependent access.
template <typename Kern, typename... Args>
static inline cudaError_t launch_dependent(Kern kern, dim3 grid, dim3 block, size_t smem, cudaStream_t stream, int cluster_z,
                                           Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int na = 0;
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
    if (cluster_z > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = 1; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = (unsigned)cluster_z;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

}  // namespace tsr
