// Programmatic dependent launch (PDL) helpers shared by every kernel of the library.
//
// Each kernel is launched with the programmatic-stream-serialization attribute, so its blocks
// may become resident while the previous kernel of the stream is still draining, and each
// kernel executes wait_for_prior_kernels() before its first access to global memory.  For the
// caller this keeps plain stream-order semantics (nothing is read or written early); what it
// removes is the launch gap between the library's own back-to-back kernels.
#pragma once
#include <cuda_runtime.h>
#include <utility>

namespace civic {

__device__ __forceinline__ void wait_for_prior_kernels()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Lets the next kernel of the stream begin its launch now (it still waits for this whole grid
// to complete before it touches memory).  Only the small grids (selection, index kernels) call
// it: early blocks of a successor would take resident-block slots away from a bandwidth-bound
// grid, and measured slower next to the persistent tensor-core kernels too.
__device__ __forceinline__ void release_next_kernel()
{
    asm volatile("griddepcontrol.launch_dependents;");
}

template <typename... KArgs, typename... Args>
cudaError_t launch(bool programmatic, void (*kernel)(KArgs...), dim3 grid, unsigned block, size_t smem,
                   cudaStream_t stream, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

}  // namespace civic
