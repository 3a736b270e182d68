// Programmatic dependent launch: every kernel of a run is launched with the "programmatic
// stream serialization" attribute, so the next kernel's CTAs may start - and run their prologue
// (barrier set-up, tensor-memory allocation, weight prefetch) - while the previous kernel drains.
// This is the stream-level analogue of the paper's pre-filled command queue (Section 3.2): no
// CPU round trip and, here, no idle gap between consecutive programs either.
//
// Rule that keeps it correct: a kernel touches no activation memory (arena, inputs, outputs)
// before pdl_wait(), which returns once every earlier kernel in the stream has completed and its
// writes are visible.  Weights are written once at bind time and may be read before the wait.
#pragma once

#include <cuda_runtime.h>

#include <utility>

namespace gi {

#if defined(__CUDACC__)
// allow the next kernel in the stream to start launching (it still waits in pdl_wait)
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// block until all earlier kernels in the stream have finished and flushed their writes
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

}  // namespace gi
