// Kernel launch helper with optional programmatic dependent launch (PDL), and the two device-side
// PDL instructions.
//
// A kernel launched with `pdl = true` may begin while the previous kernel on the stream is still
// draining: everything it does before pdl_wait() (index set-up, prefetch of weights, which no
// earlier kernel writes) overlaps that tail; pdl_wait() returns once the previous kernel has
// completed and its writes are visible.  Rule for every kernel launched this way: call
// pdl_wait() before the first read of anything an earlier kernel produced and before the first
// global write.  Launched without the attribute, both instructions do nothing.
#pragma once

#include <cuda_runtime.h>

namespace es {

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 bool pdl, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace es
