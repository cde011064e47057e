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

// Optional time stamps of a launch: slot[0] takes the earliest %globaltimer value any CTA of the launch saw at
// its start, slot[STAMP_SLOTS] the latest any warp saw at its end (nanoseconds): the slots of a pass form two
// arrays, so that one fill can reset the starts to "never" and another the ends to 0.  nullptr (the default) =
// no stamps.  The end is taken by the first thread of every CTA (the warps of a CTA of these kernels finish
// together to within a fraction of a microsecond).
// With them the time a replayed step spends in each of its kernels can be read from inside the step, with the
// programmatic overlap between consecutive kernels left as it is.
constexpr int STAMP_SLOTS = 2048;
__device__ __forceinline__ unsigned long long stamp_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void stamp_begin(unsigned long long* slot) {
  if (slot != nullptr && threadIdx.x == 0) atomicMin(slot, stamp_now());
}
// called by every thread that leaves the kernel; the first thread of each CTA records (one atomic per CTA: with one
// per warp the 2368 same-address atomics of a full grid cost microseconds per kernel)
__device__ __forceinline__ void stamp_end(unsigned long long* slot) {
  if (slot != nullptr && threadIdx.x == 0) atomicMax(slot + STAMP_SLOTS, stamp_now());
}

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
