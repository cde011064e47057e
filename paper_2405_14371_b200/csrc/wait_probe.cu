// A wait that is meant to run out: the smallest kernel with the structure of the tensor-core kernels (barrier
// initialisation, a TMEM allocation, a bounded mbarrier wait, the common teardown) whose barrier nobody ever
// arrives on.  It exists so that the path "a device-side wait gave up -> status word -> ES_ERR_DEVICE_TIMEOUT"
// can be exercised without any kernel misbehaving: the wait ends after the given limit, the CTA records the
// code, frees its TMEM and returns like any other CTA, and the context stays usable.
#include "es_internal.cuh"
#include "launch.cuh"
#include "sm100.cuh"

namespace es {

namespace {

constexpr int PROBE_CODE = 90;

__global__ void __launch_bounds__(64) wait_probe_kernel(int* status, unsigned long long limit_ns) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&tmem_slot), 32);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  // one thread waits for a phase that never completes; everybody else goes straight to the teardown
  if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0, &abort_flag, status, PROBE_CODE, limit_ns);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 32);
  }
}

}  // namespace

es_status_t launch_wait_probe(int* status, unsigned long long limit_ns, cudaStream_t s, int64_t* launches) {
  ES_CUDA_CHECK(launch_kernel(wait_probe_kernel, dim3(1), dim3(64), 0, s, false, status, limit_ns));
  if (launches) ++*launches;
  return ES_OK;
}

}  // namespace es
