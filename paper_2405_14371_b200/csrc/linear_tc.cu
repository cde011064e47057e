// Tensor-core (tcgen05 / TMEM / TMA) kernel of the linear-layer family.  Placeholder: not yet built.
#include "es_internal.cuh"

namespace es {

bool linear_tc_supported(const LinearParams&, int) { return false; }

es_status_t launch_linear_tc(const LinearParams&, int, cudaStream_t, int64_t*, int*) {
  return fail(ES_ERR_UNSUPPORTED, "tensor-core kernel not built");
}

}  // namespace es
