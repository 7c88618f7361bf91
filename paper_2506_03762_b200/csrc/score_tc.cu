// Tensor-core scoring path (placeholder until the tcgen05 kernel lands).
#include "ahakv_internal.cuh"

namespace ahakv {

bool score_tc_available() { return false; }

ahakv_status launch_score_tc(const Plan&, const void*, const void*, float*, float2*, float*, int*, int*,
                             cudaStream_t) {
  return AHAKV_ERR_UNSUPPORTED;
}

}  // namespace ahakv
