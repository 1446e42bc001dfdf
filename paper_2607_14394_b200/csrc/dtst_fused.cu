// Fused streaming kernels for the grid-side stages.
#include "dtst_fused.cuh"

namespace dtst {

bool fused_eligible(const dtst_plan*) { return false; }

void fused_workspace_elems(const dtst_plan*, int, long long* a, long long* b) {
  *a = 0;
  *b = 0;
}

dtst_status fused_forward(dtst_plan*, const float*, float2*, int, float, bool, cudaStream_t) {
  return DTST_ERR_UNSUPPORTED;
}

dtst_status fused_inverse(dtst_plan*, const float2*, float*, int, float, bool, cudaStream_t) {
  return DTST_ERR_UNSUPPORTED;
}

}  // namespace dtst
