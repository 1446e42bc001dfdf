// Fused streaming kernels for the grid-side stages (declarations).
#pragma once
#include "dtst_common.cuh"

namespace dtst {

// Workspace (in complex elements) the fused path needs for its two intermediates.
void fused_workspace_elems(const dtst_plan* p, int Cn, long long* a, long long* b);

dtst_status fused_forward(dtst_plan* p, const float* x, float2* Xhat, int Cn, float scale, bool herm,
                          cudaStream_t st);
dtst_status fused_inverse(dtst_plan* p, const float2* Yhat, float* y, int Cn, float scale, bool herm,
                          cudaStream_t st);

}  // namespace dtst
