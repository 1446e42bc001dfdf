// Instantiations of the forward plane kernel with the third dimension fused (see dtst_plane.cuh).
#include "dtst_plane.cuh"

namespace dtst {
namespace plane {
DTST_PLANE_COL_SHAPES(DTST_PLANE_COL_INSTANTIATE)
}
}  // namespace dtst
