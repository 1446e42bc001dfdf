// Instantiations of the plane kernels (group C of the supported shapes; see dtst_plane.cuh).
#include "dtst_plane.cuh"

namespace dtst {
namespace plane {
DTST_PLANE_SHAPES_C(DTST_PLANE_INSTANTIATE)
}
}  // namespace dtst
