// Instantiations of the plane kernels (group A of the supported shapes; see dtst_plane.cuh).
#include "dtst_plane.cuh"

namespace dtst {
namespace plane {
DTST_PLANE_SHAPES_A(DTST_PLANE_INSTANTIATE)
}
}  // namespace dtst
