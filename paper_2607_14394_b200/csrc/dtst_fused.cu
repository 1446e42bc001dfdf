// Dispatcher of the fused streaming kernels: which plane shapes exist, tensor-map construction, and the run-time
// selection of the instantiation for a plan's shape.  The kernels themselves are templates in dtst_plane.cuh,
// instantiated in dtst_plane_inst_*.cu.
#include <cuda.h>

#include <cstdlib>

#include "dtst_plane.cuh"

namespace dtst {

namespace plane {
DTST_PLANE_SHAPES(DTST_PLANE_EXTERN)
DTST_PLANE_COL_SHAPES(DTST_PLANE_COL_EXTERN)
}

namespace {

// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn lookup_encode_tiled() {
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult q;
  EncodeTiledFn fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
      q == cudaDriverEntryPointSuccess)
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
  (void)cudaGetLastError();
  return fn;
}

// looked up once; the initialisation of a function-local static is thread-safe, so plans on different host
// threads all see the same answer
EncodeTiledFn encode_tiled_fn() {
  static const EncodeTiledFn fn = lookup_encode_tiled();
  return fn;
}

}  // namespace

// 2-D fp32 tensor [rows][n3] viewed through [box_rows x 32] boxes with the 128-byte swizzle.
bool make_rows_map(CUtensorMap* map, const void* base, long long rows, int n3, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)n3, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)n3 * 4};
  cuuint32_t box[2] = {32, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tma_encode_available() { return encode_tiled_fn() != nullptr; }

// fp32 tensor [rows][P] with P contiguous, viewed through [box_rows x 32 floats] boxes with the 128-byte swizzle
bool make_points_map(CUtensorMap* map, const float* base, long long rows, long long P, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)P, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)P * 4};
  cuuint32_t box[2] = {32, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Shapes the plane kernels are instantiated for: (N3, k3, N2, k2).
static bool plane_supported(int N3, int K3, int N2, int K2) {
#define DTST_MATCH(a, b, c, d) if (N3 == a && K3 == b && N2 == c && K2 == d) return true;
  DTST_PLANE_SHAPES(DTST_MATCH)
#undef DTST_MATCH
  return false;
}

bool fused_eligible(const dtst_plan* p) {
  if (p->d < 2) return false;
  const int a = p->d - 1, b = p->d - 2;
  // the symmetry folding needs the whole extent of both dimensions with zero phase offset
  if (p->Nl[a] != p->Ng[a] || p->Nl[b] != p->Ng[b] || p->off[a] != 0 || p->off[b] != 0) return false;
  if (p->d == 2 && p->P > 1) return false;   // slabs would cut the second-last dimension
  if (!plane_supported((int)p->Ng[a], p->kmax[a], (int)p->Ng[b], p->kmax[b])) return false;
  long long planes = (long long)p->B;
  for (int i = 0; i < b; ++i) planes *= p->Nl[i];
  // tasks are 128 rows: with 64-row planes every tensor must hold an even number of planes
  long long pin = planes * p->C_in, pout = planes * p->C_out;
  if ((pin * p->Ng[b]) % plane::kTaskRows != 0 || (pout * p->Ng[b]) % plane::kTaskRows != 0) return false;
  if (pin * p->Ng[b] >= (1ll << 31) || pout * p->Ng[b] >= (1ll << 31)) return false;   // 32-bit TMA coordinates
  return encode_tiled_fn() != nullptr;
}

cudaError_t launch_fwd_plane(int N3, int K3, int N2, int K2, const float* x, float2* out, long long rows,
                             float scale, int herm, int* status, const RingDebug& dbg, cudaStream_t st) {
#define DTST_CALL(a, b, c, d) \
  if (N3 == a && K3 == b && N2 == c && K2 == d) return plane::plane_fwd<a, b, c, d>(x, out, rows, scale, herm, status, dbg, st);
  DTST_PLANE_SHAPES(DTST_CALL)
#undef DTST_CALL
  return cudaErrorNotSupported;
}

// N1 must be a power of two that divides 8 K1 (the unpaired mode's phase then depends on a plane's place in its
// batch of 8 only), hold both retained halves and fit the kernel's cosine table.
bool fwd_plane_col_supported(int N3, int K3, int N2, int K2, int N1, int K1) {
  static const bool off = std::getenv("DTST_NO_COLFUSE") != nullptr;   // diagnostic: keep the two-launch path
  if (off) return false;
  bool shape = false;
#define DTST_MATCH(a, b, c, d, e) if (N3 == a && K3 == b && N2 == c && K2 == d && K1 == e) shape = true;
  DTST_PLANE_COL_SHAPES(DTST_MATCH)
#undef DTST_MATCH
  return shape && N1 >= 8 && (N1 & (N1 - 1)) == 0 && N1 <= 128 && N1 >= 2 * K1 && (8 * K1) % N1 == 0;
}

cudaError_t launch_fwd_plane_col(int N3, int K3, int N2, int K2, int N1, int K1, const float* x, float2* out,
                                 long long rows, float scale, int herm, int* status, const RingDebug& dbg,
                                 cudaStream_t st) {
#define DTST_CALL(a, b, c, d, e)                                    \
  if (N3 == a && K3 == b && N2 == c && K2 == d && K1 == e)          \
    return plane::plane_fwd_col<a, b, c, d, e>(x, out, rows, N1, scale, herm, status, dbg, st);
  DTST_PLANE_COL_SHAPES(DTST_CALL)
#undef DTST_CALL
  return cudaErrorNotSupported;
}

cudaError_t launch_inv_plane(int N3, int K3, int N2, int K2, const float2* in, float* y, long long rows, float scale,
                             int herm, int* /*status*/, cudaStream_t st) {
  const plane::ColExpandArgs none{};
#define DTST_CALL(a, b, c, d) \
  if (N3 == a && K3 == b && N2 == c && K2 == d) return plane::plane_inv<a, b, c, d, 0, 1>(in, y, rows, scale, herm, none, st);
  DTST_PLANE_SHAPES(DTST_CALL)
#undef DTST_CALL
  return cudaErrorNotSupported;
}

// The helper-warp variant is built for a leading dimension of the same shape as the second plane dimension.
bool inv_plane_colexp_supported(int N3, int K3, int N2, int K2, int N1, int K1) {
  if (!plane_supported(N3, K3, N2, K2)) return false;
  return N1 == N2 && K1 == K2 && (2 * K2 * K3) % (8 * plane::kColExpandMT) == 0;
}

cudaError_t launch_inv_plane_colexp(int N3, int K3, int N2, int K2, int N1, int K1, const float2* in1, float2* ring,
                                    int ring_cols, int* counters, long long cols, float* y, long long rows,
                                    float scale, int herm, int* status, uint32_t poll_limit, cudaStream_t st) {
  if (!inv_plane_colexp_supported(N3, K3, N2, K2, N1, K1)) return cudaErrorNotSupported;
  plane::ColExpandArgs ce{};
  ce.in1 = in1;
  ce.ring = ring;
  ce.ready = counters;
  ce.done = counters + cols;
  ce.status = status;
  ce.cols = cols;
  ce.N1 = N1;
  ce.R = ring_cols < 1 ? 1 : ring_cols;
  ce.poll_limit = poll_limit;
#define DTST_CALL(a, b, c, d) \
  if (N3 == a && K3 == b && N2 == c && K2 == d) return plane::plane_inv<a, b, c, d, d, c / 32>(ring, y, rows, scale, herm, ce, st);
  DTST_PLANE_SHAPES(DTST_CALL)
#undef DTST_CALL
  return cudaErrorNotSupported;
}

}  // namespace dtst
