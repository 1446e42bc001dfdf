// Fused streaming kernels for the grid-side stages (launchers).
#pragma once
#include <cuda.h>

#include "dtst_common.cuh"

namespace dtst {

// Forward plane kernel: real rows [rows][N3] (rows = planes * N2) -> out[planes][2*K2][K3] complex,
// contracting the last two grid dimensions in one pass.  scale and the Hermitian weight (herm) are
// applied per last-dim frequency.  `status` is the plan's device status word.
cudaError_t launch_fwd_plane(int N3, int K3, int N2, int K2, const float* x, float2* out, long long rows,
                             float scale, int herm, int* status, const RingDebug& dbg, cudaStream_t st);

// The same with the third dimension (the one in front of the plane: extent N1, whole and without offset, K1 modes
// per side) contracted inside the kernel: out[columns][2 K1][2 K2][K3], columns = rows / (N2 N1).
bool fwd_plane_col_supported(int N3, int K3, int N2, int K2, int N1, int K1);
cudaError_t launch_fwd_plane_col(int N3, int K3, int N2, int K2, int N1, int K1, const float* x, float2* out,
                                 long long rows, float scale, int herm, int* status, const RingDebug& dbg,
                                 cudaStream_t st);

// Inverse plane kernel: in[planes][2*K2][K3] complex -> real rows [rows][N3].
cudaError_t launch_inv_plane(int N3, int K3, int N2, int K2, const float2* in, float* y, long long rows,
                             float scale, int herm, int* status, cudaStream_t st);

// The same with the expansion of the dimension in front of the plane (extent N1, 2 K1 retained entries) done inside
// the kernel by a helper warp per CTA: in1[cols][2 K1][2 K2 K3] is expanded column by column into `ring`
// ([ring_cols][N1][2 K2 K3], consumed from L2); `counters` holds 2 * cols ints (zeroed by the launch).
bool inv_plane_colexp_supported(int N3, int K3, int N2, int K2, int N1, int K1);
cudaError_t launch_inv_plane_colexp(int N3, int K3, int N2, int K2, int N1, int K1, const float2* in1, float2* ring,
                                    int ring_cols, int* counters, long long cols, float* y, long long rows,
                                    float scale, int herm, int* status, uint32_t poll_limit, cudaStream_t st);

// 2-D fp32 tensor [rows][n3] viewed through [box_rows x 32 floats] boxes with the 128-byte TMA swizzle.
bool make_rows_map(CUtensorMap* map, const void* base, long long rows, int n3, int box_rows);

// whether the driver's tensor-map encoder could be found (no TMA kernel runs without it)
bool tma_encode_available();
// fp32 tensor [rows][P] with P contiguous, viewed through [box_rows x 32 floats] boxes with the 128-byte swizzle
bool make_points_map(CUtensorMap* map, const float* base, long long rows, long long P, int box_rows);

// Tensor-core version of the block's forward epilogue (dtst_block_umma.cu): C_in in {8, 16, 32}, C_out in {16, 32}
bool block_umma_supported(int Ci, int Co, long long P, int B);
cudaError_t launch_block_epilogue_umma(const float* x, float* out, float* z, const float* Wb, int B, int Ci, int Co,
                                       long long P, int* status, cudaStream_t st);

// Row kernels (dtst_row.cu): the contiguous dimension alone, N3 % 32 == 0, N3 <= 256, k3 <= 16.
bool row_supported(int N3, int K3);
cudaError_t launch_row_contract(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm,
                                int* status, cudaStream_t st);
cudaError_t launch_row_expand(const float2* in, float* y, long long rows, int N3, int K3, float scale, int herm,
                              cudaStream_t st);

// Row kernels for any contiguous extent (dtst_rowg.cu): N3 <= 512 (odd extents included), k3 <= 32; cp.async-fed,
// no tensor map.  Used where row_supported() says no.  fast: single-pass TF32 instead of the hi/lo compensated products.
bool rowg_supported(int N3, int K3);
cudaError_t launch_rowg_contract(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm, bool fast,
                                 cudaStream_t st);
cudaError_t launch_rowg_expand(const float2* in, float* y, long long rows, int N3, int K3, float scale, int herm, bool fast,
                               cudaStream_t st);
// Row kernels for long contiguous extents (dtst_rowl.cu): 512 < N3 <= 16384, N3 % 8 == 0, k3 <= 32.
bool rowl_supported(int N3, int K3);
cudaError_t launch_rowl_contract(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm, bool fast,
                                 cudaStream_t st);
cudaError_t launch_rowl_expand(const float2* in, float* y, long long rows, int N3, int K3, float scale, int herm, bool fast,
                               cudaStream_t st);
// The same with the dimension in front (extent N2, whole, no offset, K2 modes per side) inside the kernel:
// x[planes][N2][N3] <-> [planes][2 K2][k3].
bool planeg_supported(int N3, int K3, int N2, int K2);
cudaError_t launch_planeg_contract(const float* x, float2* out, long long planes, int N3, int K3, int N2, int K2,
                                   float scale, int herm, bool fast, cudaStream_t st);
cudaError_t launch_planeg_expand(const float2* in, float* y, long long planes, int N3, int K3, int N2, int K2,
                                 float scale, int herm, bool fast, cudaStream_t st);

}  // namespace dtst
