// Generic kernels: one contraction/expansion along a single dimension for any
// shape, the slab-partial reduction, and the per-mode channel mixing with its
// adjoint.  They serve every shape the fused kernels do not cover.
#include "dtst_common.cuh"

namespace dtst {

// ---------------------------------------------------------------------------
// out[slab][o][r][i] = sum_q E[r][q] * in[slab][o][q][i]
// E is generated on the device from (N, k, offset) into shared memory (Eq. 18),
// or evaluated on the fly when it does not fit.
// ---------------------------------------------------------------------------
template <bool IN_REAL, bool OUT_REAL>
__global__ void __launch_bounds__(256) apply_dim_kernel(DimOp p, const void* __restrict__ in_,
                                                       void* __restrict__ out_) {
  extern __shared__ float2 Es[];
  const int slab = blockIdx.y;
  if (p.basis_in_smem) {
    const int total = p.R * p.Q;
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
      Es[e] = dimop_entry(p, e / p.Q, e % p.Q, slab);
    }
    __syncthreads();
  }
  const float* in_r = reinterpret_cast<const float*>(in_) + (long long)slab * p.in_slab_stride;
  const float2* in_c = reinterpret_cast<const float2*>(in_) + (long long)slab * p.in_slab_stride;
  float* out_r = reinterpret_cast<float*>(out_) + (long long)slab * p.out_slab_stride;
  float2* out_c = reinterpret_cast<float2*>(out_) + (long long)slab * p.out_slab_stride;

  const long long total = p.outer * p.R * p.inner;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += stride) {
    const long long i = idx % p.inner;
    const long long t = idx / p.inner;
    const int r = (int)(t % p.R);
    const long long o = t / p.R;
    const long long base = o * p.in_outer_stride + i;
    float ar = 0.f, ai = 0.f;
    for (int q = 0; q < p.Q; ++q) {
      const float2 e = p.basis_in_smem ? Es[r * p.Q + q] : dimop_entry(p, r, q, slab);
      if (IN_REAL) {
        const float v = in_r[base + (long long)q * p.inner];
        ar = fmaf(e.x, v, ar);
        ai = fmaf(e.y, v, ai);
      } else {
        const float2 v = in_c[base + (long long)q * p.inner];
        ar = fmaf(e.x, v.x, ar);
        ar = fmaf(-e.y, v.y, ar);
        if (!OUT_REAL) {
          ai = fmaf(e.x, v.y, ai);
          ai = fmaf(e.y, v.x, ai);
        }
      }
    }
    const long long oidx = o * p.out_outer_stride + (long long)r * p.inner + i;
    if (OUT_REAL) {
      out_r[oidx] = ar;
    } else {
      out_c[oidx] = make_float2(ar, ai);
    }
  }
}

cudaError_t launch_apply_dim(const DimOp& op_in, bool in_real, bool out_real, const void* in, void* out,
                             cudaStream_t st) {
  DimOp op = op_in;
  const size_t smem = (size_t)op.R * op.Q * sizeof(float2);
  op.basis_in_smem = smem <= 160 * 1024 ? 1 : 0;
  const size_t dyn = op.basis_in_smem ? smem : 0;
  const long long total = op.outer * op.R * op.inner;
  if (total <= 0) return cudaSuccess;
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)kNumSMs * 8;
  if (blocks > cap) blocks = cap;
  dim3 grid((unsigned)blocks, (unsigned)op.slabs);
  cudaError_t err = cudaSuccess;
#define DTST_LAUNCH(IR, OR)                                                                         \
  do {                                                                                              \
    if (dyn > 48 * 1024)                                                                            \
      err = cudaFuncSetAttribute(apply_dim_kernel<IR, OR>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                 (int)dyn);                                                         \
    if (err == cudaSuccess) apply_dim_kernel<IR, OR><<<grid, 256, dyn, st>>>(op, in, out);          \
  } while (0)
  if (in_real && !out_real) DTST_LAUNCH(true, false);
  else if (!in_real && out_real) DTST_LAUNCH(false, true);
  else if (!in_real && !out_real) DTST_LAUNCH(false, false);
  else return cudaErrorInvalidValue;   // real -> real never occurs: a real grid maps to a complex spectrum
#undef DTST_LAUNCH
  if (err != cudaSuccess) return err;
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Sum of P slab partial spectra in ascending slab order (Eq. 7), fixed order so
// that repeated runs are bitwise identical.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) reduce_partials_kernel(const float2* __restrict__ partial,
                                                             float2* __restrict__ out, long long n, int P) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    float2 acc = partial[i];
    for (int p = 1; p < P; ++p) {
      const float2 v = partial[(long long)p * n + i];
      acc.x += v.x;
      acc.y += v.y;
    }
    out[i] = acc;
  }
}

cudaError_t launch_reduce_partials(const float2* partial, float2* out, long long n, int P, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  long long blocks = (n + 255) / 256;
  if (blocks > (long long)kNumSMs * 8) blocks = (long long)kNumSMs * 8;
  reduce_partials_kernel<<<(unsigned)blocks, 256, 0, st>>>(partial, out, n, P);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Per-mode channel mixing (Eq. 12): Y[b,o,m] = sum_i X[b,i,m] W[i,o,m].
// One thread per (o, m); W is streamed once per chunk of up to BT batch entries.
// ---------------------------------------------------------------------------
template <int BT>
__global__ void __launch_bounds__(256) mix_kernel(const float2* __restrict__ X, const float2* __restrict__ W,
                                                 float2* __restrict__ Y, int b0, int nb, int Ci, int Co,
                                                 long long M) {
  const long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int o = blockIdx.y;
  if (m >= M) return;
  float2 acc[BT];
#pragma unroll
  for (int b = 0; b < BT; ++b) acc[b] = make_float2(0.f, 0.f);
  for (int i = 0; i < Ci; ++i) {
    const float2 w = W[((long long)i * Co + o) * M + m];
#pragma unroll
    for (int b = 0; b < BT; ++b) {
      if (b < nb) {
        const float2 x = X[((long long)(b0 + b) * Ci + i) * M + m];
        acc[b].x = fmaf(x.x, w.x, acc[b].x);
        acc[b].x = fmaf(-x.y, w.y, acc[b].x);
        acc[b].y = fmaf(x.x, w.y, acc[b].y);
        acc[b].y = fmaf(x.y, w.x, acc[b].y);
      }
    }
  }
#pragma unroll
  for (int b = 0; b < BT; ++b)
    if (b < nb) Y[((long long)(b0 + b) * Co + o) * M + m] = acc[b];
}

cudaError_t launch_mix(const float2* X, const float2* W, float2* Y, int B, int Ci, int Co, long long M,
                       cudaStream_t st, long long* launches) {
  constexpr int BT = 4;
  dim3 grid((unsigned)((M + 255) / 256), (unsigned)Co);
  for (int b0 = 0; b0 < B; b0 += BT) {
    const int nb = (B - b0 < BT) ? (B - b0) : BT;
    mix_kernel<BT><<<grid, 256, 0, st>>>(X, W, Y, b0, nb, Ci, Co, M);
    if (launches) ++*launches;
  }
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Adjoint of the mixing (Section "Backward Pass"):
//   GX[b,i,m] = sum_o GY[b,o,m] conj(W[i,o,m]);  GW[i,o,m] = sum_b conj(X[b,i,m]) GY[b,o,m]
// One thread per (i, m) walks o, so W is read once and GW written once.
// ---------------------------------------------------------------------------
template <int BT>
__global__ void __launch_bounds__(256) mix_adjoint_kernel(const float2* __restrict__ GY,
                                                         const float2* __restrict__ X,
                                                         const float2* __restrict__ W, float2* __restrict__ GX,
                                                         float2* __restrict__ GW, int b0, int nb, int B, int Ci,
                                                         int Co, long long M, int write_gw) {
  const long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int i = blockIdx.y;
  if (m >= M) return;
  float2 gx[BT];
#pragma unroll
  for (int b = 0; b < BT; ++b) gx[b] = make_float2(0.f, 0.f);
  for (int o = 0; o < Co; ++o) {
    const float2 w = W[((long long)i * Co + o) * M + m];
    if (GX != nullptr) {
#pragma unroll
      for (int b = 0; b < BT; ++b) {
        if (b < nb) {
          const float2 g = GY[((long long)(b0 + b) * Co + o) * M + m];
          // g * conj(w)
          gx[b].x = fmaf(g.x, w.x, gx[b].x);
          gx[b].x = fmaf(g.y, w.y, gx[b].x);
          gx[b].y = fmaf(g.y, w.x, gx[b].y);
          gx[b].y = fmaf(-g.x, w.y, gx[b].y);
        }
      }
    }
    if (write_gw) {
      float2 acc = make_float2(0.f, 0.f);
      for (int b = 0; b < B; ++b) {
        const float2 g = GY[((long long)b * Co + o) * M + m];
        const float2 x = X[((long long)b * Ci + i) * M + m];
        // conj(x) * g
        acc.x = fmaf(x.x, g.x, acc.x);
        acc.x = fmaf(x.y, g.y, acc.x);
        acc.y = fmaf(x.x, g.y, acc.y);
        acc.y = fmaf(-x.y, g.x, acc.y);
      }
      GW[((long long)i * Co + o) * M + m] = acc;
    }
  }
  if (GX != nullptr) {
#pragma unroll
    for (int b = 0; b < BT; ++b)
      if (b < nb) GX[((long long)(b0 + b) * Ci + i) * M + m] = gx[b];
  }
}

cudaError_t launch_mix_adjoint(const float2* GY, const float2* X, const float2* W, float2* GX, float2* GW,
                               int B, int Ci, int Co, long long M, cudaStream_t st, long long* launches) {
  constexpr int BT = 4;
  dim3 grid((unsigned)((M + 255) / 256), (unsigned)Ci);
  for (int b0 = 0; b0 < B; b0 += BT) {
    const int nb = (B - b0 < BT) ? (B - b0) : BT;
    const int write_gw = (GW != nullptr && b0 == 0) ? 1 : 0;
    if (GX == nullptr && !write_gw) break;
    mix_adjoint_kernel<BT><<<grid, 256, 0, st>>>(GY, X, W, GX, GW, b0, nb, B, Ci, Co, M, write_gw);
    if (launches) ++*launches;
    if (GX == nullptr) break;
  }
  return cudaGetLastError();
}

}  // namespace dtst
