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
  pdl_trigger();
  extern __shared__ float2 Es[];
  const int slab = blockIdx.y;
  if (p.basis_in_smem) {
    const int total = p.R * p.Q;
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
      const int r = e / p.Q, q = e % p.Q;
      Es[r * p.es_sr + q * p.es_sq] = dimop_entry(p, r, q, slab);
    }
    __syncthreads();
  }
  pdl_wait();
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
      const float2 e = p.basis_in_smem ? Es[r * p.es_sr + q * p.es_sq] : dimop_entry(p, r, q, slab);
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
  // Layout of the basis in shared memory.  With a wide inner extent the lanes of a warp share their output row r
  // and read one entry (a broadcast): rows of Q entries.  With a narrow one (the contiguous dimension itself:
  // inner = 1) neighbouring lanes own neighbouring rows and walk q together: stored [q][r] with an odd row count,
  // their reads fall into different banks (stored [r][q] they were Q entries apart - a 32-way conflict for every
  // multiple of 32, which made this kernel 20 times slower than it had to be).
  const int Rp = op.R | 1;
  const bool narrow = op.inner < 32;
  op.es_sr = narrow ? 1 : op.Q;
  op.es_sq = narrow ? Rp : 1;
  const size_t smem = (size_t)(narrow ? Rp : op.R) * op.Q * sizeof(float2);
  op.basis_in_smem = smem <= 160 * 1024 ? 1 : 0;
  const size_t dyn = op.basis_in_smem ? smem : 0;
  const long long total = op.outer * op.R * op.inner;
  if (total <= 0) return cudaSuccess;
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)num_sms() * 8;
  if (blocks > cap) blocks = cap;
  dim3 grid((unsigned)blocks, (unsigned)op.slabs);
  cudaError_t err = cudaSuccess;
#define DTST_LAUNCH(IR, OR)                                                                         \
  do {                                                                                              \
    if (dyn > 48 * 1024)                                                                            \
      err = cudaFuncSetAttribute(apply_dim_kernel<IR, OR>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                 (int)dyn);                                                         \
    if (err == cudaSuccess) err = launch_pdl(apply_dim_kernel<IR, OR>, grid, dim3(256), dyn, st, op, in, out); \
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
  pdl_trigger();
  pdl_wait();
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
  if (blocks > (long long)num_sms() * 8) blocks = (long long)num_sms() * 8;
  return launch_pdl(reduce_partials_kernel, dim3((unsigned)blocks), dim3(256), 0, st, partial, out, n, P);
}

// ---------------------------------------------------------------------------
// Per-mode channel mixing (Eq. 12): Y[b,o,m] = sum_i X[b,i,m] W[i,o,m].
// W-streaming: about B flops per byte of W, so the roof is HBM.  One thread per (o, m); W is read once
// per chunk of NB batch entries (NB is a compile-time 1..4: a run-time batch predicate inside the channel
// loop cost a third of the bandwidth).  Full occupancy (about 32 registers) is what keeps enough loads in
// flight; unrolling or 16-byte accesses measured slower.
// ---------------------------------------------------------------------------
template <int NB>
__global__ void __launch_bounds__(256) mix_kernel(const float2* __restrict__ X, const float2* __restrict__ W,
                                                 float2* __restrict__ Y, int b0, int Ci, int Co, long long M) {
  pdl_trigger();
  pdl_wait();
  const long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int o = blockIdx.y;
  if (m >= M) return;
  float2 acc[NB];
#pragma unroll
  for (int b = 0; b < NB; ++b) acc[b] = make_float2(0.f, 0.f);
  for (int i = 0; i < Ci; ++i) {
    const float2 w = __ldcs(W + ((long long)i * Co + o) * M + m);   // streamed once: do not displace the spectra in L2
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      const float2 x = __ldg(X + ((long long)(b0 + b) * Ci + i) * M + m);
      acc[b].x = fmaf(x.x, w.x, acc[b].x);
      acc[b].x = fmaf(-x.y, w.y, acc[b].x);
      acc[b].y = fmaf(x.x, w.y, acc[b].y);
      acc[b].y = fmaf(x.y, w.x, acc[b].y);
    }
  }
#pragma unroll
  for (int b = 0; b < NB; ++b) Y[((long long)(b0 + b) * Co + o) * M + m] = acc[b];
}

// The same sums for SMALL spectra (a 2-D layer with 12 modes has 288 of them): one thread per (m, o) and four batch
// entries per launch leaves most of the GPU idle and every thread waiting for one load after the other (16 x 32
// channels x 288 modes: four launches of 52 us for 3.6 MB).  Here one thread per (m, o, b), the channel loop
// unrolled so that 16 loads are in flight per thread; W (a few MB) is re-read from L2 by every batch entry.  The
// terms are added in the same order: the same bits as mix_kernel.
__global__ void __launch_bounds__(128) mix_small_kernel(const float2* __restrict__ X, const float2* __restrict__ W,
                                                       float2* __restrict__ Y, int Ci, int Co, long long M) {
  pdl_trigger();
  pdl_wait();
  const long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int o = blockIdx.y, b = blockIdx.z;
  if (m >= M) return;
  const float2* wp = W + (long long)o * M + m;
  const float2* xp = X + (long long)b * Ci * M + m;
  float2 acc = make_float2(0.f, 0.f);
#pragma unroll 8
  for (int i = 0; i < Ci; ++i) {
    const float2 w = __ldg(wp + (long long)i * Co * M);
    const float2 x = __ldg(xp + (long long)i * M);
    acc.x = fmaf(x.x, w.x, acc.x);
    acc.x = fmaf(-x.y, w.y, acc.x);
    acc.y = fmaf(x.x, w.y, acc.y);
    acc.y = fmaf(x.y, w.x, acc.y);
  }
  Y[((long long)b * Co + o) * M + m] = acc;
}

// small: few enough (m, o) pairs that mix_kernel cannot fill the GPU, and weights that stay in L2
static bool mix_is_small(int B, int Ci, int Co, long long M) {
  return M * Co < (long long)num_sms() * 2048 && (long long)Ci * Co * M * 8 <= (48ll << 20) && B <= 65535 && Co <= 65535;
}

cudaError_t launch_mix(const float2* X, const float2* W, float2* Y, int B, int Ci, int Co, long long M,
                       cudaStream_t st, long long* launches) {
  if (mix_is_small(B, Ci, Co, M)) {
    (void)launch_pdl(mix_small_kernel, dim3((unsigned)((M + 127) / 128), (unsigned)Co, (unsigned)B), dim3(128), 0, st, X, W, Y,
                     Ci, Co, M);
    if (launches) ++*launches;
    return cudaGetLastError();
  }
  dim3 grid((unsigned)((M + 255) / 256), (unsigned)Co);
  cudaError_t e = cudaSuccess;
  for (int b0 = 0; b0 < B; b0 += 4) {
    const int nb = (B - b0 < 4) ? (B - b0) : 4;
    switch (nb) {
      case 1: e = launch_pdl(mix_kernel<1>, grid, dim3(256), 0, st, X, W, Y, b0, Ci, Co, M); break;
      case 2: e = launch_pdl(mix_kernel<2>, grid, dim3(256), 0, st, X, W, Y, b0, Ci, Co, M); break;
      case 3: e = launch_pdl(mix_kernel<3>, grid, dim3(256), 0, st, X, W, Y, b0, Ci, Co, M); break;
      default: e = launch_pdl(mix_kernel<4>, grid, dim3(256), 0, st, X, W, Y, b0, Ci, Co, M); break;
    }
    if (e != cudaSuccess) return e;
    if (launches) ++*launches;
  }
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Adjoint of the mixing (Section "Backward Pass"):
//   GX[b,i,m] = sum_o GY[b,o,m] conj(W[i,o,m]);  GW[i,o,m] = sum_b conj(X[b,i,m]) GY[b,o,m]
// One thread per (i, m) walks o, so W is read once and GW written once.  NB = batch entries of this
// launch (compile time); ALLB = the launch covers the whole batch, so GW needs no second pass over b.
// ---------------------------------------------------------------------------
template <int NB, bool ALLB, bool WANT_GX, bool WANT_GW>
__global__ void __launch_bounds__(256) mix_adjoint_kernel(const float2* __restrict__ GY,
                                                         const float2* __restrict__ X,
                                                         const float2* __restrict__ W, float2* __restrict__ GX,
                                                         float2* __restrict__ GW, int b0, int B, int Ci, int Co,
                                                         long long M) {
  pdl_trigger();
  pdl_wait();
  const long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int i = blockIdx.y;
  if (m >= M) return;
  float2 gx[NB], xr[NB];
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    gx[b] = make_float2(0.f, 0.f);
    xr[b] = (WANT_GW && ALLB) ? __ldg(X + ((long long)(b0 + b) * Ci + i) * M + m) : make_float2(0.f, 0.f);
  }
  for (int o = 0; o < Co; ++o) {
    const float2 w = __ldcs(W + ((long long)i * Co + o) * M + m);   // streamed once: do not displace the spectra in L2
    float2 g[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) g[b] = __ldg(GY + ((long long)(b0 + b) * Co + o) * M + m);
    if (WANT_GX) {
#pragma unroll
      for (int b = 0; b < NB; ++b) {   // g * conj(w)
        gx[b].x = fmaf(g[b].x, w.x, gx[b].x);
        gx[b].x = fmaf(g[b].y, w.y, gx[b].x);
        gx[b].y = fmaf(g[b].y, w.x, gx[b].y);
        gx[b].y = fmaf(-g[b].x, w.y, gx[b].y);
      }
    }
    if (WANT_GW) {
      float2 acc = make_float2(0.f, 0.f);
      if (ALLB) {
#pragma unroll
        for (int b = 0; b < NB; ++b) {   // conj(x) * g
          acc.x = fmaf(xr[b].x, g[b].x, acc.x);
          acc.x = fmaf(xr[b].y, g[b].y, acc.x);
          acc.y = fmaf(xr[b].x, g[b].y, acc.y);
          acc.y = fmaf(-xr[b].y, g[b].x, acc.y);
        }
      } else {
        for (int b = 0; b < B; ++b) {
          const float2 gg = __ldg(GY + ((long long)b * Co + o) * M + m);
          const float2 xx = __ldg(X + ((long long)b * Ci + i) * M + m);
          acc.x = fmaf(xx.x, gg.x, acc.x);
          acc.x = fmaf(xx.y, gg.y, acc.x);
          acc.y = fmaf(xx.x, gg.y, acc.y);
          acc.y = fmaf(-xx.y, gg.x, acc.y);
        }
      }
      __stcs(GW + ((long long)i * Co + o) * M + m, acc);
    }
  }
  if (WANT_GX) {
#pragma unroll
    for (int b = 0; b < NB; ++b) GX[((long long)(b0 + b) * Ci + i) * M + m] = gx[b];
  }
}

// The adjoint for small spectra, as mix_small_kernel: GX with one thread per (m, i, b) walking o, GW with one thread per
// (m, o, i) walking b; the same order of terms, the same bits as mix_adjoint_kernel.
__global__ void __launch_bounds__(128) mix_adjoint_gx_small_kernel(const float2* __restrict__ GY, const float2* __restrict__ W,
                                                                  float2* __restrict__ GX, int Ci, int Co, long long M) {
  pdl_trigger();
  pdl_wait();
  const long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int i = blockIdx.y, b = blockIdx.z;
  if (m >= M) return;
  const float2* wp = W + (long long)i * Co * M + m;
  const float2* gp = GY + (long long)b * Co * M + m;
  float2 gx = make_float2(0.f, 0.f);
#pragma unroll 8
  for (int o = 0; o < Co; ++o) {   // g * conj(w)
    const float2 w = __ldg(wp + (long long)o * M);
    const float2 g = __ldg(gp + (long long)o * M);
    gx.x = fmaf(g.x, w.x, gx.x);
    gx.x = fmaf(g.y, w.y, gx.x);
    gx.y = fmaf(g.y, w.x, gx.y);
    gx.y = fmaf(-g.x, w.y, gx.y);
  }
  GX[((long long)b * Ci + i) * M + m] = gx;
}

__global__ void __launch_bounds__(128) mix_adjoint_gw_small_kernel(const float2* __restrict__ GY, const float2* __restrict__ X,
                                                                  float2* __restrict__ GW, int B, int Ci, int Co, long long M) {
  pdl_trigger();
  pdl_wait();
  const long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int o = blockIdx.y, i = blockIdx.z;
  if (m >= M) return;
  const float2* gp = GY + (long long)o * M + m;
  const float2* xp = X + (long long)i * M + m;
  float2 acc = make_float2(0.f, 0.f);
#pragma unroll 4
  for (int b = 0; b < B; ++b) {    // conj(x) * g
    const float2 g = __ldg(gp + (long long)b * Co * M);
    const float2 x = __ldg(xp + (long long)b * Ci * M);
    acc.x = fmaf(x.x, g.x, acc.x);
    acc.x = fmaf(x.y, g.y, acc.x);
    acc.y = fmaf(x.x, g.y, acc.y);
    acc.y = fmaf(-x.y, g.x, acc.y);
  }
  GW[((long long)i * Co + o) * M + m] = acc;
}

template <int NB>
void launch_mix_adjoint_nb(dim3 grid, cudaStream_t st, const float2* GY, const float2* X, const float2* W,
                           float2* GX, float2* GW, int b0, int B, int Ci, int Co, long long M, bool want_gw) {
  const bool allb = (b0 == 0 && NB == B);
  const bool gx = GX != nullptr;
#define DTST_MA(AL, WX, WW) \
  (void)launch_pdl(mix_adjoint_kernel<NB, AL, WX, WW>, grid, dim3(256), 0, st, GY, X, W, GX, GW, b0, B, Ci, Co, M)
  if (gx && want_gw) { if (allb) DTST_MA(true, true, true); else DTST_MA(false, true, true); }
  else if (gx) DTST_MA(false, true, false);
  else if (want_gw) { if (allb) DTST_MA(true, false, true); else DTST_MA(false, false, true); }
#undef DTST_MA
}

cudaError_t launch_mix_adjoint(const float2* GY, const float2* X, const float2* W, float2* GX, float2* GW,
                               int B, int Ci, int Co, long long M, cudaStream_t st, long long* launches) {
  // (up to four batch entries mix_adjoint_kernel needs ONE launch that keeps x in registers and reads GY once per
  // input channel: measured faster than the pair below, 16.7 against 22.9 us on 2 x 16 channels x 6912 modes)
  if (mix_is_small(B, Ci, Co, M) && Ci <= 65535 && B > 4) {
    const unsigned mb = (unsigned)((M + 127) / 128);
    if (GX != nullptr) {
      (void)launch_pdl(mix_adjoint_gx_small_kernel, dim3(mb, (unsigned)Ci, (unsigned)B), dim3(128), 0, st, GY, W, GX, Ci, Co, M);
      if (launches) ++*launches;
    }
    if (GW != nullptr) {
      (void)launch_pdl(mix_adjoint_gw_small_kernel, dim3(mb, (unsigned)Co, (unsigned)Ci), dim3(128), 0, st, GY, X, GW, B, Ci, Co,
                       M);
      if (launches) ++*launches;
    }
    return cudaGetLastError();
  }
  dim3 grid((unsigned)((M + 255) / 256), (unsigned)Ci);
  for (int b0 = 0; b0 < B; b0 += 4) {
    const int nb = (B - b0 < 4) ? (B - b0) : 4;
    const bool want_gw = (GW != nullptr && b0 == 0);
    if (GX == nullptr && !want_gw) break;
    switch (nb) {
      case 1: launch_mix_adjoint_nb<1>(grid, st, GY, X, W, GX, GW, b0, B, Ci, Co, M, want_gw); break;
      case 2: launch_mix_adjoint_nb<2>(grid, st, GY, X, W, GX, GW, b0, B, Ci, Co, M, want_gw); break;
      case 3: launch_mix_adjoint_nb<3>(grid, st, GY, X, W, GX, GW, b0, B, Ci, Co, M, want_gw); break;
      default: launch_mix_adjoint_nb<4>(grid, st, GY, X, W, GX, GW, b0, B, Ci, Co, M, want_gw); break;
    }
    if (launches) ++*launches;
    if (GX == nullptr) break;
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Mixing on a contiguous chunk [m0, m0 + cnt) of the flattened modes: the equal partition of the
// modes among ranks (Eq. 12 applied by rank p to its S_p).  The spectra are the full tensors
// [B][C][M] every rank holds after the reduction; the weight tensors are the rank's shards
// [C_in][C_out][cnt]; outputs are contiguous chunks [B][C][cnt], ready to be gathered.
// Not on the single-GPU hot path: plain one-thread-per-output kernels.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) mix_modes_kernel(const float2* __restrict__ X, const float2* __restrict__ W,
                                                       float2* __restrict__ Y, int Ci, int Co, long long M,
                                                       long long m0, long long cnt) {
  pdl_trigger();
  pdl_wait();
  const long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int o = blockIdx.y, b = blockIdx.z;
  if (m >= cnt) return;
  float2 acc = make_float2(0.f, 0.f);
  for (int i = 0; i < Ci; ++i) {
    const float2 w = __ldg(W + ((long long)i * Co + o) * cnt + m);
    const float2 x = __ldg(X + ((long long)b * Ci + i) * M + m0 + m);
    acc.x = fmaf(x.x, w.x, acc.x);
    acc.x = fmaf(-x.y, w.y, acc.x);
    acc.y = fmaf(x.x, w.y, acc.y);
    acc.y = fmaf(x.y, w.x, acc.y);
  }
  Y[((long long)b * Co + o) * cnt + m] = acc;
}

// G_X[b][i][m] = sum_o G_Y[b][o][m0 + m] conj(W[i][o][m])
__global__ void __launch_bounds__(256) mix_adjoint_gx_modes_kernel(const float2* __restrict__ GY,
                                                                  const float2* __restrict__ W,
                                                                  float2* __restrict__ GX, int Ci, int Co,
                                                                  long long M, long long m0, long long cnt) {
  pdl_trigger();
  pdl_wait();
  const long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int i = blockIdx.y, b = blockIdx.z;
  if (m >= cnt) return;
  float2 acc = make_float2(0.f, 0.f);
  for (int o = 0; o < Co; ++o) {
    const float2 w = __ldg(W + ((long long)i * Co + o) * cnt + m);
    const float2 g = __ldg(GY + ((long long)b * Co + o) * M + m0 + m);
    acc.x = fmaf(g.x, w.x, acc.x);
    acc.x = fmaf(g.y, w.y, acc.x);
    acc.y = fmaf(g.y, w.x, acc.y);
    acc.y = fmaf(-g.x, w.y, acc.y);
  }
  GX[((long long)b * Ci + i) * cnt + m] = acc;
}

// G_W[i][o][m] = sum_b conj(X[b][i][m0 + m]) G_Y[b][o][m0 + m]
__global__ void __launch_bounds__(256) mix_adjoint_gw_modes_kernel(const float2* __restrict__ GY,
                                                                  const float2* __restrict__ X,
                                                                  float2* __restrict__ GW, int B, int Ci, int Co,
                                                                  long long M, long long m0, long long cnt) {
  pdl_trigger();
  pdl_wait();
  const long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int o = blockIdx.y, i = blockIdx.z;
  if (m >= cnt) return;
  float2 acc = make_float2(0.f, 0.f);
  for (int b = 0; b < B; ++b) {
    const float2 x = __ldg(X + ((long long)b * Ci + i) * M + m0 + m);
    const float2 g = __ldg(GY + ((long long)b * Co + o) * M + m0 + m);
    acc.x = fmaf(x.x, g.x, acc.x);
    acc.x = fmaf(x.y, g.y, acc.x);
    acc.y = fmaf(x.x, g.y, acc.y);
    acc.y = fmaf(-x.y, g.x, acc.y);
  }
  GW[((long long)i * Co + o) * cnt + m] = acc;
}

cudaError_t launch_mix_modes(const float2* X, const float2* W, float2* Y, int B, int Ci, int Co, long long M,
                             long long m0, long long cnt, cudaStream_t st, long long* launches) {
  if (cnt <= 0 || B <= 0) return cudaSuccess;
  dim3 grid((unsigned)((cnt + 255) / 256), (unsigned)Co, (unsigned)B);
  (void)launch_pdl(mix_modes_kernel, grid, dim3(256), 0, st, X, W, Y, Ci, Co, M, m0, cnt);
  if (launches) ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_mix_adjoint_modes(const float2* GY, const float2* X, const float2* W, float2* GX, float2* GW,
                                     int B, int Ci, int Co, long long M, long long m0, long long cnt,
                                     cudaStream_t st, long long* launches) {
  if (cnt <= 0 || B <= 0) return cudaSuccess;
  if (GX != nullptr) {
    dim3 grid((unsigned)((cnt + 255) / 256), (unsigned)Ci, (unsigned)B);
    (void)launch_pdl(mix_adjoint_gx_modes_kernel, grid, dim3(256), 0, st, GY, W, GX, Ci, Co, M, m0, cnt);
    if (launches) ++*launches;
  }
  if (GW != nullptr) {
    dim3 grid((unsigned)((cnt + 255) / 256), (unsigned)Co, (unsigned)Ci);
    (void)launch_pdl(mix_adjoint_gw_modes_kernel, grid, dim3(256), 0, st, GY, X, GW, B, Ci, Co, M, m0, cnt);
    if (launches) ++*launches;
  }
  return cudaGetLastError();
}

}  // namespace dtst
