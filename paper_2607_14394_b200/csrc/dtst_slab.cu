// Two-sided middle dimension with a global phase offset and/or virtual shards (Eq. 6, 7, 18).
//
// A slab [p*nl, (p+1)*nl) of the dimension contracts with the basis B[s][off + n]: the global twiddles
// restricted to the slab's columns.  One thread owns one complex position of the reduced tensor and walks the
// slabs in ascending order: it forms slab p's partial spectrum in registers (all 2k retained frequencies) and
// adds it to the running total - the on-device reduction of the partial spectra in fixed order, without a
// round trip of the P partials through HBM.  The mirrored folding of dtst_mid.cu does not apply here (a slab
// does not contain its mirror image), so each input costs 2k complex multiply-adds; the tensor is the
// already reduced one, so this stays a small share of a step.  The basis table E[n][r] is generated on the
// device into shared memory once per persistent CTA.
#include "dtst_common.cuh"

namespace dtst {
namespace {

constexpr int kSlabThreads = 128;

template <int K>
__device__ __forceinline__ void build_slab_table(float2* tab, int Nl, int N, int off, int sign) {
  for (int e = threadIdx.x; e < Nl * 2 * K; e += blockDim.x) {
    const int n = e / (2 * K), r = e % (2 * K);
    tab[e] = twiddle(mode_at(r, K, N, 1), (long long)off + n, N, sign);
  }
}

// in[outer][Nl][inner] -> out[outer][2K][inner]
template <int K>
__global__ void __launch_bounds__(kSlabThreads) slab_contract_kernel(const float2* __restrict__ in,
                                                                     float2* __restrict__ out, long long outer,
                                                                     long long inner, int Nl, int N, int off, int P) {
  extern __shared__ float2 slab_tab[];
  build_slab_table<K>(slab_tab, Nl, N, off, -1);
  __syncthreads();
  const long long total = outer * inner;
  const int nl = Nl / P;
  for (long long p0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; p0 < total;
       p0 += (long long)gridDim.x * blockDim.x) {
    const long long o = p0 / inner, i = p0 % inner;
    const float2* src = in + o * Nl * inner + i;
    float2 tot[2 * K];
#pragma unroll
    for (int r = 0; r < 2 * K; ++r) tot[r] = make_float2(0.f, 0.f);
    for (int slab = 0; slab < P; ++slab) {
      float2 acc[2 * K];
#pragma unroll
      for (int r = 0; r < 2 * K; ++r) acc[r] = make_float2(0.f, 0.f);
      const int n0 = slab * nl;
      for (int q0 = 0; q0 < nl; q0 += 4) {
        float2 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          v[u] = (q0 + u < nl) ? __ldg(src + (long long)(n0 + q0 + u) * inner) : make_float2(0.f, 0.f);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (q0 + u >= nl) break;
          const float2* row = slab_tab + (size_t)(n0 + q0 + u) * (2 * K);
#pragma unroll
          for (int r = 0; r < 2 * K; ++r) {
            const float2 e = row[r];
            acc[r].x = fmaf(e.x, v[u].x, acc[r].x);
            acc[r].x = fmaf(-e.y, v[u].y, acc[r].x);
            acc[r].y = fmaf(e.x, v[u].y, acc[r].y);
            acc[r].y = fmaf(e.y, v[u].x, acc[r].y);
          }
        }
      }
      // Eq. 7: add this slab's partial spectrum to the total, slabs in ascending order
#pragma unroll
      for (int r = 0; r < 2 * K; ++r) {
        tot[r].x += acc[r].x;
        tot[r].y += acc[r].y;
      }
    }
    float2* dst = out + o * (2 * K) * inner + i;
#pragma unroll
    for (int r = 0; r < 2 * K; ++r) dst[(long long)r * inner] = tot[r];
  }
}

// in[outer][2K][inner] -> out[outer][Nl][inner], slab by slab with the same offsets (no reduction needed)
template <int K>
__global__ void __launch_bounds__(kSlabThreads) slab_expand_kernel(const float2* __restrict__ in,
                                                                   float2* __restrict__ out, long long outer,
                                                                   long long inner, int Nl, int N, int off, int P) {
  extern __shared__ float2 slab_tab[];
  build_slab_table<K>(slab_tab, Nl, N, off, +1);
  __syncthreads();
  const long long total = outer * inner;
  const int nl = Nl / P;
  for (long long p0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; p0 < total;
       p0 += (long long)gridDim.x * blockDim.x) {
    const long long o = p0 / inner, i = p0 % inner;
    const float2* src = in + o * (2 * K) * inner + i;
    float2 v[2 * K];
#pragma unroll
    for (int r = 0; r < 2 * K; ++r) v[r] = __ldg(src + (long long)r * inner);
    float2* dst = out + o * Nl * inner + i;
    for (int slab = 0; slab < P; ++slab) {
      for (int q = 0; q < nl; ++q) {
        const int n = slab * nl + q;
        const float2* row = slab_tab + (size_t)n * (2 * K);
        float ar = 0.f, ai = 0.f, br = 0.f, bi = 0.f;   // two chains for ILP
#pragma unroll
        for (int r = 0; r < 2 * K; r += 2) {
          const float2 e0 = row[r], e1 = row[r + 1];
          ar = fmaf(e0.x, v[r].x, ar);
          ar = fmaf(-e0.y, v[r].y, ar);
          ai = fmaf(e0.x, v[r].y, ai);
          ai = fmaf(e0.y, v[r].x, ai);
          br = fmaf(e1.x, v[r + 1].x, br);
          br = fmaf(-e1.y, v[r + 1].y, br);
          bi = fmaf(e1.x, v[r + 1].y, bi);
          bi = fmaf(e1.y, v[r + 1].x, bi);
        }
        dst[(long long)n * inner] = make_float2(ar + br, ai + bi);
      }
    }
  }
}

template <int K>
cudaError_t launch_slab_t(bool forward, const float2* in, float2* out, long long outer, long long inner, int Nl, int N,
                          int off, int P, cudaStream_t st) {
  const size_t smem = (size_t)Nl * 2 * K * sizeof(float2);
  const long long total = outer * inner;
  auto launch = [&](auto kern) -> cudaError_t {
    cudaError_t e = cudaSuccess;
    if (smem > 48 * 1024) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kSlabThreads, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    const long long want = (total + kSlabThreads - 1) / kSlabThreads;
    const long long cap = (long long)kNumSMs * per_sm;
    kern<<<(unsigned)(want < cap ? want : cap), kSlabThreads, smem, st>>>(in, out, outer, inner, Nl, N, off, P);
    return cudaGetLastError();
  };
  return forward ? launch(slab_contract_kernel<K>) : launch(slab_expand_kernel<K>);
}

}  // namespace

bool slab_supported(int Nl, int K) {
  if (!(K == 4 || K == 8 || K == 12 || K == 16)) return false;
  return (size_t)Nl * 2 * K * sizeof(float2) <= 200 * 1024;
}

cudaError_t launch_slab(bool forward, int K, const float2* in, float2* out, long long outer, long long inner, int Nl,
                        int N, int off, int P, cudaStream_t st) {
  if (outer * inner <= 0) return cudaSuccess;
  switch (K) {
    case 4: return launch_slab_t<4>(forward, in, out, outer, inner, Nl, N, off, P, st);
    case 8: return launch_slab_t<8>(forward, in, out, outer, inner, Nl, N, off, P, st);
    case 12: return launch_slab_t<12>(forward, in, out, outer, inner, Nl, N, off, P, st);
    case 16: return launch_slab_t<16>(forward, in, out, outer, inner, Nl, N, off, P, st);
    default: return cudaErrorNotSupported;
  }
}

}  // namespace dtst
