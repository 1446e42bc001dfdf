// Contraction / expansion along a two-sided middle dimension on the already reduced
// tensor [outer][Q][inner] (inner contiguous, complex64).
//
// One thread owns PT consecutive-in-memory complex positions and keeps ALL of their
// retained-frequency sums in registers, so every input element is loaded exactly once and
// every output written exactly once; consecutive lanes own consecutive positions, so all
// global accesses are coalesced 8-byte-per-lane transactions.  The basis is generated on
// the device into shared memory once per (persistent) CTA.  With the half-sample phase
// factored out (Eq. 18 with zero offset),
//     Z_{+-g} = e^{+-i psi_g/2} (A_g -+ i B_g),
//     A_g = sum_{q<Q/2} (z_q + z_{Q-1-q}) cos(psi_g (q + 1/2)),
//     B_g = sum_{q<Q/2} (z_q - z_{Q-1-q}) sin(psi_g (q + 1/2)),
// one real-coefficient FMA pair serves both +g and -g and both mirrored inputs: a fourfold
// cut of the multiply count against the plain complex matrix product.
#include <type_traits>

#include "dtst_common.cuh"

namespace dtst {
namespace {

constexpr int kMidThreads = 128;

// table[q][e]: e in [0..K] -> cos(psi_e (q+1/2)); e in [K+1..2K] -> sin(psi_{e-K} (q+1/2)); row stride TS
template <int K>
struct MidTab {
  static constexpr int TS = ((2 * K + 1 + 3) / 4) * 4;
};

template <int K>
__device__ __forceinline__ void build_mid_table(float* tab, float2* rho, int N, float scale) {
  constexpr int TS = MidTab<K>::TS;
  const int half = N / 2;
  for (int e = threadIdx.x; e < half * TS; e += blockDim.x) {
    const int q = e / TS, c = e % TS;
    float v = 0.f;
    if (c <= 2 * K) {
      const int g = c <= K ? c : c - K;
      double sn, cs;
      // psi_g (q + 1/2) = pi g (2q+1) / N, phase reduced exactly in integers
      sincospi((double)(((long long)g * (2 * q + 1)) % (2ll * N)) / (double)N, &sn, &cs);
      v = c <= K ? (float)cs : (float)sn;
    }
    tab[e] = v;
  }
  for (int g = threadIdx.x; g <= K; g += blockDim.x) {
    double sn, cs;
    sincospi((double)g / (double)N, &sn, &cs);   // e^{i psi_g / 2}
    rho[g] = make_float2((float)cs * scale, (float)sn * scale);
  }
}

// ------------------------------------------------------------------------------------------
// forward: in[outer][N][inner] -> out[outer][2K][inner]
// ------------------------------------------------------------------------------------------
template <int K, int PT, bool VEC>
__global__ void __launch_bounds__(kMidThreads) mid_contract_kernel(const float2* __restrict__ in,
                                                                   float2* __restrict__ out, long long outer,
                                                                   long long inner, int N, float scale) {
  constexpr int TS = MidTab<K>::TS;
  pdl_trigger();
  extern __shared__ float smem_mid[];
  float* tab = smem_mid;
  float2* rho = reinterpret_cast<float2*>(tab + (size_t)(N / 2) * TS);
  build_mid_table<K>(tab, rho, N, scale);
  __syncthreads();
  pdl_wait();

  const long long total = outer * inner;
  const long long per_cta = (long long)kMidThreads * PT;
  const long long tiles = (total + per_cta - 1) / per_cta;
  const int half = N / 2;
  for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    // VEC: the PT = 2 positions of a thread are adjacent in memory (one 16-byte access); otherwise they
    // are kMidThreads apart (inner odd, 8-byte accesses)
    long long ibase[PT], obase[PT];
    bool ok[PT];
#pragma unroll
    for (int t = 0; t < PT; ++t) {
      const long long p = VEC ? tile * per_cta + (long long)threadIdx.x * PT + t
                              : tile * per_cta + (long long)t * kMidThreads + threadIdx.x;
      ok[t] = p < total;
      const long long pc = ok[t] ? p : 0;
      const long long o = pc / inner, i = pc % inner;
      ibase[t] = o * N * inner + i;
      obase[t] = o * (2 * K) * inner + i;
    }
    float2 A[PT][K + 1], B[PT][K + 1];
#pragma unroll
    for (int t = 0; t < PT; ++t)
#pragma unroll
      for (int g = 0; g <= K; ++g) A[t][g] = B[t][g] = make_float2(0.f, 0.f);

    // Software pipeline over blocks of U mirrored row pairs: the loads of block b+1 are in flight while
    // block b is accumulated (a plain unrolled loop leaves only a couple of loads outstanding per warp,
    // which makes this stage latency-bound), and rows a few blocks ahead are pulled into L2.
    constexpr int U = 4;
    constexpr int NV = VEC ? 1 : PT;
    using Vec = typename std::conditional<VEC, float4, float2>::type;
    Vec nxa[U][NV], nxb[U][NV];
    auto issue = [&](int q0) {
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int q = q0 + u;
        if (q < half) {
#pragma unroll
          for (int t = 0; t < NV; ++t) {
            nxa[u][t] = __ldg(reinterpret_cast<const Vec*>(in + ibase[t] + (long long)q * inner));
            nxb[u][t] = __ldg(reinterpret_cast<const Vec*>(in + ibase[t] + (long long)(N - 1 - q) * inner));
          }
        }
      }
    };
    issue(0);
    for (int q0 = 0; q0 < half; q0 += U) {
      Vec cua[U][NV], cub[U][NV];
#pragma unroll
      for (int u = 0; u < U; ++u)
#pragma unroll
        for (int t = 0; t < NV; ++t) {
          cua[u][t] = nxa[u][t];
          cub[u][t] = nxb[u][t];
        }
      issue(q0 + U);
      if (q0 + 4 * U < half) {
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
          for (int t = 0; t < NV; ++t) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(in + ibase[t] + (long long)(q0 + 4 * U + u) * inner));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(in + ibase[t] + (long long)(N - 1 - q0 - 4 * U - u) * inner));
          }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int q = q0 + u;
        if (q >= half) break;
        float2 p[PT], m[PT];
        if constexpr (VEC) {
          const float4 a = cua[u][0], b = cub[u][0];
          p[0] = make_float2(a.x + b.x, a.y + b.y);
          m[0] = make_float2(a.x - b.x, a.y - b.y);
          p[PT - 1] = make_float2(a.z + b.z, a.w + b.w);
          m[PT - 1] = make_float2(a.z - b.z, a.w - b.w);
        } else {
#pragma unroll
          for (int t = 0; t < PT; ++t) {
            const float2 a = cua[u][t], b = cub[u][t];
            p[t] = make_float2(a.x + b.x, a.y + b.y);
            m[t] = make_float2(a.x - b.x, a.y - b.y);
          }
        }
        const float* row = tab + q * TS;
#pragma unroll
        for (int g = 0; g <= K; ++g) {
          const float c = row[g];
#pragma unroll
          for (int t = 0; t < PT; ++t) {
            A[t][g].x = fmaf(p[t].x, c, A[t][g].x);
            A[t][g].y = fmaf(p[t].y, c, A[t][g].y);
          }
        }
#pragma unroll
        for (int g = 1; g <= K; ++g) {
          const float s = row[K + g];
#pragma unroll
          for (int t = 0; t < PT; ++t) {
            B[t][g].x = fmaf(m[t].x, s, B[t][g].x);
            B[t][g].y = fmaf(m[t].y, s, B[t][g].y);
          }
        }
      }
    }
    // Z_{+g} = rho_g (A - iB), Z_{-g} = conj(rho_g) (A + iB); positions [0..K-1] hold +g, [K..2K-1] hold -(2K-r)
#pragma unroll
    for (int g = 0; g <= K; ++g) {
      const float2 r = rho[g];
      float2 zp[PT], zm[PT];
#pragma unroll
      for (int t = 0; t < PT; ++t) {
        const float2 a = A[t][g], b = B[t][g];
        const float pr = a.x + b.y, pi = a.y - b.x;   // A - iB
        const float mr = a.x - b.y, mi = a.y + b.x;   // A + iB
        zp[t] = make_float2(r.x * pr - r.y * pi, r.x * pi + r.y * pr);
        zm[t] = make_float2(r.x * mr + r.y * mi, r.x * mi - r.y * mr);
      }
      if constexpr (VEC) {
        if (ok[0]) {
          if (g < K)
            *reinterpret_cast<float4*>(out + obase[0] + (long long)g * inner) =
                make_float4(zp[0].x, zp[0].y, zp[PT - 1].x, zp[PT - 1].y);
          if (g > 0)
            *reinterpret_cast<float4*>(out + obase[0] + (long long)(2 * K - g) * inner) =
                make_float4(zm[0].x, zm[0].y, zm[PT - 1].x, zm[PT - 1].y);
        }
      } else {
#pragma unroll
        for (int t = 0; t < PT; ++t) {
          if (!ok[t]) continue;
          if (g < K) out[obase[t] + (long long)g * inner] = zp[t];
          if (g > 0) out[obase[t] + (long long)(2 * K - g) * inner] = zm[t];
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// expansion: in[outer][2K][inner] -> out[outer][N][inner]   (B^H along this dimension)
//   z_n = P_n + Q_n, z_{N-1-n} = P_n - Q_n,
//   P_n = sum_g alpha_g cos(psi_g (n+1/2)), Q_n = sum_g beta_g sin(psi_g (n+1/2)),
//   alpha_g = V'_{+g} + V'_{-g}, beta_g = i (V'_{+g} - V'_{-g}), V'_{+-g} = e^{-+i psi_g/2} V_{+-g}
// ------------------------------------------------------------------------------------------
template <int K, int PT, bool VEC>
__global__ void __launch_bounds__(kMidThreads) mid_expand_kernel(const float2* __restrict__ in,
                                                                 float2* __restrict__ out, long long outer,
                                                                 long long inner, int N, float scale) {
  constexpr int TS = MidTab<K>::TS;
  pdl_trigger();
  extern __shared__ float smem_mid[];
  float* tab = smem_mid;
  float2* rho = reinterpret_cast<float2*>(tab + (size_t)(N / 2) * TS);
  build_mid_table<K>(tab, rho, N, scale);
  __syncthreads();
  pdl_wait();

  const long long total = outer * inner;
  const long long per_cta = (long long)kMidThreads * PT;
  const long long tiles = (total + per_cta - 1) / per_cta;
  const int half = N / 2;
  for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    long long ibase[PT], obase[PT];
    bool ok[PT];
    float2 al[PT][K + 1], be[PT][K + 1];
#pragma unroll
    for (int t = 0; t < PT; ++t) {
      const long long p = VEC ? tile * per_cta + (long long)threadIdx.x * PT + t
                              : tile * per_cta + (long long)t * kMidThreads + threadIdx.x;
      ok[t] = p < total;
      const long long pc = ok[t] ? p : 0;
      const long long o = pc / inner, i = pc % inner;
      ibase[t] = o * (2 * K) * inner + i;
      obase[t] = o * N * inner + i;
    }
#pragma unroll
    for (int g = 0; g <= K; ++g) {
      const float2 r = rho[g];
      float2 vpl[PT], vmi[PT];
#pragma unroll
      for (int t = 0; t < PT; ++t) vpl[t] = vmi[t] = make_float2(0.f, 0.f);
      if constexpr (VEC) {
        if (g < K) {
          const float4 v = __ldg(reinterpret_cast<const float4*>(in + ibase[0] + (long long)g * inner));
          vpl[0] = make_float2(v.x, v.y);
          vpl[PT - 1] = make_float2(v.z, v.w);
        }
        if (g > 0) {
          const float4 v = __ldg(reinterpret_cast<const float4*>(in + ibase[0] + (long long)(2 * K - g) * inner));
          vmi[0] = make_float2(v.x, v.y);
          vmi[PT - 1] = make_float2(v.z, v.w);
        }
      } else {
#pragma unroll
        for (int t = 0; t < PT; ++t) {
          if (g < K) vpl[t] = __ldg(in + ibase[t] + (long long)g * inner);
          if (g > 0) vmi[t] = __ldg(in + ibase[t] + (long long)(2 * K - g) * inner);
        }
      }
#pragma unroll
      for (int t = 0; t < PT; ++t) {
        const float2 v = vpl[t], u = vmi[t];
        const float2 vp = make_float2(v.x * r.x + v.y * r.y, v.y * r.x - v.x * r.y);   // v * conj(rho)
        const float2 vm = make_float2(u.x * r.x - u.y * r.y, u.y * r.x + u.x * r.y);   // u * rho
        al[t][g] = make_float2(vp.x + vm.x, vp.y + vm.y);
        be[t][g] = make_float2(-(vp.y - vm.y), vp.x - vm.x);                           // i (vp - vm)
      }
    }
#pragma unroll 2
    for (int n = 0; n < half; ++n) {
      const float* row = tab + n * TS;
      float2 P[PT], Q[PT];
#pragma unroll
      for (int t = 0; t < PT; ++t) P[t] = Q[t] = make_float2(0.f, 0.f);
#pragma unroll
      for (int g = 0; g <= K; ++g) {
        const float c = row[g];
#pragma unroll
        for (int t = 0; t < PT; ++t) {
          P[t].x = fmaf(al[t][g].x, c, P[t].x);
          P[t].y = fmaf(al[t][g].y, c, P[t].y);
        }
      }
#pragma unroll
      for (int g = 1; g <= K; ++g) {
        const float s = row[K + g];
#pragma unroll
        for (int t = 0; t < PT; ++t) {
          Q[t].x = fmaf(be[t][g].x, s, Q[t].x);
          Q[t].y = fmaf(be[t][g].y, s, Q[t].y);
        }
      }
      if constexpr (VEC) {
        if (ok[0]) {
          *reinterpret_cast<float4*>(out + obase[0] + (long long)n * inner) =
              make_float4(P[0].x + Q[0].x, P[0].y + Q[0].y, P[PT - 1].x + Q[PT - 1].x, P[PT - 1].y + Q[PT - 1].y);
          *reinterpret_cast<float4*>(out + obase[0] + (long long)(N - 1 - n) * inner) =
              make_float4(P[0].x - Q[0].x, P[0].y - Q[0].y, P[PT - 1].x - Q[PT - 1].x, P[PT - 1].y - Q[PT - 1].y);
        }
      } else {
#pragma unroll
        for (int t = 0; t < PT; ++t) {
          if (!ok[t]) continue;
          out[obase[t] + (long long)n * inner] = make_float2(P[t].x + Q[t].x, P[t].y + Q[t].y);
          out[obase[t] + (long long)(N - 1 - n) * inner] = make_float2(P[t].x - Q[t].x, P[t].y - Q[t].y);
        }
      }
    }
  }
}

template <int K, int PT, bool VEC>
cudaError_t launch_mid_t(bool forward, const float2* in, float2* out, long long outer, long long inner, int N,
                         float scale, cudaStream_t st) {
  const size_t smem = (size_t)(N / 2) * MidTab<K>::TS * 4 + (size_t)(K + 1) * 8;
  const long long total = outer * inner;
  const long long tiles = (total + (long long)kMidThreads * PT - 1) / ((long long)kMidThreads * PT);
  // persistent CTAs: exactly as many as are resident at once, so that no CTA starts late
  auto launch = [&](auto kern) -> cudaError_t {
    cudaError_t e = cudaSuccess;
    if (smem > 48 * 1024) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kMidThreads, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    const long long cap = (long long)num_sms() * per_sm;
    const int grid = (int)(tiles < cap ? tiles : cap);
    (void)launch_pdl(kern, dim3(grid), dim3(kMidThreads), smem, st, in, out, outer, inner, N, scale);
    return cudaGetLastError();
  };
  return forward ? launch(mid_contract_kernel<K, PT, VEC>) : launch(mid_expand_kernel<K, PT, VEC>);
}

}  // namespace

// the double-folded FFMA kernels of this file
static bool mid_ffma_supported(int N, int K) {
  if (N % 2 != 0 || 2 * K > N) return false;
  if (!(K == 4 || K == 8 || K == 12 || K == 16)) return false;
  const size_t smem = (size_t)(N / 2) * (((2 * K + 1 + 3) / 4) * 4) * 4 + (size_t)(K + 1) * 8;
  return smem <= 200 * 1024;
}

// some folded kernel serves this extent and mode count: the ones of this file, their tensor-core versions
// (dtst_midmma.cu) or the ones for any extent and any mode count up to 32 (dtst_midg.cu)
bool mid_supported(int N, int K) { return mid_ffma_supported(N, K) || midg_supported(N, K); }

cudaError_t launch_mid(bool forward, int K, const float2* in, float2* out, long long outer, long long inner, int N,
                       float scale, bool fast, cudaStream_t st) {
  if (outer * inner <= 0) return cudaSuccess;
  const bool aligned16 = ((reinterpret_cast<uintptr_t>(in) | reinterpret_cast<uintptr_t>(out)) & 15u) == 0;
  if (aligned16 && mid_mma_supported(N, K, inner)) return launch_mid_mma(forward, K, in, out, outer, inner, N, scale, st);
  if (!mid_ffma_supported(N, K)) return launch_midg(forward, K, in, out, outer, inner, N, scale, fast, st);
  // The kernels below run one thread per two positions: a tensor with few of them (a 2-D layer: batch x channels x
  // k3) leaves most of the GPU idle (4 x 32 x 1024 x 12: six CTAs, 147 us); the kernels for any extent split such a
  // tensor along the contracted dimension as well.
  if (outer * inner < 65536 && midg_supported(N, K)) return launch_midg(forward, K, in, out, outer, inner, N, scale, fast, st);
  // two adjacent positions per thread need an even inner extent (then every pair is 16-byte aligned and
  // never straddles two outer slices) and 16-byte aligned tensors
  const bool vec = (inner % 2 == 0) && ((reinterpret_cast<uintptr_t>(in) | reinterpret_cast<uintptr_t>(out)) & 15u) == 0;
#define DTST_MID_CASE(KK)                                                                          \
  case KK:                                                                                         \
    return vec ? launch_mid_t<KK, 2, true>(forward, in, out, outer, inner, N, scale, st)           \
               : launch_mid_t<KK, 2, false>(forward, in, out, outer, inner, N, scale, st);
  switch (K) {
    DTST_MID_CASE(4)
    DTST_MID_CASE(8)
    DTST_MID_CASE(12)
    DTST_MID_CASE(16)
    default: return cudaErrorNotSupported;
  }
#undef DTST_MID_CASE
}

}  // namespace dtst
