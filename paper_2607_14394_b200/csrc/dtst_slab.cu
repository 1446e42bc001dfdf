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
#include "dtst_mma.cuh"

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
  pdl_trigger();
  extern __shared__ float2 slab_tab[];
  build_slab_table<K>(slab_tab, Nl, N, off, -1);
  __syncthreads();
  pdl_wait();
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
  pdl_trigger();
  extern __shared__ float2 slab_tab[];
  build_slab_table<K>(slab_tab, Nl, N, off, +1);
  __syncthreads();
  pdl_wait();
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

// ------------------------------------------------------------------------------------------
// The contraction on the tensor cores, for slabs whose row count is a multiple of 8 (and inner % 4 == 0).
// No fold is possible, so this is the plain complex product written with real MMAs:
//   M = 16 real columns = 8 complex positions (real parts | imaginary parts), the data as A operand;
//   K = 8 rows of the slab per step;  N = 8 of the 2k retained frequencies, cos and sin tables as B operands.
// A slab's partial spectrum is accumulated from zero (C = sum x cos, S = sum x sin; Z = (C_re + S_im) + i (C_im -
// S_re)) and then added to the running total: Eq. 7, slabs in ascending order.  The input streams through a
// per-warp cp.async ring as in the folded kernel.
// ------------------------------------------------------------------------------------------
constexpr int kSMT = 1;                       // m-tiles per task: 8 complex positions = 64 bytes per row
constexpr int kSPos = 8 * kSMT;
constexpr int kSWarps = 16;
constexpr int kSStages = 6;
constexpr int kSRow = 2 * kSPos + 8;          // floats per staged row (8 mod 32: conflict-free 8-byte loads)
constexpr int kSStageFloats = 8 * kSRow;

__device__ __forceinline__ void slab_cp_async16(float* smem_dst, const float* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}

template <int K>
__global__ void __launch_bounds__(kSWarps * 32, 1)
slab_contract_mma_kernel(const float* __restrict__ in, float2* __restrict__ out, long long outer, long long inner,
                         int Nl, int N, int off, int P) {
  // +g and -g share their sums: C_g = sum_n z_n cos(phi_g (off + n)), S_g = sum_n z_n sin(phi_g (off + n)),
  // Z_{+g} = C_g - i S_g, Z_{-g} = C_g + i S_g, phi_g = 2 pi g / N.  The MMA n-tiles cover g = 0..K-1; g = K (only
  // -K is retained) runs on FFMA.
  pdl_trigger();
  constexpr int NT = (K + 7) / 8;
  extern __shared__ float4 slab_smem4[];
  const int KS = Nl / 8;                        // k-steps over all local rows
  const int ksl = KS / P;                       // k-steps per slab
  float4* btab = slab_smem4;                    // [KS][NT][cos | sin][lane]
  float2* tK = reinterpret_cast<float2*>(btab + (size_t)KS * NT * 2 * 32);   // (cos, sin)(phi_K (off + n)), n < Nl
  float* ringbase = reinterpret_cast<float*>(tK + Nl);

  for (int e = threadIdx.x; e < KS * NT * 2 * 32; e += blockDim.x) {
    const int l = e & 31, sn_tab = (e >> 5) & 1, nt = (e >> 6) % NT, ks = (e >> 6) / NT;
    const int lg = l >> 2, lt = l & 3;          // B fragment: k = row lt (+4), n = frequency slot lg
    const int g = 8 * nt + lg;
    uint32_t hi[2], lo[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float2 t = twiddle(g, (long long)off + 8 * ks + lt + 4 * h, N, +1);   // (cos, sin) of the phase
      split_tf32_rna(g < K ? (sn_tab ? t.y : t.x) : 0.f, hi[h], lo[h]);
    }
    btab[e] = make_float4(__uint_as_float(hi[0]), __uint_as_float(hi[1]), __uint_as_float(lo[0]), __uint_as_float(lo[1]));
  }
  for (int n = threadIdx.x; n < Nl; n += blockDim.x) tK[n] = twiddle(K, (long long)off + n, N, +1);
  __syncthreads();
  pdl_wait();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g8 = lane >> 2, t4 = lane & 3;
  const long long cblocks = (inner + kSPos - 1) / kSPos;
  const long long tasks = outer * cblocks;
  const long long rs = 2 * inner;               // floats per row
  const long long tstride = (long long)gridDim.x * kSWarps;
  float* ring = ringbase + (size_t)warp * kSStages * kSStageFloats;

  long long ptask = (long long)blockIdx.x * kSWarps + warp;
  int pks = 0, pstage = 0;
  const float* ptb = in;
  bool pchunk_ok = false;
  auto issue = [&]() {
    if (ptask < tasks) {
      if (pks == 0) {
        const long long o = ptask / cblocks, cb = ptask % cblocks;
        const long long left = inner - cb * kSPos;
        const int nch = left >= kSPos ? kSPos / 2 : (int)(left / 2);
        ptb = in + o * Nl * rs + cb * (2 * kSPos) + 4 * (lane & 7);
        pchunk_ok = (lane & 7) < nch;
      }
      if (pchunk_ok) {
        float* dst = ring + pstage * kSStageFloats + (lane >> 3) * kSRow + 4 * (lane & 7);
        const int n = 8 * pks + (lane >> 3);
        slab_cp_async16(dst, ptb + (long long)n * rs);
        slab_cp_async16(dst + 4 * kSRow, ptb + (long long)(n + 4) * rs);
      }
      if (++pks == KS) {
        pks = 0;
        ptask += tstride;
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    pstage = pstage + 1 == kSStages ? 0 : pstage + 1;
  };
#pragma unroll
  for (int i = 0; i < kSStages - 1; ++i) issue();

  int cstage = 0;
  for (long long task = (long long)blockIdx.x * kSWarps + warp; task < tasks; task += tstride) {
    const long long o = task / cblocks, cb = task % cblocks;
    const long long left = inner - cb * kSPos;
    const int mtv = left >= kSPos ? kSMT : (int)((left + 7) / 8);
    // totals: Z_{+g} and Z_{-g} as (re, slot 2 t4) (re, slot 2 t4 + 1) (im, 2 t4) (im, 2 t4 + 1); Z_{-K} as (re, im)
    float totp[kSMT][NT][4], totm[kSMT][NT][4], totK[kSMT][2];
#pragma unroll
    for (int mt = 0; mt < kSMT; ++mt) {
      totK[mt][0] = totK[mt][1] = 0.f;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) totp[mt][nt][e] = totm[mt][nt][e] = 0.f;
    }

#pragma unroll 1
    for (int slab = 0; slab < P; ++slab) {
      float aC[kSMT][NT][4], aS[kSMT][NT][4], cK[kSMT][2], sK[kSMT][2];
#pragma unroll
      for (int mt = 0; mt < kSMT; ++mt) {
        cK[mt][0] = cK[mt][1] = sK[mt][0] = sK[mt][1] = 0.f;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) aC[mt][nt][e] = aS[mt][nt][e] = 0.f;
      }
#pragma unroll 1
      for (int k = 0; k < ksl; ++k) {
        const int ks = slab * ksl + k;
        asm volatile("cp.async.wait_group %0;" ::"n"(kSStages - 2) : "memory");
        __syncwarp();
        issue();
        const float* S = ring + cstage * kSStageFloats + t4 * kSRow + 2 * g8;
        const float4* bt = btab + (size_t)(ks * NT * 2) * 32 + lane;
        const float2 tk0 = tK[8 * ks + t4], tk1 = tK[8 * ks + t4 + 4];
#pragma unroll
        for (int mt = 0; mt < kSMT; ++mt) {
          if (mt < mtv) {
            const float2 lo_row = *reinterpret_cast<const float2*>(S + 16 * mt);
            const float2 hi_row = *reinterpret_cast<const float2*>(S + 4 * kSRow + 16 * mt);
            cK[mt][0] = fmaf(lo_row.x, tk0.x, fmaf(hi_row.x, tk1.x, cK[mt][0]));
            cK[mt][1] = fmaf(lo_row.y, tk0.x, fmaf(hi_row.y, tk1.x, cK[mt][1]));
            sK[mt][0] = fmaf(lo_row.x, tk0.y, fmaf(hi_row.x, tk1.y, sK[mt][0]));
            sK[mt][1] = fmaf(lo_row.y, tk0.y, fmaf(hi_row.y, tk1.y, sK[mt][1]));
            uint32_t ah[4], al[4];
            split_tf32_round(lo_row.x, ah[0], al[0]);
            split_tf32_round(lo_row.y, ah[1], al[1]);
            split_tf32_round(hi_row.x, ah[2], al[2]);
            split_tf32_round(hi_row.y, ah[3], al[3]);
            // the three compensated products of an accumulator depend on one another: issue them interleaved
            // over the 2 NT accumulators
            float4 bc[NT], bs[NT];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              bc[nt] = bt[(nt * 2 + 0) * 32];
              bs[nt] = bt[(nt * 2 + 1) * 32];
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              mma_m16n8k8_tf32(aC[mt][nt], ah, __float_as_uint(bc[nt].x), __float_as_uint(bc[nt].y));
              mma_m16n8k8_tf32(aS[mt][nt], ah, __float_as_uint(bs[nt].x), __float_as_uint(bs[nt].y));
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              mma_m16n8k8_tf32(aC[mt][nt], al, __float_as_uint(bc[nt].x), __float_as_uint(bc[nt].y));
              mma_m16n8k8_tf32(aS[mt][nt], al, __float_as_uint(bs[nt].x), __float_as_uint(bs[nt].y));
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              mma_m16n8k8_tf32(aC[mt][nt], ah, __float_as_uint(bc[nt].z), __float_as_uint(bc[nt].w));
              mma_m16n8k8_tf32(aS[mt][nt], ah, __float_as_uint(bs[nt].z), __float_as_uint(bs[nt].w));
            }
          }
        }
        cstage = cstage + 1 == kSStages ? 0 : cstage + 1;
      }
      // Eq. 7: this slab's partial spectrum, then onto the totals (slabs in ascending order).
#pragma unroll
      for (int mt = 0; mt < kSMT; ++mt) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          // Z_{+g} = C - iS: (C_re + S_im, C_im - S_re);  Z_{-g} = C + iS: (C_re - S_im, C_im + S_re)
          totp[mt][nt][0] += aC[mt][nt][0] + aS[mt][nt][2];
          totp[mt][nt][1] += aC[mt][nt][1] + aS[mt][nt][3];
          totp[mt][nt][2] += aC[mt][nt][2] - aS[mt][nt][0];
          totp[mt][nt][3] += aC[mt][nt][3] - aS[mt][nt][1];
          totm[mt][nt][0] += aC[mt][nt][0] - aS[mt][nt][2];
          totm[mt][nt][1] += aC[mt][nt][1] - aS[mt][nt][3];
          totm[mt][nt][2] += aC[mt][nt][2] + aS[mt][nt][0];
          totm[mt][nt][3] += aC[mt][nt][3] + aS[mt][nt][1];
        }
        // Z_{-K} of this slab: the quad's lanes covered rows t4, t4 + 4 of every k-step
        float cr = cK[mt][0], ci = cK[mt][1], sr = sK[mt][0], si = sK[mt][1];
#pragma unroll
        for (int m = 1; m <= 2; m <<= 1) {
          cr += __shfl_xor_sync(0xffffffffu, cr, m);
          ci += __shfl_xor_sync(0xffffffffu, ci, m);
          sr += __shfl_xor_sync(0xffffffffu, sr, m);
          si += __shfl_xor_sync(0xffffffffu, si, m);
        }
        totK[mt][0] += cr - si;
        totK[mt][1] += ci + sr;
      }
    }
#pragma unroll
    for (int mt = 0; mt < kSMT; ++mt) {
      const long long pos = cb * kSPos + 8 * mt + g8;
      if (mt < mtv && pos < inner) {
        float2* dst = out + o * (2 * K) * inner + pos;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const int g = 8 * nt + 2 * t4 + q;
            if (g < K) {
              dst[(long long)g * inner] = make_float2(totp[mt][nt][q], totp[mt][nt][2 + q]);
              if (g > 0) dst[(long long)(2 * K - g) * inner] = make_float2(totm[mt][nt][q], totm[mt][nt][2 + q]);
            }
          }
        if (t4 == 0) dst[(long long)K * inner] = make_float2(totK[mt][0], totK[mt][1]);
      }
    }
  }
}

template <int K>
size_t slab_mma_smem(int Nl) {
  return (size_t)(Nl / 8) * ((K + 7) / 8) * 2 * 32 * 16 + (size_t)Nl * 8 + (size_t)kSWarps * kSStages * kSStageFloats * 4;
}

template <int K>
cudaError_t launch_slab_mma_t(const float2* in, float2* out, long long outer, long long inner, int Nl, int N, int off,
                              int P, cudaStream_t st) {
  const size_t smem = slab_mma_smem<K>(Nl);
  auto kern = slab_contract_mma_kernel<K>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const long long tasks = outer * ((inner + kSPos - 1) / kSPos);
  const long long want = (tasks + kSWarps - 1) / kSWarps;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3(kSWarps * 32), smem, st, reinterpret_cast<const float*>(in), out, outer, inner, Nl, N, off, P);
  return cudaGetLastError();
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
    const long long cap = (long long)num_sms() * per_sm;
    (void)launch_pdl(kern, dim3((unsigned)(want < cap ? want : cap)), dim3(kSlabThreads), smem, st, in, out, outer, inner, Nl, N, off, P);
    return cudaGetLastError();
  };
  return forward ? launch(slab_contract_kernel<K>) : launch(slab_expand_kernel<K>);
}

}  // namespace

// the kernels of this file
static bool slab_own_supported(int Nl, int K) {
  if (!(K == 4 || K == 8 || K == 12 || K == 16)) return false;
  return (size_t)Nl * 2 * K * sizeof(float2) <= 200 * 1024;
}

// ... or, for other mode counts, the folded kernels of dtst_midg.cu on the local rows with their global phases
bool slab_supported(int Nl, int K) { return slab_own_supported(Nl, K) || midg_local_supported(Nl, K); }

cudaError_t launch_slab(bool forward, int K, const float2* in, float2* out, long long outer, long long inner, int Nl,
                        int N, int off, int P, bool fast, cudaStream_t st) {
  if (outer * inner <= 0) return cudaSuccess;
  // Slabs of one device are consecutive rows with consecutive global indices: taken together they are ONE local
  // block that starts at `off` (the sum over the slabs is then part of the contraction's own sum).
  if (!slab_own_supported(Nl, K)) return launch_midg_local(forward, K, in, out, outer, inner, Nl, N, off, 1.0f, fast, st);
  // contraction of slabs that are whole k-steps of 8 rows: tensor-core kernel
  const bool aligned16 = ((reinterpret_cast<uintptr_t>(in) | reinterpret_cast<uintptr_t>(out)) & 15u) == 0;
  if (forward && aligned16 && inner % 4 == 0 && P >= 1 && Nl % P == 0 && (Nl / P) % 8 == 0) {
    const size_t lim = 227 * 1024;
    switch (K) {
      case 4: if (slab_mma_smem<4>(Nl) <= lim) return launch_slab_mma_t<4>(in, out, outer, inner, Nl, N, off, P, st); break;
      case 8: if (slab_mma_smem<8>(Nl) <= lim) return launch_slab_mma_t<8>(in, out, outer, inner, Nl, N, off, P, st); break;
      case 12: if (slab_mma_smem<12>(Nl) <= lim) return launch_slab_mma_t<12>(in, out, outer, inner, Nl, N, off, P, st); break;
      case 16: if (slab_mma_smem<16>(Nl) <= lim) return launch_slab_mma_t<16>(in, out, outer, inner, Nl, N, off, P, st); break;
      default: break;
    }
  }
  switch (K) {
    case 4: return launch_slab_t<4>(forward, in, out, outer, inner, Nl, N, off, P, st);
    case 8: return launch_slab_t<8>(forward, in, out, outer, inner, Nl, N, off, P, st);
    case 12: return launch_slab_t<12>(forward, in, out, outer, inner, Nl, N, off, P, st);
    case 16: return launch_slab_t<16>(forward, in, out, outer, inner, Nl, N, off, P, st);
    default: return cudaErrorNotSupported;
  }
}

}  // namespace dtst
