// Row kernels for ANY contiguous extent: the contiguous (rfft) dimension alone, for grids whose last extent is not
// a multiple of 32 (the paper's own time axis of 30 points, Section "cuBLAS vs cuFFT"), whose rows are therefore not
// 16-byte aligned and cannot be described to the TMA unit as a 2-D tensor.  The remaining dimensions run on the
// reduced tensor (dtst_midmma.cu / dtst_mid.cu).
//
//   rowg_contract_kernel:  x[rows][N3] real  ->  out[rows][k3] complex   (Eq. 5 along the last dimension)
//   rowg_expand_kernel:    in[rows][k3] complex -> y[rows][N3] real      (Eq. 14 along the last dimension)
//
// One fold about the half-sample point (valid for every N3, odd ones included): with theta_{f,j} = 2 pi f (j + 1/2) / N3,
//     X_f = e^{+i pi f / N3} ( sum_j s_j cos theta_{f,j}  -  i sum_j d_j sin theta_{f,j} ),
//     s_j = x_j + x_{N3-1-j},  d_j = x_j - x_{N3-1-j},  j < N3 / 2     (odd N3: the middle sample is s alone, its sine is 0)
// and the two sums are [rows x pairs] x [pairs x frequencies] products on the tensor cores (warp-level m16n8k8 TF32,
// hi/lo compensated, fp32 accumulate), the basis from a fragment-ordered shared table built once per persistent CTA.
// A task is 16 or 32 consecutive rows: a CONTIGUOUS piece of the grid whose start and length are multiples of
// 16 bytes whatever N3 is, so it is staged with 16-byte cp.async requests (contraction: a per-warp ring of three
// stages, two tasks in flight per warp; two stages where three do not fit) and written back with 16-byte stores
// from a per-warp staging area.
#include "dtst_fused.cuh"
#include "dtst_mma.cuh"

namespace dtst {

namespace {

constexpr size_t kGSmemLimit = 227 * 1024;
constexpr int kGMaxWarps = 12;

__device__ __forceinline__ void g_cp_async16(float* smem_dst, const float* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}
__device__ __forceinline__ void g_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void g_cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// hi = the value with its low 13 mantissa bits cleared, lo = the exact rest (the tensor core drops lo's low bits)
__device__ __forceinline__ void g_split(float v, uint32_t& hi, uint32_t& lo) {
  hi = __float_as_uint(v) & 0xffffe000u;
  lo = __float_as_uint(v - __uint_as_float(hi));
}

// cos (part 0) or sin (part 1) of 2 pi f (j + 1/2) / N, the phase reduced exactly in integers
__device__ __forceinline__ float g_basis(int part, int f, int j, int N) {
  double s, c;
  sincospi((double)(((long long)f * (2 * j + 1)) % (2ll * N)) / (double)N, &s, &c);
  return part == 0 ? (float)c : (float)s;
}

// ---------------------------------------------------------------------------------------------
// contraction.  MT m-tiles of 16 rows per task, NT n-tiles of 8 frequencies (k3 <= 8 NT).
// ---------------------------------------------------------------------------------------------
template <int MT, int NT, int ST>
__global__ void __launch_bounds__(kGMaxWarps * 32, 1)
rowg_contract_kernel(const float* __restrict__ x, float2* __restrict__ out, long long rows, int N3, int K3, float scale,
                     int herm, int stage_floats) {
  pdl_trigger();
  constexpr int TR = 16 * MT;
  extern __shared__ float4 rg_smem[];
  const int half = N3 / 2, H = (N3 + 1) / 2, KS = (H + 7) / 8;   // pairs (odd N3: + the middle sample), k-steps
  const bool odd = (N3 & 1) != 0;
  float4* btab = rg_smem;                                          // [part][ks][nt][lane] = (b0 hi, b1 hi, b0 lo, b1 lo)
  float* ring = reinterpret_cast<float*>(btab + (size_t)2 * KS * NT * 32);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;
  const int W = blockDim.x >> 5;

  for (int e = threadIdx.x; e < 2 * KS * NT * 32; e += blockDim.x) {
    const int l = e & 31;
    int r = e >> 5;
    const int nt = r % NT;
    r /= NT;
    const int ks = r % KS, part = r / KS;
    const int f = 8 * nt + (l >> 2);                               // B fragment: k = l & 3 (+4), n = l >> 2
    uint32_t hi[2], lo[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int j = 8 * ks + (l & 3) + 4 * h;
      split_tf32_rna((f < K3 && j < H) ? g_basis(part, f, j, N3) : 0.f, hi[h], lo[h]);
    }
    btab[e] = make_float4(__uint_as_float(hi[0]), __uint_as_float(hi[1]), __uint_as_float(lo[0]), __uint_as_float(lo[1]));
  }
  // rotation of this lane's frequencies f = 8 nt + 2 t4 + q: the deferred half-sample phase, scale, Hermitian weight
  float2 rot[NT][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int f = 8 * nt + 2 * t4 + q;
      double sn, cs;
      sincospi((double)f / (double)N3, &sn, &cs);
      const float wgt = scale * (herm ? herm_weight(f, N3) : 1.0f);
      rot[nt][q] = make_float2((float)cs * wgt, (float)sn * wgt);
    }
  __syncthreads();
  pdl_wait();   // everything above is independent of the preceding kernel

  float* S = ring + (size_t)warp * ST * stage_floats;
  const long long tasks = (rows + TR - 1) / TR;
  const long long stride = (long long)W * gridDim.x;
  auto load = [&](long long t, int s) {
    if (t < tasks) {
      const long long r0 = t * TR;
      const long long nr = rows - r0 < TR ? rows - r0 : TR;
      const int nf = (int)(nr * N3);                               // floats of this task: contiguous, 16-byte aligned start
      const float* src = x + r0 * N3;
      float* dst = S + (size_t)s * stage_floats;
      for (int i = lane; i < (nf >> 2); i += 32) g_cp_async16(dst + 4 * i, src + 4 * i);
      const int done = nf & ~3;
      if (lane < (nf & 3)) dst[done + lane] = __ldg(src + done + lane);   // a ragged last task only
    }
    g_cp_async_commit();   // one group per call, empty past the end: the wait below counts groups
  };
  long long t = (long long)warp * gridDim.x + blockIdx.x;
#pragma unroll
  for (int q = 0; q < ST - 1; ++q) load(t + q * stride, q);
  int s = 0;
  for (; t < tasks; t += stride, s = s == ST - 1 ? 0 : s + 1) {
    load(t + (ST - 1) * stride, s == 0 ? ST - 1 : s - 1);
    g_cp_async_wait<ST - 1>();
    __syncwarp();
    const float* T = S + (size_t)s * stage_floats;
    float accC[MT][NT][4], accS[MT][NT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) accC[mt][nt][e] = accS[mt][nt][e] = 0.f;
#pragma unroll 2
    for (int ks = 0; ks < KS; ++ks) {
      float4 bc[NT], bs[NT];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        bc[nt] = btab[((size_t)(0 * KS + ks) * NT + nt) * 32 + lane];
        bs[nt] = btab[((size_t)(1 * KS + ks) * NT + nt) * 32 + lane];
      }
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        uint32_t sh[4], sl[4], dh[4], dl[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {                              // A fragment: row g8 (+8), pair t4 (+4)
          const int row = 16 * mt + g8 + 8 * (e & 1);
          const int j = 8 * ks + t4 + 4 * (e >> 1);
          const bool in = j < half, mid = odd && j == half;
          const int ja = (in || mid) ? j : 0, jb = in ? N3 - 1 - j : ja;
          const float a = T[row * N3 + ja], b = T[row * N3 + jb];
          g_split(in ? a + b : (mid ? a : 0.f), sh[e], sl[e]);
          g_split(in ? a - b : 0.f, dh[e], dl[e]);
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          mma3_tf32(accC[mt][nt], sh, sl, __float_as_uint(bc[nt].x), __float_as_uint(bc[nt].y), __float_as_uint(bc[nt].z),
                    __float_as_uint(bc[nt].w));
          mma3_tf32(accS[mt][nt], dh, dl, __float_as_uint(bs[nt].x), __float_as_uint(bs[nt].y), __float_as_uint(bs[nt].z),
                    __float_as_uint(bs[nt].w));
        }
      }
    }
    // X_f = rot_f (C_f - i S_f); a C fragment holds rows g8, g8 + 8 and the frequencies 8 nt + 2 t4, + 1
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const long long row = t * TR + 16 * mt + g8 + 8 * h;
        if (row >= rows) continue;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int f0 = 8 * nt + 2 * t4;
          float2 r[2];
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const float C = accC[mt][nt][2 * h + q], Sv = accS[mt][nt][2 * h + q];
            r[q] = make_float2(rot[nt][q].x * C + rot[nt][q].y * Sv, rot[nt][q].y * C - rot[nt][q].x * Sv);
          }
          float2* dst = out + row * K3 + f0;
          if (f0 + 1 < K3 && (K3 & 1) == 0) {
            *reinterpret_cast<float4*>(dst) = make_float4(r[0].x, r[0].y, r[1].x, r[1].y);
          } else {
            if (f0 < K3) dst[0] = r[0];
            if (f0 + 1 < K3) dst[1] = r[1];
          }
        }
      }
    __syncwarp();   // every lane is done with this stage before it is filled again
  }
}

// ---------------------------------------------------------------------------------------------
// expansion.  y_j = P_j - Q_j, y_{N3-1-j} = P_j + Q_j with P_j = sum_f Re z'_f cos theta_{f,j},
// Q_j = sum_f Im z'_f sin theta_{f,j}, z'_f = scale c_f e^{-i pi f / N3} in_f.  MT m-tiles of 16 rows per task,
// KSF k-steps of 8 frequencies (k3 <= 8 KSF).
// ---------------------------------------------------------------------------------------------
template <int MT, int KSF>
__global__ void __launch_bounds__(kGMaxWarps * 32, 1)
rowg_expand_kernel(const float2* __restrict__ in, float* __restrict__ y, long long rows, int N3, int K3, float scale,
                   int herm, int stage_floats) {
  pdl_trigger();
  constexpr int TR = 16 * MT;
  extern __shared__ float4 rg_smem[];
  const int half = N3 / 2, H = (N3 + 1) / 2, NTJ = (H + 7) / 8;
  const bool odd = (N3 & 1) != 0;
  float4* btab = rg_smem;                                          // [part][ks][ntj][lane]
  float* stg = reinterpret_cast<float*>(btab + (size_t)2 * KSF * NTJ * 32);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;
  const int W = blockDim.x >> 5;

  for (int e = threadIdx.x; e < 2 * KSF * NTJ * 32; e += blockDim.x) {
    const int l = e & 31;
    int r = e >> 5;
    const int ntj = r % NTJ;
    r /= NTJ;
    const int ks = r % KSF, part = r / KSF;
    const int j = 8 * ntj + (l >> 2);                              // B fragment: k = frequency l & 3 (+4), n = pair l >> 2
    uint32_t hi[2], lo[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int f = 8 * ks + (l & 3) + 4 * h;
      split_tf32_rna((f < K3 && j < H) ? g_basis(part, f, j, N3) : 0.f, hi[h], lo[h]);
    }
    btab[e] = make_float4(__uint_as_float(hi[0]), __uint_as_float(hi[1]), __uint_as_float(lo[0]), __uint_as_float(lo[1]));
  }
  // rotation of this lane's A-fragment frequencies f = 8 ks + t4 + 4 hf
  float2 rot[KSF][2];
#pragma unroll
  for (int ks = 0; ks < KSF; ++ks)
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const int f = 8 * ks + t4 + 4 * hf;
      double sn, cs;
      sincospi((double)f / (double)N3, &sn, &cs);
      const float wgt = (f < K3) ? scale * (herm ? herm_weight(f, N3) : 1.0f) : 0.f;
      rot[ks][hf] = make_float2((float)cs * wgt, -(float)sn * wgt);
    }
  __syncthreads();
  pdl_wait();

  float* st = stg + (size_t)warp * stage_floats;
  const long long tasks = (rows + TR - 1) / TR;
  const long long stride = (long long)W * gridDim.x;
  float2 vin[MT][KSF][4];   // the NEXT task's values: requested a task ahead
  auto load_inputs = [&](long long t) {
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int ks = 0; ks < KSF; ++ks)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const long long row = t * TR + 16 * mt + g8 + 8 * (e & 1);
          const int f = 8 * ks + t4 + 4 * (e >> 1);
          vin[mt][ks][e] = (t < tasks && row < rows && f < K3) ? __ldg(in + row * K3 + f) : make_float2(0.f, 0.f);
        }
  };
  long long t = (long long)warp * gridDim.x + blockIdx.x;
  load_inputs(t);
  for (; t < tasks; t += stride) {
    uint32_t rh[MT][KSF][4], rl[MT][KSF][4], ih[MT][KSF][4], il[MT][KSF][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int ks = 0; ks < KSF; ++ks)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 v = vin[mt][ks][e];
          const float2 r = rot[ks][e >> 1];
          g_split(v.x * r.x - v.y * r.y, rh[mt][ks][e], rl[mt][ks][e]);
          g_split(v.x * r.y + v.y * r.x, ih[mt][ks][e], il[mt][ks][e]);
        }
    load_inputs(t + stride);
#pragma unroll 1
    for (int ntj = 0; ntj < NTJ; ++ntj) {
      float4 bc[KSF], bs[KSF];
#pragma unroll
      for (int ks = 0; ks < KSF; ++ks) {
        bc[ks] = btab[((size_t)(0 * KSF + ks) * NTJ + ntj) * 32 + lane];
        bs[ks] = btab[((size_t)(1 * KSF + ks) * NTJ + ntj) * 32 + lane];
      }
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        float P[4] = {0.f, 0.f, 0.f, 0.f}, Q[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < KSF; ++ks) {
          mma3_tf32(P, rh[mt][ks], rl[mt][ks], __float_as_uint(bc[ks].x), __float_as_uint(bc[ks].y),
                    __float_as_uint(bc[ks].z), __float_as_uint(bc[ks].w));
          mma3_tf32(Q, ih[mt][ks], il[mt][ks], __float_as_uint(bs[ks].x), __float_as_uint(bs[ks].y),
                    __float_as_uint(bs[ks].z), __float_as_uint(bs[ks].w));
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float* srow = st + (16 * mt + g8 + 8 * h) * N3;
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const int j = 8 * ntj + 2 * t4 + q;
            const float p = P[2 * h + q], qv = Q[2 * h + q];
            if (j < half) {
              srow[j] = p - qv;
              srow[N3 - 1 - j] = p + qv;
            } else if (odd && j == half) {
              srow[j] = p;
            }
          }
        }
      }
    }
    __syncwarp();
    {
      const long long r0 = t * TR;
      const long long nr = rows - r0 < TR ? rows - r0 : TR;
      const int nf = (int)(nr * N3);
      float* dst = y + r0 * N3;
      for (int i = lane; i < (nf >> 2); i += 32)
        __stcs(reinterpret_cast<float4*>(dst) + i, *reinterpret_cast<const float4*>(st + 4 * i));
      const int done = nf & ~3;
      if (lane < (nf & 3)) dst[done + lane] = st[done + lane];
    }
    __syncwarp();   // the staging area is read out before the next task writes to it
  }
}

// =============================================================================================
// The same two kernels with the dimension in front of the contiguous one (extent N2, whole, no offset, K2 modes
// per side) contracted / expanded inside: where the contiguous stage does not compress (the paper's time axis keeps
// 16 of its 16 one-sided modes), the reduced tensor of the row stage is as large as the grid, and writing and
// re-reading it tripled the traffic of a transform.  A warp takes whole planes (N2 rows).
//
//   planeg_contract_kernel:  x[planes][N2][N3] real -> out[planes][2 K2][k3] complex
//   planeg_expand_kernel:    in[planes][2 K2][k3] complex -> y[planes][N2][N3] real
//
// Contraction.  The row stage runs TRANSPOSED, eight rows at a time: [16 frequencies x pairs] x [pairs x 8 rows], so
// that its C fragment (frequency g8 / g8 + 8, rows 2 t4 / 2 t4 + 1) is, after the rotation, exactly the column
// operand of the second stage's k-step over these eight rows - [modes x 8 rows] x [8 rows x real columns] - once the
// MMA's k index is read as row 2 k (k < 4) or 2 (k - 4) + 1 and the four n-tiles as (re, im) x (f < 8, f >= 8):
// a sum does not care how its terms or its columns are named, and the basis table is built with the same naming.
// Nothing is transposed through shared memory; the plane's [2 K2][k3] sums live in C fragments until its last row.
//
// Expansion.  The second dimension first: [16 rows x modes] x [modes x (re, im) columns] from the plane's spectrum
// (a padded copy in shared memory, fetched one plane ahead); its C fragment (rows g8 / g8 + 8, the complex value of
// frequency 4 nc + t4) is exactly the row operand of the contiguous stage (frequency 8 ks + t4 + 4 half <-> n-tile
// 2 ks + half), which then runs as in rowg_expand_kernel.
// =============================================================================================
__device__ __forceinline__ void g_cp_async8(float* smem_dst, const float2* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}

// cos (part 0) or sin (part 1) of 2 pi k_p n / N2 for the retained position p of a two-sided dimension
__device__ __forceinline__ float g_basis2(int part, int p, int n, int N2, int K2) {
  const long long k = p < K2 ? p : N2 - (2 * K2 - p);
  double s, c;
  sincospi(2.0 * (double)((k * n) % N2) / (double)N2, &s, &c);
  return part == 0 ? (float)c : (float)s;
}

__device__ __forceinline__ void g_split4(const float4& v, uint32_t (&hi)[4], uint32_t (&lo)[4]) {
  g_split(v.x, hi[0], lo[0]);
  g_split(v.y, hi[1], lo[1]);
  g_split(v.z, hi[2], lo[2]);
  g_split(v.w, hi[3], lo[3]);
}

// MT: 16-row tiles per task; NC: n-tiles of the second stage (2 for k3 <= 8, else 4); MTM: 16-mode tiles (2 K2 <= 16 MTM)
template <int MT, int NC, int MTM, int ST>
__global__ void __launch_bounds__(kGMaxWarps * 32, 1)
planeg_contract_kernel(const float* __restrict__ x, float2* __restrict__ out, long long planes, int N3, int K3, int N2,
                       int K2, float scale, int herm, int stage_floats) {
  pdl_trigger();
  constexpr int TR = 16 * MT, GPT = 2 * MT;   // rows and 8-row groups per task
  extern __shared__ float4 rg_smem[];
  const int half = N3 / 2, H = (N3 + 1) / 2, KS = (H + 7) / 8;
  const bool odd = (N3 & 1) != 0;
  const int NG = N2 / 8, TP = N2 / TR;
  float4* atab = rg_smem;                                   // [part][ks][hi | lo][lane]: the row stage's 16-row operand
  float4* a2tab = atab + (size_t)2 * KS * 2 * 32;           // [part][group][mtm][lane]: the second stage's, unsplit
  float* ring = reinterpret_cast<float*>(a2tab + (size_t)2 * NG * MTM * 32);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;
  const int W = blockDim.x >> 5;

  for (int e = threadIdx.x; e < 2 * KS * 32; e += blockDim.x) {
    const int l = e & 31, ks = (e >> 5) % KS, part = (e >> 5) / KS;
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {                           // A fragment: frequency l >> 2 (+8), pair l & 3 (+4)
      const int f = (l >> 2) + 8 * (q & 1), j = 8 * ks + (l & 3) + 4 * (q >> 1);
      split_tf32_rna((f < K3 && j < H) ? g_basis(part, f, j, N3) : 0.f, hi[q], lo[q]);
    }
    atab[((size_t)(part * KS + ks) * 2 + 0) * 32 + l] =
        make_float4(__uint_as_float(hi[0]), __uint_as_float(hi[1]), __uint_as_float(hi[2]), __uint_as_float(hi[3]));
    atab[((size_t)(part * KS + ks) * 2 + 1) * 32 + l] =
        make_float4(__uint_as_float(lo[0]), __uint_as_float(lo[1]), __uint_as_float(lo[2]), __uint_as_float(lo[3]));
  }
  for (int e = threadIdx.x; e < 2 * NG * MTM * 32; e += blockDim.x) {
    const int l = e & 31;
    int r = e >> 5;
    const int mtm = r % MTM;
    r /= MTM;
    const int grp = r % NG, part = r / NG;
    float v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {                           // A fragment: mode l >> 2 (+8), row 2 (l & 3) (+1)
      const int pm = 16 * mtm + (l >> 2) + 8 * (q & 1), n = 8 * grp + 2 * (l & 3) + (q >> 1);
      v[q] = pm < 2 * K2 ? g_basis2(part, pm, n, N2, K2) : 0.f;
    }
    a2tab[e] = make_float4(v[0], v[1], v[2], v[3]);
  }
  float2 rot[2];                                            // frequencies g8 and g8 + 8
#pragma unroll
  for (int fh = 0; fh < 2; ++fh) {
    const int f = g8 + 8 * fh;
    double sn, cs;
    sincospi((double)f / (double)N3, &sn, &cs);
    const float wgt = scale * (herm ? herm_weight(f, N3) : 1.0f);
    rot[fh] = make_float2((float)cs * wgt, (float)sn * wgt);
  }
  __syncthreads();
  pdl_wait();

  float* S = ring + (size_t)warp * ST * stage_floats;
  const long long stride = (long long)W * gridDim.x;
  long long pl = (long long)warp * gridDim.x + blockIdx.x;
  long long apl = pl;                                       // the task staged next: plane and place within it
  int aj = 0;
  auto load = [&](int s) {
    if (apl < planes) {
      const float* src = x + (apl * N2 + (long long)aj * TR) * N3;
      float* dst = S + (size_t)s * stage_floats;
      for (int i = lane; i < (TR * N3) / 4; i += 32) g_cp_async16(dst + 4 * i, src + 4 * i);
    }
    g_cp_async_commit();
    if (++aj == TP) {
      aj = 0;
      apl += stride;
    }
  };
#pragma unroll
  for (int q = 0; q < ST - 1; ++q) load(q);
  int s = 0;
  for (; pl < planes; pl += stride) {
    float P[MTM][NC][4], Q[MTM][NC][4];
#pragma unroll
    for (int mtm = 0; mtm < MTM; ++mtm)
#pragma unroll
      for (int nc = 0; nc < NC; ++nc)
#pragma unroll
        for (int e = 0; e < 4; ++e) P[mtm][nc][e] = Q[mtm][nc][e] = 0.f;
    for (int j = 0; j < TP; ++j) {
      load(s == 0 ? ST - 1 : s - 1);
      g_cp_async_wait<ST - 1>();
      __syncwarp();
      const float* T = S + (size_t)s * stage_floats;
#pragma unroll 1
      for (int gq = 0; gq < GPT; ++gq) {
        const float* Trow = T + (8 * gq + g8) * N3;         // this lane's row of the group (the B operand's n index)
        float accC[4] = {0.f, 0.f, 0.f, 0.f}, accS[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 2
        for (int ks = 0; ks < KS; ++ks) {
          const float4 ch = atab[((size_t)(0 * KS + ks) * 2 + 0) * 32 + lane], cl = atab[((size_t)(0 * KS + ks) * 2 + 1) * 32 + lane];
          const float4 sh = atab[((size_t)(1 * KS + ks) * 2 + 0) * 32 + lane], sl = atab[((size_t)(1 * KS + ks) * 2 + 1) * 32 + lane];
          uint32_t bsh[2], bsl[2], bdh[2], bdl[2];
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {                  // B fragment: pair t4 (+4)
            const int jj = 8 * ks + t4 + 4 * hh;
            const bool in = jj < half, mid = odd && jj == half;
            const int ja = (in || mid) ? jj : 0, jb = in ? N3 - 1 - jj : ja;
            const float a = Trow[ja], b = Trow[jb];
            g_split(in ? a + b : (mid ? a : 0.f), bsh[hh], bsl[hh]);
            g_split(in ? a - b : 0.f, bdh[hh], bdl[hh]);
          }
          const uint32_t chv[4] = {__float_as_uint(ch.x), __float_as_uint(ch.y), __float_as_uint(ch.z), __float_as_uint(ch.w)};
          const uint32_t clv[4] = {__float_as_uint(cl.x), __float_as_uint(cl.y), __float_as_uint(cl.z), __float_as_uint(cl.w)};
          const uint32_t shv[4] = {__float_as_uint(sh.x), __float_as_uint(sh.y), __float_as_uint(sh.z), __float_as_uint(sh.w)};
          const uint32_t slv[4] = {__float_as_uint(sl.x), __float_as_uint(sl.y), __float_as_uint(sl.z), __float_as_uint(sl.w)};
          mma3_tf32(accC, chv, clv, bsh[0], bsh[1], bsl[0], bsl[1]);
          mma3_tf32(accS, shv, slv, bdh[0], bdh[1], bdl[0], bdl[1]);
        }
        // X = rot (C - i S) of (frequency g8 + 8 fh, row 2 t4 + q): the second stage's column operand
        uint32_t bh[NC][2], bl[NC][2];
#pragma unroll
        for (int fh = 0; fh < NC / 2; ++fh)
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const float C = accC[2 * fh + q], Sv = accS[2 * fh + q];
            g_split(rot[fh].x * C + rot[fh].y * Sv, bh[2 * fh][q], bl[2 * fh][q]);          // real part
            g_split(rot[fh].y * C - rot[fh].x * Sv, bh[2 * fh + 1][q], bl[2 * fh + 1][q]);  // imaginary part
          }
        const int grp = j * GPT + gq;
#pragma unroll
        for (int mtm = 0; mtm < MTM; ++mtm) {
          uint32_t ch2[4], cl2[4], sh2[4], sl2[4];
          g_split4(a2tab[((size_t)(0 * NG + grp) * MTM + mtm) * 32 + lane], ch2, cl2);
          g_split4(a2tab[((size_t)(1 * NG + grp) * MTM + mtm) * 32 + lane], sh2, sl2);
#pragma unroll
          for (int nc = 0; nc < NC; ++nc) {
            mma3_tf32(P[mtm][nc], ch2, cl2, bh[nc][0], bh[nc][1], bl[nc][0], bl[nc][1]);
            mma3_tf32(Q[mtm][nc], sh2, sl2, bh[nc][0], bh[nc][1], bl[nc][0], bl[nc][1]);
          }
        }
      }
      __syncwarp();   // every lane is done with this stage before it is filled again
      s = s == ST - 1 ? 0 : s + 1;
    }
    // sum_n (cos - i sin)(Tr + i Ti) = (P_re + Q_im) + i (P_im - Q_re); a C fragment: modes g8 (+8), columns 2 t4 (+1)
    float2* ob = out + pl * (2 * K2) * K3;
#pragma unroll
    for (int mtm = 0; mtm < MTM; ++mtm)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int pm = 16 * mtm + g8 + 8 * h;
        if (pm >= 2 * K2) continue;
#pragma unroll
        for (int fh = 0; fh < NC / 2; ++fh) {
          const int f0 = 8 * fh + 2 * t4;
          float2 r[2];
#pragma unroll
          for (int q = 0; q < 2; ++q)
            r[q] = make_float2(P[mtm][2 * fh][2 * h + q] + Q[mtm][2 * fh + 1][2 * h + q],
                               P[mtm][2 * fh + 1][2 * h + q] - Q[mtm][2 * fh][2 * h + q]);
          float2* dst = ob + (long long)pm * K3 + f0;
          if (f0 + 1 < K3 && (K3 & 1) == 0) {
            *reinterpret_cast<float4*>(dst) = make_float4(r[0].x, r[0].y, r[1].x, r[1].y);
          } else {
            if (f0 < K3) dst[0] = r[0];
            if (f0 + 1 < K3) dst[1] = r[1];
          }
        }
      }
  }
}

constexpr int kGVS = 40;   // floats per row of the padded spectrum copy: 8 mod 32, conflict-free fragment loads

// MT: 16-row tiles per task; KSF: k-steps of 8 frequencies (k3 <= 8 KSF); KS2: k-steps of 8 modes (2 K2 <= 8 KS2)
template <int MT, int KSF, int KS2>
__global__ void __launch_bounds__(kGMaxWarps * 32, 1)
planeg_expand_kernel(const float2* __restrict__ in, float* __restrict__ y, long long planes, int N3, int K3, int N2,
                     int K2, float scale, int herm, int stage_floats) {
  pdl_trigger();
  constexpr int TR = 16 * MT, NC = 2 * KSF, VROWS = 8 * KS2;
  extern __shared__ float4 rg_smem[];
  const int half = N3 / 2, H = (N3 + 1) / 2, NTJ = (H + 7) / 8;
  const bool odd = (N3 & 1) != 0;
  const int NM = N2 / 16, TP = N2 / TR;
  float4* btab = rg_smem;                                   // [part][ks][ntj][lane], split: the contiguous stage's basis
  float4* a2e = btab + (size_t)2 * KSF * NTJ * 32;          // [part][16-row tile][ks2][lane], unsplit
  float* warp_area = reinterpret_cast<float*>(a2e + (size_t)2 * NM * KS2 * 32);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;
  const int W = blockDim.x >> 5;
  const int area_floats = stage_floats + 2 * VROWS * kGVS;
  float* st = warp_area + (size_t)warp * area_floats;       // output staging of a task
  float* Vs = st + stage_floats;                            // [2][VROWS][kGVS]: this plane's and the next plane's spectrum

  for (int e = threadIdx.x; e < 2 * KSF * NTJ * 32; e += blockDim.x) {
    const int l = e & 31;
    int r = e >> 5;
    const int ntj = r % NTJ;
    r /= NTJ;
    const int ks = r % KSF, part = r / KSF;
    const int j = 8 * ntj + (l >> 2);
    uint32_t hi[2], lo[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int f = 8 * ks + (l & 3) + 4 * h;
      split_tf32_rna((f < K3 && j < H) ? g_basis(part, f, j, N3) : 0.f, hi[h], lo[h]);
    }
    btab[e] = make_float4(__uint_as_float(hi[0]), __uint_as_float(hi[1]), __uint_as_float(lo[0]), __uint_as_float(lo[1]));
  }
  for (int e = threadIdx.x; e < 2 * NM * KS2 * 32; e += blockDim.x) {
    const int l = e & 31;
    int r = e >> 5;
    const int ks2 = r % KS2;
    r /= KS2;
    const int tile = r % NM, part = r / NM;
    float v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {                           // A fragment: row l >> 2 (+8), mode l & 3 (+4)
      const int n = 16 * tile + (l >> 2) + 8 * (q & 1), pm = 8 * ks2 + (l & 3) + 4 * (q >> 1);
      v[q] = pm < 2 * K2 ? g_basis2(part, pm, n, N2, K2) : 0.f;
    }
    a2e[e] = make_float4(v[0], v[1], v[2], v[3]);
  }
  // the padding of the spectrum copies (modes past 2 K2, columns past 2 k3) meets zero basis entries: it must be finite
  for (int e = lane; e < 2 * VROWS * kGVS; e += 32) Vs[e] = 0.f;
  float2 rot[KSF][2];
#pragma unroll
  for (int ks = 0; ks < KSF; ++ks)
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const int f = 8 * ks + t4 + 4 * hf;
      double sn, cs;
      sincospi((double)f / (double)N3, &sn, &cs);
      const float wgt = (f < K3) ? scale * (herm ? herm_weight(f, N3) : 1.0f) : 0.f;
      rot[ks][hf] = make_float2((float)cs * wgt, -(float)sn * wgt);
    }
  __syncthreads();
  pdl_wait();

  const long long stride = (long long)W * gridDim.x;
  const int npieces = 2 * K2 * K3;                          // complex values of a plane's spectrum
  auto fetch = [&](long long plane, int buf) {
    if (plane < planes) {
      const float2* src = in + plane * npieces;
      float* dst = Vs + (size_t)buf * VROWS * kGVS;
      for (int i = lane; i < npieces; i += 32) g_cp_async8(dst + (i / K3) * kGVS + 2 * (i % K3), src + i);
    }
    g_cp_async_commit();
  };
  long long pl = (long long)warp * gridDim.x + blockIdx.x;
  fetch(pl, 0);
  int vb = 0;
  for (; pl < planes; pl += stride, vb ^= 1) {
    fetch(pl + stride, vb ^ 1);
    g_cp_async_wait<1>();
    __syncwarp();
    const float* V = Vs + (size_t)vb * VROWS * kGVS;
    for (int j = 0; j < TP; ++j) {
#pragma unroll 1
      for (int mt = 0; mt < MT; ++mt) {
        const int tile = j * MT + mt;
        // the second dimension: U[row][f] = sum_p e^{+i phi} V[p][f]
        float P[NC][4], Q[NC][4];
#pragma unroll
        for (int nc = 0; nc < NC; ++nc)
#pragma unroll
          for (int e = 0; e < 4; ++e) P[nc][e] = Q[nc][e] = 0.f;
#pragma unroll
        for (int ks2 = 0; ks2 < KS2; ++ks2) {
          uint32_t ch2[4], cl2[4], sh2[4], sl2[4];
          g_split4(a2e[((size_t)(0 * NM + tile) * KS2 + ks2) * 32 + lane], ch2, cl2);
          g_split4(a2e[((size_t)(1 * NM + tile) * KS2 + ks2) * 32 + lane], sh2, sl2);
#pragma unroll
          for (int nc = 0; nc < NC; ++nc) {
            uint32_t b0h, b0l, b1h, b1l;
            g_split(V[(8 * ks2 + t4) * kGVS + 8 * nc + g8], b0h, b0l);
            g_split(V[(8 * ks2 + t4 + 4) * kGVS + 8 * nc + g8], b1h, b1l);
            mma3_tf32(P[nc], ch2, cl2, b0h, b1h, b0l, b1l);
            mma3_tf32(Q[nc], sh2, sl2, b0h, b1h, b0l, b1l);
          }
        }
        // (cos + i sin)(Vr + i Vi): U_re = P_re - Q_im, U_im = P_im + Q_re; rotated, it is the contiguous stage's row operand
        uint32_t rh[KSF][4], rl[KSF][4], ih[KSF][4], il[KSF][4];
#pragma unroll
        for (int ks = 0; ks < KSF; ++ks)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int nc = 2 * ks + (e >> 1), h = e & 1;
            const float ur = P[nc][2 * h] - Q[nc][2 * h + 1], ui = P[nc][2 * h + 1] + Q[nc][2 * h];
            const float2 r = rot[ks][e >> 1];
            g_split(ur * r.x - ui * r.y, rh[ks][e], rl[ks][e]);
            g_split(ur * r.y + ui * r.x, ih[ks][e], il[ks][e]);
          }
#pragma unroll 1
        for (int ntj = 0; ntj < NTJ; ++ntj) {
          float Pj[4] = {0.f, 0.f, 0.f, 0.f}, Qj[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int ks = 0; ks < KSF; ++ks) {
            const float4 bc = btab[((size_t)(0 * KSF + ks) * NTJ + ntj) * 32 + lane];
            const float4 bs = btab[((size_t)(1 * KSF + ks) * NTJ + ntj) * 32 + lane];
            mma3_tf32(Pj, rh[ks], rl[ks], __float_as_uint(bc.x), __float_as_uint(bc.y), __float_as_uint(bc.z), __float_as_uint(bc.w));
            mma3_tf32(Qj, ih[ks], il[ks], __float_as_uint(bs.x), __float_as_uint(bs.y), __float_as_uint(bs.z), __float_as_uint(bs.w));
          }
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float* srow = st + (16 * mt + g8 + 8 * h) * N3;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const int jj = 8 * ntj + 2 * t4 + q;
              const float pv = Pj[2 * h + q], qv = Qj[2 * h + q];
              if (jj < half) {
                srow[jj] = pv - qv;
                srow[N3 - 1 - jj] = pv + qv;
              } else if (odd && jj == half) {
                srow[jj] = pv;
              }
            }
          }
        }
      }
      __syncwarp();
      {
        float* dst = y + (pl * N2 + (long long)j * TR) * N3;
        for (int i = lane; i < (TR * N3) / 4; i += 32)
          __stcs(reinterpret_cast<float4*>(dst) + i, *reinterpret_cast<const float4*>(st + 4 * i));
      }
      __syncwarp();   // the staging area is read out before the next task writes to it
    }
    __syncwarp();     // this plane's spectrum copy is not needed any more: the plane after next may land in it
  }
}

struct GCfg {
  int warps;
  size_t smem;
};

// the most warps (<= 12) whose per-warp areas fit next to the basis table
GCfg g_cfg(size_t table_bytes, size_t per_warp_bytes) {
  GCfg c{0, 0};
  if (table_bytes + 2 * per_warp_bytes > kGSmemLimit) return c;
  int w = (int)((kGSmemLimit - table_bytes) / per_warp_bytes);
  if (w > kGMaxWarps) w = kGMaxWarps;
  c.warps = w;
  c.smem = table_bytes + (size_t)w * per_warp_bytes;
  return c;
}

int g_mt(int N3) { return N3 <= 64 ? 2 : 1; }
int g_stage_floats(int N3, int mt) { return (16 * mt * N3 + 3) & ~3; }

// three ring stages where at least four warps of them fit, else two
int g_stages(size_t table_bytes, size_t stage_bytes) { return g_cfg(table_bytes, 3 * stage_bytes).warps >= 4 ? 3 : 2; }

template <int MT, int NT, int ST>
cudaError_t launch_contract_s(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm,
                              cudaStream_t st) {
  const int H = (N3 + 1) / 2, KS = (H + 7) / 8;
  const int sf = g_stage_floats(N3, MT);
  const GCfg c = g_cfg((size_t)2 * KS * NT * 32 * 16, (size_t)ST * sf * 4);
  if (c.warps < 2) return cudaErrorInvalidConfiguration;
  auto kern = rowg_contract_kernel<MT, NT, ST>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem);
  if (e != cudaSuccess) return e;
  const long long tasks = (rows + 16 * MT - 1) / (16 * MT);
  const long long want = (tasks + c.warps - 1) / c.warps;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3(c.warps * 32), c.smem, st, x, out, rows, N3, K3, scale, herm, sf);
  return cudaGetLastError();
}

template <int MT, int NT>
cudaError_t launch_contract_t(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm,
                              cudaStream_t st) {
  const int H = (N3 + 1) / 2, KS = (H + 7) / 8;
  const size_t sb = (size_t)g_stage_floats(N3, MT) * 4;
  return g_stages((size_t)2 * KS * NT * 32 * 16, sb) == 3 ? launch_contract_s<MT, NT, 3>(x, out, rows, N3, K3, scale, herm, st)
                                                          : launch_contract_s<MT, NT, 2>(x, out, rows, N3, K3, scale, herm, st);
}

template <int MT, int KSF>
cudaError_t launch_expand_t(const float2* in, float* y, long long rows, int N3, int K3, float scale, int herm,
                            cudaStream_t st) {
  const int H = (N3 + 1) / 2, NTJ = (H + 7) / 8;
  const int sf = g_stage_floats(N3, MT);
  const GCfg c = g_cfg((size_t)2 * KSF * NTJ * 32 * 16, (size_t)sf * 4);
  if (c.warps < 2) return cudaErrorInvalidConfiguration;
  auto kern = rowg_expand_kernel<MT, KSF>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem);
  if (e != cudaSuccess) return e;
  const long long tasks = (rows + 16 * MT - 1) / (16 * MT);
  const long long want = (tasks + c.warps - 1) / c.warps;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3(c.warps * 32), c.smem, st, in, y, rows, N3, K3, scale, herm, sf);
  return cudaGetLastError();
}

// shared memory of the two plane kernels: tables, then per-warp areas
size_t pg_contract_table(int N3, int N2, int MTM) {
  const int KS = ((N3 + 1) / 2 + 7) / 8;
  return ((size_t)2 * KS * 2 + (size_t)2 * (N2 / 8) * MTM) * 32 * 16;
}
size_t pg_expand_table(int N3, int N2, int KSF, int KS2) {
  const int NTJ = ((N3 + 1) / 2 + 7) / 8;
  return ((size_t)2 * KSF * NTJ + (size_t)2 * (N2 / 16) * KS2) * 32 * 16;
}

template <int MT, int NC, int MTM, int ST>
cudaError_t launch_pg_contract_s(const float* x, float2* out, long long planes, int N3, int K3, int N2, int K2,
                                 float scale, int herm, cudaStream_t st) {
  const int sf = g_stage_floats(N3, MT);
  const GCfg c = g_cfg(pg_contract_table(N3, N2, MTM), (size_t)ST * sf * 4);
  if (c.warps < 2) return cudaErrorInvalidConfiguration;
  auto kern = planeg_contract_kernel<MT, NC, MTM, ST>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem);
  if (e != cudaSuccess) return e;
  const long long want = (planes + c.warps - 1) / c.warps;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3(c.warps * 32), c.smem, st, x, out, planes, N3, K3, N2, K2, scale, herm, sf);
  return cudaGetLastError();
}

template <int MT, int NC, int MTM>
cudaError_t launch_pg_contract_t(const float* x, float2* out, long long planes, int N3, int K3, int N2, int K2,
                                 float scale, int herm, cudaStream_t st) {
  const size_t sb = (size_t)g_stage_floats(N3, MT) * 4;
  return g_stages(pg_contract_table(N3, N2, MTM), sb) == 3
             ? launch_pg_contract_s<MT, NC, MTM, 3>(x, out, planes, N3, K3, N2, K2, scale, herm, st)
             : launch_pg_contract_s<MT, NC, MTM, 2>(x, out, planes, N3, K3, N2, K2, scale, herm, st);
}

template <int MT, int KSF, int KS2>
cudaError_t launch_pg_expand_t(const float2* in, float* y, long long planes, int N3, int K3, int N2, int K2,
                               float scale, int herm, cudaStream_t st) {
  const int sf = g_stage_floats(N3, MT);
  const GCfg c = g_cfg(pg_expand_table(N3, N2, KSF, KS2), ((size_t)sf + 2 * 8 * KS2 * kGVS) * 4);
  if (c.warps < 2) return cudaErrorInvalidConfiguration;
  auto kern = planeg_expand_kernel<MT, KSF, KS2>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem);
  if (e != cudaSuccess) return e;
  const long long want = (planes + c.warps - 1) / c.warps;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3(c.warps * 32), c.smem, st, in, y, planes, N3, K3, N2, K2, scale, herm, sf);
  return cudaGetLastError();
}

}  // namespace

// The plane kernels of this file: any contiguous extent up to 256 with up to 16 one-sided modes, a second extent that
// is a whole number of tasks (16 rows; 32 for N3 <= 64) up to 256 with 1..16 modes per side; both kernels must
// have room for four warps.
bool planeg_supported(int N3, int K3, int N2, int K2) {
  if (N3 < 2 || N3 > 256 || K3 < 1 || K3 > 16 || K3 > N3 / 2 + 1) return false;
  const int mt = g_mt(N3);
  if (N2 < 16 * mt || N2 > 256 || N2 % (16 * mt) != 0 || K2 < 1 || K2 > 16 || 2 * K2 > N2) return false;
  const int MTM = (2 * K2 + 15) / 16, KS2 = (2 * K2 + 7) / 8, KSF = (K3 + 7) / 8;
  const size_t sf = (size_t)g_stage_floats(N3, mt) * 4;
  const size_t ct = pg_contract_table(N3, N2, MTM), et = pg_expand_table(N3, N2, KSF, KS2);
  if (ct + 4 * 2 * sf > kGSmemLimit) return false;
  return g_cfg(ct, g_stages(ct, sf) * sf).warps >= 4 && g_cfg(et, sf + (size_t)2 * 8 * KS2 * kGVS * 4).warps >= 4;
}

cudaError_t launch_planeg_contract(const float* x, float2* out, long long planes, int N3, int K3, int N2, int K2,
                                   float scale, int herm, cudaStream_t st) {
  const bool two = g_mt(N3) == 2, wide = K3 > 8, tall = 2 * K2 > 16;
#define DTST_PG(MT, NC, MTM) return launch_pg_contract_t<MT, NC, MTM>(x, out, planes, N3, K3, N2, K2, scale, herm, st)
  if (two) {
    if (wide) { if (tall) DTST_PG(2, 4, 2); DTST_PG(2, 4, 1); }
    if (tall) DTST_PG(2, 2, 2);
    DTST_PG(2, 2, 1);
  }
  if (wide) { if (tall) DTST_PG(1, 4, 2); DTST_PG(1, 4, 1); }
  if (tall) DTST_PG(1, 2, 2);
  DTST_PG(1, 2, 1);
#undef DTST_PG
}

cudaError_t launch_planeg_expand(const float2* in, float* y, long long planes, int N3, int K3, int N2, int K2,
                                 float scale, int herm, cudaStream_t st) {
  const bool two = g_mt(N3) == 2;
  const int KSF = (K3 + 7) / 8, KS2 = (2 * K2 + 7) / 8;
#define DTST_PG(MT, A, B) \
  if (two == (MT == 2) && KSF == A && KS2 == B) return launch_pg_expand_t<MT, A, B>(in, y, planes, N3, K3, N2, K2, scale, herm, st);
  DTST_PG(2, 1, 1) DTST_PG(2, 1, 2) DTST_PG(2, 1, 3) DTST_PG(2, 1, 4)
  DTST_PG(2, 2, 1) DTST_PG(2, 2, 2) DTST_PG(2, 2, 3) DTST_PG(2, 2, 4)
  DTST_PG(1, 1, 1) DTST_PG(1, 1, 2) DTST_PG(1, 1, 3) DTST_PG(1, 1, 4)
  DTST_PG(1, 2, 1) DTST_PG(1, 2, 2) DTST_PG(1, 2, 3) DTST_PG(1, 2, 4)
#undef DTST_PG
  return cudaErrorNotSupported;
}

// Any extent up to 512 and up to 32 retained one-sided modes (the Nyquist mode of an even extent included); the
// extent times 64 bytes must leave room for two warps' areas beside the basis table.
bool rowg_supported(int N3, int K3) {
  if (N3 < 2 || N3 > 512 || K3 < 1 || K3 > 32 || K3 > N3 / 2 + 1) return false;
  const int H = (N3 + 1) / 2, KS = (H + 7) / 8, NT = (K3 + 7) / 8;
  const int mt = (NT > 2) ? 1 : g_mt(N3);
  const size_t sf = (size_t)g_stage_floats(N3, mt) * 4;
  const size_t table = (size_t)2 * KS * NT * 32 * 16;
  return g_cfg(table, g_stages(table, sf) * sf).warps >= 2 && g_cfg(table, sf).warps >= 2;
}

cudaError_t launch_rowg_contract(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm,
                                 cudaStream_t st) {
  const int NT = (K3 + 7) / 8;
  const bool two = g_mt(N3) == 2;
  switch (NT) {
    case 1: return two ? launch_contract_t<2, 1>(x, out, rows, N3, K3, scale, herm, st)
                       : launch_contract_t<1, 1>(x, out, rows, N3, K3, scale, herm, st);
    case 2: return two ? launch_contract_t<2, 2>(x, out, rows, N3, K3, scale, herm, st)
                       : launch_contract_t<1, 2>(x, out, rows, N3, K3, scale, herm, st);
    case 3: return launch_contract_t<1, 3>(x, out, rows, N3, K3, scale, herm, st);
    default: return launch_contract_t<1, 4>(x, out, rows, N3, K3, scale, herm, st);
  }
}

cudaError_t launch_rowg_expand(const float2* in, float* y, long long rows, int N3, int K3, float scale, int herm,
                               cudaStream_t st) {
  const int KSF = (K3 + 7) / 8;
  const bool two = g_mt(N3) == 2;
  switch (KSF) {
    case 1: return two ? launch_expand_t<2, 1>(in, y, rows, N3, K3, scale, herm, st)
                       : launch_expand_t<1, 1>(in, y, rows, N3, K3, scale, herm, st);
    case 2: return two ? launch_expand_t<2, 2>(in, y, rows, N3, K3, scale, herm, st)
                       : launch_expand_t<1, 2>(in, y, rows, N3, K3, scale, herm, st);
    case 3: return launch_expand_t<1, 3>(in, y, rows, N3, K3, scale, herm, st);
    default: return launch_expand_t<1, 4>(in, y, rows, N3, K3, scale, herm, st);
  }
}

}  // namespace dtst
