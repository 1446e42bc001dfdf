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
constexpr int kGMaxWarps = 16;

__device__ __forceinline__ void g_cp_async16(float* smem_dst, const float* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}
__device__ __forceinline__ void g_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void g_cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// hi = the value with its low 13 mantissa bits cleared, lo = the exact rest (the tensor core drops lo's low bits).
// FAST (single-pass TF32, a plan option): the value rounded to the 11 bits the tensor core reads (it ignores the
// low 13 bits, so adding half a unit of the last kept bit rounds); no lo part - every use of it below disappears.
template <bool FAST>
__device__ __forceinline__ void g_split(float v, uint32_t& hi, uint32_t& lo) {
  if (FAST) {
    hi = __float_as_uint(v) + 0x1000u;
    lo = 0u;
  } else {
    hi = __float_as_uint(v) & 0xffffe000u;
    lo = __float_as_uint(v - __uint_as_float(hi));
  }
}
// one product: compensated (three MMAs, d += (ahi + alo)(bhi + blo) without lo * lo) or, FAST, the hi parts alone
template <bool FAST>
__device__ __forceinline__ void g_mma3(float (&d)[4], const uint32_t (&ahi)[4], const uint32_t (&alo)[4], uint32_t bh0,
                                       uint32_t bh1, uint32_t bl0, uint32_t bl1) {
  if (FAST) mma_m16n8k8_tf32(d, ahi, bh0, bh1);
  else mma3_tf32(d, ahi, alo, bh0, bh1, bl0, bl1);
}

__device__ __forceinline__ void g_bits(const float4& v, uint32_t (&o)[4]) {
  o[0] = __float_as_uint(v.x);
  o[1] = __float_as_uint(v.y);
  o[2] = __float_as_uint(v.z);
  o[3] = __float_as_uint(v.w);
}
// one compensated product with the 8-column operand as a table entry (b0 hi, b1 hi, b0 lo, b1 lo)
template <bool FAST>
__device__ __forceinline__ void g_mma3q(float (&d)[4], const uint32_t (&ahi)[4], const uint32_t (&alo)[4], const float4& b) {
  g_mma3<FAST>(d, ahi, alo, __float_as_uint(b.x), __float_as_uint(b.y), __float_as_uint(b.z), __float_as_uint(b.w));
}

// cos (part 0) or sin (part 1) of 2 pi f (j + 1/2) / N, the phase reduced exactly in integers
__device__ __forceinline__ float g_basis(int part, int f, int j, int N) {
  double s, c;
  sincospi((double)(((long long)f * (2 * j + 1)) % (2ll * N)) / (double)N, &s, &c);
  return part == 0 ? (float)c : (float)s;
}
// The same for the CONTRACTION tables.  The kernels form s_j = x_j + x_{N-1-j}, d_j = x_j - x_{N-1-j} for every pair
// index without looking at it: the middle sample of an odd extent pairs with itself (s = 2 x, d = 0), so its cosine
// carries the weight 1/2; pair indices past the end are clamped to the last pair and meet zero table entries.
__device__ __forceinline__ float g_basis_c(int part, int f, int j, int N) {
  const float v = g_basis(part, f, j, N);
  return ((N & 1) && j == N / 2 && part == 0) ? 0.5f * v : v;
}

// ---------------------------------------------------------------------------------------------
// contraction.  MT m-tiles of 16 rows per task, NT n-tiles of 8 frequencies (k3 <= 8 NT).
// ---------------------------------------------------------------------------------------------
template <int MT, int NT, int ST, bool FAST>
__global__ void __launch_bounds__(kGMaxWarps * 32, 1)
rowg_contract_kernel(const float* __restrict__ x, float2* __restrict__ out, long long rows, int N3, int K3, float scale,
                     int herm, int stage_floats) {
  pdl_trigger();
  constexpr int TR = 16 * MT;
  extern __shared__ float4 rg_smem[];
  const int H = (N3 + 1) / 2, KS = (H + 7) / 8;   // pairs (odd N3: + the middle sample), k-steps
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
      split_tf32_rna((f < K3 && j < H) ? g_basis_c(part, f, j, N3) : 0.f, hi[h], lo[h]);
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
          const int j = min(8 * ks + t4 + 4 * (e >> 1), H - 1);   // past the end: any pair, its table entries are zero
          const float a = T[row * N3 + j], b = T[row * N3 + N3 - 1 - j];
          g_split<FAST>(a + b, sh[e], sl[e]);
          g_split<FAST>(a - b, dh[e], dl[e]);
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          g_mma3q<FAST>(accC[mt][nt], sh, sl, bc[nt]);
          g_mma3q<FAST>(accS[mt][nt], dh, dl, bs[nt]);
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
// contraction of LONG rows (N3 > 256, e.g. a 421 x 421 grid): tasks of 8 rows, so that a stage is half as large and
// twice as many warps fit an SM (with 16-row tasks three).  The product runs transposed - [16 frequencies x pairs] x
// [pairs x 8 rows], as the first stage of planeg_contract_kernel below - and a C fragment holds the frequencies
// g8 / g8 + 8 of the rows 2 t4, 2 t4 + 1.  MTF: 16-frequency tiles (k3 <= 16 MTF).
// ---------------------------------------------------------------------------------------------
template <int MTF, int ST, bool FAST>
__global__ void __launch_bounds__(kGMaxWarps * 32, 1)
rowg_contract8_kernel(const float* __restrict__ x, float2* __restrict__ out, long long rows, int N3, int K3, float scale,
                      int herm, int stage_floats) {
  pdl_trigger();
  extern __shared__ float4 rg_smem[];
  const int H = (N3 + 1) / 2, KS = (H + 7) / 8;
  float4* atab = rg_smem;                                          // [part][ks][mtf][hi | lo][lane]
  float* ring = reinterpret_cast<float*>(atab + (size_t)2 * KS * MTF * 2 * 32);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;
  const int W = blockDim.x >> 5;

  for (int e = threadIdx.x; e < 2 * KS * MTF * 32; e += blockDim.x) {
    const int l = e & 31;
    int r = e >> 5;
    const int mtf = r % MTF;
    r /= MTF;
    const int ks = r % KS, part = r / KS;
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {                                  // A fragment: frequency l >> 2 (+8), pair l & 3 (+4)
      const int f = 16 * mtf + (l >> 2) + 8 * (q & 1), j = 8 * ks + (l & 3) + 4 * (q >> 1);
      split_tf32_rna((f < K3 && j < H) ? g_basis_c(part, f, j, N3) : 0.f, hi[q], lo[q]);
    }
    float4* dst = atab + ((size_t)((part * KS + ks) * MTF + mtf) * 2) * 32 + l;
    dst[0] = make_float4(__uint_as_float(hi[0]), __uint_as_float(hi[1]), __uint_as_float(hi[2]), __uint_as_float(hi[3]));
    dst[32] = make_float4(__uint_as_float(lo[0]), __uint_as_float(lo[1]), __uint_as_float(lo[2]), __uint_as_float(lo[3]));
  }
  float2 rot[MTF][2];                                              // frequencies 16 mtf + g8 (+8)
#pragma unroll
  for (int mtf = 0; mtf < MTF; ++mtf)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int f = 16 * mtf + g8 + 8 * h;
      double sn, cs;
      sincospi((double)f / (double)N3, &sn, &cs);
      const float wgt = scale * (herm ? herm_weight(f, N3) : 1.0f);
      rot[mtf][h] = make_float2((float)cs * wgt, (float)sn * wgt);
    }
  __syncthreads();
  pdl_wait();

  float* S = ring + (size_t)warp * ST * stage_floats;
  const long long tasks = (rows + 7) / 8;
  const long long stride = (long long)W * gridDim.x;
  auto load = [&](long long t, int s) {
    if (t < tasks) {
      const long long r0 = t * 8;
      const long long nr = rows - r0 < 8 ? rows - r0 : 8;
      const int nf = (int)(nr * N3);
      const float* src = x + r0 * N3;
      float* dst = S + (size_t)s * stage_floats;
      for (int i = lane; i < (nf >> 2); i += 32) g_cp_async16(dst + 4 * i, src + 4 * i);
      const int done = nf & ~3;
      if (lane < (nf & 3)) dst[done + lane] = __ldg(src + done + lane);
    }
    g_cp_async_commit();
  };
  const int jl0 = min(8 * (KS - 1) + t4, H - 1), jl1 = min(8 * (KS - 1) + t4 + 4, H - 1);
  long long t = (long long)warp * gridDim.x + blockIdx.x;
#pragma unroll
  for (int q = 0; q < ST - 1; ++q) load(t + q * stride, q);
  int s = 0;
  for (; t < tasks; t += stride, s = s == ST - 1 ? 0 : s + 1) {
    load(t + (ST - 1) * stride, s == 0 ? ST - 1 : s - 1);
    g_cp_async_wait<ST - 1>();
    __syncwarp();
    const float* Trow = S + (size_t)s * stage_floats + g8 * N3;   // this lane's row (the B operand's n index)
    // accC / accS: the running sums; cC / cS: the sums of up to eight k-steps, added to them with ordinary fp32
    // additions (the tensor core's accumulate step truncates: one chain through all k-steps of a 512-point row cost
    // half of the error budget)
    float accC[MTF][4], accS[MTF][4], cC[MTF][4], cS[MTF][4];
#pragma unroll
    for (int mtf = 0; mtf < MTF; ++mtf)
#pragma unroll
      for (int e = 0; e < 4; ++e) accC[mtf][e] = accS[mtf][e] = cC[mtf][e] = cS[mtf][e] = 0.f;
    auto flush = [&]() {
#pragma unroll
      for (int mtf = 0; mtf < MTF; ++mtf)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          accC[mtf][e] += cC[mtf][e];
          accS[mtf][e] += cS[mtf][e];
          cC[mtf][e] = cS[mtf][e] = 0.f;
        }
    };
    auto step = [&](int ks, int j0, int j1) {
      const float a0 = Trow[j0], b0 = Trow[N3 - 1 - j0], a1 = Trow[j1], b1 = Trow[N3 - 1 - j1];
      uint32_t bsh[2], bsl[2], bdh[2], bdl[2];
      g_split<FAST>(a0 + b0, bsh[0], bsl[0]);
      g_split<FAST>(a0 - b0, bdh[0], bdl[0]);
      g_split<FAST>(a1 + b1, bsh[1], bsl[1]);
      g_split<FAST>(a1 - b1, bdh[1], bdl[1]);
#pragma unroll
      for (int mtf = 0; mtf < MTF; ++mtf) {
        const float4* ac = atab + ((ks * MTF + mtf) * 2) * 32 + lane;
        const float4* as = atab + (((KS + ks) * MTF + mtf) * 2) * 32 + lane;
        uint32_t chv[4], clv[4], shv[4], slv[4];
        g_bits(ac[0], chv);
        g_bits(ac[32], clv);
        g_bits(as[0], shv);
        g_bits(as[32], slv);
        g_mma3<FAST>(cC[mtf], chv, clv, bsh[0], bsh[1], bsl[0], bsl[1]);
        g_mma3<FAST>(cS[mtf], shv, slv, bdh[0], bdh[1], bdl[0], bdl[1]);
      }
    };
    for (int k0 = 0; k0 < KS - 1; k0 += 8) {
      const int k1 = k0 + 8 < KS - 1 ? k0 + 8 : KS - 1;
#pragma unroll 2
      for (int ks = k0; ks < k1; ++ks) step(ks, 8 * ks + t4, 8 * ks + t4 + 4);
      flush();
    }
    step(KS - 1, jl0, jl1);
    flush();
    // X_f = rot_f (C_f - i S_f): frequency 16 mtf + g8 + 8 h of the rows 2 t4 + q
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const long long row = t * 8 + 2 * t4 + q;
      if (row >= rows) continue;
#pragma unroll
      for (int mtf = 0; mtf < MTF; ++mtf)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int f = 16 * mtf + g8 + 8 * h;
          const float C = accC[mtf][2 * h + q], Sv = accS[mtf][2 * h + q];
          if (f < K3)
            out[row * K3 + f] = make_float2(rot[mtf][h].x * C + rot[mtf][h].y * Sv, rot[mtf][h].y * C - rot[mtf][h].x * Sv);
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
template <int MT, int KSF, bool FAST>
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
          g_split<FAST>(v.x * r.x - v.y * r.y, rh[mt][ks][e], rl[mt][ks][e]);
          g_split<FAST>(v.x * r.y + v.y * r.x, ih[mt][ks][e], il[mt][ks][e]);
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
          g_mma3q<FAST>(P, rh[mt][ks], rl[mt][ks], bc[ks]);
          g_mma3q<FAST>(Q, ih[mt][ks], il[mt][ks], bs[ks]);
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
// Nothing is transposed through shared memory; the plane's sums live in C fragments until its last row.
// The second stage is folded over the sign of the mode: cos(k phi) serves +k and -k, sin(k phi) too up to its sign, so
// its 16-row operand holds [cos k phi, k < K2 | sin k phi, k = 1..K2] (2 K2 rows, ONE product instead of a cosine and a
// sine product over all 2 K2 modes) and Z_{+k} = A_k - i B_k, Z_{-k} = A_k + i B_k are formed at the plane's end; the
// one term left over, A_{K2} = sum cos(K2 phi) T of the unpaired mode -K2, runs on FFMA.
//
// Expansion.  The second dimension first: [16 rows x modes] x [modes x (re, im) columns] from the plane's spectrum
// (a padded copy in shared memory, fetched one plane ahead); its C fragment (rows g8 / g8 + 8, the complex value of
// frequency 4 nc + t4) is exactly the row operand of the contiguous stage (frequency 8 ks + t4 + 4 half <-> n-tile
// 2 ks + half), which then runs as in rowg_expand_kernel.  The same fold: U = sum_k cos(k phi) E_k + sin(k phi) (i O_k)
// with E_k = V_k + V_{-k}, O_k = V_k - V_{-k} formed once per plane in shared memory (the factor i is a swap of the
// real and imaginary columns), one product over 2 K2 entries; cos(K2 phi) V_{-K2} is added on FFMA.
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

// entry r of the folded second-stage basis at row n: cos(2 pi r n / N2) for r < K2, sin(2 pi (r - K2 + 1) n / N2) for
// K2 <= r < 2 K2, zero beyond
__device__ __forceinline__ float g_basis2f(int r, int n, int N2, int K2) {
  if (r >= 2 * K2) return 0.f;
  const long long k = r < K2 ? r : r - K2 + 1;
  double s, c;
  sincospi(2.0 * (double)((k * n) % N2) / (double)N2, &s, &c);
  return r < K2 ? (float)c : (float)s;
}

template <bool FAST>
__device__ __forceinline__ void g_split4(const float4& v, uint32_t (&hi)[4], uint32_t (&lo)[4]) {
  g_split<FAST>(v.x, hi[0], lo[0]);
  g_split<FAST>(v.y, hi[1], lo[1]);
  g_split<FAST>(v.z, hi[2], lo[2]);
  g_split<FAST>(v.w, hi[3], lo[3]);
}

// MT: 16-row tiles per task; NC: n-tiles of the second stage (2 for k3 <= 8, else 4); MTM: 16-mode tiles (2 K2 <= 16 MTM)
template <int MT, int NC, int MTM, int ST, bool FAST>
__global__ void __launch_bounds__(kGMaxWarps * 32, 1)
planeg_contract_kernel(const float* __restrict__ x, float2* __restrict__ out, long long planes, int N3, int K3, int N2,
                       int K2, float scale, int herm, int stage_floats) {
  pdl_trigger();
  constexpr int TR = 16 * MT, GPT = 2 * MT;   // rows and 8-row groups per task
  extern __shared__ float4 rg_smem[];
  const int H = (N3 + 1) / 2, KS = (H + 7) / 8;
  const int NG = N2 / 8, TP = N2 / TR;
  float4* atab = rg_smem;                                   // [part][ks][hi | lo][lane]: the row stage's 16-row operand
  float4* a2tab = atab + (size_t)2 * KS * 2 * 32;           // [group][mtm][lane]: the second stage's, folded, unsplit
  float* cK = reinterpret_cast<float*>(a2tab + (size_t)NG * MTM * 32);   // cos(2 pi K2 n / N2)
  float* ring = cK + ((N2 + 3) & ~3);
  constexpr int SCW = 34, SCRF = ((16 * MTM + 1) * SCW + 3) & ~3;   // per-warp scratch of the plane's end: rows of 34 floats
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;
  const int W = blockDim.x >> 5;

  for (int e = threadIdx.x; e < 2 * KS * 32; e += blockDim.x) {
    const int l = e & 31, ks = (e >> 5) % KS, part = (e >> 5) / KS;
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {                           // A fragment: frequency l >> 2 (+8), pair l & 3 (+4)
      const int f = (l >> 2) + 8 * (q & 1), j = 8 * ks + (l & 3) + 4 * (q >> 1);
      split_tf32_rna((f < K3 && j < H) ? g_basis_c(part, f, j, N3) : 0.f, hi[q], lo[q]);
    }
    atab[((size_t)(part * KS + ks) * 2 + 0) * 32 + l] =
        make_float4(__uint_as_float(hi[0]), __uint_as_float(hi[1]), __uint_as_float(hi[2]), __uint_as_float(hi[3]));
    atab[((size_t)(part * KS + ks) * 2 + 1) * 32 + l] =
        make_float4(__uint_as_float(lo[0]), __uint_as_float(lo[1]), __uint_as_float(lo[2]), __uint_as_float(lo[3]));
  }
  for (int e = threadIdx.x; e < NG * MTM * 32; e += blockDim.x) {
    const int l = e & 31, mtm = (e >> 5) % MTM, grp = (e >> 5) / MTM;
    float v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)                             // A fragment: basis row l >> 2 (+8), grid row 2 (l & 3) (+1)
      v[q] = g_basis2f(16 * mtm + (l >> 2) + 8 * (q & 1), 8 * grp + 2 * (l & 3) + (q >> 1), N2, K2);
    a2tab[e] = make_float4(v[0], v[1], v[2], v[3]);
  }
  for (int n = threadIdx.x; n < N2; n += blockDim.x) cK[n] = g_basis2(0, K2, n, N2, K2);   // position K2 is the mode -K2
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

  float* S = ring + (size_t)warp * (ST * stage_floats + SCRF);
  float* scr = S + (size_t)ST * stage_floats;
  const int jl0 = min(8 * (KS - 1) + t4, H - 1), jl1 = min(8 * (KS - 1) + t4 + 4, H - 1);
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
    float P[MTM][NC][4];
    float lw[NC];                                           // this lane's share of the left-over sums A_{K2}
#pragma unroll
    for (int nc = 0; nc < NC; ++nc) lw[nc] = 0.f;
#pragma unroll
    for (int mtm = 0; mtm < MTM; ++mtm)
#pragma unroll
      for (int nc = 0; nc < NC; ++nc)
#pragma unroll
        for (int e = 0; e < 4; ++e) P[mtm][nc][e] = 0.f;
    for (int j = 0; j < TP; ++j) {
      load(s == 0 ? ST - 1 : s - 1);
      g_cp_async_wait<ST - 1>();
      __syncwarp();
      const float* T = S + (size_t)s * stage_floats;
#pragma unroll 1
      for (int gq = 0; gq < GPT; ++gq) {
        const float* Trow = T + (8 * gq + g8) * N3;         // this lane's row of the group (the B operand's n index)
        float accC[4] = {0.f, 0.f, 0.f, 0.f}, accS[4] = {0.f, 0.f, 0.f, 0.f};
        // one k-step: the pairs at the columns (j0, N3-1-j0) and (j1, N3-1-j1)
        auto step = [&](int ks, int j0, int j1) {
          const float4* at = atab + ks * 64 + lane;
          const float4 ch = at[0], cl = at[32], sh = at[KS * 64], sl = at[KS * 64 + 32];
          const float a0 = Trow[j0], b0 = Trow[N3 - 1 - j0], a1 = Trow[j1], b1 = Trow[N3 - 1 - j1];
          uint32_t bsh[2], bsl[2], bdh[2], bdl[2];
          g_split<FAST>(a0 + b0, bsh[0], bsl[0]);
          g_split<FAST>(a0 - b0, bdh[0], bdl[0]);
          g_split<FAST>(a1 + b1, bsh[1], bsl[1]);
          g_split<FAST>(a1 - b1, bdh[1], bdl[1]);
          uint32_t chv[4], clv[4], shv[4], slv[4];
          g_bits(ch, chv);
          g_bits(cl, clv);
          g_bits(sh, shv);
          g_bits(sl, slv);
          g_mma3<FAST>(accC, chv, clv, bsh[0], bsh[1], bsl[0], bsl[1]);
          g_mma3<FAST>(accS, shv, slv, bdh[0], bdh[1], bdl[0], bdl[1]);
        };
#pragma unroll 2
        for (int ks = 0; ks < KS - 1; ++ks) step(ks, 8 * ks + t4, 8 * ks + t4 + 4);
        step(KS - 1, jl0, jl1);                             // the last k-step: pair indices clamped (zero table entries)
        // X = rot (C - i S) of (frequency g8 + 8 fh, row 2 t4 + q): the second stage's column operand
        uint32_t bh[NC][2], bl[NC][2];
        const int grp = j * GPT + gq;
        const float ck0 = cK[8 * grp + 2 * t4], ck1 = cK[8 * grp + 2 * t4 + 1];
#pragma unroll
        for (int fh = 0; fh < NC / 2; ++fh) {
          float re[2], im[2];
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const float C = accC[2 * fh + q], Sv = accS[2 * fh + q];
            re[q] = rot[fh].x * C + rot[fh].y * Sv;
            im[q] = rot[fh].y * C - rot[fh].x * Sv;
            g_split<FAST>(re[q], bh[2 * fh][q], bl[2 * fh][q]);
            g_split<FAST>(im[q], bh[2 * fh + 1][q], bl[2 * fh + 1][q]);
          }
          lw[2 * fh] = fmaf(ck0, re[0], fmaf(ck1, re[1], lw[2 * fh]));
          lw[2 * fh + 1] = fmaf(ck0, im[0], fmaf(ck1, im[1], lw[2 * fh + 1]));
        }
#pragma unroll
        for (int mtm = 0; mtm < MTM; ++mtm) {
          uint32_t ah2[4], al2[4];
          g_split4<FAST>(a2tab[(grp * MTM + mtm) * 32 + lane], ah2, al2);
#pragma unroll
          for (int nc = 0; nc < NC; ++nc) g_mma3<FAST>(P[mtm][nc], ah2, al2, bh[nc][0], bh[nc][1], bl[nc][0], bl[nc][1]);
        }
      }
      __syncwarp();   // every lane is done with this stage before it is filled again
      s = s == ST - 1 ? 0 : s + 1;
    }
    // The plane's end.  Rows of the product: A_k = sum cos(k phi) T (k < K2), then B_k = sum sin(k phi) T (k = 1..K2);
    // a C fragment holds rows g8 (+8) and the columns 2 t4 (+1) of its tile (tile 2 fh + part: frequency 8 fh + column,
    // real or imaginary part).  Through the warp's scratch rows, so that every output can pick up its A and its B.
#pragma unroll
    for (int mtm = 0; mtm < MTM; ++mtm)
#pragma unroll
      for (int nc = 0; nc < NC; ++nc)
#pragma unroll
        for (int e = 0; e < 4; ++e)
          scr[(16 * mtm + g8 + 8 * (e >> 1)) * SCW + 2 * (8 * (nc >> 1) + 2 * t4 + (e & 1)) + (nc & 1)] = P[mtm][nc][e];
#pragma unroll
    for (int nc = 0; nc < NC; ++nc) {                       // the left-over row: add the four lanes that share a column
      float v = lw[nc];
      v += __shfl_xor_sync(0xffffffffu, v, 1);
      v += __shfl_xor_sync(0xffffffffu, v, 2);
      if (t4 == 0) scr[16 * MTM * SCW + 2 * (8 * (nc >> 1) + g8) + (nc & 1)] = v;
    }
    __syncwarp();
    // Z_{+k} = A_k - i B_k at position k, Z_{-k} = A_k + i B_k at position 2 K2 - k (B_0 = 0, A_{K2} = the left-over row)
    float2* ob = out + pl * (2 * K2) * K3;
    for (int idx = lane; idx < 2 * K2 * K3; idx += 32) {
      const int pm = idx / K3, f = idx - pm * K3;
      const int k = pm < K2 ? pm : 2 * K2 - pm;
      const float sg = pm < K2 ? -1.f : 1.f;
      const float* ar = scr + (k < K2 ? k : 16 * MTM) * SCW + 2 * f;
      float2 v = make_float2(ar[0], ar[1]);
      if (k > 0) {
        const float* br = scr + (K2 + k - 1) * SCW + 2 * f;
        v.x -= sg * br[1];
        v.y += sg * br[0];
      }
      ob[idx] = v;
    }
    __syncwarp();   // the scratch rows are read before the next plane's end writes them
  }
}

constexpr int kGVS = 40;   // floats per row of the padded spectrum copy: 8 mod 32, conflict-free fragment loads

// MT: 16-row tiles per task; KSF: k-steps of 8 frequencies (k3 <= 8 KSF); KS2: k-steps of 8 modes (2 K2 <= 8 KS2)
template <int MT, int KSF, int KS2, bool FAST>
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
  float4* a2e = btab + (size_t)2 * KSF * NTJ * 32;          // [16-row tile][ks2][lane]: folded basis, unsplit
  float* cK = reinterpret_cast<float*>(a2e + (size_t)NM * KS2 * 32);   // cos(2 pi K2 n / N2)
  float* warp_area = cK + ((N2 + 3) & ~3);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;
  const int W = blockDim.x >> 5;
  const int area_floats = stage_floats + (3 * VROWS + 1) * kGVS;
  float* st = warp_area + (size_t)warp * area_floats;       // output staging of a task
  float* Vs = st + stage_floats;                            // [2][VROWS][kGVS]: this plane's and the next plane's spectrum
  float* Bm = Vs + 2 * VROWS * kGVS;                        // [VROWS + 1][kGVS]: E_k, i O_k and, last row, V_{-K2}

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
  for (int e = threadIdx.x; e < NM * KS2 * 32; e += blockDim.x) {
    const int l = e & 31, ks2 = (e >> 5) % KS2, tile = (e >> 5) / KS2;
    float v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)                             // A fragment: grid row l >> 2 (+8), basis entry l & 3 (+4)
      v[q] = g_basis2f(8 * ks2 + (l & 3) + 4 * (q >> 1), 16 * tile + (l >> 2) + 8 * (q & 1), N2, K2);
    a2e[e] = make_float4(v[0], v[1], v[2], v[3]);
  }
  for (int n = threadIdx.x; n < N2; n += blockDim.x) cK[n] = g_basis2(0, K2, n, N2, K2);
  // the padding of the spectrum copies (entries past 2 K2, columns past 2 k3) meets zero basis entries: it must be finite
  for (int e = lane; e < (3 * VROWS + 1) * kGVS; e += 32) Vs[e] = 0.f;
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
    {
      // E_0 = V_0, E_k = V_k + V_{-k}; i O_k with O_k = V_k - V_{-k} (k < K2), O_{K2} = -V_{-K2}; position of -k: 2 K2 - k
      const float* V = Vs + (size_t)vb * VROWS * kGVS;
      for (int idx = lane; idx < 2 * K2 * K3; idx += 32) {
        const int r = idx / K3, f = idx - r * K3;
        const int k = r < K2 ? r : r - K2 + 1;
        const float2 vp = (k < K2) ? *reinterpret_cast<const float2*>(V + k * kGVS + 2 * f) : make_float2(0.f, 0.f);
        const float2 vm = (k > 0) ? *reinterpret_cast<const float2*>(V + (2 * K2 - k) * kGVS + 2 * f) : make_float2(0.f, 0.f);
        float2 o;
        if (r < K2) o = make_float2(vp.x + vm.x, vp.y + vm.y);
        else o = make_float2(-(vp.y - vm.y), vp.x - vm.x);
        *reinterpret_cast<float2*>(Bm + r * kGVS + 2 * f) = o;
      }
      for (int c = lane; c < 2 * K3; c += 32) Bm[VROWS * kGVS + c] = V[K2 * kGVS + c];
    }
    __syncwarp();
    float lv[NC][2];                                        // V_{-K2} at this lane's columns 8 nc + 2 t4 (+1)
#pragma unroll
    for (int nc = 0; nc < NC; ++nc)
#pragma unroll
      for (int q = 0; q < 2; ++q) lv[nc][q] = Bm[VROWS * kGVS + 8 * nc + 2 * t4 + q];
    for (int j = 0; j < TP; ++j) {
#pragma unroll 1
      for (int mt = 0; mt < MT; ++mt) {
        const int tile = j * MT + mt;
        // the second dimension: U[row][f] = cos(K2 phi_row) V_{-K2}[f] + sum_r basis[row][r] Bm[r][f]
        float P[NC][4];
        {
          const float c0 = cK[16 * tile + g8], c1 = cK[16 * tile + g8 + 8];
#pragma unroll
          for (int nc = 0; nc < NC; ++nc)
#pragma unroll
            for (int e = 0; e < 4; ++e) P[nc][e] = ((e >> 1) ? c1 : c0) * lv[nc][e & 1];
        }
#pragma unroll
        for (int ks2 = 0; ks2 < KS2; ++ks2) {
          uint32_t ah2[4], al2[4];
          g_split4<FAST>(a2e[(tile * KS2 + ks2) * 32 + lane], ah2, al2);
#pragma unroll
          for (int nc = 0; nc < NC; ++nc) {
            uint32_t b0h, b0l, b1h, b1l;
            g_split<FAST>(Bm[(8 * ks2 + t4) * kGVS + 8 * nc + g8], b0h, b0l);
            g_split<FAST>(Bm[(8 * ks2 + t4 + 4) * kGVS + 8 * nc + g8], b1h, b1l);
            g_mma3<FAST>(P[nc], ah2, al2, b0h, b1h, b0l, b1l);
          }
        }
        // a C fragment holds the complex value of frequency 4 nc + t4 for the rows g8 (+8): rotated, it is the
        // contiguous stage's row operand
        uint32_t rh[KSF][4], rl[KSF][4], ih[KSF][4], il[KSF][4];
#pragma unroll
        for (int ks = 0; ks < KSF; ++ks)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int nc = 2 * ks + (e >> 1), h = e & 1;
            const float ur = P[nc][2 * h], ui = P[nc][2 * h + 1];
            const float2 r = rot[ks][e >> 1];
            g_split<FAST>(ur * r.x - ui * r.y, rh[ks][e], rl[ks][e]);
            g_split<FAST>(ur * r.y + ui * r.x, ih[ks][e], il[ks][e]);
          }
        // one tile of 8 pairs: y_j = P - Q, y_{N3-1-j} = P + Q; `last`: pairs past the end go to the dump slot behind the
        // task's floats, the middle sample of an odd extent is P alone
        auto tile_j = [&](int ntj, bool last) {
          float Pj[4] = {0.f, 0.f, 0.f, 0.f}, Qj[4] = {0.f, 0.f, 0.f, 0.f};
          const float4* bt = btab + ntj * 32 + lane;
#pragma unroll
          for (int ks = 0; ks < KSF; ++ks) {
            const float4 bc = bt[ks * NTJ * 32], bs = bt[(KSF + ks) * NTJ * 32];
            g_mma3q<FAST>(Pj, rh[ks], rl[ks], bc);
            g_mma3q<FAST>(Qj, ih[ks], il[ks], bs);
          }
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int rowoff = (16 * mt + g8 + 8 * h) * N3;
            float* srow = st + rowoff;
            const int dump = TR * N3 - rowoff;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const int jj = 8 * ntj + 2 * t4 + q;
              const float pv = Pj[2 * h + q], qv = Qj[2 * h + q];
              if (!last) {
                srow[jj] = pv - qv;
                srow[N3 - 1 - jj] = pv + qv;
              } else {
                const bool in = jj < half;
                srow[in ? jj : ((odd && jj == half) ? jj : dump)] = in ? pv - qv : pv;
                srow[in ? N3 - 1 - jj : dump] = pv + qv;
              }
            }
          }
        };
#pragma unroll 1
        for (int ntj = 0; ntj < NTJ - 1; ++ntj) tile_j(ntj, false);
        tile_j(NTJ - 1, true);
      }
      __syncwarp();
      {
        float* dst = y + (pl * N2 + (long long)j * TR) * N3;
        for (int i = lane; i < (TR * N3) / 4; i += 32)
          __stcs(reinterpret_cast<float4*>(dst) + i, *reinterpret_cast<const float4*>(st + 4 * i));
      }
      __syncwarp();   // the staging area is read out before the next task writes to it
    }
    __syncwarp();     // this plane's operand rows are not needed any more: the next plane's are formed over them
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
cudaError_t launch_contract_s(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm, bool fast,
                              cudaStream_t st) {
  const int H = (N3 + 1) / 2, KS = (H + 7) / 8;
  const int sf = g_stage_floats(N3, MT);
  const GCfg c = g_cfg((size_t)2 * KS * NT * 32 * 16, (size_t)ST * sf * 4);
  if (c.warps < 2) return cudaErrorInvalidConfiguration;
  auto kern = fast ? rowg_contract_kernel<MT, NT, ST, true> : rowg_contract_kernel<MT, NT, ST, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem);
  if (e != cudaSuccess) return e;
  const long long tasks = (rows + 16 * MT - 1) / (16 * MT);
  const long long want = (tasks + c.warps - 1) / c.warps;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3(c.warps * 32), c.smem, st, x, out, rows, N3, K3, scale, herm, sf);
  return cudaGetLastError();
}

template <int MT, int NT>
cudaError_t launch_contract_t(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm, bool fast,
                              cudaStream_t st) {
  const int H = (N3 + 1) / 2, KS = (H + 7) / 8;
  const size_t sb = (size_t)g_stage_floats(N3, MT) * 4;
  return g_stages((size_t)2 * KS * NT * 32 * 16, sb) == 3 ? launch_contract_s<MT, NT, 3>(x, out, rows, N3, K3, scale, herm, fast, st)
                                                          : launch_contract_s<MT, NT, 2>(x, out, rows, N3, K3, scale, herm, fast, st);
}

template <int MTF, int ST>
cudaError_t launch_contract8_s(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm, bool fast,
                               cudaStream_t st) {
  const int H = (N3 + 1) / 2, KS = (H + 7) / 8;
  const int sf = (8 * N3 + 3) & ~3;
  const GCfg c = g_cfg((size_t)2 * KS * MTF * 2 * 32 * 16, (size_t)ST * sf * 4);
  if (c.warps < 2) return cudaErrorInvalidConfiguration;
  auto kern = fast ? rowg_contract8_kernel<MTF, ST, true> : rowg_contract8_kernel<MTF, ST, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem);
  if (e != cudaSuccess) return e;
  const long long tasks = (rows + 7) / 8;
  const long long want = (tasks + c.warps - 1) / c.warps;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3(c.warps * 32), c.smem, st, x, out, rows, N3, K3, scale, herm, sf);
  return cudaGetLastError();
}

template <int MTF>
cudaError_t launch_contract8_t(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm, bool fast,
                               cudaStream_t st) {
  const int H = (N3 + 1) / 2, KS = (H + 7) / 8;
  const size_t sb = (size_t)((8 * N3 + 3) & ~3) * 4, table = (size_t)2 * KS * MTF * 2 * 32 * 16;
  // long rows leave room for few warps: three stages only where eight warps of them fit, else two stages and more warps
  const bool three = g_cfg(table, 3 * sb).warps >= 8 || g_cfg(table, 2 * sb).warps <= g_cfg(table, 3 * sb).warps;
  return three ? launch_contract8_s<MTF, 3>(x, out, rows, N3, K3, scale, herm, fast, st)
               : launch_contract8_s<MTF, 2>(x, out, rows, N3, K3, scale, herm, fast, st);
}

template <int MT, int KSF>
cudaError_t launch_expand_t(const float2* in, float* y, long long rows, int N3, int K3, float scale, int herm, bool fast,
                            cudaStream_t st) {
  const int H = (N3 + 1) / 2, NTJ = (H + 7) / 8;
  const int sf = g_stage_floats(N3, MT);
  const GCfg c = g_cfg((size_t)2 * KSF * NTJ * 32 * 16, (size_t)sf * 4);
  if (c.warps < 2) return cudaErrorInvalidConfiguration;
  auto kern = fast ? rowg_expand_kernel<MT, KSF, true> : rowg_expand_kernel<MT, KSF, false>;
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
  return ((size_t)2 * KS * 2 + (size_t)(N2 / 8) * MTM) * 32 * 16 + (size_t)((N2 + 3) & ~3) * 4;
}
size_t pg_contract_scratch(int MTM) { return (size_t)(((16 * MTM + 1) * 34 + 3) & ~3) * 4; }
size_t pg_expand_table(int N3, int N2, int KSF, int KS2) {
  const int NTJ = ((N3 + 1) / 2 + 7) / 8;
  return ((size_t)2 * KSF * NTJ + (size_t)(N2 / 16) * KS2) * 32 * 16 + (size_t)((N2 + 3) & ~3) * 4;
}
size_t pg_expand_rows(int KS2) { return (size_t)(3 * 8 * KS2 + 1) * kGVS * 4; }

template <int MT, int NC, int MTM, int ST>
cudaError_t launch_pg_contract_s(const float* x, float2* out, long long planes, int N3, int K3, int N2, int K2,
                                 float scale, int herm, bool fast, cudaStream_t st) {
  const int sf = g_stage_floats(N3, MT);
  const GCfg c = g_cfg(pg_contract_table(N3, N2, MTM), (size_t)ST * sf * 4 + pg_contract_scratch(MTM));
  if (c.warps < 2) return cudaErrorInvalidConfiguration;
  auto kern = fast ? planeg_contract_kernel<MT, NC, MTM, ST, true> : planeg_contract_kernel<MT, NC, MTM, ST, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem);
  if (e != cudaSuccess) return e;
  const long long want = (planes + c.warps - 1) / c.warps;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3(c.warps * 32), c.smem, st, x, out, planes, N3, K3, N2, K2, scale, herm, sf);
  return cudaGetLastError();
}

template <int MT, int NC, int MTM>
cudaError_t launch_pg_contract_t(const float* x, float2* out, long long planes, int N3, int K3, int N2, int K2,
                                 float scale, int herm, bool fast, cudaStream_t st) {
  const size_t sb = (size_t)g_stage_floats(N3, MT) * 4;
  return g_stages(pg_contract_table(N3, N2, MTM) + kGMaxWarps * pg_contract_scratch(MTM), sb) == 3
             ? launch_pg_contract_s<MT, NC, MTM, 3>(x, out, planes, N3, K3, N2, K2, scale, herm, fast, st)
             : launch_pg_contract_s<MT, NC, MTM, 2>(x, out, planes, N3, K3, N2, K2, scale, herm, fast, st);
}

template <int MT, int KSF, int KS2>
cudaError_t launch_pg_expand_t(const float2* in, float* y, long long planes, int N3, int K3, int N2, int K2,
                               float scale, int herm, bool fast, cudaStream_t st) {
  const int sf = g_stage_floats(N3, MT) + 4;   // + the dump slot
  const GCfg c = g_cfg(pg_expand_table(N3, N2, KSF, KS2), (size_t)sf * 4 + pg_expand_rows(KS2));
  if (c.warps < 2) return cudaErrorInvalidConfiguration;
  auto kern = fast ? planeg_expand_kernel<MT, KSF, KS2, true> : planeg_expand_kernel<MT, KSF, KS2, false>;
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
  const size_t scr = pg_contract_scratch(MTM), sfd = sf + 16;   // the expansion's staging carries a dump slot
  return g_cfg(ct, g_stages(ct + kGMaxWarps * scr, sf) * sf + scr).warps >= 4 && g_cfg(et, sfd + pg_expand_rows(KS2)).warps >= 4;
}

cudaError_t launch_planeg_contract(const float* x, float2* out, long long planes, int N3, int K3, int N2, int K2,
                                   float scale, int herm, bool fast, cudaStream_t st) {
  const bool two = g_mt(N3) == 2, wide = K3 > 8, tall = 2 * K2 > 16;
#define DTST_PG(MT, NC, MTM) return launch_pg_contract_t<MT, NC, MTM>(x, out, planes, N3, K3, N2, K2, scale, herm, fast, st)
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
                                 float scale, int herm, bool fast, cudaStream_t st) {
  const bool two = g_mt(N3) == 2;
  const int KSF = (K3 + 7) / 8, KS2 = (2 * K2 + 7) / 8;
#define DTST_PG(MT, A, B) \
  if (two == (MT == 2) && KSF == A && KS2 == B) return launch_pg_expand_t<MT, A, B>(in, y, planes, N3, K3, N2, K2, scale, herm, fast, st);
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

cudaError_t launch_rowg_contract(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm, bool fast,
                                 cudaStream_t st) {
  const int NT = (K3 + 7) / 8;
  const bool two = g_mt(N3) == 2;
  if (N3 > 256)   // long rows: 8-row tasks
    return K3 <= 16 ? launch_contract8_t<1>(x, out, rows, N3, K3, scale, herm, fast, st)
                    : launch_contract8_t<2>(x, out, rows, N3, K3, scale, herm, fast, st);
  switch (NT) {
    case 1: return two ? launch_contract_t<2, 1>(x, out, rows, N3, K3, scale, herm, fast, st)
                       : launch_contract_t<1, 1>(x, out, rows, N3, K3, scale, herm, fast, st);
    case 2: return two ? launch_contract_t<2, 2>(x, out, rows, N3, K3, scale, herm, fast, st)
                       : launch_contract_t<1, 2>(x, out, rows, N3, K3, scale, herm, fast, st);
    case 3: return launch_contract_t<1, 3>(x, out, rows, N3, K3, scale, herm, fast, st);
    default: return launch_contract_t<1, 4>(x, out, rows, N3, K3, scale, herm, fast, st);
  }
}

cudaError_t launch_rowg_expand(const float2* in, float* y, long long rows, int N3, int K3, float scale, int herm, bool fast,
                               cudaStream_t st) {
  const int KSF = (K3 + 7) / 8;
  const bool two = g_mt(N3) == 2;
  switch (KSF) {
    case 1: return two ? launch_expand_t<2, 1>(in, y, rows, N3, K3, scale, herm, fast, st)
                       : launch_expand_t<1, 1>(in, y, rows, N3, K3, scale, herm, fast, st);
    case 2: return two ? launch_expand_t<2, 2>(in, y, rows, N3, K3, scale, herm, fast, st)
                       : launch_expand_t<1, 2>(in, y, rows, N3, K3, scale, herm, fast, st);
    case 3: return launch_expand_t<1, 3>(in, y, rows, N3, K3, scale, herm, fast, st);
    default: return launch_expand_t<1, 4>(in, y, rows, N3, K3, scale, herm, fast, st);
  }
}

}  // namespace dtst
