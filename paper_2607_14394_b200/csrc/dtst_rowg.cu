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

}  // namespace

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
