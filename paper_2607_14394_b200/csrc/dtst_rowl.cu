// Row kernels for LONG contiguous extents (512 < N3 <= 16384, N3 a multiple of 8, up to 32 one-sided modes): the
// contiguous (rfft) dimension alone - a 1-D signal of 8192 points, a 1024 x 1024 grid.  Same fold and same TF32x3
// products as dtst_rowg.cu (X_f = e^{i pi f/N3} (sum_j s_j cos theta_fj - i sum_j d_j sin theta_fj), s_j, d_j =
// x_j +- x_{N3-1-j}, theta_fj = 2 pi f (j + 1/2) / N3), but a row no longer fits a warp's share of the shared memory
// and its basis no table:
//   * a task is 8 rows, streamed in CHUNKS of 64 pairs: the 64 columns from the left and the 64 mirrored columns
//     from the right (two 256-byte segments per row, 16-byte aligned because N3 is a multiple of 4; the last chunk
//     may be shorter, a multiple of 4 pairs), through a per-warp cp.async ring of 4 KB stages - 16 warps per SM
//     whatever N3 is;
//   * the basis of chunk c is the product of two small exact tables, e^{i theta} = T1[f][j - 64 c] * T2[c][f] with
//     T1 = e^{2 pi i f (jl + 1/2) / N3} (32 x 64 entries) and T2 = e^{2 pi i f 64 c / N3} (one row per chunk), both
//     built once per CTA from integer-reduced phases in double precision: one complex multiplication per entry, no
//     recurrence, no drift.
//
//   rowl_contract_kernel:  x[rows][N3] real  ->  out[rows][k3] complex   (Eq. 5 along the last dimension)
//   rowl_expand_kernel:    in[rows][k3] complex -> y[rows][N3] real      (Eq. 14 along the last dimension)
//
// Both run the product transposed (8 rows are the 8-wide operand), as rowg_contract8_kernel does.
#include "dtst_fused.cuh"
#include "dtst_mma.cuh"

namespace dtst {

namespace {

constexpr size_t kLSmemLimit = 227 * 1024;
constexpr int kLMaxWarps = 16;
constexpr int kLStages = 3;
constexpr int kLPairs = 64;          // pairs per chunk = 8 k-steps
constexpr int kLRow = 132;           // floats per staged row: [64 left | 64 right | 4]: rows land 4 banks apart
constexpr int kLStage = 8 * kLRow;   // floats per stage
constexpr int kLT1 = 68;             // float2 per T1 row: rows land 4 eight-byte slots apart
constexpr int kLMaxF = 32;

__device__ __forceinline__ void l_cp_async16(float* smem_dst, const float* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}
__device__ __forceinline__ void l_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void l_cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// hi/lo operand parts (truncating split); FAST: the value rounded to the 11 bits the tensor core reads, no lo part
template <bool FAST>
__device__ __forceinline__ void l_split(float v, uint32_t& hi, uint32_t& lo) {
  if (FAST) {
    hi = __float_as_uint(v) + 0x1000u;
    lo = 0u;
  } else {
    hi = __float_as_uint(v) & 0xffffe000u;
    lo = __float_as_uint(v - __uint_as_float(hi));
  }
}
template <bool FAST>
__device__ __forceinline__ void l_mma3(float (&d)[4], const uint32_t (&ahi)[4], const uint32_t (&alo)[4], uint32_t bh0,
                                       uint32_t bh1, uint32_t bl0, uint32_t bl1) {
  if (FAST) mma_m16n8k8_tf32(d, ahi, bh0, bh1);
  else mma3_tf32(d, ahi, alo, bh0, bh1, bl0, bl1);
}

// the two tables: T1[f][jl] = e^{2 pi i f (jl + 1/2) / N3}, T2[c][f] = e^{2 pi i f 64 c / N3}
__device__ __forceinline__ void l_build_tables(float2* T1, float2* T2, int N3, int NCK) {
  for (int e = threadIdx.x; e < kLMaxF * kLPairs; e += blockDim.x) {
    const int f = e / kLPairs, jl = e % kLPairs;
    double s, c;
    sincospi((double)(((long long)f * (2 * jl + 1)) % (2ll * N3)) / (double)N3, &s, &c);
    T1[f * kLT1 + jl] = make_float2((float)c, (float)s);
  }
  for (int e = threadIdx.x; e < NCK * kLMaxF; e += blockDim.x) {
    const int c = e / kLMaxF, f = e % kLMaxF;
    double s, cs;
    sincospi(2.0 * (double)(((long long)f * kLPairs * c) % N3) / (double)N3, &s, &cs);
    T2[e] = make_float2((float)cs, (float)s);
  }
}

// MTF: 16-frequency tiles (k3 <= 16 MTF).  SPLIT: a task belongs to the whole CTA - warp w takes the chunks w, w + W, ..
// and the warps' sums are added in warp order at the task's end (a fixed order: the same bits on every run).  For
// tensors with fewer 8-row tasks than the GPU has warps: a batch of 1-D signals.
template <int MTF, bool FAST, bool SPLIT>
__global__ void __launch_bounds__(kLMaxWarps * 32, 1)
rowl_contract_kernel(const float* __restrict__ x, float2* __restrict__ out, long long rows, int N3, int K3, float scale,
                     int herm) {
  pdl_trigger();
  extern __shared__ float4 rl_smem[];
  const int H = N3 / 2, NCK = (H + kLPairs - 1) / kLPairs;          // pairs, chunks of 64 pairs (the last: H - 64 c, a multiple of 4)
  float2* T1 = reinterpret_cast<float2*>(rl_smem);
  float2* T2 = T1 + kLMaxF * kLT1;
  float* ring = reinterpret_cast<float*>(T2 + (size_t)NCK * kLMaxF);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;
  const int W = blockDim.x >> 5;
  l_build_tables(T1, T2, N3, NCK);
  float* S = ring + (size_t)warp * kLStages * kLStage;
  float* red = ring + (size_t)W * kLStages * kLStage;               // SPLIT: [warp][MTF][8][lane]
  for (int e = lane; e < kLStages * kLStage; e += 32) S[e] = 0.f;   // rows of a ragged last task are never copied
  float2 rot[MTF][2];                                               // frequencies 16 mtf + g8 (+8)
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

  const long long tasks = (rows + 7) / 8;
  const long long stride = SPLIT ? (long long)gridDim.x : (long long)W * gridDim.x;
  long long t = SPLIT ? (long long)blockIdx.x : (long long)warp * gridDim.x + blockIdx.x;
  const int c_first = SPLIT ? warp : 0, c_step = SPLIT ? W : 1;     // this warp's chunks of a task
  long long at = t;                                                 // the chunk staged next: task and chunk within it
  int ac = c_first;
  if (ac >= NCK) at = tasks;                                        // a warp beyond the chunks of a task stages nothing
  auto load = [&](int s) {
    if (at < tasks) {
      const long long r0 = at * 8;
      const int nr = (int)(rows - r0 < 8 ? rows - r0 : 8);
      const int L = H - kLPairs * ac < kLPairs ? H - kLPairs * ac : kLPairs;   // pairs of this chunk = floats per segment
      const float* src = x + r0 * N3;
      float* dst = S + (size_t)s * kLStage;
      const int ppr = L >> 2;                                       // 16-byte pieces per segment
      for (int i = lane; i < nr * 2 * ppr; i += 32) {
        const int r = i / (2 * ppr), q = i - r * 2 * ppr;
        if (q < ppr) l_cp_async16(dst + r * kLRow + 4 * q, src + (long long)r * N3 + kLPairs * ac + 4 * q);
        else l_cp_async16(dst + r * kLRow + 128 - L + 4 * (q - ppr),
                          src + (long long)r * N3 + N3 - kLPairs * ac - L + 4 * (q - ppr));
      }
    }
    l_cp_async_commit();
    ac += c_step;
    if (ac >= NCK) {
      ac = c_first;
      at += stride;
    }
  };
#pragma unroll
  for (int q = 0; q < kLStages - 1; ++q) load(q);
  int s = 0;
  for (; t < tasks; t += stride) {
    float accC[MTF][4], accS[MTF][4];
#pragma unroll
    for (int mtf = 0; mtf < MTF; ++mtf)
#pragma unroll
      for (int e = 0; e < 4; ++e) accC[mtf][e] = accS[mtf][e] = 0.f;
    for (int c = c_first; c < NCK; c += c_step) {
      load(s == 0 ? kLStages - 1 : s - 1);
      l_cp_async_wait<kLStages - 1>();
      __syncwarp();
      const float* Trow = S + (size_t)s * kLStage + g8 * kLRow;     // this lane's row (the 8-wide operand's n index)
      const int L = H - kLPairs * c < kLPairs ? H - kLPairs * c : kLPairs;
      const int nk = (L + 7) >> 3;                                  // k-steps; the last may hold 4 pairs only
      float2 t2[MTF][2];
#pragma unroll
      for (int mtf = 0; mtf < MTF; ++mtf)
#pragma unroll
        for (int h = 0; h < 2; ++h) t2[mtf][h] = T2[c * kLMaxF + 16 * mtf + g8 + 8 * h];
      // The chunk's products are summed in fresh fragments and added to the running sums with ordinary fp32 additions:
      // the tensor core's accumulate step truncates, and one chain through the 1536 MMAs of an 8192-point row left the
      // spectrum at 6e-5 of the oracle.
      float cC[MTF][4], cS[MTF][4];
#pragma unroll
      for (int mtf = 0; mtf < MTF; ++mtf)
#pragma unroll
        for (int e = 0; e < 4; ++e) cC[mtf][e] = cS[mtf][e] = 0.f;
#pragma unroll 2
      for (int kk = 0; kk < nk; ++kk) {
        const int jl = 8 * kk + t4;
        const float a0 = Trow[jl], b0 = Trow[127 - jl];
        const bool v1 = jl + 4 < L;                                 // pairs past the chunk's end (only t4 + 4 can be) count zero
        const float a1 = v1 ? Trow[jl + 4] : 0.f, b1 = v1 ? Trow[123 - jl] : 0.f;
        uint32_t bsh[2], bsl[2], bdh[2], bdl[2];
        l_split<FAST>(a0 + b0, bsh[0], bsl[0]);
        l_split<FAST>(a0 - b0, bdh[0], bdl[0]);
        l_split<FAST>(a1 + b1, bsh[1], bsl[1]);
        l_split<FAST>(a1 - b1, bdh[1], bdl[1]);
#pragma unroll
        for (int mtf = 0; mtf < MTF; ++mtf) {
          uint32_t ch[4], cl[4], sh[4], sl[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {                             // A fragment: frequency g8 (+8), pair t4 (+4)
            const float2 e1 = T1[(16 * mtf + g8 + 8 * (q & 1)) * kLT1 + jl + 4 * (q >> 1)];
            const float2 e2 = t2[mtf][q & 1];
            l_split<FAST>(e1.x * e2.x - e1.y * e2.y, ch[q], cl[q]);
            l_split<FAST>(e1.x * e2.y + e1.y * e2.x, sh[q], sl[q]);
          }
          l_mma3<FAST>(cC[mtf], ch, cl, bsh[0], bsh[1], bsl[0], bsl[1]);
          l_mma3<FAST>(cS[mtf], sh, sl, bdh[0], bdh[1], bdl[0], bdl[1]);
        }
      }
#pragma unroll
      for (int mtf = 0; mtf < MTF; ++mtf)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          accC[mtf][e] += cC[mtf][e];
          accS[mtf][e] += cS[mtf][e];
        }
      __syncwarp();   // every lane is done with this stage before it is filled again
      s = s == kLStages - 1 ? 0 : s + 1;
    }
    if (SPLIT) {
      // the warps' sums, added in warp order by warp 0
#pragma unroll
      for (int mtf = 0; mtf < MTF; ++mtf)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          red[((warp * MTF + mtf) * 8 + e) * 32 + lane] = accC[mtf][e];
          red[((warp * MTF + mtf) * 8 + 4 + e) * 32 + lane] = accS[mtf][e];
        }
      __syncthreads();
      if (warp == 0) {
#pragma unroll
        for (int mtf = 0; mtf < MTF; ++mtf)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float c = 0.f, sv = 0.f;
            for (int w = 0; w < W; ++w) {
              c += red[((w * MTF + mtf) * 8 + e) * 32 + lane];
              sv += red[((w * MTF + mtf) * 8 + 4 + e) * 32 + lane];
            }
            accC[mtf][e] = c;
            accS[mtf][e] = sv;
          }
      }
      __syncthreads();   // the sums are read before the next task's are written
      if (warp != 0) continue;
    }
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
  }
}

// y_j = P_j - Q_j, y_{N3-1-j} = P_j + Q_j with P_j = sum_f Re z'_f cos theta_fj, Q_j = sum_f Im z'_f sin theta_fj,
// z'_f = scale c_f e^{-i pi f / N3} in_f.  KSF: k-steps of 8 frequencies (k3 <= 8 KSF).
template <int KSF, bool FAST>
__global__ void __launch_bounds__(kLMaxWarps * 32, 1)
rowl_expand_kernel(const float2* __restrict__ in, float* __restrict__ y, long long rows, int N3, int K3, float scale,
                   int herm, int cpt) {
  pdl_trigger();
  extern __shared__ float4 rl_smem[];
  const int H = N3 / 2, NCK = (H + kLPairs - 1) / kLPairs;
  float2* T1 = reinterpret_cast<float2*>(rl_smem);
  float2* T2 = T1 + kLMaxF * kLT1;
  float* stg = reinterpret_cast<float*>(T2 + (size_t)NCK * kLMaxF);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;
  const int W = blockDim.x >> 5;
  l_build_tables(T1, T2, N3, NCK);
  float* st = stg + (size_t)warp * kLStage;                         // a chunk of 8 rows: [64 left | 64 right] per row
  float2 rot[KSF][2];                                               // frequencies 8 ks + t4 (+4)
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

  // a task: 8 rows and `cpt` chunks of them (all chunks when there are row blocks enough to fill the GPU)
  const int NCG = (NCK + cpt - 1) / cpt;
  const long long tasks = ((rows + 7) / 8) * NCG;
  const long long stride = (long long)W * gridDim.x;
  float2 vin[KSF][2];                                               // the NEXT task's values of row g8
  auto load_inputs = [&](long long task) {
#pragma unroll
    for (int ks = 0; ks < KSF; ++ks)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const long long row = (task / NCG) * 8 + g8;
        const int f = 8 * ks + t4 + 4 * hf;
        vin[ks][hf] = (task < tasks && row < rows && f < K3) ? __ldg(in + row * K3 + f) : make_float2(0.f, 0.f);
      }
  };
  long long t = (long long)warp * gridDim.x + blockIdx.x;
  load_inputs(t);
  for (; t < tasks; t += stride) {
    // the 8-wide operand: z'[f = 8 ks + t4 (+4)][row g8], real and imaginary parts
    uint32_t rh[KSF][2], rl[KSF][2], ih[KSF][2], il[KSF][2];
#pragma unroll
    for (int ks = 0; ks < KSF; ++ks)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const float2 v = vin[ks][hf], r = rot[ks][hf];
        l_split<FAST>(v.x * r.x - v.y * r.y, rh[ks][hf], rl[ks][hf]);
        l_split<FAST>(v.x * r.y + v.y * r.x, ih[ks][hf], il[ks][hf]);
      }
    load_inputs(t + stride);
    const long long r0 = (t / NCG) * 8;
    const int cg = (int)(t % NCG);
    const int nr = (int)(rows - r0 < 8 ? rows - r0 : 8);
    const int c_end = (cg + 1) * cpt < NCK ? (cg + 1) * cpt : NCK;
    for (int c = cg * cpt; c < c_end; ++c) {
      const int L = H - kLPairs * c < kLPairs ? H - kLPairs * c : kLPairs;   // pairs of this chunk
      float2 t2[KSF][2];
#pragma unroll
      for (int ks = 0; ks < KSF; ++ks)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) t2[ks][hf] = T2[c * kLMaxF + 8 * ks + t4 + 4 * hf];
#pragma unroll 1
      for (int mtj = 0; 16 * mtj < L; ++mtj) {                      // 16 pairs per product
        float P[4] = {0.f, 0.f, 0.f, 0.f}, Q[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < KSF; ++ks) {
          uint32_t ch[4], cl[4], sh[4], sl[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {                             // A fragment: pair g8 (+8), frequency t4 (+4)
            const float2 e1 = T1[(8 * ks + t4 + 4 * (q >> 1)) * kLT1 + 16 * mtj + g8 + 8 * (q & 1)];
            const float2 e2 = t2[ks][q >> 1];
            l_split<FAST>(e1.x * e2.x - e1.y * e2.y, ch[q], cl[q]);
            l_split<FAST>(e1.x * e2.y + e1.y * e2.x, sh[q], sl[q]);
          }
          l_mma3<FAST>(P, ch, cl, rh[ks][0], rh[ks][1], rl[ks][0], rl[ks][1]);
          l_mma3<FAST>(Q, sh, sl, ih[ks][0], ih[ks][1], il[ks][0], il[ks][1]);
        }
        // a C fragment: pairs 16 mtj + g8 (+8 h), rows 2 t4 + q
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int jl = 16 * mtj + g8 + 8 * h;
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            float* srow = st + (2 * t4 + q) * kLRow;
            srow[jl] = P[2 * h + q] - Q[2 * h + q];
            srow[127 - jl] = P[2 * h + q] + Q[2 * h + q];
          }
        }
      }
      __syncwarp();
      {
        float* dst = y + r0 * N3;
        const int ppr = L >> 2;
        for (int i = lane; i < nr * 2 * ppr; i += 32) {
          const int r = i / (2 * ppr), q = i - r * 2 * ppr;
          if (q < ppr)
            __stcs(reinterpret_cast<float4*>(dst + (long long)r * N3 + kLPairs * c + 4 * q),
                   *reinterpret_cast<const float4*>(st + r * kLRow + 4 * q));
          else
            __stcs(reinterpret_cast<float4*>(dst + (long long)r * N3 + N3 - kLPairs * c - L + 4 * (q - ppr)),
                   *reinterpret_cast<const float4*>(st + r * kLRow + 128 - L + 4 * (q - ppr)));
        }
      }
      __syncwarp();   // the staging area is read out before the next chunk writes to it
    }
  }
}

size_t l_table_bytes(int N3) {
  const int NCK = (N3 / 2 + kLPairs - 1) / kLPairs;
  return ((size_t)kLMaxF * kLT1 + (size_t)NCK * kLMaxF) * sizeof(float2);
}
int l_warps(size_t table, size_t per_warp) {
  if (table + 4 * per_warp > kLSmemLimit) return 0;
  const int w = (int)((kLSmemLimit - table) / per_warp);
  return w > kLMaxWarps ? kLMaxWarps : w;
}

template <int MTF>
cudaError_t launch_contract_t(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm, bool fast,
                              cudaStream_t st) {
  const size_t table = l_table_bytes(N3), pw = (size_t)kLStages * kLStage * 4 + (size_t)MTF * 8 * 32 * 4;
  const int w = l_warps(table, pw);
  if (w < 4) return cudaErrorInvalidConfiguration;
  const size_t smem = table + (size_t)w * pw;
  const long long tasks = (rows + 7) / 8;
  const bool split = tasks < (long long)w * num_sms();   // fewer tasks than warps on the GPU: a CTA per task
  auto kern = split ? (fast ? rowl_contract_kernel<MTF, true, true> : rowl_contract_kernel<MTF, false, true>)
                    : (fast ? rowl_contract_kernel<MTF, true, false> : rowl_contract_kernel<MTF, false, false>);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const long long want = split ? tasks : (tasks + w - 1) / w;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3(w * 32), smem, st, x, out, rows, N3, K3, scale, herm);
  return cudaGetLastError();
}

template <int KSF>
cudaError_t launch_expand_t(const float2* in, float* y, long long rows, int N3, int K3, float scale, int herm, bool fast,
                            cudaStream_t st) {
  const size_t table = l_table_bytes(N3), pw = (size_t)kLStage * 4;
  const int w = l_warps(table, pw);
  if (w < 4) return cudaErrorInvalidConfiguration;
  const size_t smem = table + (size_t)w * pw;
  auto kern = fast ? rowl_expand_kernel<KSF, true> : rowl_expand_kernel<KSF, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  // chunks per task: all of them when there are row blocks enough to fill the GPU twice, else fewer
  const long long blocks = (rows + 7) / 8;
  const int NCK = (N3 / 2 + kLPairs - 1) / kLPairs;
  long long groups = (2ll * w * num_sms() + blocks - 1) / blocks;
  if (groups > NCK) groups = NCK;
  if (groups < 1) groups = 1;
  const int cpt = (int)((NCK + groups - 1) / groups);
  const long long tasks = blocks * ((NCK + cpt - 1) / cpt);
  const long long want = (tasks + w - 1) / w;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3(w * 32), smem, st, in, y, rows, N3, K3, scale, herm, cpt);
  return cudaGetLastError();
}

}  // namespace

bool rowl_supported(int N3, int K3) {
  if (N3 <= 512 || N3 > 16384 || N3 % 8 != 0 || K3 < 1 || K3 > 32 || K3 > N3 / 2 + 1) return false;
  return l_warps(l_table_bytes(N3), (size_t)kLStages * kLStage * 4 + 2 * 8 * 32 * 4) >= 4;
}

cudaError_t launch_rowl_contract(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm,
                                 bool fast, cudaStream_t st) {
  return K3 <= 16 ? launch_contract_t<1>(x, out, rows, N3, K3, scale, herm, fast, st)
                  : launch_contract_t<2>(x, out, rows, N3, K3, scale, herm, fast, st);
}

cudaError_t launch_rowl_expand(const float2* in, float* y, long long rows, int N3, int K3, float scale, int herm, bool fast,
                               cudaStream_t st) {
  switch ((K3 + 7) / 8) {
    case 1: return launch_expand_t<1>(in, y, rows, N3, K3, scale, herm, fast, st);
    case 2: return launch_expand_t<2>(in, y, rows, N3, K3, scale, herm, fast, st);
    case 3: return launch_expand_t<3>(in, y, rows, N3, K3, scale, herm, fast, st);
    default: return launch_expand_t<4>(in, y, rows, N3, K3, scale, herm, fast, st);
  }
}

}  // namespace dtst
