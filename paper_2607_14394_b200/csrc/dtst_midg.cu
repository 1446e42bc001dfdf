// Two-sided middle dimension for ANY extent and ANY mode count up to 32: the kernels behind the folded ones of
// dtst_midmma.cu / dtst_mid.cu (which are built for k in {4, 8, 12, 16} and extents that are multiples of 32).
//
//   midg_contract_kernel:  in[outer][N][inner] complex -> out[outer][2K][inner] complex   (Eq. 5 along one dimension)
//   midg_expand_kernel:    in[outer][2K][inner] complex -> out[outer][N][inner] complex   (Eq. 14 along one dimension)
//
// Folded over the sign of the mode: with phi_n = 2 pi n / N,
//     A_k = sum_n cos(k phi_n) z_n (k = 0..K),   B_k = sum_n sin(k phi_n) z_n (k = 1..K),
//     Z_{+k} = A_k - i B_k (k < K),   Z_{-k} = A_k + i B_k (k = 1..K)
// so one real product [cos k | sin k] (2K rows) x [N x real columns] serves all 2K modes; the one row left over,
// A_K of the unpaired mode -K, runs on FFMA.  The product is warp-level m16n8k8 TF32 with hi/lo compensation; a
// complex position is two adjacent real columns, which a C fragment holds in one lane.  A task is one outer index
// and a block of 16 complex positions (128 bytes per row); the contraction streams its N rows in chunks of 32
// through a per-warp cp.async ring and keeps the sums in C fragments, the expansion builds
// E_k = V_k + V_{-k}, i O_k = i (V_k - V_{-k}) once per task in shared memory and forms 16 output rows per product.
#include "dtst_common.cuh"
#include "dtst_mma.cuh"

namespace dtst {

namespace {

constexpr size_t kMgSmemLimit = 227 * 1024;
constexpr int kMgMaxWarps = 12;
constexpr int kMgStages = 3;
constexpr int kMgPos = 16;            // complex positions per task
constexpr int kMgRow = 36;            // floats per staged row of the contraction: rows 2 t4 apart land 8 t4 banks apart
constexpr int kMgRowE = 40;           // floats per operand row of the expansion: rows t4 apart land 8 t4 banks apart
constexpr int kMgChunk = 32;          // rows per ring stage
constexpr int kMgScw = 34;            // floats per scratch row

__device__ __forceinline__ void mg_cp16(float* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}
__device__ __forceinline__ void mg_cp8(float* smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}
__device__ __forceinline__ void mg_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void mg_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// hi = v rounded to the 11 significant bits the tensor core reads, lo = the exact rest (at most 2^-12 |v|, of which the
// hardware drops 2^-23 |v|): half the error of a truncating split, which the short sums of small extents need
// FAST (single-pass TF32, a plan option): the rounded value alone; every use of the lo part disappears.
template <bool FAST>
__device__ __forceinline__ void mg_split(float v, uint32_t& hi, uint32_t& lo) {
  hi = (__float_as_uint(v) + 0x1000u) & 0xffffe000u;
  lo = FAST ? 0u : __float_as_uint(v - __uint_as_float(hi));
}
template <bool FAST>
__device__ __forceinline__ void mg_split4(const float4& v, uint32_t (&hi)[4], uint32_t (&lo)[4]) {
  mg_split<FAST>(v.x, hi[0], lo[0]);
  mg_split<FAST>(v.y, hi[1], lo[1]);
  mg_split<FAST>(v.z, hi[2], lo[2]);
  mg_split<FAST>(v.w, hi[3], lo[3]);
}
template <bool FAST>
__device__ __forceinline__ void mg_mma3(float (&d)[4], const uint32_t (&ahi)[4], const uint32_t (&alo)[4], uint32_t bh0,
                                        uint32_t bh1, uint32_t bl0, uint32_t bl1) {
  if (FAST) mma_m16n8k8_tf32(d, ahi, bh0, bh1);
  else mma3_tf32(d, ahi, alo, bh0, bh1, bl0, bl1);
}

// entry r of the folded basis at local row n (global index off + n of an extent Ng, Eq. 18): cos(k phi) for r < K
// (k = r), sin(k phi) for K <= r < 2K (k = r - K + 1), phi = 2 pi (off + n) / Ng; zero beyond and for rows past the
// local extent N
__device__ __forceinline__ float mg_basis(int r, int n, int N, int Ng, int off, int K) {
  if (r >= 2 * K || n >= N) return 0.f;
  const long long k = r < K ? r : r - K + 1;
  // the phase is reduced exactly in integers to [0, 2); single precision from there on (1 ulp of the fp32 entry): in
  // double precision the tables of a short-running launch took longer to build than its data to process
  float s, c;
  sincospif(2.0f * (float)((k * (off + n)) % Ng) / (float)Ng, &s, &c);
  return r < K ? c : s;
}
__device__ __forceinline__ float mg_cosK(int n, int N, int Ng, int off, int K) {
  if (n >= N) return 0.f;
  return cospif(2.0f * (float)(((long long)K * (off + n)) % Ng) / (float)Ng);
}

// MTM: 16-row tiles of the folded basis (2K <= 16 MTM).  VEC: 16-byte copies (inner even, 16-byte aligned tensors).
// SPLIT: a task belongs to the whole CTA - warp w takes the row chunks w, w + W, .. and the warps' sums are added in
// warp order at the task's end (through their scratch rows; a fixed order: the same bits on every run).  For
// tensors with fewer tasks than the GPU has warps: a 2-D layer has batch x channels of them.
template <int MTM, bool VEC, bool FAST, bool SPLIT>
__global__ void __launch_bounds__(kMgMaxWarps * 32, 1)
midg_contract_kernel(const float2* __restrict__ in, float2* __restrict__ out, long long outer, long long inner, int N,
                     int Ng, int off, int K, float scale) {
  pdl_trigger();
  extern __shared__ float4 mg_smem[];
  const int NCH = (N + kMgChunk - 1) / kMgChunk, NG = 4 * NCH;
  float4* a2tab = mg_smem;                                          // [group of 8 rows][mtm][lane], unsplit
  float* cK = reinterpret_cast<float*>(a2tab + (size_t)NG * MTM * 32);   // cos(2 pi K n / N), zero past the extent
  float* areas = cK + NCH * kMgChunk;
  constexpr int STAGE = kMgChunk * kMgRow;
  constexpr int SCRF = ((16 * MTM + 1) * kMgScw + 3) & ~3;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;
  const int W = blockDim.x >> 5;
  float* S = areas + (size_t)warp * (kMgStages * STAGE + SCRF);
  float* scr = S + kMgStages * STAGE;

  for (int e = threadIdx.x; e < NG * MTM * 32; e += blockDim.x) {
    const int l = e & 31, mtm = (e >> 5) % MTM, grp = (e >> 5) / MTM;
    float v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)                                     // A fragment: basis row l >> 2 (+8), row 2 (l & 3) (+1)
      v[q] = mg_basis(16 * mtm + (l >> 2) + 8 * (q & 1), 8 * grp + 2 * (l & 3) + (q >> 1), N, Ng, off, K);
    a2tab[e] = make_float4(v[0], v[1], v[2], v[3]);
  }
  for (int n = threadIdx.x; n < NCH * kMgChunk; n += blockDim.x) cK[n] = mg_cosK(n, N, Ng, off, K);
  // rows and columns a copy never reaches (past the extent, past a ragged block) meet zero basis entries or are not
  // stored: they must be finite
  for (int e = lane; e < kMgStages * STAGE; e += 32) S[e] = 0.f;
  __syncthreads();
  pdl_wait();

  const long long CB = (inner + kMgPos - 1) / kMgPos;
  const long long tasks = outer * CB;
  const long long stride = SPLIT ? (long long)gridDim.x : (long long)W * gridDim.x;
  long long t = SPLIT ? (long long)blockIdx.x : (long long)warp * gridDim.x + blockIdx.x;
  const int c_first = SPLIT ? warp : 0, c_step = SPLIT ? W : 1;   // this warp's chunks of a task
  // the chunk staged next: task (as outer index and block, advanced by additions) and chunk within it
  long long at = t, ao = t / CB, acb = t % CB;
  const long long sdiv = stride / CB, smod = stride % CB;
  int ac = c_first;
  if (ac >= NCH) at = tasks;                                   // a warp beyond the chunks of a task stages nothing
  auto load = [&](int s) {
    if (at < tasks) {
      const long long o = ao, cb = acb;
      const int valid = (int)(inner - cb * kMgPos < kMgPos ? inner - cb * kMgPos : kMgPos);   // complex positions
      const int rows = N - ac * kMgChunk < kMgChunk ? N - ac * kMgChunk : kMgChunk;
      const float2* src = in + (o * N + (long long)ac * kMgChunk) * inner + cb * kMgPos;
      float* dst = S + (size_t)s * STAGE;
      if (VEC) {
        const int ppr = valid >> 1;                                 // 16-byte pieces per row
        for (int i = lane; i < rows * 8; i += 32) {
          const int r = i >> 3, c = i & 7;
          if (c < ppr) mg_cp16(dst + r * kMgRow + 4 * c, src + (long long)r * inner + 2 * c);
        }
      } else {
        for (int i = lane; i < rows * 16; i += 32) {
          const int r = i >> 4, c = i & 15;
          if (c < valid) mg_cp8(dst + r * kMgRow + 2 * c, src + (long long)r * inner + c);
        }
      }
    }
    mg_commit();
    ac += c_step;
    if (ac >= NCH) {
      ac = c_first;
      at += stride;
      ao += sdiv;
      acb += smod;
      if (acb >= CB) {
        acb -= CB;
        ++ao;
      }
    }
  };
#pragma unroll
  for (int q = 0; q < kMgStages - 1; ++q) load(q);
  int s = 0;
  for (; t < tasks; t += stride) {
    float P[MTM][4][4];
    float lw[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int mtm = 0; mtm < MTM; ++mtm)
#pragma unroll
      for (int nc = 0; nc < 4; ++nc)
#pragma unroll
        for (int e = 0; e < 4; ++e) P[mtm][nc][e] = 0.f;
    for (int ch = c_first; ch < NCH; ch += c_step) {
      load(s == 0 ? kMgStages - 1 : s - 1);
      mg_wait<kMgStages - 1>();
      __syncwarp();
      const float* T = S + (size_t)s * STAGE;
#pragma unroll 1
      for (int g = 0; g < 4; ++g) {
        const int grp = 4 * ch + g;
        const float* r0 = T + (8 * g + 2 * t4) * kMgRow + g8;       // B fragment: rows 2 t4, 2 t4 + 1 of the group, column g8
        const float ck0 = cK[8 * grp + 2 * t4], ck1 = cK[8 * grp + 2 * t4 + 1];
        uint32_t bh[4][2], bl[4][2];
#pragma unroll
        for (int nc = 0; nc < 4; ++nc) {
          const float v0 = r0[8 * nc], v1 = r0[kMgRow + 8 * nc];
          mg_split<FAST>(v0, bh[nc][0], bl[nc][0]);
          mg_split<FAST>(v1, bh[nc][1], bl[nc][1]);
          lw[nc] = fmaf(ck0, v0, fmaf(ck1, v1, lw[nc]));
        }
#pragma unroll
        for (int mtm = 0; mtm < MTM; ++mtm) {
          uint32_t ah[4], al[4];
          mg_split4<FAST>(a2tab[(grp * MTM + mtm) * 32 + lane], ah, al);
#pragma unroll
          for (int nc = 0; nc < 4; ++nc) mg_mma3<FAST>(P[mtm][nc], ah, al, bh[nc][0], bh[nc][1], bl[nc][0], bl[nc][1]);
        }
      }
      __syncwarp();   // every lane is done with this stage before it is filled again
      s = s == kMgStages - 1 ? 0 : s + 1;
    }
    // The task's end: rows A_k (k < K), then B_k (k = 1..K), the left-over row A_K; a C fragment holds rows g8 (+8) and
    // the real columns 8 nc + 2 t4 (+1) = the complex position 4 nc + t4.
#pragma unroll
    for (int mtm = 0; mtm < MTM; ++mtm)
#pragma unroll
      for (int nc = 0; nc < 4; ++nc)
#pragma unroll
        for (int e = 0; e < 4; ++e) scr[(16 * mtm + g8 + 8 * (e >> 1)) * kMgScw + 8 * nc + 2 * t4 + (e & 1)] = P[mtm][nc][e];
#pragma unroll
    for (int nc = 0; nc < 4; ++nc) {
      float v = lw[nc];
      v += __shfl_xor_sync(0xffffffffu, v, 1);
      v += __shfl_xor_sync(0xffffffffu, v, 2);
      if (t4 == 0) scr[16 * MTM * kMgScw + 8 * nc + g8] = v;
    }
    if (SPLIT) __syncthreads();
    else __syncwarp();
    {
      const long long o = t / CB, cb = t - o * CB;
      const int valid = (int)(inner - cb * kMgPos < kMgPos ? inner - cb * kMgPos : kMgPos);
      float2* ob = out + o * (2 * K) * inner + cb * kMgPos;
      const int nw = SPLIT ? W : 1;                                 // scratch areas to add, in warp order
      const float* sbase = SPLIT ? areas + kMgStages * STAGE : scr;
      const int wstride = kMgStages * STAGE + SCRF;
      for (int idx = SPLIT ? (int)threadIdx.x : lane; idx < 2 * K * kMgPos; idx += SPLIT ? (int)blockDim.x : 32) {
        const int pm = idx >> 4, i = idx & 15;
        if (i >= valid) continue;
        const int k = pm < K ? pm : 2 * K - pm;
        const float sg = pm < K ? -1.f : 1.f;
        float2 a = make_float2(0.f, 0.f), bq = make_float2(0.f, 0.f);
        for (int w = 0; w < nw; ++w) {
          const float* ar = sbase + (size_t)w * wstride + (k < K ? k : 16 * MTM) * kMgScw + 2 * i;
          a.x += ar[0];
          a.y += ar[1];
          if (k > 0) {
            const float* br = sbase + (size_t)w * wstride + (K + k - 1) * kMgScw + 2 * i;
            bq.x += br[0];
            bq.y += br[1];
          }
        }
        ob[(long long)pm * inner + i] = make_float2((a.x - sg * bq.y) * scale, (a.y + sg * bq.x) * scale);
      }
    }
    if (SPLIT) __syncthreads();   // the scratch rows are read before the next task's end writes them
    else __syncwarp();
  }
}

// U_n = cos(K phi_n) V_{-K} + sum_r basis[n][r] Bm[r]: Bm = E_k (k < K), then i O_k (k = 1..K).
template <bool VEC, bool FAST>
__global__ void __launch_bounds__(kMgMaxWarps * 32, 1)
midg_expand_kernel(const float2* __restrict__ in, float2* __restrict__ out, long long outer, long long inner, int N,
                   int Ng, int off, int K, float scale, int tpt) {
  pdl_trigger();
  extern __shared__ float4 mg_smem[];
  const int NM = (N + 15) / 16, KS2 = (2 * K + 7) / 8, VROWS = 8 * KS2;
  float4* a2e = mg_smem;                                            // [16-row tile][ks2][lane], unsplit
  float* cK = reinterpret_cast<float*>(a2e + (size_t)NM * KS2 * 32);
  float* areas = cK + NM * 16;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;
  const int W = blockDim.x >> 5;
  const int area = (3 * VROWS + 1) * kMgRowE;
  float* Vs = areas + (size_t)warp * area;                          // [2][VROWS][kMgRowE]: this task's and the next task's input
  float* Bm = Vs + 2 * VROWS * kMgRowE;                              // [VROWS + 1][kMgRowE]

  for (int e = threadIdx.x; e < NM * KS2 * 32; e += blockDim.x) {
    const int l = e & 31, ks2 = (e >> 5) % KS2, tile = (e >> 5) / KS2;
    float v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)                                     // A fragment: row l >> 2 (+8), basis entry l & 3 (+4)
      v[q] = mg_basis(8 * ks2 + (l & 3) + 4 * (q >> 1), 16 * tile + (l >> 2) + 8 * (q & 1), N, Ng, off, K);
    a2e[e] = make_float4(v[0], v[1], v[2], v[3]);
  }
  for (int n = threadIdx.x; n < NM * 16; n += blockDim.x) cK[n] = mg_cosK(n, N, Ng, off, K);
  for (int e = lane; e < area; e += 32) Vs[e] = 0.f;                // padding meets zero basis entries: finite
  __syncthreads();
  pdl_wait();

  // a task: one outer index, one block of positions and `tpt` 16-row tiles of the output (a few tasks per column
  // block when there are not enough blocks to fill the GPU: a 2-D layer has batch x channels of them)
  const long long CB = (inner + kMgPos - 1) / kMgPos;
  const int NRG = (NM + tpt - 1) / tpt;
  const long long tasks = outer * CB * NRG;
  const long long stride = (long long)W * gridDim.x;
  auto fetch = [&](long long task, int buf) {
    if (task < tasks) {
      const long long ocb = task / NRG;
      const long long o = ocb / CB, cb = ocb - o * CB;
      const int valid = (int)(inner - cb * kMgPos < kMgPos ? inner - cb * kMgPos : kMgPos);
      const float2* src = in + o * (2 * K) * inner + cb * kMgPos;
      float* dst = Vs + (size_t)buf * VROWS * kMgRowE;
      if (VEC) {
        const int ppr = valid >> 1;
        for (int i = lane; i < 2 * K * 8; i += 32) {
          const int r = i >> 3, c = i & 7;
          if (c < ppr) mg_cp16(dst + r * kMgRowE + 4 * c, src + (long long)r * inner + 2 * c);
        }
      } else {
        for (int i = lane; i < 2 * K * 16; i += 32) {
          const int r = i >> 4, c = i & 15;
          if (c < valid) mg_cp8(dst + r * kMgRowE + 2 * c, src + (long long)r * inner + c);
        }
      }
    }
    mg_commit();
  };
  long long t = (long long)warp * gridDim.x + blockIdx.x;
  fetch(t, 0);
  int vb = 0;
  for (; t < tasks; t += stride, vb ^= 1) {
    fetch(t + stride, vb ^ 1);
    mg_wait<1>();
    __syncwarp();
    const long long ocb = t / NRG;
    const int rg = (int)(t - ocb * NRG);
    const long long o = ocb / CB, cb = ocb - o * CB;
    const int valid = (int)(inner - cb * kMgPos < kMgPos ? inner - cb * kMgPos : kMgPos);
    {
      // E_0 = V_0, E_k = V_k + V_{-k}; i O_k with O_k = V_k - V_{-k} (k < K), O_K = -V_{-K}; position of -k: 2K - k
      const float* V = Vs + (size_t)vb * VROWS * kMgRowE;
      for (int idx = lane; idx < 2 * K * kMgPos; idx += 32) {
        const int r = idx >> 4, i = idx & 15;
        const int k = r < K ? r : r - K + 1;
        const float2 vp = (k < K) ? *reinterpret_cast<const float2*>(V + k * kMgRowE + 2 * i) : make_float2(0.f, 0.f);
        const float2 vm = (k > 0) ? *reinterpret_cast<const float2*>(V + (2 * K - k) * kMgRowE + 2 * i) : make_float2(0.f, 0.f);
        float2 ov;
        if (r < K) ov = make_float2(vp.x + vm.x, vp.y + vm.y);
        else ov = make_float2(-(vp.y - vm.y), vp.x - vm.x);
        *reinterpret_cast<float2*>(Bm + r * kMgRowE + 2 * i) = ov;
      }
      Bm[VROWS * kMgRowE + lane] = V[K * kMgRowE + lane];             // V_{-K}: 32 real columns, one per lane
    }
    __syncwarp();
    float lv[4][2];                                                 // V_{-K} at this lane's columns 8 nc + 2 t4 (+1)
#pragma unroll
    for (int nc = 0; nc < 4; ++nc)
#pragma unroll
      for (int q = 0; q < 2; ++q) lv[nc][q] = Bm[VROWS * kMgRowE + 8 * nc + 2 * t4 + q];
    float2* ob = out + o * N * inner + cb * kMgPos;
    const int tile_end = (rg + 1) * tpt < NM ? (rg + 1) * tpt : NM;
#pragma unroll 1
    for (int tile = rg * tpt; tile < tile_end; ++tile) {
      float P[4][4];
      {
        const float c0 = cK[16 * tile + g8], c1 = cK[16 * tile + g8 + 8];
#pragma unroll
        for (int nc = 0; nc < 4; ++nc)
#pragma unroll
          for (int e = 0; e < 4; ++e) P[nc][e] = ((e >> 1) ? c1 : c0) * lv[nc][e & 1];
      }
#pragma unroll 1
      for (int ks2 = 0; ks2 < KS2; ++ks2) {
        uint32_t ah[4], al[4];
        mg_split4<FAST>(a2e[(tile * KS2 + ks2) * 32 + lane], ah, al);
        const float* b0 = Bm + (8 * ks2 + t4) * kMgRowE + g8;
#pragma unroll
        for (int nc = 0; nc < 4; ++nc) {
          uint32_t b0h, b0l, b1h, b1l;
          mg_split<FAST>(b0[8 * nc], b0h, b0l);
          mg_split<FAST>(b0[4 * kMgRowE + 8 * nc], b1h, b1l);
          mg_mma3<FAST>(P[nc], ah, al, b0h, b1h, b0l, b1l);
        }
      }
      // a C fragment: rows g8 (+8), the complex position 4 nc + t4
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int n = 16 * tile + g8 + 8 * h;
        if (n >= N) continue;
#pragma unroll
        for (int nc = 0; nc < 4; ++nc) {
          const int i = 4 * nc + t4;
          if (i < valid) ob[(long long)n * inner + i] = make_float2(P[nc][2 * h] * scale, P[nc][2 * h + 1] * scale);
        }
      }
    }
    __syncwarp();   // this task's operand rows are not needed any more: the next task's are formed over them
  }
}

struct MgCfg {
  int warps;
  size_t smem;
};
MgCfg mg_cfg(size_t table_bytes, size_t per_warp_bytes) {
  MgCfg c{0, 0};
  if (table_bytes + 2 * per_warp_bytes > kMgSmemLimit) return c;
  int w = (int)((kMgSmemLimit - table_bytes) / per_warp_bytes);
  if (w > kMgMaxWarps) w = kMgMaxWarps;
  c.warps = w;
  c.smem = table_bytes + (size_t)w * per_warp_bytes;
  return c;
}
size_t mg_contract_table(int N, int MTM) {
  const int NCH = (N + kMgChunk - 1) / kMgChunk;
  return (size_t)4 * NCH * MTM * 32 * 16 + (size_t)NCH * kMgChunk * 4;
}
size_t mg_contract_warp(int MTM) {
  return ((size_t)kMgStages * kMgChunk * kMgRow + (((16 * MTM + 1) * kMgScw + 3) & ~3)) * 4;
}
size_t mg_expand_table(int N, int K) {
  const int NM = (N + 15) / 16, KS2 = (2 * K + 7) / 8;
  return (size_t)NM * KS2 * 32 * 16 + (size_t)NM * 16 * 4;
}
size_t mg_expand_warp(int K) { return (size_t)(3 * 8 * ((2 * K + 7) / 8) + 1) * kMgRowE * 4; }

template <int MTM, bool VEC>
cudaError_t launch_contract_t(const float2* in, float2* out, long long outer, long long inner, int N, int Ng, int off,
                              int K, float scale, bool fast, cudaStream_t st) {
  const MgCfg c = mg_cfg(mg_contract_table(N, MTM), mg_contract_warp(MTM));
  if (c.warps < 2) return cudaErrorInvalidConfiguration;
  const long long tasks = outer * ((inner + kMgPos - 1) / kMgPos);
  // fewer tasks than warps on the GPU (and more than one chunk of rows to share): a CTA per task
  const bool split = tasks < (long long)c.warps * num_sms() && N > kMgChunk;
  auto kern = split ? (fast ? midg_contract_kernel<MTM, VEC, true, true> : midg_contract_kernel<MTM, VEC, false, true>)
                    : (fast ? midg_contract_kernel<MTM, VEC, true, false> : midg_contract_kernel<MTM, VEC, false, false>);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem);
  if (e != cudaSuccess) return e;
  const long long want = split ? tasks : (tasks + c.warps - 1) / c.warps;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3(c.warps * 32), c.smem, st, in, out, outer, inner, N, Ng, off, K, scale);
  return cudaGetLastError();
}

template <bool VEC>
cudaError_t launch_expand_t(const float2* in, float2* out, long long outer, long long inner, int N, int Ng, int off, int K,
                            float scale, bool fast, cudaStream_t st) {
  const MgCfg c = mg_cfg(mg_expand_table(N, K), mg_expand_warp(K));
  if (c.warps < 2) return cudaErrorInvalidConfiguration;
  auto kern = fast ? midg_expand_kernel<VEC, true> : midg_expand_kernel<VEC, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem);
  if (e != cudaSuccess) return e;
  // 16-row tiles per task: all of them when there are column blocks enough to fill the GPU twice, else fewer
  const long long blocks = outer * ((inner + kMgPos - 1) / kMgPos);
  const int NM = (N + 15) / 16;
  long long groups = (2ll * c.warps * num_sms() + blocks - 1) / blocks;
  if (groups > NM) groups = NM;
  if (groups < 1) groups = 1;
  const int tpt = (int)((NM + groups - 1) / groups);
  const long long tasks = blocks * ((NM + tpt - 1) / tpt);
  const long long want = (tasks + c.warps - 1) / c.warps;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3(c.warps * 32), c.smem, st, in, out, outer, inner, N, Ng, off, K, scale, tpt);
  return cudaGetLastError();
}

}  // namespace

// Any extent with 2K <= N and any K up to 32 whose tables leave room for four warps (N up to ~1000).
bool midg_supported(int N, int K) { return N >= 2 && 2 * K <= N && midg_local_supported(N, K); }

// The same for Nl local rows of a longer dimension (a rank's block, or the slabs of virtual shards taken together):
// the rows carry their global phases, the local extent may be shorter than 2K.
bool midg_local_supported(int Nl, int K) {
  if (K < 1 || K > 32 || Nl < 1) return false;
  const int MTM = (2 * K + 15) / 16;
  return mg_cfg(mg_contract_table(Nl, MTM), mg_contract_warp(MTM)).warps >= 4 &&
         mg_cfg(mg_expand_table(Nl, K), mg_expand_warp(K)).warps >= 4;
}

cudaError_t launch_midg_local(bool forward, int K, const float2* in, float2* out, long long outer, long long inner, int Nl,
                              int Ng, int off, float scale, bool fast, cudaStream_t st) {
  if (outer * inner <= 0) return cudaSuccess;
  const bool vec = (inner % 2 == 0) && ((reinterpret_cast<uintptr_t>(in) | reinterpret_cast<uintptr_t>(out)) & 15u) == 0;
  if (!forward) return vec ? launch_expand_t<true>(in, out, outer, inner, Nl, Ng, off, K, scale, fast, st)
                           : launch_expand_t<false>(in, out, outer, inner, Nl, Ng, off, K, scale, fast, st);
  switch ((2 * K + 15) / 16) {
#define DTST_MG(M) \
  case M: return vec ? launch_contract_t<M, true>(in, out, outer, inner, Nl, Ng, off, K, scale, fast, st) \
                     : launch_contract_t<M, false>(in, out, outer, inner, Nl, Ng, off, K, scale, fast, st);
    DTST_MG(1) DTST_MG(2) DTST_MG(3) DTST_MG(4)
#undef DTST_MG
    default: return cudaErrorNotSupported;
  }
}

cudaError_t launch_midg(bool forward, int K, const float2* in, float2* out, long long outer, long long inner, int N,
                        float scale, bool fast, cudaStream_t st) {
  return launch_midg_local(forward, K, in, out, outer, inner, N, N, 0, scale, fast, st);
}

}  // namespace dtst
