// Fused streaming kernels for the grid-side stages of the truncated spectral layer: the kernel templates.
// Included by the translation units that instantiate them for the supported plane shapes
// (dtst_plane_inst_*.cu, split so that they compile in parallel) and by the dispatcher (dtst_fused.cu).
//
// Forward ("plane") kernel: contracts the last two grid dimensions in one pass.  The real
// grid is read from HBM exactly once through a TMA-fed shared-memory ring; each consumer
// warp owns a task of 128 consecutive rows (one or two [N2 x N3] planes), contracts the
// contiguous dimension with one thread per row (folded FFMA with immediate coefficients),
// then the next dimension on the tensor cores (TF32 hi/lo compensated warp MMAs), and writes
// only the [2*k2 x k3] complex result of each plane.
//
// Both contractions use the symmetries of the DFT basis (Eq. 18 with zero offset): with the
// half-sample phase factored out,
//     sum_n x[n] e^{-i phi n} = e^{+i phi/2} sum_n x[n] e^{-i phi (n + 1/2)},
// the cos/sin factors are even/odd about the centre of the row and again (up to (-1)^f)
// about the centre of each half, so four inputs (n, N/2-1-n, N/2+n, N-1-n) are folded with
// 8 additions and then need one multiply-add per retained frequency and parity class instead
// of four.  Frequencies +g and -g of a two-sided dimension share their cos and sin sums.
// This cuts the multiply count roughly fourfold and keeps the arithmetic in exact fp32 FMAs,
// which is what lets an HBM-bound kernel afford a dense contraction with only 8..16 output
// columns (far too narrow for the tensor cores to help: the MMA would be bound by reading
// its 128 x 8 A tile from shared memory, which costs as much as the FMAs done here).
#pragma once
#include <cuda.h>

#include "dtst_fused.cuh"
#include "dtst_mma.cuh"
#include "dtst_sm100.cuh"

namespace dtst {
namespace plane {

using namespace sm100;

constexpr int kTaskRows = 128;       // rows of the contiguous dimension per warp task
constexpr int kColAccWarps = 4;      // accumulator warps of the forward kernel's fused third dimension
constexpr int kStageBytes = 16384;   // one ring slot
constexpr int kSmemLimit = 232448;   // 227 KB opt-in limit per CTA

// Stage-1 coefficients cos/sin(2 pi f (j + 1/2) / N3), j < N3/4, as COMPILE-TIME constants: the row code is fully
// unrolled over (j, f), so every FMA carries its coefficient as a 32-bit immediate.  No table in HBM, shared or
// constant memory, no load instruction, no register: a shared-memory operand would cost LDS bandwidth this kernel
// does not have, and a constant-bank table costs one uniform load per four coefficients (measured: 9 % of the
// forward kernel's instructions, 22 % of the inverse kernel's).
namespace ct {
constexpr double kPi = 3.14159265358979323846264338327950288;
// Taylor series on |x| <= pi/4 (terms to x^27: below 1e-19)
constexpr double sin_small(double x) {
  const double x2 = x * x;
  double term = x, sum = x;
  for (int k = 1; k <= 13; ++k) {
    term *= -x2 / (double)((2 * k) * (2 * k + 1));
    sum += term;
  }
  return sum;
}
constexpr double cos_small(double x) {
  const double x2 = x * x;
  double term = 1.0, sum = 1.0;
  for (int k = 1; k <= 13; ++k) {
    term *= -x2 / (double)((2 * k - 1) * (2 * k));
    sum += term;
  }
  return sum;
}
// cos(pi num / den), sin(pi num / den): the argument is reduced exactly in integers to the first octant
constexpr double cospi_ratio(long long num, long long den) {
  num %= 2 * den;
  if (num < 0) num += 2 * den;
  if (num > den) num = 2 * den - num;          // cos(2 pi - a) = cos a
  double sign = 1.0;
  if (2 * num > den) {                         // cos(pi - a) = -cos a
    num = den - num;
    sign = -1.0;
  }
  if (4 * num <= den) return sign * cos_small(kPi * (double)num / (double)den);
  return sign * sin_small(kPi * (double)(den - 2 * num) / (double)(2 * den));   // cos a = sin(pi/2 - a)
}
constexpr double sinpi_ratio(long long num, long long den) {
  num %= 2 * den;
  if (num < 0) num += 2 * den;
  double sign = 1.0;
  if (num > den) {                             // sin(2 pi - a) = -sin a
    num = 2 * den - num;
    sign = -1.0;
  }
  if (2 * num > den) num = den - num;          // sin(pi - a) = sin a
  if (4 * num <= den) return sign * sin_small(kPi * (double)num / (double)den);
  return sign * cos_small(kPi * (double)(den - 2 * num) / (double)(2 * den));   // sin a = cos(pi/2 - a)
}
// phase (2j+1) f / (2 N3) turns = pi (2j+1) f / N3
template <int N3, int J, int F>
struct Coef {
  static constexpr float cs = (float)cospi_ratio((long long)(2 * J + 1) * F, N3);
  static constexpr float sn = (float)sinpi_ratio((long long)(2 * J + 1) * F, N3);
};
}  // namespace ct

template <int N3, int K3, int N2, int K2>
struct PlaneCfg {
  static constexpr int ROWS_PER_STAGE = kStageBytes / (N3 * 4);
  static constexpr int SPT = kTaskRows / ROWS_PER_STAGE;      // ring slots per task
  static constexpr int BOXES = N3 / 32;                       // 128-byte column panels per row
  static constexpr int G = kTaskRows / N2;                    // planes per task
  static constexpr int QUADS = N2 / 4;                        // row quadruples per plane
  static constexpr int NC = 2 * K3;                           // real columns after stage 1 (C | S)
  static constexpr int LPP = 2 * K2;                          // output rows (modes) per plane
  static constexpr int NKS = QUADS / 8;                       // MMA k-steps over the quadruples
  static constexpr int MT = G * NC / 16;                      // MMA m-tiles over (plane, column)
  static constexpr int MT2 = 2;                               // inverse: MMA m-tiles over the 32 quadruples
  static constexpr int GT = K2 / 2;                           // frequencies per parity class
  static constexpr int NS = 4 * NC + 8;                       // floats per combo row: 4 classes x NC, +8 pad
  static constexpr int ABS = NC + 1;                          // floats between A/B entries (odd: scalar accesses)
  static constexpr int ABP = (2 * K2 + 1) * ABS;
  // forward kernel: one parity class at a time, row stride NSC = 8 mod 16 words (conflict-free fragment loads)
  static constexpr int NSC = (NC % 16 == 8) ? NC : NC + 8;
  // per-warp buffer (class combos, later the A/B entries), a multiple of 128 bytes so that every warp's
  // region stays 16-byte aligned for the vector stores
  static constexpr int COMBO_FLOATS = (((32 * NSC > G * ABP ? 32 * NSC : G * ABP) + 31) / 32) * 32;
  static constexpr int BTAB_FLOAT4 = 5 * NKS * 32;            // stage-2 basis fragments, CTA-shared
  static_assert(N3 % 32 == 0 && (N3 == 32 || N3 == 64), "N3");
  static_assert(kTaskRows % N2 == 0 && G * QUADS == 32, "one lane per row quadruple");
  static_assert(G * LPP <= 32 && (G * NC) % 16 == 0, "stage-2 mapping");
  static_assert(K3 % 2 == 0 && NC % 8 == 0 && K2 % 2 == 0 && GT <= 8 && QUADS % 8 == 0, "shape");
  static_assert(NS % 32 == 8, "combo row stride must be 8 mod 32 words for conflict-free fragment loads");
  static_assert(SPT == 1 || SPT == 2, "SPT");
};

struct SmemPlan {
  int stages;
  size_t ring, combos, rot, bars, total;
};

template <typename Cfg, int K2, int K3, int W>
SmemPlan smem_plan(size_t extra = 0) {   // extra: bytes behind the barrier block (fused third dimension)
  SmemPlan s;
  const size_t combos = (size_t)W * Cfg::COMBO_FLOATS * 4 + (size_t)Cfg::BTAB_FLOAT4 * 16;
  const size_t rot = (size_t)2 * K2 * K3 * 8;
  const size_t fixed = 1024 /*alignment slack*/ + combos + rot + 512 /*barriers*/ + extra;
  s.stages = (int)((kSmemLimit - fixed) / kStageBytes);
  if (s.stages > 12) s.stages = 12;
  s.ring = 0;
  s.combos = (size_t)s.stages * kStageBytes;
  s.rot = s.combos + combos;
  s.bars = s.rot + rot;
  s.total = s.bars + 512 + extra + 1024;
  return s;
}

// 16-byte shared-memory access by 32-bit shared-space address (+ immediate byte offset).  Volatile: a ring
// slot is refilled by the TMA engine between two reads of the same address, which the compiler cannot see.
template <int IMM>
__device__ __forceinline__ float4 lds128_s(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4+%5];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "r"(addr), "n"(IMM));
  return v;
}
template <int IMM>
__device__ __forceinline__ void sts128_s(uint32_t addr, float a, float b, float c, float d) {
  asm volatile("st.shared.v4.f32 [%0+%1], {%2,%3,%4,%5};" ::"r"(addr), "n"(IMM), "f"(a), "f"(b), "f"(c), "f"(d)
               : "memory");
}

// fp32 -> (hi, lo) TF32 pair for the error-compensated product hi*hi + lo*hi + hi*lo: the truncating split
// (two instructions) for operands split in the inner loop, the rounding one for the basis tables built once
__device__ __forceinline__ void split_tf32(float v, uint32_t& hi, uint32_t& lo) { split_tf32_trunc(v, hi, lo); }

// D += A(16x8, row) * B(8x8, col), TF32 inputs, fp32 accumulate
__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Forward row code, one quadruple j: o[f] += folded input * coefficient(j, f), f = F .. K3-1 (compile-time recursion
// so that j and f are constant expressions and the coefficients become immediates).
template <int N3, int K3, int J, int F>
__device__ __forceinline__ void s1_freqs(float uu, float ud, float vs, float vd, float (&o)[2 * K3]) {
  if constexpr (F < K3) {
    constexpr float cs = ct::Coef<N3, J, F>::cs, sn = ct::Coef<N3, J, F>::sn;
    if constexpr ((F & 1) == 0) {
      o[F] = (J == 0) ? uu * cs : fmaf(uu, cs, o[F]);
      if constexpr (F > 0) o[K3 + F] = (J == 0) ? vd * sn : fmaf(vd, sn, o[K3 + F]);
    } else {
      o[F] = (J == 0) ? ud * cs : fmaf(ud, cs, o[F]);
      o[K3 + F] = (J == 0) ? vs * sn : fmaf(vs, sn, o[K3 + F]);
    }
    s1_freqs<N3, K3, J, F + 1>(uu, ud, vs, vd, o);
  }
}

// chunks C, CH/2-1-C, CH/2+C, CH-1-C of the row: four quadruples j = 4C .. 4C+3
template <int N3, int K3, int BOXR, int C>
__device__ __forceinline__ void s1_chunks(uint32_t rx, float (&o)[2 * K3]) {
  constexpr int CH = N3 / 4;
  if constexpr (C < CH / 4) {
    constexpr int P = BOXR * 128;
    constexpr int c0 = C, c1 = CH / 2 - 1 - C, c2 = CH / 2 + C, c3 = CH - 1 - C;
    // (the panel offset is an immediate, the XOR constant depends on the chunk only)
    const float4 A = lds128_s<(c0 / 8) * P>(rx ^ (uint32_t)((c0 % 8) << 4));
    const float4 Bq = lds128_s<(c1 / 8) * P>(rx ^ (uint32_t)((c1 % 8) << 4));
    const float4 Cq = lds128_s<(c2 / 8) * P>(rx ^ (uint32_t)((c2 % 8) << 4));
    const float4 D = lds128_s<(c3 / 8) * P>(rx ^ (uint32_t)((c3 % 8) << 4));
#define DTST_QUAD(E, av, bv, cv, dv)                                               \
    {                                                                              \
      const float u = (av) + (dv), v = (av) - (dv);                                \
      const float up = (bv) + (cv), vp = (bv) - (cv);                              \
      s1_freqs<N3, K3, 4 * C + (E), 0>(u + up, u - up, v + vp, v - vp, o);         \
    }
    DTST_QUAD(0, A.x, Bq.w, Cq.x, D.w)
    DTST_QUAD(1, A.y, Bq.z, Cq.y, D.z)
    DTST_QUAD(2, A.z, Bq.y, Cq.z, D.y)
    DTST_QUAD(3, A.w, Bq.x, Cq.w, D.x)
#undef DTST_QUAD
    s1_chunks<N3, K3, BOXR, C + 1>(rx, o);
  }
}

// One row of N3 reals -> C_f = sum u cos, S_f = sum v sin for f < K3 (half-sample phase deferred).
// `stage` is the 32-bit shared address of the slot (1024-byte aligned), BOXR its rows per 128-byte panel.
template <int N3, int K3, int BOXR>
__device__ __forceinline__ void stage1_row(uint32_t stage, int row, float (&o)[2 * K3]) {
  o[K3] = 0.f;   // the sine sum of f = 0 has no terms
  // chunk c of this row sits at row*128 + ((c ^ (row & 7)) << 4) (+ one panel for c >= 8); the row base has
  // zeros in bits 4..6, so the swizzle is a single XOR of a precomputed base with a constant
  const uint32_t rx = stage + (uint32_t)row * 128u + (((uint32_t)row & 7u) << 4);
  s1_chunks<N3, K3, BOXR, 0>(rx, o);
}

// Consumer side of the ring: wait until fill number q (0-based) of `slot` has landed.
// Every lane of the warp calls it; the lanes poll independently but leave with ONE verdict (a lane whose barrier
// completed just as another warp raised the abort flag must not go on alone into the warp-synchronous MMA code).
__device__ __forceinline__ bool wait_fill(volatile uint32_t* fill_seq, uint64_t* full, int slot, uint32_t q,
                                          volatile int* abort_flag, uint32_t limit) {
  bool ok = true;
  for (uint32_t it = 0; fill_seq[slot] < q + 1u; ++it) {
    if ((it & 63u) == 63u) {
      if (*abort_flag) {
        ok = false;
        break;
      }
      __nanosleep(64);
    }
    if (it > limit) {
      *abort_flag = 1;
      ok = false;
      break;
    }
  }
  if (ok) ok = mbar_wait_bounded(&full[slot], q & 1u, abort_flag, limit);
  return __all_sync(0xffffffffu, ok) != 0;
}

// All lanes of a warp wait for a phase of an mbarrier and leave with one verdict.
__device__ __forceinline__ bool wait_bar_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag, uint32_t limit) {
  const bool ok = mbar_wait_bounded(bar, parity, abort_flag, limit);
  return __all_sync(0xffffffffu, ok) != 0;
}

// K1 > 0: the THIRD dimension (the one in front of the plane, extent N1, K1 retained modes per side) is contracted
// inside this kernel too.  A CTA then takes whole columns (the N1 consecutive planes that share their leading
// indices); the consumer warps put each finished plane - [2 k2][k3] complex, 2 KB - into a double-buffered batch of
// 8 planes in shared memory instead of writing it to HBM, and kColAccWarps further warps contract every complete
// batch into the column's [2 k1][2 k2][k3] accumulator, which lives in their MMA C fragments:
//   C_g[m] += sum_k cos(2 pi g n_k / N1) v_k[m],  S_g[m] += sum_k sin(..) v_k[m]     (TF32 hi/lo, 16 x 8 x 8 MMAs)
//   Z_{+g} = C_g - i S_g,  Z_{-g} = C_g + i S_g  at the column's end;  Z_{-K1} = sum_n v_n e^{+2 pi i K1 n / N1} in FFMA.
// The reduced tensor of the plane stage ([planes][2 k2][k3], 6 % of the bytes of a transform, written and read once)
// and the launch that contracted it disappear.  Twelve warps: every warp is capped at 168 registers.
template <int N3, int K3, int N2, int K2, int W, int K1>
__global__ void __launch_bounds__((W + 1 + (K1 > 0 ? kColAccWarps : 0)) * 32, 1)
fwd_plane_kernel(const __grid_constant__ CUtensorMap in_map, float2* __restrict__ out, long long num_tasks, float scale, int herm, int stages,
                 int* __restrict__ status, uint32_t poll_limit, long long withhold_after, int N1) {
  using Cfg = PlaneCfg<N3, K3, N2, K2>;
  constexpr int NC = Cfg::NC, QUADS = Cfg::QUADS, G = Cfg::G, LPP = Cfg::LPP;
  constexpr int SPT = Cfg::SPT, RPS = Cfg::ROWS_PER_STAGE;
  constexpr bool COLS = K1 > 0;
  constexpr int PCOLS = 2 * (2 * K2) * K3;   // floats of one finished plane
  static_assert(!COLS || (G == 1 && K1 == 16 && PCOLS % (64 * kColAccWarps) == 0), "fused third dimension: shape");

  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment for the TMA swizzle, by pointer arithmetic on the shared array itself (an integer
  // round trip would make the compiler lose the address space and emit generic loads and stores)
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* ring = smem;
  const uint32_t ring_s = smem_u32(ring);
  float4* btab = reinterpret_cast<float4*>(smem + (size_t)stages * kStageBytes);
  float* combos_all = reinterpret_cast<float*>(btab + Cfg::BTAB_FLOAT4);
  float2* rot = reinterpret_cast<float2*>(combos_all + (size_t)W * Cfg::COMBO_FLOATS);
  uint64_t* full = reinterpret_cast<uint64_t*>(rot + 2 * K2 * K3);
  uint64_t* empty = full + 16;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(empty + 16);
  // fill_seq[slot] = number of fills the producer has armed for that slot.  A parity wait can only
  // tell "this phase" from "the previous one", so a consumer that is a whole lap of the ring ahead
  // must first see its fill armed (which implies every earlier fill of the slot has landed).
  volatile uint32_t* fill_seq = reinterpret_cast<volatile uint32_t*>(empty + 16) + 4;
  // fused third dimension: batch complete / batch consumed barriers (inside the 512-byte barrier block), the two
  // batches of finished planes and the cosine table cos(2 pi j / N1)
  uint64_t* pfull = full + 44;
  uint64_t* pfree = full + 46;
  float* pbuf = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(full) + 512);
  float* ctab = pbuf + 2 * 8 * PCOLS;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
      fill_seq[s] = 0;
    }
    *abort_flag = 0;
    if constexpr (COLS) {
      for (int i = 0; i < 2; ++i) {
        mbar_init(&pfull[i], 8);
        mbar_init(&pfree[i], kColAccWarps);
      }
    }
    fence_barrier_init();
    prefetch_tensormap(&in_map);
  }
  if constexpr (COLS)
    for (int e = threadIdx.x; e < N1; e += blockDim.x) ctab[e] = (float)cospi(2.0 * (double)e / (double)N1);
  // Stage-2 basis as MMA B fragments (k = quadruple n, n = frequency slot of the parity class), TF32 hi/lo,
  // generated once per CTA: entry [cls][ks][lane] = (b0 hi, b1 hi, b0 lo, b1 lo).  Classes: 0 = A even (pp,
  // cos), 1 = A odd (pd, cos), 2 = B odd (ms, sin), 3 = B even (md, sin); 4 = the unpaired A_{K2} (cos, shares
  // the pp operand), in column 0 only.
  for (int e = threadIdx.x; e < Cfg::BTAB_FLOAT4; e += blockDim.x) {
    const int l = e & 31, ks = (e >> 5) % Cfg::NKS, cls = (e >> 5) / Cfg::NKS;
    const int lg = l >> 2, lt = l & 3;
    uint32_t hi[2], lo[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int n = 8 * ks + lt + 4 * h;
      int g = 0;
      bool valid = lg < Cfg::GT;
      if (cls == 0) g = 2 * lg;
      else if (cls == 1 || cls == 2) g = 2 * lg + 1;
      else if (cls == 3) g = 2 * lg + 2;
      else { g = K2; valid = (lg == 0); }
      double sn, cs;
      sincospi((double)(((long long)g * (2 * n + 1)) % (2 * N2)) / (double)N2, &sn, &cs);
      const float v = valid ? ((cls == 2 || cls == 3) ? (float)sn : (float)cs) : 0.f;
      split_tf32_rna(v, hi[h], lo[h]);
    }
    btab[e] = make_float4(__uint_as_float(hi[0]), __uint_as_float(hi[1]), __uint_as_float(lo[0]), __uint_as_float(lo[1]));
  }
  // rotation table: the deferred half-sample phases of both dimensions, the scale and the
  // Hermitian weight, one complex factor per (mode position r, last-dim frequency f)
  for (int e = threadIdx.x; e < 2 * K2 * K3; e += blockDim.x) {
    const int r = e / K3, f = e % K3;
    const int sg = (r < K2) ? r : -(2 * K2 - r);
    // angle / pi = sg / N2 + f / N3, reduced as an exact rational
    const long long num = (long long)sg * N3 + (long long)f * N2;
    double sn, cs;
    sincospi((double)num / (double)((long long)N2 * N3), &sn, &cs);
    const float w = scale * (herm ? herm_weight(f, N3) : 1.0f);
    rot[f * (2 * K2) + r] = make_float2((float)cs * w, (float)sn * w);   // [f][r]: lanes (r) read conflict-free
  }
  __syncthreads();
  pdl_wait();   // everything above is independent of the preceding kernel

  const long long first = blockIdx.x;
  long long n_local;
  if constexpr (COLS) {
    // a task is one plane; this CTA takes the columns first, first + grid, ..: N1 consecutive planes each
    const long long cols = num_tasks / N1;
    n_local = first < cols ? ((cols - first + gridDim.x - 1) / gridDim.x) * N1 : 0;
  } else {
    n_local = first < num_tasks ? (num_tasks - first + gridDim.x - 1) / gridDim.x : 0;
  }

  if (warp == 0) {
    // ---------------- producer: one thread feeds the ring in task order ----------------
    if (lane == 0) {
      // slot and lap (fill number of that slot) advance incrementally: no division on the thread every load of
      // this CTA waits for.  The diagnostic of dtst_plan_debug_ring_fault shortens the loop instead of testing
      // inside it: after `withhold_after` fills (rounded down to whole tasks) the ring is fed no more and the
      // consumers' bounded waits run out.
      const long long n_feed = (withhold_after >= 0 && withhold_after / SPT < n_local) ? withhold_after / SPT : n_local;
      uint32_t slot = 0, lap = 0;
      long long pcol0 = first * N1;   // fused third dimension: first plane of the current column, plane within it
      int pn = 0;
      for (long long tl = 0; tl < n_feed; ++tl) {
        int row0;
        if constexpr (COLS) {
          row0 = (int)((pcol0 + pn) * kTaskRows);
          if (++pn == N1) {
            pn = 0;
            pcol0 += (long long)gridDim.x * N1;
          }
        } else {
          row0 = (int)((first + tl * gridDim.x) * kTaskRows);
        }
#pragma unroll
        for (int s = 0; s < SPT; ++s) {
          if (!mbar_wait_bounded(&empty[slot], (lap & 1u) ^ 1u, abort_flag)) goto producer_done;
          fill_seq[slot] = lap + 1u;
          mbar_arrive_expect_tx(&full[slot], (uint32_t)kStageBytes);
#pragma unroll
          for (int h = 0; h < Cfg::BOXES; ++h)
            tma_load_2d(ring + (size_t)slot * kStageBytes + (size_t)h * RPS * 128, &in_map, h * 32, row0 + s * RPS,
                        &full[slot]);
          if (++slot == (uint32_t)stages) {
            slot = 0;
            ++lap;
          }
        }
      }
    }
  producer_done:
    __syncwarp();
  } else if (!COLS || warp <= W) {
    // ---------------- consumers: one warp per task ----------------
    const int w = warp - 1;
    int ct = w;   // fused third dimension: this warp's task as a CTA-local count (batch = ct / 8, place = ct % 8)
    float* combo = combos_all + (size_t)w * Cfg::COMBO_FLOATS;

    // stage-1 role: lane = (plane in task, row quadruple)
    const int pl1 = lane / QUADS, n1 = lane % QUADS;
    // epilogue role: lane = (plane, mode position r)
    const bool act2 = lane < G * LPP;
    const int pl2 = act2 ? lane / LPP : 0;
    const int l2 = lane % LPP;
    // MMA fragment coordinates
    const int g8 = lane >> 2, t4 = lane & 3;

    // this warp's position in the ring, advanced by W tasks per trip (no division in the loop)
    uint32_t slot0 = (uint32_t)((w * SPT) % stages), lap0 = (uint32_t)((w * SPT) / stages);
    for (long long tl = w; tl < n_local; tl += W) {
      const long long task = first + tl * gridDim.x;
      uint32_t slot1 = slot0, lap1 = lap0;
      if (SPT == 2 && ++slot1 == (uint32_t)stages) {
        slot1 = 0;
        ++lap1;
      }
      constexpr bool kSplit = (SPT == 2 && N2 == 128);   // rows a, b in the first slot, c, d in the second

      // ---- stage 1: the four rows of this lane's quadruple, accumulated straight into the four
      // parity combos  pp = a+d+b+c, pd = a+d-b-c, ms = a-d+b-c, md = a-d-b+c  (one copy of the row code)
      float cpp[NC], cpd[NC], cms[NC], cmd[NC];
#pragma unroll
      for (int c = 0; c < NC; ++c) cpp[c] = cpd[c] = cms[c] = cmd[c] = 0.f;
      if constexpr (!kSplit) {
        if (!wait_fill(fill_seq, full, slot0, lap0, abort_flag, poll_limit)) break;
        if (SPT == 2 && !wait_fill(fill_seq, full, slot1, lap1, abort_flag, poll_limit)) break;
      }
      bool alive = true;
#pragma unroll 1
      for (int r4 = 0; r4 < 4; ++r4) {
        if constexpr (kSplit) {
          if (r4 == 0) alive = wait_fill(fill_seq, full, slot0, lap0, abort_flag, poll_limit);
          if (r4 == 2) {
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[slot0]);
            alive = wait_fill(fill_seq, full, slot1, lap1, abort_flag, poll_limit);
          }
          if (!alive) break;
        }
        // order a, b, c, d = rows n, N2/2-1-n, N2/2+n, N2-1-n of the plane
        const int rowq = (r4 == 0) ? n1 : (r4 == 1) ? (N2 / 2 - 1 - n1) : (r4 == 2) ? (N2 / 2 + n1) : (N2 - 1 - n1);
        const float s1 = (r4 == 0 || r4 == 3) ? 1.f : -1.f;
        const float s2 = (r4 <= 1) ? 1.f : -1.f;
        const float s3 = (r4 == 0 || r4 == 2) ? 1.f : -1.f;
        const int trow = pl1 * N2 + rowq;
        const int sl = (trow / RPS) ? slot1 : slot0;
        const uint32_t st = ring_s + (uint32_t)sl * kStageBytes;
        float o[NC];
        stage1_row<N3, K3, RPS>(st, trow % RPS, o);
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          cpp[c] += o[c];
          cpd[c] = fmaf(s1, o[c], cpd[c]);
          cms[c] = fmaf(s2, o[c], cms[c]);
          cmd[c] = fmaf(s3, o[c], cmd[c]);
        }
      }
      if (!alive) break;
      __syncwarp();
      if (lane == 0) {
        if constexpr (kSplit) {
          mbar_arrive(&empty[slot1]);
        } else {
          mbar_arrive(&empty[slot0]);
          if (SPT == 2) mbar_arrive(&empty[slot1]);
        }
      }

      // ---- stage 2 on the tensor cores (legacy warp-level MMA, TF32 with hi/lo error compensation), one
      // parity class at a time through a small per-warp buffer:
      //   out[(plane, column)][frequency slot] = sum_n combo_cls[n][(plane, column)] * basis_cls[n][slot]
      // The class's combos are published as rows (plane, n) of NC floats, 16-byte chunks swapped pairwise on
      // odd groups of four rows so that both the stores and the fragment loads are bank-conflict free.
      float acc[5][Cfg::MT][4];
#pragma unroll
      for (int cls = 0; cls < 5; ++cls)
#pragma unroll
        for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[cls][mt][e] = 0.f;
#pragma unroll
      for (int cls = 0; cls < 4; ++cls) {
        __syncwarp();   // the previous class's fragment loads (or the previous task's epilogue reads) are done
        {
          float* dst = combo + (size_t)lane * Cfg::NSC;
          const int sw = ((n1 >> 2) & 1);
#pragma unroll
          for (int c4 = 0; c4 < NC / 4; ++c4) {
            const int cc = 4 * (c4 ^ sw);
            const float* srcv = (cls == 0) ? cpp : (cls == 1) ? cpd : (cls == 2) ? cms : cmd;
            *reinterpret_cast<float4*>(dst + cc) =
                make_float4(srcv[4 * c4], srcv[4 * c4 + 1], srcv[4 * c4 + 2], srcv[4 * c4 + 3]);
          }
        }
        __syncwarp();
#pragma unroll
        for (int ks = 0; ks < Cfg::NKS; ++ks) {
          const float4 bf = btab[(cls * Cfg::NKS + ks) * 32 + lane];
          const uint32_t bh0 = __float_as_uint(bf.x), bh1 = __float_as_uint(bf.y);
          const uint32_t bl0 = __float_as_uint(bf.z), bl1 = __float_as_uint(bf.w);
          float4 bx = make_float4(0.f, 0.f, 0.f, 0.f);
          if (cls == 0) bx = btab[(4 * Cfg::NKS + ks) * 32 + lane];
#pragma unroll
          for (int mt = 0; mt < Cfg::MT; ++mt) {
            uint32_t ahi[4], alo[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int m = 16 * mt + g8 + 8 * (e & 1);
              const int n = 8 * ks + t4 + 4 * (e >> 1);
              const int pl = m / NC, c = m % NC;
              const float v = combo[(size_t)(pl * QUADS + n) * Cfg::NSC + (c ^ ((e >> 1) << 2))];
              split_tf32(v, ahi[e], alo[e]);
            }
            mma_tf32(acc[cls][mt], ahi, bh0, bh1);
            mma_tf32(acc[cls][mt], alo, bh0, bh1);
            mma_tf32(acc[cls][mt], ahi, bl0, bl1);
            if (cls == 0) {   // the pp operand also feeds the unpaired A_{K2}
              mma_tf32(acc[4][mt], ahi, __float_as_uint(bx.x), __float_as_uint(bx.y));
              mma_tf32(acc[4][mt], alo, __float_as_uint(bx.x), __float_as_uint(bx.y));
              mma_tf32(acc[4][mt], ahi, __float_as_uint(bx.z), __float_as_uint(bx.w));
            }
          }
        }
      }
      __syncwarp();

      // A/B sums -> shared: entry g for A_g (g <= K2), entry K2+g for B_g (g >= 1)
#pragma unroll
      for (int cls = 0; cls < 5; ++cls)
#pragma unroll
        for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int m = 16 * mt + g8 + 8 * (e >> 1);
            const int gi = 2 * t4 + (e & 1);
            const int pl = m / NC, c = m % NC;
            int entry;
            bool valid = gi < Cfg::GT;
            if (cls == 0) entry = 2 * gi;
            else if (cls == 1) entry = 2 * gi + 1;
            else if (cls == 2) entry = K2 + 2 * gi + 1;
            else if (cls == 3) entry = K2 + 2 * gi + 2;
            else { entry = K2; valid = (gi == 0); }
            if (valid) combo[pl * Cfg::ABP + entry * Cfg::ABS + c] = acc[cls][mt][e];
          }
      __syncwarp();

      if constexpr (COLS) {
        // the accumulator warps must be done with the batch that used this buffer before
        const int u = ct >> 4;
        if (u > 0 && !wait_bar_warp(&pfree[(ct >> 3) & 1], (uint32_t)(u - 1) & 1u, abort_flag, poll_limit)) break;
      }
      // epilogue: Z_{+g} = rho (A - iB), Z_{-g} = rho (A + iB) with A = AC - i AS, B = BC - i BS
      if (act2) {
        const int r = l2;
        const bool pos = r < K2;
        const int g = pos ? r : 2 * K2 - r;
        const float* A = combo + pl2 * Cfg::ABP + g * Cfg::ABS;
        const float* Bp = combo + pl2 * Cfg::ABP + (K2 + g) * Cfg::ABS;
        float2* dst = out + ((task * G + pl2) * (2 * K2) + r) * K3;
        // fused third dimension: place ct % 8 of batch ct / 8; the 8-float groups of a plane are permuted by its
        // place so that the accumulator warps' fragment loads (four planes x eight columns per request) hit 32
        // different banks
        float* prow = pbuf + (size_t)(((ct >> 3) & 1) * 8 + (ct & 7)) * PCOLS;
        const int swz = (ct & 3) << 3;
        const float2* rr = rot + r;
#pragma unroll
        for (int f2 = 0; f2 < K3 / 2; ++f2) {
          float res[4];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int f = 2 * f2 + e;
            const float AC = A[f], AS = A[K3 + f];
            const float BC = g > 0 ? Bp[f] : 0.f, BS = g > 0 ? Bp[K3 + f] : 0.f;
            const float wr = pos ? AC - BS : AC + BS;
            const float wi = pos ? -(AS + BC) : BC - AS;
            const float2 ro = rr[f * (2 * K2)];
            res[2 * e] = ro.x * wr - ro.y * wi;
            res[2 * e + 1] = ro.x * wi + ro.y * wr;
          }
          if constexpr (COLS)
            *reinterpret_cast<float4*>(prow + ((r * 2 * K3 + 4 * f2) ^ swz)) = make_float4(res[0], res[1], res[2], res[3]);
          else
            *reinterpret_cast<float4*>(dst + 2 * f2) = make_float4(res[0], res[1], res[2], res[3]);
        }
      }
      __syncwarp();   // the next task's combos overwrite the A/B entries read above
      if constexpr (COLS) {
        if (lane == 0) mbar_arrive(&pfull[(ct >> 3) & 1]);   // this plane is in its batch (release after the __syncwarp)
        ct += W;
      }
      slot0 += (uint32_t)(W * SPT);
      while (slot0 >= (uint32_t)stages) {
        slot0 -= (uint32_t)stages;
        ++lap0;
      }
    }
  } else {
    if constexpr (COLS) {
      // ---------------- accumulator warps: contract every complete batch of 8 planes along the third dimension ---
      const int a = warp - (W + 1);
      const int g8 = lane >> 2, t4 = lane & 3;
      constexpr int NTW = (PCOLS / 8) / kColAccWarps;   // n-tiles of 8 real columns per warp
      constexpr int INNER = PCOLS / 2;                  // complex values per plane
      const int qN = N1 - (N1 >> 2);                    // sin x = cos(x - pi/2): index shift in the cosine table
      const int nm = N1 - 1;                            // N1 is a power of two: indices reduce with a mask
      float accC[NTW][4], accS[NTW][4];
      float z16[4];                                     // Z_{-K1} of this lane's two complex columns
#pragma unroll
      for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) accC[nt][e] = accS[nt][e] = 0.f;
      z16[0] = z16[1] = z16[2] = z16[3] = 0.f;
      const int nb = (int)(n_local >> 3), bpc = N1 >> 3;
      long long col = first;
      int bc = 0;                                       // batch within the column
      for (int b = 0; b < nb; ++b) {
        const int buf = b & 1;
        if (!wait_bar_warp(&pfull[buf], (uint32_t)(b >> 1) & 1u, abort_flag, poll_limit)) break;
        const float* pb = pbuf + (size_t)buf * 8 * PCOLS;
        // basis fragments of this batch: rows = frequencies g8, g8 + 8; columns = planes n = 8 bc + t4, + 4
        uint32_t chi[4], clo[4], shi[4], slo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int g = g8 + 8 * (e & 1), n = 8 * bc + t4 + 4 * (e >> 1);
          const int idx = (g * n) & nm;
          split_tf32_rna(ctab[idx], chi[e], clo[e]);
          split_tf32_rna(ctab[(idx + qN) & nm], shi[e], slo[e]);
        }
        const int sw = t4 << 3;   // planes t4 and t4 + 4 carry the same permutation
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt) {
          const int c0 = (8 * (NTW * a + nt) + g8) ^ sw;
          uint32_t bh0, bl0, bh1, bl1;
          split_tf32_round(pb[t4 * PCOLS + c0], bh0, bl0);
          split_tf32_round(pb[(t4 + 4) * PCOLS + c0], bh1, bl1);
          mma3_tf32(accC[nt], chi, clo, bh0, bh1, bl0, bl1);
          mma3_tf32(accS[nt], shi, slo, bh0, bh1, bl0, bl1);
        }
        // the unpaired mode -K1: e^{+2 pi i K1 n / N1} depends on the place in the batch only (8 K1 / N1 is whole)
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int idx = (K1 * k) & nm;
          const float cs = ctab[idx], sn = ctab[(idx + qN) & nm];
          const float4 v = *reinterpret_cast<const float4*>(pb + k * PCOLS + ((2 * INNER / kColAccWarps * a + 4 * lane) ^ ((k & 3) << 3)));
          z16[0] = fmaf(v.x, cs, fmaf(-v.y, sn, z16[0]));
          z16[1] = fmaf(v.x, sn, fmaf(v.y, cs, z16[1]));
          z16[2] = fmaf(v.z, cs, fmaf(-v.w, sn, z16[2]));
          z16[3] = fmaf(v.z, sn, fmaf(v.w, cs, z16[3]));
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&pfree[buf]);
        if (++bc == bpc) {
          // the column is complete: Z_{+g} = C_g - i S_g (position g), Z_{-g} = C_g + i S_g (position 2 K1 - g)
          float2* ob = out + col * (2 * K1) * INNER;
#pragma unroll
          for (int nt = 0; nt < NTW; ++nt) {
            const int m = 4 * (NTW * a + nt) + t4;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int g = g8 + 8 * h;
              const float cx = accC[nt][2 * h], cy = accC[nt][2 * h + 1];
              const float sx = accS[nt][2 * h], sy = accS[nt][2 * h + 1];
              ob[(long long)g * INNER + m] = make_float2(cx + sy, cy - sx);
              if (g > 0) ob[(long long)(2 * K1 - g) * INNER + m] = make_float2(cx - sy, cy + sx);
              accC[nt][2 * h] = accC[nt][2 * h + 1] = accS[nt][2 * h] = accS[nt][2 * h + 1] = 0.f;
            }
          }
          *reinterpret_cast<float4*>(ob + (long long)K1 * INNER + INNER / kColAccWarps * a + 2 * lane) =
              make_float4(z16[0], z16[1], z16[2], z16[3]);
          z16[0] = z16[1] = z16[2] = z16[3] = 0.f;
          bc = 0;
          col += gridDim.x;
        }
      }
    }
  }

  // the dependent kernel may be scheduled from here on: triggering at the start of this kernel instead was measured
  // slower (its blocks become resident beside this kernel's and compete for the issue slots of a kernel that needs them)
  pdl_trigger();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    // the pipeline gave up: loads that were armed but never consumed may still be in flight, and this CTA's
    // shared memory must not be handed to the next one while the TMA engine writes to it
    for (int s = 0; s < stages; ++s)
      if (fill_seq[s] > 0) mbar_wait_plain(&full[s], (fill_seq[s] - 1u) & 1u, 1u << 16);
    atomicExch(status, 1);
  }
}

// ---------------------------------------------------------------------------------------------
// Inverse plane kernel: the transpose of the forward one.  in[planes][2*K2][K3] complex ->
// real rows [planes*N2][N3].  Each warp owns a task of 128 output rows: it pre-rotates the plane's
// modes, forms alpha_g = V'_{+g} + V'_{-g}, beta_g = i (V'_{+g} - V'_{-g}), expands them to the
// four rows of each row quadruple (one lane per quadruple), expands every row to N3 reals with
// the same folded basis, stages the rows in shared memory (TMA swizzle) and stores them with TMA.
// Inverse row code, one quadruple j: the four class sums over f = F .. K3-1 with immediate coefficients.
template <int N3, int K3, int J, int F>
__device__ __forceinline__ void e1_freqs(const float (&z)[2 * K3], float& Ea, float& Oa, float& Eb, float& Ob) {
  if constexpr (F < K3) {
    constexpr float cs = ct::Coef<N3, J, F>::cs, sn = ct::Coef<N3, J, F>::sn;
    if constexpr ((F & 1) == 0) {
      Ea = (F == 0) ? z[F] * cs : fmaf(z[F], cs, Ea);
      if constexpr (F > 0) Eb = (F == 2) ? z[K3 + F] * sn : fmaf(z[K3 + F], sn, Eb);
    } else {
      Oa = (F == 1) ? z[F] * cs : fmaf(z[F], cs, Oa);
      Ob = (F == 1) ? z[K3 + F] * sn : fmaf(z[K3 + F], sn, Ob);
    }
    e1_freqs<N3, K3, J, F + 1>(z, Ea, Oa, Eb, Ob);
  }
}

template <int N3, int K3, int J>
__device__ __forceinline__ void e1_quad(const float (&z)[2 * K3], float& ya, float& yb, float& yc, float& yd) {
  float Ea = 0.f, Oa = 0.f, Eb = 0.f, Ob = 0.f;
  e1_freqs<N3, K3, J, 0>(z, Ea, Oa, Eb, Ob);
  const float sa = Ea + Oa, da = Ea - Oa, sb = Eb + Ob, db = Eb - Ob;
  ya = sa - sb;   // y[j]
  yd = sa + sb;   // y[N3-1-j]
  yb = da + db;   // y[N3/2-1-j]
  yc = da - db;   // y[N3/2+j]
}

template <int N3, int K3, int BOXR, int C>
__device__ __forceinline__ void e1_chunks(uint32_t rx, const float (&z)[2 * K3]) {
  constexpr int CH = N3 / 4;
  if constexpr (C < CH / 4) {
    constexpr int P = BOXR * 128;
    constexpr int c0 = C, c1 = CH / 2 - 1 - C, c2 = CH / 2 + C, c3 = CH - 1 - C;
    float a[4], b[4], cc[4], d[4];
    e1_quad<N3, K3, 4 * C + 0>(z, a[0], b[0], cc[0], d[0]);
    e1_quad<N3, K3, 4 * C + 1>(z, a[1], b[1], cc[1], d[1]);
    e1_quad<N3, K3, 4 * C + 2>(z, a[2], b[2], cc[2], d[2]);
    e1_quad<N3, K3, 4 * C + 3>(z, a[3], b[3], cc[3], d[3]);
    sts128_s<(c0 / 8) * P>(rx ^ (uint32_t)((c0 % 8) << 4), a[0], a[1], a[2], a[3]);
    sts128_s<(c1 / 8) * P>(rx ^ (uint32_t)((c1 % 8) << 4), b[3], b[2], b[1], b[0]);
    sts128_s<(c2 / 8) * P>(rx ^ (uint32_t)((c2 % 8) << 4), cc[0], cc[1], cc[2], cc[3]);
    sts128_s<(c3 / 8) * P>(rx ^ (uint32_t)((c3 % 8) << 4), d[3], d[2], d[1], d[0]);
    e1_chunks<N3, K3, BOXR, C + 1>(rx, z);
  }
}

template <int N3, int K3, int BOXR>
__device__ __forceinline__ void expand_row(uint32_t stage, int row, const float (&z)[2 * K3]) {
  // same single-XOR swizzled addressing as the forward kernel's row loads
  const uint32_t rx = stage + (uint32_t)row * 128u + (((uint32_t)row & 7u) << 4);
  e1_chunks<N3, K3, BOXR, 0>(rx, z);
}

template <int N3, int K3, int N2, int K2>
struct InvCfg {
  using P = PlaneCfg<N3, K3, N2, K2>;
  static constexpr int ABS = P::NC + 4;                     // floats between entries
  static constexpr int ENTRIES = 2 * K2 + 2;                // alpha_0..alpha_K2, beta_0..beta_K2 (beta_0 unused)
  static constexpr int ABP = ENTRIES * ABS + 4;             // floats between planes
  static constexpr int AB_FLOATS = ((P::G * ABP + 3) / 4) * 4;
  static constexpr int COMBO_FLOATS = 32 * P::NS;           // expanded combos, one row per quadruple
  static constexpr int NT = P::NC / 8;                      // MMA n-tiles over the columns
  static constexpr int STAGING_BYTES = kTaskRows * N3 * 4;  // 128 output rows
  // With two staging blocks that are stored one after the other (rows a, b then rows c, d) the small
  // alpha/beta and combo buffers live inside the first block: its store is issued half a task before the
  // next task needs the space, so one bounded wait on that store group is all the aliasing costs.
  static constexpr bool ALIAS = (P::SPT == 2 && N2 == 128) && ((AB_FLOATS + COMBO_FLOATS) * 4 <= kStageBytes);
  static constexpr int WARP_BYTES =
      ALIAS ? STAGING_BYTES : STAGING_BYTES + (((AB_FLOATS + COMBO_FLOATS) * 4 + 1023) / 1024) * 1024;
};

// ---------------------------------------------------------------------------------------------
// Column expansion inside the inverse plane kernel.  The dimension in front of the two the plane kernel expands
// (extent N1, 2 K1 retained entries) is expanded by ONE EXTRA WARP per CTA, column by column (a column = all N1
// planes that share their leading indices), a few microseconds before the worker warps consume the planes:
//   in1[col][2 K1][inner]  ->  ring[col % R][N1][inner],   inner = 2 K2 * K3 complex values per plane.
// The expanded planes are then read while they are still in L2, and the separate expansion launch with its
// full-size intermediate in HBM disappears.  Flow control is two counters per column in global memory:
//   ready[col]  += 1 by the helper that finished one block of positions;
//               a worker loads a plane of column col only after all blocks of the column are there;
//   done[col]   += planes by a worker once its planes of column col are in its registers; a helper overwrites
//               ring slot col % R only after done[col - R] == N1.
// Helpers walk the (column, block) pairs in ascending order and workers walk the planes in ascending order, so
// the smallest blocked column can always make progress as long as all CTAs are resident (one per SM).  Every
// wait is a bounded poll that raises the status word and makes its warp leave.
// The arithmetic is the folded expansion of the middle-dimension kernels (same fold, same TF32 hi/lo MMAs), with
// the basis fragments in registers instead of shared memory: this kernel's shared memory is all staging.
__device__ __forceinline__ bool poll_counter(const int* ctr, int want, uint32_t limit, int* status) {
  for (uint32_t it = 0; it < limit; ++it) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
    if (v >= want) return true;
    __nanosleep(100);
    if ((it & 255u) == 255u && *reinterpret_cast<volatile int*>(status) != 0) return false;   // someone gave up
  }
  atomicExch(status, 1);
  return false;
}

template <int K1, int NT1>
struct ColBasis {
  float4 bf[NT1][4];      // B fragments (b0 hi, b1 hi, b0 lo, b1 lo) per tile of 8 row quadruples and parity class
  float c0[NT1], c1[NT1]; // cos(psi_K1 (n + 1/2)) of this lane's two quadruples per tile
  float2 rho[7];          // e^{i psi_g / 2} of this lane's six frequencies; [6] = frequency K1
  __device__ __forceinline__ void init(int N1, int lane) {
    const int lg = lane >> 2, lt = lane & 3;
#pragma unroll
    for (int nt = 0; nt < NT1; ++nt) {
#pragma unroll
      for (int cls = 0; cls < 4; ++cls) {
        uint32_t hi[2], lo[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int slot = lt + 4 * h;
          float cs, sn;
          basis_cs(class_freq(cls, slot), 8 * nt + lg, N1, cs, sn);
          const float v = slot < K1 / 2 ? ((cls == 0 || cls == 1) ? cs : sn) : 0.f;
          split_tf32_rna(v, hi[h], lo[h]);
        }
        bf[nt][cls] = make_float4(__uint_as_float(hi[0]), __uint_as_float(hi[1]), __uint_as_float(lo[0]),
                                  __uint_as_float(lo[1]));
      }
      float sn;
      basis_cs(K1, 8 * nt + 2 * lt, N1, c0[nt], sn);
      basis_cs(K1, 8 * nt + 2 * lt + 1, N1, c1[nt], sn);
    }
#pragma unroll
    for (int j = 0; j < 7; ++j) {
      const int g = j < 6 ? 2 * lt + (j % 3) + 8 * (j / 3) : K1;
      double s, c;
      sincospi((double)g / (double)N1, &s, &c);
      rho[j] = make_float2((float)c, (float)s);
    }
  }
};

// one block of 8 MT complex positions of one column: src[2 K1][inner] -> dst[N1][inner] (both already offset to the block)
template <int K1, int NT1, int MT>
__device__ __forceinline__ void col_expand_block(const ColBasis<K1, NT1>& cb, const float2* __restrict__ src,
                                                 float2* __restrict__ dst, long long inner, int N1, int lane) {
  const int g8 = lane >> 2, t4 = lane & 3;
  uint32_t ah[MT][4][4], al[MT][4][4];
  float2 aKv[MT];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    const float2* sp = src + 8 * mt + g8;
    float2 alpha[6], beta[6];
#pragma unroll
    for (int j = 0; j < 6; ++j) {
      const int g = 2 * t4 + (j % 3) + 8 * (j / 3);
      float2 v = make_float2(0.f, 0.f), u = make_float2(0.f, 0.f);
      if (g < K1) v = __ldcs(sp + (long long)g * inner);
      if (g > 0 && g <= K1) u = __ldcs(sp + (long long)(2 * K1 - g) * inner);
      const float2 r = cb.rho[j];
      const float2 vp = make_float2(v.x * r.x + v.y * r.y, v.y * r.x - v.x * r.y);   // v * conj(rho)
      const float2 vm = make_float2(u.x * r.x - u.y * r.y, u.y * r.x + u.x * r.y);   // u * rho
      alpha[j] = make_float2(vp.x + vm.x, vp.y + vm.y);
      beta[j] = make_float2(-(vp.y - vm.y), vp.x - vm.x);                            // i (vp - vm)
    }
    {
      const float2 u = __ldcs(sp + (long long)K1 * inner);                           // V_{-K1}
      const float2 r = cb.rho[6];
      aKv[mt] = make_float2(u.x * r.x - u.y * r.y, u.y * r.x + u.x * r.y);           // alpha_K1 = rho_K1 V_{-K1}
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      split_tf32_round(alpha[3 * h + 0].x, ah[mt][0][2 * h], al[mt][0][2 * h]);
      split_tf32_round(alpha[3 * h + 0].y, ah[mt][0][2 * h + 1], al[mt][0][2 * h + 1]);
      split_tf32_round(alpha[3 * h + 1].x, ah[mt][1][2 * h], al[mt][1][2 * h]);
      split_tf32_round(alpha[3 * h + 1].y, ah[mt][1][2 * h + 1], al[mt][1][2 * h + 1]);
      split_tf32_round(beta[3 * h + 1].x, ah[mt][2][2 * h], al[mt][2][2 * h]);
      split_tf32_round(beta[3 * h + 1].y, ah[mt][2][2 * h + 1], al[mt][2][2 * h + 1]);
      split_tf32_round(beta[3 * h + 2].x, ah[mt][3][2 * h], al[mt][3][2 * h]);
      split_tf32_round(beta[3 * h + 2].y, ah[mt][3][2 * h + 1], al[mt][3][2 * h + 1]);
    }
  }
  float2* ob = dst + g8;
#pragma unroll
  for (int nt = 0; nt < NT1; ++nt) {
    const int n0 = 8 * nt + 2 * t4;                      // this lane's two quadruples: n0, n0 + 1
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      float acc[4][4];
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[c][e] = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c)
        mma3_tf32(acc[c], ah[mt][c], al[mt][c], __float_as_uint(cb.bf[nt][c].x), __float_as_uint(cb.bf[nt][c].y),
                  __float_as_uint(cb.bf[nt][c].z), __float_as_uint(cb.bf[nt][c].w));
      acc[0][0] = fmaf(aKv[mt].x, cb.c0[nt], acc[0][0]);
      acc[0][1] = fmaf(aKv[mt].x, cb.c1[nt], acc[0][1]);
      acc[0][2] = fmaf(aKv[mt].y, cb.c0[nt], acc[0][2]);
      acc[0][3] = fmaf(aKv[mt].y, cb.c1[nt], acc[0][3]);
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int n = n0 + q;
        const float per = acc[0][q], pei = acc[0][2 + q], por = acc[1][q], poi = acc[1][2 + q];
        const float qor = acc[2][q], qoi = acc[2][2 + q], qer = acc[3][q], qei = acc[3][2 + q];
        const float spr = per + por, dpr = per - por, sqr = qor + qer, dqr = qor - qer;
        const float spi = pei + poi, dpi = pei - poi, sqi = qoi + qei, dqi = qoi - qei;
        float2* d = ob + 8 * mt;
        d[(long long)n * inner] = make_float2(spr + sqr, spi + sqi);                  // z_n         = Pe+Po+Qo+Qe
        d[(long long)(N1 / 2 - 1 - n) * inner] = make_float2(dpr + dqr, dpi + dqi);   // z_{N/2-1-n} = Pe-Po+Qo-Qe
        d[(long long)(N1 / 2 + n) * inner] = make_float2(dpr - dqr, dpi - dqi);       // z_{N/2+n}   = Pe-Po-Qo+Qe
        d[(long long)(N1 - 1 - n) * inner] = make_float2(spr - sqr, spi - sqi);       // z_{N-1-n}   = Pe+Po-Qo-Qe
      }
    }
  }
}

constexpr int kColExpandMT = 2;   // positions per helper block / 8 (blocks of 8 positions were measured slower: the
                                  // per-block overhead makes the helper the bottleneck)
constexpr int kColExpandHelpers = 1;   // helper warps per CTA: a ninth warp would cap every warp at 168 registers (three warps
                                       // on one scheduler's register file) and the workers need 255

// what the helper warp and the waits of the workers need (all zero / null when the kernel runs without a helper)
struct ColExpandArgs {
  const float2* in1;     // [cols][2 K1][inner]: the tensor before this dimension's expansion
  float2* ring;          // [R][N1][inner]
  int* ready;            // [cols]
  int* done;             // [cols]
  int* status;
  long long cols;
  int N1, R;
  uint32_t poll_limit;
};

template <int N3, int K3, int N2, int K2, int W, int K1, int NT1>
__global__ void __launch_bounds__((W + (K1 > 0 ? kColExpandHelpers : 0)) * 32, 1)
inv_plane_kernel(const __grid_constant__ CUtensorMap out_map, const float2* __restrict__ in, long long num_tasks, float scale, int herm,
                 const ColExpandArgs ce) {
  constexpr bool HELP = K1 > 0;
  using Cfg = PlaneCfg<N3, K3, N2, K2>;
  using IC = InvCfg<N3, K3, N2, K2>;
  constexpr int NC = Cfg::NC, QUADS = Cfg::QUADS, G = Cfg::G, LPP = Cfg::LPP;
  constexpr int SPT = Cfg::SPT, RPS = Cfg::ROWS_PER_STAGE;

  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment for the TMA swizzle, by pointer arithmetic on the shared array itself (an integer
  // round trip would make the compiler lose the address space and emit generic loads and stores)
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  char* staging = reinterpret_cast<char*>(smem) + (size_t)(warp < W ? warp : 0) * IC::WARP_BYTES;
  const uint32_t staging_s = smem_u32(staging);
  float* ab = reinterpret_cast<float*>(IC::ALIAS ? staging : staging + IC::STAGING_BYTES);
  float2* rot = reinterpret_cast<float2*>(smem + (size_t)W * IC::WARP_BYTES);

  if (threadIdx.x == 0) prefetch_tensormap(&out_map);
  // conjugate rotation table: exp(-i pi (sg/N2 + f/N3)) * scale * Hermitian weight
  for (int e = threadIdx.x; e < 2 * K2 * K3; e += blockDim.x) {
    const int r = e / K3, f = e % K3;
    const int sg = (r < K2) ? r : -(2 * K2 - r);
    const long long num = (long long)sg * N3 + (long long)f * N2;
    double sn, cs;
    sincospi((double)num / (double)((long long)N2 * N3), &sn, &cs);
    const float w = scale * (herm ? herm_weight(f, N3) : 1.0f);
    rot[f * (2 * K2) + r] = make_float2((float)cs * w, -(float)sn * w);   // [f][r]
  }
  __syncthreads();

  if constexpr (HELP) {
    if (warp >= W) {
      // ---------------- helper warp: expands the columns ahead of the workers ----------------
      constexpr int inner = 2 * K2 * K3;               // complex values per plane
      constexpr int CMT = kColExpandMT;                // m-tiles (8 positions) per block
      constexpr int BLK = inner / (8 * CMT);           // blocks per column
      ColBasis<K1, NT1> cb;
      cb.init(ce.N1, lane);
      pdl_wait();
      const long long total = ce.cols * BLK;
      const long long hstride = (long long)gridDim.x * kColExpandHelpers;
      for (long long s = (long long)blockIdx.x * kColExpandHelpers + (warp - W); s < total; s += hstride) {
        const long long col = s / BLK;
        const int blk = (int)(s % BLK);
        {   // the next block's input rows into L2 while this one runs
          const long long nx = s + hstride;
          if (nx < total) {
            const float2* nsrc = ce.in1 + (nx / BLK) * (2 * K1) * inner + (nx % BLK) * (8 * CMT);
            for (int r = lane; r < 2 * K1; r += 32) asm volatile("prefetch.global.L2 [%0];" ::"l"(nsrc + (long long)r * inner));
          }
        }
        bool ok = true;
        if (col >= ce.R) {
          if (lane == 0) ok = poll_counter(ce.done + (col - ce.R), ce.N1, ce.poll_limit, ce.status);
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
        if (!ok) break;
        col_expand_block<K1, NT1, CMT>(cb, ce.in1 + col * (2 * K1) * inner + blk * (8 * CMT),
                                       ce.ring + (col % ce.R) * (long long)ce.N1 * inner + blk * (8 * CMT), inner,
                                       ce.N1, lane);
        __threadfence();     // this lane's rows are visible device-wide ...
        __syncwarp();        // ... for every lane, before the block is published
        if (lane == 0) asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(ce.ready + col), "r"(1) : "memory");
      }
      return;
    }
  }

  // roles: row quadruple (stage 1 / unfold), MMA fragment coordinates, mode loader
  const int pl1 = lane / QUADS, n1 = lane % QUADS;
  const int g8 = lane >> 2, t4 = lane & 3;
  float* combo = ab + IC::AB_FLOATS;

  // Second-dimension basis as MMA A fragments (row = quadruple n, col = frequency slot of the parity class),
  // TF32 hi/lo.  Classes: 0 = Pe (even g, cos), 1 = Po (odd g, cos), 2 = Qo (odd g, sin), 3 = Qe (even g, sin);
  // index 4 = the unpaired g = K2 cosine, which adds into Pe through one extra k-step.
  uint32_t ahi[5][Cfg::MT2][4], alo[5][Cfg::MT2][4];
#pragma unroll
  for (int cls = 0; cls < 5; ++cls)
#pragma unroll
    for (int mt = 0; mt < Cfg::MT2; ++mt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int n = (16 * mt + g8 + 8 * (e & 1)) % QUADS;
        const int gi = t4 + 4 * (e >> 1);
        int g = 0;
        bool valid = gi < Cfg::GT;
        if (cls == 0) g = 2 * gi;
        else if (cls == 1 || cls == 2) g = 2 * gi + 1;
        else if (cls == 3) g = 2 * gi + 2;
        else { g = K2; valid = (gi == 0); }
        double sn, cs;
        sincospi((double)(((long long)g * (2 * n + 1)) % (2 * N2)) / (double)N2, &sn, &cs);
        const float v = valid ? ((cls == 2 || cls == 3) ? (float)sn : (float)cs) : 0.f;
        split_tf32_rna(v, ahi[cls][mt][e], alo[cls][mt][e]);
      }

  // loader role: lane = (plane, mode position r)
  const bool actl = lane < G * LPP;
  const int pll = actl ? lane / LPP : 0, rl = lane % LPP;

  const long long tstride = (long long)gridDim.x * W;
  long long task = (long long)blockIdx.x + (long long)warp * gridDim.x;
  float4 vin[K3 / 2];
  pdl_wait();   // everything above is independent of the preceding kernel
  // where the modes of this lane's plane of task t live: the reduced tensor itself, or (with the helper warp) the
  // slot of the plane's column in the ring
  auto plane_src = [&](long long t) -> const float4* {
    long long p = t * G + pll;
    if constexpr (HELP) p = ((p / ce.N1) % ce.R) * ce.N1 + p % ce.N1;
    return reinterpret_cast<const float4*>((HELP ? ce.ring : in) + (p * (2 * K2) + rl) * K3);
  };
  // with the helper warp: wait until the column of task t has been expanded (one verdict for the warp).  `early`
  // is the counter value lane 0 fetched a while ago (the load travels while the warp works), so that in the usual
  // case - the helpers are ahead - the check costs no round trip to L2.
  auto fetch_ready = [&](long long t) -> int {
    int v = 0;
    if constexpr (HELP) {
      if (lane == 0 && t < num_tasks)
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ce.ready + (t * G) / ce.N1) : "memory");
    }
    return v;
  };
  auto column_ready = [&](long long t, int early) -> bool {
    if constexpr (HELP) {
      bool ok = true;
      if (lane == 0 && early < 2 * K2 * K3 / (8 * kColExpandMT))
        ok = poll_counter(ce.ready + (t * G) / ce.N1, 2 * K2 * K3 / (8 * kColExpandMT), ce.poll_limit, ce.status);
      return __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    } else {
      return true;
    }
  };
  bool alive = true;
  if (task < num_tasks) {
    alive = column_ready(task, 0);
    if (alive && actl) {
      const float4* src = plane_src(task);
      // ring slots are rewritten during the kernel: read them from L2 (an L1 line could be a stale earlier column)
#pragma unroll
      for (int i = 0; i < K3 / 2; ++i) vin[i] = HELP ? __ldcg(src + i) : __ldcs(src + i);
    }
  }

  for (; alive && task < num_tasks; task += tstride) {
    const int ready_early = fetch_ready(task + tstride);
    if constexpr (IC::ALIAS) {
      // the store of the previous task's first block (committed second to last) must have read its rows
      if (lane == 0) tma_store_wait_read<1>();
      __syncwarp();
    }
    // ---- rotate this task's modes, publish V'
    if (actl) {
      float* dst = ab + pll * IC::ABP + rl * IC::ABS;
      const float2* rr = rot + rl;
      float re[K3], im[K3];
#pragma unroll
      for (int i = 0; i < K3 / 2; ++i) {
        const float2 r0 = rr[(2 * i) * (2 * K2)], r1 = rr[(2 * i + 1) * (2 * K2)];
        re[2 * i] = vin[i].x * r0.x - vin[i].y * r0.y;
        im[2 * i] = vin[i].x * r0.y + vin[i].y * r0.x;
        re[2 * i + 1] = vin[i].z * r1.x - vin[i].w * r1.y;
        im[2 * i + 1] = vin[i].z * r1.y + vin[i].w * r1.x;
      }
#pragma unroll
      for (int i = 0; i < K3 / 4; ++i) {
        *reinterpret_cast<float4*>(dst + 4 * i) = make_float4(re[4 * i], re[4 * i + 1], re[4 * i + 2], re[4 * i + 3]);
        *reinterpret_cast<float4*>(dst + K3 + 4 * i) =
            make_float4(im[4 * i], im[4 * i + 1], im[4 * i + 2], im[4 * i + 3]);
      }
    }
    if constexpr (HELP) {
      // this task's planes are in registers (their values were just used): their ring slots may be reused
      __syncwarp();
      if (lane == 0)   // release: ordered after this warp's loads of the planes (made cumulative by the __syncwarp)
        asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(ce.done + (task * G) / ce.N1), "r"(G) : "memory");
    }
    // prefetch the next task's modes while this one is expanded
    {
      const long long nt = task + tstride;
      if (nt < num_tasks) {
        alive = column_ready(nt, ready_early);
        if (alive && actl) {
          const float4* src = plane_src(nt);
#pragma unroll
          for (int i = 0; i < K3 / 2; ++i) vin[i] = HELP ? __ldcg(src + i) : __ldcs(src + i);
        }
      }
    }
    __syncwarp();
    // ---- alpha_g = V'_{+g} + V'_{-g}, beta_g = i (V'_{+g} - V'_{-g}); lane (plane, g), g = 0..K2
    {
      const bool acta = lane < G * LPP && (lane % LPP) <= K2;
      const int pla = acta ? lane / LPP : 0, g = acta ? lane % LPP : 0;
      float vp[NC], vm[NC];
      const float* srcp = ab + pla * IC::ABP + g * IC::ABS;
      const float* srcm = ab + pla * IC::ABP + ((2 * K2 - g) % (2 * K2)) * IC::ABS;
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        vp[c] = (g < K2) ? srcp[c] : 0.f;
        vm[c] = (g > 0) ? srcm[c] : 0.f;
      }
      __syncwarp();
      if (acta) {
        float* da = ab + pla * IC::ABP + g * IC::ABS;
        float* db = ab + pla * IC::ABP + (K2 + 1 + g) * IC::ABS;
#pragma unroll
        for (int f = 0; f < K3; ++f) {
          const float pr = vp[f], pi = vp[K3 + f], mr = vm[f], mi = vm[K3 + f];
          da[f] = pr + mr;
          da[K3 + f] = pi + mi;
          // i * ((pr - mr) + i (pi - mi)) = -(pi - mi) + i (pr - mr)
          db[f] = -(pi - mi);
          db[K3 + f] = pr - mr;
        }
      }
    }
    __syncwarp();

    // ---- expand the second dimension on the tensor cores (warp-level MMA, TF32 hi/lo compensated):
    // combo_cls[quadruple n][(plane, column)] = sum_slot basis_cls[n][slot] * (alpha|beta)_cls[slot][column]
#pragma unroll
    for (int cls = 0; cls < 4; ++cls)
#pragma unroll
      for (int nt = 0; nt < IC::NT; ++nt)
#pragma unroll
        for (int mt = 0; mt < Cfg::MT2; ++mt) {
          const int pl = (16 * mt) / QUADS;
          float acc[4] = {0.f, 0.f, 0.f, 0.f};
          const int c = 8 * nt + g8;
          {
            uint32_t bh[2], bl[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int gi = t4 + 4 * h;
              int entry = 0;
              if (cls == 0) entry = 2 * gi;
              else if (cls == 1) entry = 2 * gi + 1;
              else if (cls == 2) entry = K2 + 1 + 2 * gi + 1;
              else entry = K2 + 1 + 2 * gi + 2;
              const float v = (gi < Cfg::GT) ? ab[pl * IC::ABP + entry * IC::ABS + c] : 0.f;
              split_tf32(v, bh[h], bl[h]);
            }
            mma_tf32(acc, ahi[cls][mt], bh[0], bh[1]);
            mma_tf32(acc, alo[cls][mt], bh[0], bh[1]);
            mma_tf32(acc, ahi[cls][mt], bl[0], bl[1]);
          }
          if (cls == 0) {   // unpaired g = K2: slot 0 of an extra k-step, all other slots are zero
            uint32_t bh[2], bl[2];
            const float v = (t4 == 0) ? ab[pl * IC::ABP + K2 * IC::ABS + c] : 0.f;
            split_tf32(v, bh[0], bl[0]);
            bh[1] = 0u;
            bl[1] = 0u;
            mma_tf32(acc, ahi[4][mt], bh[0], bh[1]);
            mma_tf32(acc, alo[4][mt], bh[0], bh[1]);
            mma_tf32(acc, ahi[4][mt], bl[0], bl[1]);
          }
          // C fragment -> combos row (quadruple), 16-byte chunks swapped pairwise on odd groups of four rows
          const int colp = (8 * nt + 2 * t4) ^ (((g8 >> 2) & 1) << 2);
          float* d0 = combo + (size_t)(16 * mt + g8) * Cfg::NS + cls * NC + colp;
          *reinterpret_cast<float2*>(d0) = make_float2(acc[0], acc[1]);
          *reinterpret_cast<float2*>(d0 + 8 * Cfg::NS) = make_float2(acc[2], acc[3]);
        }
    __syncwarp();

    // this lane's quadruple: Pe, Po, Qo, Qe
    float Pe[NC], Po[NC], Qo[NC], Qe[NC];
    {
      const float* src = combo + (size_t)lane * Cfg::NS;
      const int sw = (n1 >> 2) & 1;
#pragma unroll
      for (int c4 = 0; c4 < NC / 4; ++c4) {
        const int cc = 4 * (c4 ^ sw);
        const float4 v0 = *reinterpret_cast<const float4*>(src + 0 * NC + cc);
        const float4 v1 = *reinterpret_cast<const float4*>(src + 1 * NC + cc);
        const float4 v2 = *reinterpret_cast<const float4*>(src + 2 * NC + cc);
        const float4 v3 = *reinterpret_cast<const float4*>(src + 3 * NC + cc);
        Pe[4 * c4] = v0.x; Pe[4 * c4 + 1] = v0.y; Pe[4 * c4 + 2] = v0.z; Pe[4 * c4 + 3] = v0.w;
        Po[4 * c4] = v1.x; Po[4 * c4 + 1] = v1.y; Po[4 * c4 + 2] = v1.z; Po[4 * c4 + 3] = v1.w;
        Qo[4 * c4] = v2.x; Qo[4 * c4 + 1] = v2.y; Qo[4 * c4 + 2] = v2.z; Qo[4 * c4 + 3] = v2.w;
        Qe[4 * c4] = v3.x; Qe[4 * c4 + 1] = v3.y; Qe[4 * c4 + 2] = v3.z; Qe[4 * c4 + 3] = v3.w;
      }
    }
    // the previous task's TMA stores must have finished reading the staging rows before they are rewritten
    // (aliased layout: the first block is already free, and every lane has its combos in registers now)
    if constexpr (!IC::ALIAS) {
      if (lane == 0) tma_store_wait_read<0>();
    }
    __syncwarp();

    // ---- unfold to the four rows (a: n, b: N2/2-1-n, c: N2/2+n, d: N2-1-n) and expand each along the
    // contiguous dimension; one copy of the row code, signs select the row
    constexpr bool kSplit = (SPT == 2 && N2 == 128);   // rows a, b fill the first staging block: store it early
#pragma unroll 1
    for (int r4 = 0; r4 < 4; ++r4) {
      if constexpr (kSplit) {
        if (r4 == 2) {
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
#pragma unroll
            for (int h = 0; h < Cfg::BOXES; ++h)
              tma_store_2d(&out_map, h * 32, (int)(task * kTaskRows), staging + (size_t)h * RPS * 128);
            tma_store_commit();
            // rows c, d go to the second block: the previous task's store of it must be done reading
            if constexpr (IC::ALIAS) tma_store_wait_read<1>();
          }
          if constexpr (IC::ALIAS) __syncwarp();
        }
      }
      const int rowq = (r4 == 0) ? n1 : (r4 == 1) ? (N2 / 2 - 1 - n1) : (r4 == 2) ? (N2 / 2 + n1) : (N2 - 1 - n1);
      const float sPo = (r4 == 0 || r4 == 3) ? 1.f : -1.f;   // a, d: +Po;  b, c: -Po
      const float sQe = (r4 == 0 || r4 == 2) ? 1.f : -1.f;   // a, c: +Qe;  b, d: -Qe
      const float sQo = (r4 <= 1) ? 1.f : -1.f;              // a, b: +Qo;  c, d: -Qo
      float z[NC];
#pragma unroll
      for (int c = 0; c < NC; ++c) z[c] = fmaf(sQo, Qo[c], fmaf(sQe, Qe[c], fmaf(sPo, Po[c], Pe[c])));
      const int trow = pl1 * N2 + rowq;
      expand_row<N3, K3, RPS>(staging_s + (uint32_t)(trow / RPS) * kStageBytes, trow % RPS, z);
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
#pragma unroll
      for (int rb = kSplit ? 1 : 0; rb < SPT; ++rb)
#pragma unroll
        for (int h = 0; h < Cfg::BOXES; ++h)
          tma_store_2d(&out_map, h * 32, (int)(task * kTaskRows + (long long)rb * RPS),
                       staging + (size_t)rb * kStageBytes + (size_t)h * RPS * 128);
      tma_store_commit();
    }
  }
  pdl_trigger();   // late, as in the forward kernel
  if (lane == 0) tma_store_wait_all<0>();
}

// ---------------------------------------------------------------------------------------------
// Launchers, one pair per plane shape (N3, k3, N2, k2); explicitly instantiated in dtst_plane_inst_*.cu.
template <int N3, int K3, int N2, int K2>
cudaError_t plane_fwd(const float* x, float2* out, long long rows, float scale, int herm, int* status,
                               const RingDebug& dbg, cudaStream_t st) {
  // consumer warps (+ the producer warp = 2 warps per scheduler; 8 or 10 consumers measured slower on the HBM-bound
  // shapes).  With half of the contiguous extent retained (k3 = N3 / 2) the kernel is bound by its arithmetic and
  // 11 warps at 168 registers are 4 % faster than 7 at 232.
  constexpr int W = (N3 == 32 && K3 == 16) ? 11 : 7;
  using Cfg = PlaneCfg<N3, K3, N2, K2>;
  const SmemPlan sp = smem_plan<Cfg, K2, K3, W>();
  if (sp.stages < 2 * Cfg::SPT) return cudaErrorInvalidConfiguration;
  CUtensorMap map;
  if (!make_rows_map(&map, x, rows, N3, Cfg::ROWS_PER_STAGE)) return cudaErrorNotSupported;
  auto kern = fwd_plane_kernel<N3, K3, N2, K2, W, 0>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sp.total);
  if (e != cudaSuccess) return e;
  const long long tasks = rows / kTaskRows;
  const int grid = (int)(tasks < num_sms() ? tasks : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3((W + 1) * 32), sp.total, st, map, out, tasks, scale, herm, sp.stages, status,
                   dbg.poll_limit, dbg.withhold_after, 0);
  return cudaGetLastError();
}

// The forward kernel with the third dimension (extent N1, K1 modes per side) contracted on chip: x rows as above,
// out [columns][2 K1][2 k2][k3] complex, columns = rows / (N2 N1).
template <int N3, int K3, int N2, int K2, int K1>
cudaError_t plane_fwd_col(const float* x, float2* out, long long rows, int N1, float scale, int herm, int* status,
                          const RingDebug& dbg, cudaStream_t st) {
  constexpr int W = 7;
  using Cfg = PlaneCfg<N3, K3, N2, K2>;
  static_assert(Cfg::G == 1, "one plane per task");
  const size_t extra = (size_t)2 * 8 * (2 * 2 * K2 * K3) * 4 + 512;   // two batches of 8 planes, the cosine table
  const SmemPlan sp = smem_plan<Cfg, K2, K3, W>(extra);
  if (sp.stages < 2 * Cfg::SPT || N1 > 128) return cudaErrorInvalidConfiguration;
  CUtensorMap map;
  if (!make_rows_map(&map, x, rows, N3, Cfg::ROWS_PER_STAGE)) return cudaErrorNotSupported;
  auto kern = fwd_plane_kernel<N3, K3, N2, K2, W, K1>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sp.total);
  if (e != cudaSuccess) return e;
  const long long tasks = rows / kTaskRows;   // planes
  const long long cols = tasks / N1;
  const int grid = (int)(cols < num_sms() ? cols : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3((W + 1 + kColAccWarps) * 32), sp.total, st, map, out, tasks, scale, herm,
                   sp.stages, status, dbg.poll_limit, dbg.withhold_after, N1);
  return cudaGetLastError();
}

template <int N3, int K3, int N2, int K2, int K1, int NT1>
cudaError_t plane_inv(const float2* in, float* y, long long rows, float scale, int herm,
                               const ColExpandArgs& ce, cudaStream_t st) {
  using IC = InvCfg<N3, K3, N2, K2>;
  constexpr int W = (IC::WARP_BYTES * 7 + 2 * K2 * K3 * 8 + 1024 <= kSmemLimit) ? 7
                    : (IC::WARP_BYTES * 6 + 2 * K2 * K3 * 8 + 1024 <= kSmemLimit) ? 6 : 5;
  const size_t total = (size_t)W * IC::WARP_BYTES + (size_t)2 * K2 * K3 * 8 + 1024;
  static_assert((size_t)W * IC::WARP_BYTES + (size_t)2 * K2 * K3 * 8 + 1024 <= kSmemLimit, "shared memory");
  CUtensorMap map;
  if (!make_rows_map(&map, y, rows, N3, PlaneCfg<N3, K3, N2, K2>::ROWS_PER_STAGE)) return cudaErrorNotSupported;
  auto kern = inv_plane_kernel<N3, K3, N2, K2, W, K1, NT1>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)total);
  if (e != cudaSuccess) return e;
  const long long tasks = rows / kTaskRows;
  const long long want = (tasks + W - 1) / W;
  const int grid = (int)(want < num_sms() ? want : num_sms());
  if (K1 > 0) {
    // the column counters start every launch at zero
    e = cudaMemsetAsync(ce.ready, 0, (size_t)2 * ce.cols * sizeof(int), st);
    if (e != cudaSuccess) return e;
  }
  (void)launch_pdl(kern, dim3(grid), dim3((W + (K1 > 0 ? kColExpandHelpers : 0)) * 32), total, st, map, in, tasks, scale, herm, ce);
  return cudaGetLastError();
}


// The shapes the library is built for.  X(N3, k3, N2, k2): contiguous extent and its retained one-sided modes, the
// extent in front of it and its retained modes per side.  The in-kernel column expansion variant of the inverse
// kernel is built for a leading dimension of the same shape as the second one (K1 = k2, N1 = N2).
#define DTST_PLANE_SHAPES_A(X) X(64, 8, 128, 16) X(64, 8, 128, 8)
#define DTST_PLANE_SHAPES_B(X) X(32, 4, 64, 8) X(64, 8, 64, 8) X(32, 8, 64, 8) X(32, 16, 64, 8)
#define DTST_PLANE_SHAPES_C(X) X(32, 8, 128, 16) X(32, 8, 128, 8) X(64, 4, 64, 8)
#define DTST_PLANE_SHAPES(X) DTST_PLANE_SHAPES_A(X) DTST_PLANE_SHAPES_B(X) DTST_PLANE_SHAPES_C(X)

#define DTST_PLANE_INSTANTIATE(N3, K3, N2, K2)                                                                          \
  template cudaError_t plane_fwd<N3, K3, N2, K2>(const float*, float2*, long long, float, int, int*, const RingDebug&,   \
                                                  cudaStream_t);                                                        \
  template cudaError_t plane_inv<N3, K3, N2, K2, 0, 1>(const float2*, float*, long long, float, int,                    \
                                                        const ColExpandArgs&, cudaStream_t);                            \
  template cudaError_t plane_inv<N3, K3, N2, K2, K2, N2 / 32>(const float2*, float*, long long, float, int,             \
                                                               const ColExpandArgs&, cudaStream_t);
#define DTST_PLANE_EXTERN(N3, K3, N2, K2)                                                                                \
  extern template cudaError_t plane_fwd<N3, K3, N2, K2>(const float*, float2*, long long, float, int, int*,              \
                                                         const RingDebug&, cudaStream_t);                                \
  extern template cudaError_t plane_inv<N3, K3, N2, K2, 0, 1>(const float2*, float*, long long, float, int,              \
                                                               const ColExpandArgs&, cudaStream_t);                      \
  extern template cudaError_t plane_inv<N3, K3, N2, K2, K2, N2 / 32>(const float2*, float*, long long, float, int,       \
                                                                      const ColExpandArgs&, cudaStream_t);

// The forward kernel with the third dimension fused is built for the largest benchmark shape.
#define DTST_PLANE_COL_SHAPES(X) X(64, 8, 128, 16, 16)
#define DTST_PLANE_COL_INSTANTIATE(N3, K3, N2, K2, K1)                                                                  \
  template cudaError_t plane_fwd_col<N3, K3, N2, K2, K1>(const float*, float2*, long long, int, float, int, int*,       \
                                                          const RingDebug&, cudaStream_t);
#define DTST_PLANE_COL_EXTERN(N3, K3, N2, K2, K1)                                                                       \
  extern template cudaError_t plane_fwd_col<N3, K3, N2, K2, K1>(const float*, float2*, long long, int, float, int,      \
                                                                 int*, const RingDebug&, cudaStream_t);

}  // namespace plane
}  // namespace dtst
