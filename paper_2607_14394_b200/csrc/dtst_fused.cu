// Fused streaming kernels for the grid-side stages of the truncated spectral layer.
//
// Forward ("plane") kernel: contracts the last two grid dimensions in one pass.  The real
// grid is read from HBM exactly once through a TMA-fed shared-memory ring; each consumer
// warp owns a task of 128 consecutive rows (one or two [N2 x N3] planes), contracts the
// contiguous dimension with one thread per row, then the next dimension with one thread
// per retained frequency, and writes only the [2*k2 x k3] complex result of each plane.
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
#include <cuda.h>

#include "dtst_fused.cuh"
#include "dtst_sm100.cuh"

namespace dtst {

using namespace sm100;

namespace {

constexpr int kTaskRows = 128;       // rows of the contiguous dimension per warp task
constexpr int kStageBytes = 16384;   // one ring slot
constexpr int kSmemLimit = 232448;   // 227 KB opt-in limit per CTA

// Stage-1 coefficients cos/sin(2 pi f (j + 1/2) / N3), j < N3/4, delivered in the kernel
// parameter constant bank so that every FMA takes its coefficient as a constant operand
// (a shared-memory operand would cost LDS bandwidth this kernel does not have).
template <int N3, int K3>
struct Stage1Table {
  float cs[N3 / 4][K3];
  float sn[N3 / 4][K3];
};

template <int N3, int K3, int N2, int K2>
struct PlaneCfg {
  static constexpr int ROWS_PER_STAGE = kStageBytes / (N3 * 4);
  static constexpr int SPT = kTaskRows / ROWS_PER_STAGE;      // ring slots per task
  static constexpr int BOXES = N3 / 32;                       // 128-byte column panels per row
  static constexpr int G = kTaskRows / N2;                    // planes per task
  static constexpr int QUADS = N2 / 4;                        // row quadruples per plane
  static constexpr int NC = 2 * K3;                           // real columns after stage 1 (C | S)
  static constexpr int LPP = 2 * K2;                          // stage-2 lanes per plane
  static constexpr int CSTRIDE = NC + 4;                      // floats between parity classes
  static constexpr int NSTRIDE = 4 * CSTRIDE + 4;             // floats between quadruples
  static constexpr int PSTRIDE = QUADS * NSTRIDE + 16;        // floats between planes
  static constexpr int ABS = NC + 4;                          // floats between A/B entries
  static constexpr int ABP = (2 * K2 + 1) * ABS;
  static constexpr int COMBO_FLOATS = (G * PSTRIDE > G * ABP ? G * PSTRIDE : G * ABP);
  static_assert(N3 % 32 == 0 && (N3 == 32 || N3 == 64), "N3");
  static_assert(kTaskRows % N2 == 0 && G * QUADS == 32, "one lane per row quadruple");
  static_assert(G * LPP <= 32 && G * NC <= 32, "stage-2 lane mapping");
  static_assert(K3 % 2 == 0 && NC % 4 == 0, "K3");
  static_assert(SPT == 1 || SPT == 2, "SPT");
};

struct SmemPlan {
  int stages;
  size_t ring, combos, rot, bars, total;
};

template <typename Cfg, int K2, int K3, int W>
SmemPlan smem_plan() {
  SmemPlan s;
  const size_t combos = (size_t)W * Cfg::COMBO_FLOATS * 4;
  const size_t rot = (size_t)2 * K2 * K3 * 8;
  const size_t fixed = 1024 /*alignment slack*/ + combos + rot + 512 /*barriers*/;
  s.stages = (int)((kSmemLimit - fixed) / kStageBytes);
  if (s.stages > 12) s.stages = 12;
  s.ring = 0;
  s.combos = (size_t)s.stages * kStageBytes;
  s.rot = s.combos + combos;
  s.bars = s.rot + rot;
  s.total = s.bars + 512 + 1024;
  return s;
}

__device__ __forceinline__ float4 lds128(const char* p) { return *reinterpret_cast<const float4*>(p); }

// One row of N3 reals -> C_f = sum u cos, S_f = sum v sin for f < K3 (half-sample phase deferred).
template <int N3, int K3>
__device__ __forceinline__ void stage1_row(const char* stage, int box_rows, int row,
                                           const Stage1Table<N3, K3>& tab, float (&o)[2 * K3]) {
  constexpr int CH = N3 / 4;
#pragma unroll
  for (int i = 0; i < 2 * K3; ++i) o[i] = 0.f;
  const uint32_t sw = (uint32_t)(row & 7);
  const char* rbase = stage + (size_t)row * 128;
#pragma unroll
  for (int c = 0; c < CH / 4; ++c) {
    const int c0 = c, c1 = CH / 2 - 1 - c, c2 = CH / 2 + c, c3 = CH - 1 - c;
    const float4 A = lds128(rbase + (size_t)(c0 / 8) * box_rows * 128 + (((uint32_t)(c0 % 8) ^ sw) << 4));
    const float4 Bq = lds128(rbase + (size_t)(c1 / 8) * box_rows * 128 + (((uint32_t)(c1 % 8) ^ sw) << 4));
    const float4 Cq = lds128(rbase + (size_t)(c2 / 8) * box_rows * 128 + (((uint32_t)(c2 % 8) ^ sw) << 4));
    const float4 D = lds128(rbase + (size_t)(c3 / 8) * box_rows * 128 + (((uint32_t)(c3 % 8) ^ sw) << 4));
    const float a[4] = {A.x, A.y, A.z, A.w};
    const float b[4] = {Bq.w, Bq.z, Bq.y, Bq.x};
    const float cc[4] = {Cq.x, Cq.y, Cq.z, Cq.w};
    const float d[4] = {D.w, D.z, D.y, D.x};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int j = 4 * c + e;
      const float u = a[e] + d[e], v = a[e] - d[e];
      const float up = b[e] + cc[e], vp = b[e] - cc[e];
      const float uu = u + up, ud = u - up, vs = v + vp, vd = v - vp;
#pragma unroll
      for (int f = 0; f < K3; ++f) {
        if ((f & 1) == 0) {
          o[f] = fmaf(uu, tab.cs[j][f], o[f]);
          if (f > 0) o[K3 + f] = fmaf(vd, tab.sn[j][f], o[K3 + f]);
        } else {
          o[f] = fmaf(ud, tab.cs[j][f], o[f]);
          o[K3 + f] = fmaf(vs, tab.sn[j][f], o[K3 + f]);
        }
      }
    }
  }
}

// Consumer side of the ring: wait until fill number q (0-based) of `slot` has landed.
__device__ __forceinline__ bool wait_fill(volatile uint32_t* fill_seq, uint64_t* full, int slot, uint32_t q,
                                          volatile int* abort_flag) {
  for (uint32_t it = 0; fill_seq[slot] < q + 1u; ++it) {
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      __nanosleep(64);
    }
    if (it > (1u << 24)) {
      *abort_flag = 1;
      return false;
    }
  }
  return mbar_wait_bounded(&full[slot], q & 1u, abort_flag);
}

template <int N3, int K3, int N2, int K2, int W>
__global__ void __launch_bounds__((W + 1) * 32, 1)
fwd_plane_kernel(const __grid_constant__ CUtensorMap in_map, const __grid_constant__ Stage1Table<N3, K3> tab,
                 float2* __restrict__ out, long long num_tasks, float scale, int herm, int stages,
                 int* __restrict__ status) {
  using Cfg = PlaneCfg<N3, K3, N2, K2>;
  constexpr int NC = Cfg::NC, QUADS = Cfg::QUADS, G = Cfg::G, LPP = Cfg::LPP;
  constexpr int SPT = Cfg::SPT, RPS = Cfg::ROWS_PER_STAGE;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* ring = smem;
  float* combos_all = reinterpret_cast<float*>(smem + (size_t)stages * kStageBytes);
  float2* rot = reinterpret_cast<float2*>(combos_all + (size_t)W * Cfg::COMBO_FLOATS);
  uint64_t* full = reinterpret_cast<uint64_t*>(rot + 2 * K2 * K3);
  uint64_t* empty = full + 16;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(empty + 16);
  // fill_seq[slot] = number of fills the producer has armed for that slot.  A parity wait can only
  // tell "this phase" from "the previous one", so a consumer that is a whole lap of the ring ahead
  // must first see its fill armed (which implies every earlier fill of the slot has landed).
  volatile uint32_t* fill_seq = reinterpret_cast<volatile uint32_t*>(empty + 16) + 4;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
      fill_seq[s] = 0;
    }
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tensormap(&in_map);
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
    rot[e] = make_float2((float)cs * w, (float)sn * w);
  }
  __syncthreads();

  const long long first = blockIdx.x;
  const long long n_local = first < num_tasks ? (num_tasks - first + gridDim.x - 1) / gridDim.x : 0;

  if (warp == 0) {
    // ---------------- producer: one thread feeds the ring in task order ----------------
    if (lane == 0) {
      long long k = 0;
      for (long long tl = 0; tl < n_local; ++tl) {
        const long long task = first + tl * gridDim.x;
        for (int s = 0; s < SPT; ++s, ++k) {
          const int slot = (int)(k % stages);
          const uint32_t ph = (uint32_t)((k / stages) & 1);
          if (!mbar_wait_bounded(&empty[slot], ph ^ 1u, abort_flag)) goto producer_done;
          fill_seq[slot] = (uint32_t)(k / stages) + 1u;
          mbar_arrive_expect_tx(&full[slot], (uint32_t)kStageBytes);
#pragma unroll
          for (int h = 0; h < Cfg::BOXES; ++h)
            tma_load_2d(ring + (size_t)slot * kStageBytes + (size_t)h * RPS * 128, &in_map, h * 32,
                        (int)(task * kTaskRows + (long long)s * RPS), &full[slot]);
        }
      }
    }
  producer_done:
    __syncwarp();
  } else {
    // ---------------- consumers: one warp per task ----------------
    const int w = warp - 1;
    float* combo = combos_all + (size_t)w * Cfg::COMBO_FLOATS;

    // stage-1 role: lane = (plane in task, row quadruple)
    const int pl1 = lane / QUADS, n1 = lane % QUADS;
    // stage-2 role: lane = (plane, A_g or B_g)
    const bool act2 = lane < G * LPP;
    const int pl2 = act2 ? lane / LPP : 0;
    const int l2 = lane % LPP;
    const bool isB = l2 >= K2;
    const int g2 = isB ? l2 - K2 + 1 : l2;
    const int cls2 = isB ? ((g2 & 1) ? 2 : 3) : ((g2 & 1) ? 1 : 0);
    // the unpaired cosine sum A_{K2} (needed by mode -K2 only) is spread over lanes by column
    const bool actx = lane < G * NC;
    const int plx = actx ? lane / NC : 0, cx = lane % NC;
    constexpr int clsx = (K2 & 1) ? 1 : 0;

    float coef[QUADS], coefx[QUADS];
#pragma unroll
    for (int n = 0; n < QUADS; ++n) {
      double sn, cs;
      sincospi((double)(((long long)g2 * (2 * n + 1)) % (2 * N2)) / (double)N2, &sn, &cs);
      coef[n] = isB ? (float)sn : (float)cs;
      sincospi((double)(((long long)K2 * (2 * n + 1)) % (2 * N2)) / (double)N2, &sn, &cs);
      coefx[n] = (float)cs;
    }

    for (long long tl = w; tl < n_local; tl += W) {
      const long long task = first + tl * gridDim.x;
      const long long k0 = tl * SPT;
      float ra[NC], rb[NC], rc[NC], rd[NC];

      if constexpr (SPT == 1) {
        const int slot = (int)(k0 % stages);
        if (!wait_fill(fill_seq, full, slot, (uint32_t)(k0 / stages), abort_flag)) break;
        const char* st = reinterpret_cast<const char*>(ring) + (size_t)slot * kStageBytes;
        const int base = pl1 * N2;
        stage1_row<N3, K3>(st, RPS, base + n1, tab, ra);
        stage1_row<N3, K3>(st, RPS, base + N2 - 1 - n1, tab, rd);
        stage1_row<N3, K3>(st, RPS, base + N2 / 2 - 1 - n1, tab, rb);
        stage1_row<N3, K3>(st, RPS, base + N2 / 2 + n1, tab, rc);
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[slot]);
      } else if constexpr (N2 == 128) {
        // rows n, 63-n live in the first slot; 64+n, 127-n in the second: release each early
        {
          const int slot = (int)(k0 % stages);
          if (!wait_fill(fill_seq, full, slot, (uint32_t)(k0 / stages), abort_flag)) break;
          const char* st = reinterpret_cast<const char*>(ring) + (size_t)slot * kStageBytes;
          stage1_row<N3, K3>(st, RPS, n1, tab, ra);
          stage1_row<N3, K3>(st, RPS, 63 - n1, tab, rb);
          __syncwarp();
          if (lane == 0) mbar_arrive(&empty[slot]);
        }
        {
          const long long k1 = k0 + 1;
          const int slot = (int)(k1 % stages);
          if (!wait_fill(fill_seq, full, slot, (uint32_t)(k1 / stages), abort_flag)) break;
          const char* st = reinterpret_cast<const char*>(ring) + (size_t)slot * kStageBytes;
          stage1_row<N3, K3>(st, RPS, n1, tab, rc);
          stage1_row<N3, K3>(st, RPS, 63 - n1, tab, rd);
          __syncwarp();
          if (lane == 0) mbar_arrive(&empty[slot]);
        }
      } else {
        // two planes of 64 rows, one per slot: a lane's four rows all sit in its plane's slot
        const int slot0 = (int)(k0 % stages), slot1 = (int)((k0 + 1) % stages);
        if (!wait_fill(fill_seq, full, slot0, (uint32_t)(k0 / stages), abort_flag)) break;
        if (!wait_fill(fill_seq, full, slot1, (uint32_t)((k0 + 1) / stages), abort_flag)) break;
        const char* st = reinterpret_cast<const char*>(ring) + (size_t)(pl1 ? slot1 : slot0) * kStageBytes;
        stage1_row<N3, K3>(st, RPS, n1, tab, ra);
        stage1_row<N3, K3>(st, RPS, N2 - 1 - n1, tab, rd);
        stage1_row<N3, K3>(st, RPS, N2 / 2 - 1 - n1, tab, rb);
        stage1_row<N3, K3>(st, RPS, N2 / 2 + n1, tab, rc);
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&empty[slot0]);
          mbar_arrive(&empty[slot1]);
        }
      }

      // fold the four rows of the quadruple (second dimension) and publish the four combos
      {
        float* dst = combo + pl1 * Cfg::PSTRIDE + n1 * Cfg::NSTRIDE;
#pragma unroll
        for (int c4 = 0; c4 < NC / 4; ++c4) {
          float pp[4], pd[4], ms[4], md[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int c = 4 * c4 + e;
            const float p = ra[c] + rd[c], m = ra[c] - rd[c];
            const float pq = rb[c] + rc[c], mq = rb[c] - rc[c];
            pp[e] = p + pq;
            pd[e] = p - pq;
            ms[e] = m + mq;
            md[e] = m - mq;
          }
          *reinterpret_cast<float4*>(dst + 0 * Cfg::CSTRIDE + 4 * c4) = make_float4(pp[0], pp[1], pp[2], pp[3]);
          *reinterpret_cast<float4*>(dst + 1 * Cfg::CSTRIDE + 4 * c4) = make_float4(pd[0], pd[1], pd[2], pd[3]);
          *reinterpret_cast<float4*>(dst + 2 * Cfg::CSTRIDE + 4 * c4) = make_float4(ms[0], ms[1], ms[2], ms[3]);
          *reinterpret_cast<float4*>(dst + 3 * Cfg::CSTRIDE + 4 * c4) = make_float4(md[0], md[1], md[2], md[3]);
        }
      }
      __syncwarp();

      // stage 2: A_g = sum_n (pp|pd)[n] cos, B_g = sum_n (md|ms)[n] sin, one lane per (g, A/B)
      float acc[NC];
      float accx = 0.f;
#pragma unroll
      for (int c = 0; c < NC; ++c) acc[c] = 0.f;
      {
        const float* cb = combo + pl2 * Cfg::PSTRIDE + cls2 * Cfg::CSTRIDE;
        const float* cbx = combo + plx * Cfg::PSTRIDE + clsx * Cfg::CSTRIDE + cx;
#pragma unroll
        for (int n = 0; n < QUADS; ++n) {
#pragma unroll
          for (int c4 = 0; c4 < NC / 4; ++c4) {
            const float4 v = *reinterpret_cast<const float4*>(cb + n * Cfg::NSTRIDE + 4 * c4);
            acc[4 * c4 + 0] = fmaf(coef[n], v.x, acc[4 * c4 + 0]);
            acc[4 * c4 + 1] = fmaf(coef[n], v.y, acc[4 * c4 + 1]);
            acc[4 * c4 + 2] = fmaf(coef[n], v.z, acc[4 * c4 + 2]);
            acc[4 * c4 + 3] = fmaf(coef[n], v.w, acc[4 * c4 + 3]);
          }
          accx = fmaf(coefx[n], cbx[n * Cfg::NSTRIDE], accx);
        }
      }
      __syncwarp();

      // A/B sums -> shared, entry g for A_g (g <= K2), entry K2+g for B_g (g >= 1)
      if (act2) {
        float* ab = combo + pl2 * Cfg::ABP + (isB ? K2 + g2 : g2) * Cfg::ABS;
#pragma unroll
        for (int c4 = 0; c4 < NC / 4; ++c4)
          *reinterpret_cast<float4*>(ab + 4 * c4) =
              make_float4(acc[4 * c4], acc[4 * c4 + 1], acc[4 * c4 + 2], acc[4 * c4 + 3]);
      }
      if (actx) combo[plx * Cfg::ABP + K2 * Cfg::ABS + cx] = accx;
      __syncwarp();

      // epilogue: Z_{+g} = rho (A - iB), Z_{-g} = rho (A + iB) with A = AC - i AS, B = BC - i BS
      if (act2) {
        const int r = l2;
        const bool pos = r < K2;
        const int g = pos ? r : 2 * K2 - r;
        const float* A = combo + pl2 * Cfg::ABP + g * Cfg::ABS;
        const float* Bp = combo + pl2 * Cfg::ABP + (K2 + g) * Cfg::ABS;
        float2* dst = out + ((task * G + pl2) * (2 * K2) + r) * K3;
        const float2* rr = rot + r * K3;
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
            const float2 ro = rr[f];
            res[2 * e] = ro.x * wr - ro.y * wi;
            res[2 * e + 1] = ro.x * wi + ro.y * wr;
          }
          *reinterpret_cast<float4*>(dst + 2 * f2) = make_float4(res[0], res[1], res[2], res[3]);
        }
      }
      __syncwarp();   // the next task's combos overwrite the A/B entries read above
    }
  }

  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, 1);
}

// ---------------------------------------------------------------------------------------------
// Inverse plane kernel: the transpose of the forward one.  in[planes][2*K2][K3] complex ->
// real rows [planes*N2][N3].  Each warp owns a task of 128 output rows: it pre-rotates the plane's
// modes, forms alpha_g = V'_{+g} + V'_{-g}, beta_g = i (V'_{+g} - V'_{-g}), expands them to the
// four rows of each row quadruple (one lane per quadruple), expands every row to N3 reals with
// the same folded basis, stages the rows in shared memory (TMA swizzle) and stores them with TMA.
template <int N3, int K3>
__device__ __forceinline__ void expand_row(char* stage, int box_rows, int row, const Stage1Table<N3, K3>& tab,
                                           const float (&z)[2 * K3]) {
  constexpr int CH = N3 / 4;
  const uint32_t sw = (uint32_t)(row & 7);
  char* rbase = stage + (size_t)row * 128;
#pragma unroll
  for (int c = 0; c < CH / 4; ++c) {
    float a[4], b[4], cc[4], d[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int j = 4 * c + e;
      float Ea = 0.f, Oa = 0.f, Eb = 0.f, Ob = 0.f;
#pragma unroll
      for (int f = 0; f < K3; ++f) {
        if ((f & 1) == 0) {
          Ea = fmaf(z[f], tab.cs[j][f], Ea);
          if (f > 0) Eb = fmaf(z[K3 + f], tab.sn[j][f], Eb);
        } else {
          Oa = fmaf(z[f], tab.cs[j][f], Oa);
          Ob = fmaf(z[K3 + f], tab.sn[j][f], Ob);
        }
      }
      const float sa = Ea + Oa, da = Ea - Oa, sb = Eb + Ob, db = Eb - Ob;
      a[e] = sa - sb;    // y[j]
      d[e] = sa + sb;    // y[N3-1-j]
      b[e] = da + db;    // y[N3/2-1-j]
      cc[e] = da - db;   // y[N3/2+j]
    }
    const int c0 = c, c1 = CH / 2 - 1 - c, c2 = CH / 2 + c, c3 = CH - 1 - c;
    *reinterpret_cast<float4*>(rbase + (size_t)(c0 / 8) * box_rows * 128 + (((uint32_t)(c0 % 8) ^ sw) << 4)) =
        make_float4(a[0], a[1], a[2], a[3]);
    *reinterpret_cast<float4*>(rbase + (size_t)(c1 / 8) * box_rows * 128 + (((uint32_t)(c1 % 8) ^ sw) << 4)) =
        make_float4(b[3], b[2], b[1], b[0]);
    *reinterpret_cast<float4*>(rbase + (size_t)(c2 / 8) * box_rows * 128 + (((uint32_t)(c2 % 8) ^ sw) << 4)) =
        make_float4(cc[0], cc[1], cc[2], cc[3]);
    *reinterpret_cast<float4*>(rbase + (size_t)(c3 / 8) * box_rows * 128 + (((uint32_t)(c3 % 8) ^ sw) << 4)) =
        make_float4(d[3], d[2], d[1], d[0]);
  }
}

template <int N3, int K3, int N2, int K2>
struct InvCfg {
  using P = PlaneCfg<N3, K3, N2, K2>;
  static constexpr int ABS = P::NC + 4;                     // floats between entries
  static constexpr int ENTRIES = 2 * K2 + 2;                // alpha_0..alpha_K2, beta_0..beta_K2 (beta_0 unused)
  static constexpr int ABP = ENTRIES * ABS + 4;             // floats between planes (offset banks)
  static constexpr int AB_FLOATS = ((P::G * ABP + 3) / 4) * 4;
  static constexpr int STAGING_BYTES = kTaskRows * N3 * 4;  // 128 output rows
  static constexpr int WARP_BYTES = STAGING_BYTES + ((AB_FLOATS * 4 + 1023) / 1024) * 1024;
};

template <int N3, int K3, int N2, int K2, int W>
__global__ void __launch_bounds__(W * 32, 1)
inv_plane_kernel(const __grid_constant__ CUtensorMap out_map, const __grid_constant__ Stage1Table<N3, K3> tab,
                 const float2* __restrict__ in, long long num_tasks, float scale, int herm) {
  using Cfg = PlaneCfg<N3, K3, N2, K2>;
  using IC = InvCfg<N3, K3, N2, K2>;
  constexpr int NC = Cfg::NC, QUADS = Cfg::QUADS, G = Cfg::G, LPP = Cfg::LPP;
  constexpr int SPT = Cfg::SPT, RPS = Cfg::ROWS_PER_STAGE;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  char* staging = reinterpret_cast<char*>(smem) + (size_t)warp * IC::WARP_BYTES;
  float* ab = reinterpret_cast<float*>(staging + IC::STAGING_BYTES);
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
    rot[e] = make_float2((float)cs * w, -(float)sn * w);
  }
  __syncthreads();

  // stage-2 role (one lane per row quadruple) and its basis values, kept in registers
  const int pl1 = lane / QUADS, n1 = lane % QUADS;
  float cosc[K2 + 1], sinc[K2 + 1];
#pragma unroll
  for (int g = 0; g <= K2; ++g) {
    double sn, cs;
    sincospi((double)(((long long)g * (2 * n1 + 1)) % (2 * N2)) / (double)N2, &sn, &cs);
    cosc[g] = (float)cs;
    sinc[g] = (float)sn;
  }
  // loader role: lane = (plane, mode position r)
  const bool actl = lane < G * LPP;
  const int pll = actl ? lane / LPP : 0, rl = lane % LPP;

  const long long tstride = (long long)gridDim.x * W;
  long long task = (long long)blockIdx.x + (long long)warp * gridDim.x;
  float4 vin[K3 / 2];
  if (task < num_tasks && actl) {
    const float4* src = reinterpret_cast<const float4*>(in + ((task * G + pll) * (2 * K2) + rl) * K3);
#pragma unroll
    for (int i = 0; i < K3 / 2; ++i) vin[i] = __ldg(src + i);
  }

  for (; task < num_tasks; task += tstride) {
    // ---- A. rotate this task's modes, publish V'
    if (actl) {
      float* dst = ab + pll * IC::ABP + rl * IC::ABS;
      const float2* rr = rot + rl * K3;
      float re[K3], im[K3];
#pragma unroll
      for (int i = 0; i < K3 / 2; ++i) {
        const float2 r0 = rr[2 * i], r1 = rr[2 * i + 1];
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
    // prefetch the next task's modes while this one is expanded
    {
      const long long nt = task + tstride;
      if (nt < num_tasks && actl) {
        const float4* src = reinterpret_cast<const float4*>(in + ((nt * G + pll) * (2 * K2) + rl) * K3);
#pragma unroll
        for (int i = 0; i < K3 / 2; ++i) vin[i] = __ldg(src + i);
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

    // ---- B. expand the second dimension for this lane's row quadruple
    float Pe[NC], Po[NC], Qe[NC], Qo[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) Pe[c] = Po[c] = Qe[c] = Qo[c] = 0.f;
    {
      const float* al = ab + pl1 * IC::ABP;
      const float* be = ab + pl1 * IC::ABP + (K2 + 1) * IC::ABS;
#pragma unroll
      for (int g = 0; g <= K2; ++g) {
#pragma unroll
        for (int c4 = 0; c4 < NC / 4; ++c4) {
          const float4 av = *reinterpret_cast<const float4*>(al + g * IC::ABS + 4 * c4);
          if ((g & 1) == 0) {
            Pe[4 * c4] = fmaf(cosc[g], av.x, Pe[4 * c4]);
            Pe[4 * c4 + 1] = fmaf(cosc[g], av.y, Pe[4 * c4 + 1]);
            Pe[4 * c4 + 2] = fmaf(cosc[g], av.z, Pe[4 * c4 + 2]);
            Pe[4 * c4 + 3] = fmaf(cosc[g], av.w, Pe[4 * c4 + 3]);
          } else {
            Po[4 * c4] = fmaf(cosc[g], av.x, Po[4 * c4]);
            Po[4 * c4 + 1] = fmaf(cosc[g], av.y, Po[4 * c4 + 1]);
            Po[4 * c4 + 2] = fmaf(cosc[g], av.z, Po[4 * c4 + 2]);
            Po[4 * c4 + 3] = fmaf(cosc[g], av.w, Po[4 * c4 + 3]);
          }
          if (g > 0) {
            const float4 bv = *reinterpret_cast<const float4*>(be + g * IC::ABS + 4 * c4);
            if ((g & 1) == 0) {
              Qe[4 * c4] = fmaf(sinc[g], bv.x, Qe[4 * c4]);
              Qe[4 * c4 + 1] = fmaf(sinc[g], bv.y, Qe[4 * c4 + 1]);
              Qe[4 * c4 + 2] = fmaf(sinc[g], bv.z, Qe[4 * c4 + 2]);
              Qe[4 * c4 + 3] = fmaf(sinc[g], bv.w, Qe[4 * c4 + 3]);
            } else {
              Qo[4 * c4] = fmaf(sinc[g], bv.x, Qo[4 * c4]);
              Qo[4 * c4 + 1] = fmaf(sinc[g], bv.y, Qo[4 * c4 + 1]);
              Qo[4 * c4 + 2] = fmaf(sinc[g], bv.z, Qo[4 * c4 + 2]);
              Qo[4 * c4 + 3] = fmaf(sinc[g], bv.w, Qo[4 * c4 + 3]);
            }
          }
        }
      }
    }
    // the previous task's TMA stores must have finished reading the staging rows before they are rewritten
    if (lane == 0) tma_store_wait_read<0>();
    __syncwarp();

    // ---- C/D. unfold to the four rows and expand each along the contiguous dimension
    {
      float z[NC];
      const int base = pl1 * N2;
      auto row_ptr = [&](int r) -> char* { return staging + (size_t)(r / RPS) * kStageBytes; };
#pragma unroll
      for (int c = 0; c < NC; ++c) z[c] = (Pe[c] + Po[c]) + (Qe[c] + Qo[c]);
      expand_row<N3, K3>(row_ptr(base + n1), RPS, (base + n1) % RPS, tab, z);
#pragma unroll
      for (int c = 0; c < NC; ++c) z[c] = (Pe[c] + Po[c]) - (Qe[c] + Qo[c]);
      expand_row<N3, K3>(row_ptr(base + N2 - 1 - n1), RPS, (base + N2 - 1 - n1) % RPS, tab, z);
#pragma unroll
      for (int c = 0; c < NC; ++c) z[c] = (Pe[c] - Po[c]) - (Qe[c] - Qo[c]);
      expand_row<N3, K3>(row_ptr(base + N2 / 2 - 1 - n1), RPS, (base + N2 / 2 - 1 - n1) % RPS, tab, z);
#pragma unroll
      for (int c = 0; c < NC; ++c) z[c] = (Pe[c] - Po[c]) + (Qe[c] - Qo[c]);
      expand_row<N3, K3>(row_ptr(base + N2 / 2 + n1), RPS, (base + N2 / 2 + n1) % RPS, tab, z);
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
#pragma unroll
      for (int rb = 0; rb < SPT; ++rb)
#pragma unroll
        for (int h = 0; h < Cfg::BOXES; ++h)
          tma_store_2d(&out_map, h * 32, (int)(task * kTaskRows + (long long)rb * RPS),
                       staging + (size_t)rb * kStageBytes + (size_t)h * RPS * 128);
      tma_store_commit();
    }
  }
  if (lane == 0) tma_store_wait_all<0>();
}

// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
    (void)cudaGetLastError();
  }
  return fn;
}

// 2-D fp32 tensor [rows][n3] viewed through [box_rows x 32] boxes with the 128-byte swizzle.
bool make_rows_map(CUtensorMap* map, const void* base, long long rows, int n3, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)n3, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)n3 * 4};
  cuuint32_t box[2] = {32, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int N3, int K3>
void fill_stage1_table(Stage1Table<N3, K3>* t) {
  for (int j = 0; j < N3 / 4; ++j)
    for (int f = 0; f < K3; ++f) {
      // phase (2j+1) f / (2 N3) turns, reduced exactly before the double-precision evaluation
      const long long num = ((long long)(2 * j + 1) * f) % (2ll * N3);
      const double ang = 3.14159265358979323846 * (double)num / (double)N3;
      t->cs[j][f] = (float)cos(ang);
      t->sn[j][f] = (float)sin(ang);
    }
}

template <int N3, int K3, int N2, int K2>
cudaError_t launch_fwd_plane_t(const float* x, float2* out, long long rows, float scale, int herm, int* status,
                               cudaStream_t st) {
  constexpr int W = 6;
  using Cfg = PlaneCfg<N3, K3, N2, K2>;
  const SmemPlan sp = smem_plan<Cfg, K2, K3, W>();
  if (sp.stages < 2 * Cfg::SPT) return cudaErrorInvalidConfiguration;
  CUtensorMap map;
  if (!make_rows_map(&map, x, rows, N3, Cfg::ROWS_PER_STAGE)) return cudaErrorNotSupported;
  Stage1Table<N3, K3> tab;
  fill_stage1_table(&tab);
  auto kern = fwd_plane_kernel<N3, K3, N2, K2, W>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sp.total);
  if (e != cudaSuccess) return e;
  const long long tasks = rows / kTaskRows;
  const int grid = (int)(tasks < kNumSMs ? tasks : kNumSMs);
  kern<<<grid, (W + 1) * 32, sp.total, st>>>(map, tab, out, tasks, scale, herm, sp.stages, status);
  return cudaGetLastError();
}

template <int N3, int K3, int N2, int K2>
cudaError_t launch_inv_plane_t(const float2* in, float* y, long long rows, float scale, int herm, cudaStream_t st) {
  using IC = InvCfg<N3, K3, N2, K2>;
  constexpr int W = (IC::WARP_BYTES * 6 + 2 * K2 * K3 * 8 + 2048 <= kSmemLimit) ? 6 : 5;
  const size_t total = (size_t)W * IC::WARP_BYTES + (size_t)2 * K2 * K3 * 8 + 1024;
  static_assert((size_t)W * IC::WARP_BYTES + (size_t)2 * K2 * K3 * 8 + 1024 <= kSmemLimit, "shared memory");
  CUtensorMap map;
  if (!make_rows_map(&map, y, rows, N3, PlaneCfg<N3, K3, N2, K2>::ROWS_PER_STAGE)) return cudaErrorNotSupported;
  Stage1Table<N3, K3> tab;
  fill_stage1_table(&tab);
  auto kern = inv_plane_kernel<N3, K3, N2, K2, W>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)total);
  if (e != cudaSuccess) return e;
  const long long tasks = rows / kTaskRows;
  const long long want = (tasks + W - 1) / W;
  const int grid = (int)(want < kNumSMs ? want : kNumSMs);
  kern<<<grid, W * 32, total, st>>>(map, tab, in, tasks, scale, herm);
  return cudaGetLastError();
}

}  // namespace

// Shapes the plane kernels are instantiated for: (N3, k3, N2, k2).
static bool plane_supported(int N3, int K3, int N2, int K2) {
  return (N3 == 64 && K3 == 8 && N2 == 128 && K2 == 16) || (N3 == 32 && K3 == 4 && N2 == 64 && K2 == 8) ||
         (N3 == 64 && K3 == 8 && N2 == 64 && K2 == 8);
}

bool fused_eligible(const dtst_plan* p) {
  if (p->d < 2) return false;
  const int a = p->d - 1, b = p->d - 2;
  // the symmetry folding needs the whole extent of both dimensions with zero phase offset
  if (p->Nl[a] != p->Ng[a] || p->Nl[b] != p->Ng[b] || p->off[a] != 0 || p->off[b] != 0) return false;
  if (p->d == 2 && p->P > 1) return false;   // slabs would cut the second-last dimension
  if (!plane_supported((int)p->Ng[a], p->kmax[a], (int)p->Ng[b], p->kmax[b])) return false;
  const int Cmin = 1;
  long long planes = (long long)p->B * Cmin;
  for (int i = 0; i < b; ++i) planes *= p->Nl[i];
  // tasks are 128 rows: with 64-row planes every tensor must hold an even number of planes
  long long pin = planes * p->C_in, pout = planes * p->C_out;
  if ((pin * p->Ng[b]) % kTaskRows != 0 || (pout * p->Ng[b]) % kTaskRows != 0) return false;
  if (pin * p->Ng[b] >= (1ll << 31) || pout * p->Ng[b] >= (1ll << 31)) return false;   // 32-bit TMA coordinates
  return encode_tiled_fn() != nullptr;
}

cudaError_t launch_fwd_plane(int N3, int K3, int N2, int K2, const float* x, float2* out, long long rows,
                             float scale, int herm, int* status, cudaStream_t st) {
  if (N3 == 64 && K3 == 8 && N2 == 128 && K2 == 16)
    return launch_fwd_plane_t<64, 8, 128, 16>(x, out, rows, scale, herm, status, st);
  if (N3 == 32 && K3 == 4 && N2 == 64 && K2 == 8)
    return launch_fwd_plane_t<32, 4, 64, 8>(x, out, rows, scale, herm, status, st);
  if (N3 == 64 && K3 == 8 && N2 == 64 && K2 == 8)
    return launch_fwd_plane_t<64, 8, 64, 8>(x, out, rows, scale, herm, status, st);
  return cudaErrorNotSupported;
}

}  // namespace dtst

namespace dtst {
cudaError_t launch_inv_plane(int N3, int K3, int N2, int K2, const float2* in, float* y, long long rows, float scale,
                             int herm, int* /*status*/, cudaStream_t st) {
  if (N3 == 64 && K3 == 8 && N2 == 128 && K2 == 16) return launch_inv_plane_t<64, 8, 128, 16>(in, y, rows, scale, herm, st);
  if (N3 == 32 && K3 == 4 && N2 == 64 && K2 == 8) return launch_inv_plane_t<32, 4, 64, 8>(in, y, rows, scale, herm, st);
  if (N3 == 64 && K3 == 8 && N2 == 64 && K2 == 8) return launch_inv_plane_t<64, 8, 64, 8>(in, y, rows, scale, herm, st);
  return cudaErrorNotSupported;
}
}  // namespace dtst
