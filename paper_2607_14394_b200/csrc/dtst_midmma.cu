// Two-sided middle dimension on the tensor cores: the folded contraction / expansion of dtst_mid.cu
// (Eq. 18 with zero offset, half-sample phase factored out),
//     A_g = sum_{q<N/2} (z_q + z_{N-1-q}) cos(psi_g (q + 1/2)),   B_g = sum_{q<N/2} (z_q - z_{N-1-q}) sin(psi_g (q + 1/2)),
//     Z_{+-g} = e^{+-i psi_g/2} (A_g -+ i B_g),
// folded a second time about the quarter points (even g: cosine even, sine odd; odd g the other way round), with the
// sums over the row quadruples as warp-level TF32 MMAs (hi/lo compensated, fp32 accumulate).  The folded DATA is
// the 16-row operand (8 complex positions: real parts in rows 0..7, imaginary parts in rows 8..15, so that a C
// fragment holds whole complex values); the BASIS of one parity class (even cos, odd cos, odd sin, even sin:
// K/2 <= 8 frequencies each) is the 8-column operand from a fragment-ordered shared table built once per persistent
// CTA; the one frequency left over, cos K, runs on FFMA.
//
// The FFMA version of this stage was issue-bound (half of all instructions were the multiply-adds, the other half
// their bookkeeping); a first MMA version with one fold and the frequencies as the 16-row operand needed twice the
// MMAs and was bound by the tensor pipe of the warp-level path.  Shapes: N % 32 == 0, K in {4, 8, 12, 16},
// inner % 4 == 0.
#include "dtst_common.cuh"
#include "dtst_mma.cuh"

namespace dtst {
namespace {


// ------------------------------------------------------------------------------------------
// contraction: in[outer][N][inner] -> out[outer][2K][inner]
//
// Second fold: psi_g (N/2-1-q + 1/2) = pi g - psi_g (q + 1/2), so the cosine is even (odd) and the sine odd (even)
// about the quarter points for even (odd) g.  The four rows a = z_q, b = z_{N/2-1-q}, c = z_{N/2+q}, d = z_{N-1-q}
// (q < N/4) fold into
//     uu = (a+d)+(b+c) -> A_g, g even      ud = (a+d)-(b+c) -> A_g, g odd
//     vs = (a-d)+(b-c) -> B_g, g odd       vd = (a-d)-(b-c) -> B_g, g even
// and each of the four parity classes has K/2 <= 8 frequencies: exactly one MMA n-tile.  MMA roles:
//   M = 16 real columns = 8 complex positions (rows 0..7 = real parts, 8..15 = imaginary parts: a C fragment
//       then holds whole complex values), the folded DATA as A operand;
//   K = 8 row quadruples per k-step;  N = the class's frequency slots, the BASIS as B operand (shared table).
// Half the MMAs of the single fold (which needs two 16-row frequency tiles per 8 columns), and half the row pairs.
// The left-over cos K (even class, ninth slot) runs on FFMA.
//
// The input streams through a per-warp ring of shared-memory stages filled with cp.async (16 bytes per lane and
// request): one stage = one k-step of one task = 4 x 8 rows of 128 bytes.  The ring runs ahead across task
// boundaries, so several kilobytes per warp are in flight at all times without holding them in registers (with
// register double-buffering this stage was bound by load latency).
// ------------------------------------------------------------------------------------------
constexpr int kCMT = 2;                       // MMA m-tiles per task: 16 complex positions = 128 bytes per row
constexpr int kCPos = 8 * kCMT;
constexpr int kCWarps = 12;
constexpr int kCThreads = kCWarps * 32;
constexpr int kCStages = 3;
constexpr int kCRow = 2 * kCPos + 8;          // floats per staged row: 40 = 8 mod 32, conflict-free 8-byte loads
constexpr int kCStageFloats = 32 * kCRow;     // [a | b | c | d][8 quadruples]

__device__ __forceinline__ void cp_async16(float* smem_dst, const float* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// One k-step (8 quadruples) of one m-tile (8 complex positions) from a filled stage.
__device__ __forceinline__ void contract_step(const float* S, const float4* bt, float ck0, float ck1,
                                              float (&acc)[4][4], float (&aK)[2]) {
  // S points at this lane's (quadruple t4, position g8): rows of group g sit 8 * kCRow floats apart
  float X[4][4];   // [class][A-fragment element: (re, t4) (im, t4) (re, t4+4) (im, t4+4)]
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const float2 a = *reinterpret_cast<const float2*>(S + (0 * 8 + 4 * h) * kCRow);
    const float2 b = *reinterpret_cast<const float2*>(S + (1 * 8 + 4 * h) * kCRow);
    const float2 c = *reinterpret_cast<const float2*>(S + (2 * 8 + 4 * h) * kCRow);
    const float2 d = *reinterpret_cast<const float2*>(S + (3 * 8 + 4 * h) * kCRow);
    {
      const float u = a.x + d.x, v = a.x - d.x, up = b.x + c.x, vp = b.x - c.x;
      X[0][2 * h] = u + up;
      X[1][2 * h] = u - up;
      X[2][2 * h] = v + vp;
      X[3][2 * h] = v - vp;
    }
    {
      const float u = a.y + d.y, v = a.y - d.y, up = b.y + c.y, vp = b.y - c.y;
      X[0][2 * h + 1] = u + up;
      X[1][2 * h + 1] = u - up;
      X[2][2 * h + 1] = v + vp;
      X[3][2 * h + 1] = v - vp;
    }
  }
  aK[0] = fmaf(X[0][0], ck0, fmaf(X[0][2], ck1, aK[0]));
  aK[1] = fmaf(X[0][1], ck0, fmaf(X[0][3], ck1, aK[1]));
#pragma unroll
  for (int cls = 0; cls < 4; ++cls) {
    uint32_t ah[4], al[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) split_tf32_round(X[cls][e], ah[e], al[e]);
    const float4 b = bt[cls * 32];   // (b0 hi, b1 hi, b0 lo, b1 lo)
    mma_m16n8k8_tf32(acc[cls], ah, __float_as_uint(b.x), __float_as_uint(b.y));
    mma_m16n8k8_tf32(acc[cls], al, __float_as_uint(b.x), __float_as_uint(b.y));
    mma_m16n8k8_tf32(acc[cls], ah, __float_as_uint(b.z), __float_as_uint(b.w));
  }
}

template <int K>
__global__ void __launch_bounds__(kCThreads, 1)
mid_contract_mma_kernel(const float* __restrict__ in, float2* __restrict__ out, long long outer, long long inner,
                        int N, float scale) {
  static_assert(K % 4 == 0 && K <= 16, "parity classes of K/2 <= 8 frequencies");
  pdl_trigger();
  extern __shared__ float4 mm_smem[];
  const int KS = N / 32;                                    // k-steps of 8 row quadruples
  float4* btab = mm_smem;                                   // [KS][class][lane]
  float* cK = reinterpret_cast<float*>(btab + (size_t)KS * 4 * 32);   // cos(psi_K (q + 1/2)), q < N/4

  for (int e = threadIdx.x; e < KS * 4 * 32; e += blockDim.x) {
    const int l = e & 31, cls = (e >> 5) & 3, ks = e >> 7;
    const int lg = l >> 2, lt = l & 3;                      // B fragment: k = lt (+4), n = lg
    const int g = class_freq(cls, lg);
    const bool valid = lg < K / 2;
    uint32_t hi[2], lo[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float cs, sn;
      basis_cs(g, 8 * ks + lt + 4 * h, N, cs, sn);
      const float v = valid ? ((cls == 0 || cls == 1) ? cs : sn) : 0.f;
      split_tf32_rna(v, hi[h], lo[h]);
    }
    btab[e] = make_float4(__uint_as_float(hi[0]), __uint_as_float(hi[1]), __uint_as_float(lo[0]), __uint_as_float(lo[1]));
  }
  for (int q = threadIdx.x; q < N / 4; q += blockDim.x) {
    float cs, sn;
    basis_cs(K, q, N, cs, sn);
    cK[q] = cs;
  }
  __syncthreads();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g8 = lane >> 2, t4 = lane & 3;
  // e^{i psi_g / 2} * scale for this lane's frequencies 4 t4 .. 4 t4 + 3 and for K
  float2 rho[5];
#pragma unroll
  for (int j = 0; j < 5; ++j) {
    double s, c;
    sincospi((double)(j < 4 ? 4 * t4 + j : K) / (double)N, &s, &c);
    rho[j] = make_float2((float)c * scale, (float)s * scale);
  }

  const long long cblocks = (inner + kCPos - 1) / kCPos;
  const long long tasks = outer * cblocks;
  const long long rs = 2 * inner;   // floats per row
  const long long tstride = (long long)gridDim.x * kCWarps;
  float* ring = cK + N / 4 + (size_t)warp * kCStages * kCStageFloats;   // this warp's stages (16-byte aligned)
  pdl_wait();   // everything above is independent of the preceding kernel

  // producer cursor: (task, k-step) of the next stage to request; lane = (row lane / 8, 16-byte chunk lane % 8)
  long long ptask = (long long)blockIdx.x * kCWarps + warp;
  int pks = 0, pstage = 0;
  const float* ptb = in;
  bool pchunk_ok = false;
  auto issue = [&]() {
    if (ptask < tasks) {
      if (pks == 0) {
        const long long o = ptask / cblocks, cb = ptask % cblocks;
        const long long left = inner - cb * kCPos;
        const int nch = left >= kCPos ? kCPos / 2 : (int)(left / 2);   // valid 16-byte chunks per row
        ptb = in + o * N * rs + cb * (2 * kCPos) + 4 * (lane & 7);
        pchunk_ok = (lane & 7) < nch;
      }
      if (pchunk_ok) {
        float* dst = ring + pstage * kCStageFloats + (lane >> 3) * kCRow + 4 * (lane & 7);
        const int q = 8 * pks + (lane >> 3);
        // staged rows: group a = rows q, b = N/2-1-q, c = N/2+q, d = N-1-q (8 quadruples each; this lane: q, q+4)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int qq = q + 4 * h;
          cp_async16(dst + (0 * 8 + 4 * h) * kCRow, ptb + (long long)qq * rs);
          cp_async16(dst + (1 * 8 + 4 * h) * kCRow, ptb + (long long)(N / 2 - 1 - qq) * rs);
          cp_async16(dst + (2 * 8 + 4 * h) * kCRow, ptb + (long long)(N / 2 + qq) * rs);
          cp_async16(dst + (3 * 8 + 4 * h) * kCRow, ptb + (long long)(N - 1 - qq) * rs);
        }
      }
      if (++pks == KS) {
        pks = 0;
        ptask += tstride;
      }
    }
    cp_async_commit();   // one group per call, also when nothing was requested: the wait below counts groups
    pstage = pstage + 1 == kCStages ? 0 : pstage + 1;
  };
#pragma unroll
  for (int i = 0; i < kCStages - 1; ++i) issue();

  int cstage = 0;
  for (long long task = (long long)blockIdx.x * kCWarps + warp; task < tasks; task += tstride) {
    const long long o = task / cblocks, cb = task % cblocks;
    const long long left = inner - cb * kCPos;
    const int mtv = left >= kCPos ? kCMT : (int)((left + 7) / 8);   // m-tiles with at least one valid position

    float acc[kCMT][4][4], aK[kCMT][2];
#pragma unroll
    for (int mt = 0; mt < kCMT; ++mt) {
      aK[mt][0] = aK[mt][1] = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[mt][c][e] = 0.f;
    }

#pragma unroll 1
    for (int ks = 0; ks < KS; ++ks) {
      cp_async_wait<kCStages - 2>();   // this k-step's stage has landed (for this lane's requests) ...
      __syncwarp();                    // ... and for everyone's; all lanes are done with the previous stage
      issue();                         // refill the stage read in the previous k-step
      const float* S = ring + cstage * kCStageFloats + t4 * kCRow + 2 * g8;
      const float4* bt = btab + (size_t)(ks * 4) * 32 + lane;
      const float ck0 = cK[8 * ks + t4], ck1 = cK[8 * ks + t4 + 4];
#pragma unroll
      for (int mt = 0; mt < kCMT; ++mt)
        if (mt < mtv) contract_step(S + 16 * mt, bt, ck0, ck1, acc[mt], aK[mt]);
      cstage = cstage + 1 == kCStages ? 0 : cstage + 1;
    }

    // ---- epilogue.  acc[mt][cls] = (re, slot 2 t4), (re, slot 2 t4 + 1), (im, 2 t4), (im, 2 t4 + 1) of position g8.
    // Z_{+g} = rho_g (A_g - i B_g) -> row g (g < K);  Z_{-g} = conj(rho_g) (A_g + i B_g) -> row 2K - g (g >= 1)
#pragma unroll
    for (int mt = 0; mt < kCMT; ++mt) {
      // A_K: sum the quad's partial sums (each lane covered the quadruples t4, t4 + 4 of every k-step)
      float aKr = aK[mt][0], aKi = aK[mt][1];
      aKr += __shfl_xor_sync(0xffffffffu, aKr, 1);
      aKr += __shfl_xor_sync(0xffffffffu, aKr, 2);
      aKi += __shfl_xor_sync(0xffffffffu, aKi, 1);
      aKi += __shfl_xor_sync(0xffffffffu, aKi, 2);
      // B of the even frequency 4 t4 is the even-sine slot 2 t4 - 1: the second slot of the lane below
      float bpr = __shfl_up_sync(0xffffffffu, acc[mt][3][1], 1);
      float bpi = __shfl_up_sync(0xffffffffu, acc[mt][3][3], 1);
      if (t4 == 0) bpr = bpi = 0.f;   // B_0 = 0
      const long long pos = cb * kCPos + 8 * mt + g8;
      if (mt < mtv && pos < inner) {
        float2* dst = out + o * (2 * K) * inner + pos;
        auto emit = [&](int g, float2 r, float ax, float ay, float bx, float by) {
          const float pr = ax + by, pi = ay - bx;   // A - iB
          const float mr = ax - by, mi = ay + bx;   // A + iB
          if (g < K) dst[(long long)g * inner] = make_float2(r.x * pr - r.y * pi, r.x * pi + r.y * pr);
          if (g > 0) dst[(long long)(2 * K - g) * inner] = make_float2(r.x * mr + r.y * mi, r.x * mi - r.y * mr);
        };
        const int g0 = 4 * t4;
        if (g0 < K) {
          emit(g0, rho[0], acc[mt][0][0], acc[mt][0][2], bpr, bpi);                                   // even, slot 2 t4
          emit(g0 + 1, rho[1], acc[mt][1][0], acc[mt][1][2], acc[mt][2][0], acc[mt][2][2]);           // odd
          emit(g0 + 2, rho[2], acc[mt][0][1], acc[mt][0][3], acc[mt][3][0], acc[mt][3][2]);           // even, slot 2 t4 + 1
          emit(g0 + 3, rho[3], acc[mt][1][1], acc[mt][1][3], acc[mt][2][1], acc[mt][2][3]);           // odd
        }
        if (t4 == K / 4 - 1) emit(K, rho[4], aKr, aKi, acc[mt][3][1], acc[mt][3][3]);                 // -K only
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// expansion: in[outer][2K][inner] -> out[outer][N][inner]   (B^H along this dimension), the transpose of the
// contraction above with the same two folds.  With
//   alpha_g = V'_{+g} + V'_{-g}, beta_g = i (V'_{+g} - V'_{-g}), V'_{+-g} = e^{-+i psi_g/2} V_{+-g}
// and, for a row quadruple n < N/4, the four class sums
//   Pe = sum_{g even} alpha_g cos(psi_g (n+1/2)),  Po = sum_{g odd} alpha_g cos,
//   Qo = sum_{g odd} beta_g sin(psi_g (n+1/2)),    Qe = sum_{g even} beta_g sin,
// the four output rows are
//   z_n = Pe+Po+Qo+Qe,  z_{N/2-1-n} = Pe-Po+Qo-Qe,  z_{N/2+n} = Pe-Po-Qo+Qe,  z_{N-1-n} = Pe+Po-Qo-Qe.
// MMA roles: M = 16 real columns = 8 complex positions (real parts | imaginary parts), alpha / beta of a class as
// the A operand, built once per task straight from global memory into registers; K = the class's 8 frequency
// slots; N = 8 row quadruples, the basis as B operand from a fragment-ordered shared table.  The left-over
// alpha_K cos(psi_K (n+1/2)) is added on FFMA.  Rows are written from the C fragments, 64 contiguous bytes per row
// and store instruction.
// ------------------------------------------------------------------------------------------
constexpr int kEMT = 2;                       // m-tiles per task: 16 complex positions
constexpr int kEPos = 8 * kEMT;
constexpr int kEWarps = 12;
constexpr int kEThreads = kEWarps * 32;

template <int K>
__global__ void __launch_bounds__(kEThreads, 1)
mid_expand_mma_kernel(const float2* __restrict__ in, float2* __restrict__ out, long long outer, long long inner,
                      int N, float scale, int streaming) {
  static_assert(K % 4 == 0 && K <= 16, "parity classes of K/2 <= 8 frequencies");
  pdl_trigger();
  extern __shared__ float4 mm_smem[];
  const int NT = N / 32;                                   // n-tiles of 8 row quadruples
  float4* btab = mm_smem;                                  // [NT][class][lane]
  float* cK = reinterpret_cast<float*>(btab + (size_t)NT * 4 * 32);   // cos(psi_K (n + 1/2)), n < N/4

  for (int e = threadIdx.x; e < NT * 4 * 32; e += blockDim.x) {
    const int l = e & 31, cls = (e >> 5) & 3, nt = e >> 7;
    const int lg = l >> 2, lt = l & 3;                      // B fragment: k = slot lt (+4), n = quadruple lg
    uint32_t hi[2], lo[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int slot = lt + 4 * h;
      float cs, sn;
      basis_cs(class_freq(cls, slot), 8 * nt + lg, N, cs, sn);
      const float v = slot < K / 2 ? ((cls == 0 || cls == 1) ? cs : sn) : 0.f;
      split_tf32_rna(v, hi[h], lo[h]);
    }
    btab[e] = make_float4(__uint_as_float(hi[0]), __uint_as_float(hi[1]), __uint_as_float(lo[0]), __uint_as_float(lo[1]));
  }
  for (int n = threadIdx.x; n < N / 4; n += blockDim.x) {
    float cs, sn;
    basis_cs(K, n, N, cs, sn);
    cK[n] = cs;
  }
  __syncthreads();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g8 = lane >> 2, t4 = lane & 3;
  // the six frequencies whose alpha / beta this lane turns into A fragments: 2 t4 + {0, 1, 2} and the same + 8
  float2 rho[7];   // e^{i psi_g / 2} * scale; [6] = frequency K
#pragma unroll
  for (int j = 0; j < 7; ++j) {
    const int g = j < 6 ? 2 * t4 + (j % 3) + 8 * (j / 3) : K;
    double s, c;
    sincospi((double)g / (double)N, &s, &c);
    rho[j] = make_float2((float)c * scale, (float)s * scale);
  }

  const long long cblocks = (inner + kEPos - 1) / kEPos;
  const long long tasks = outer * cblocks;
  const long long tstride = (long long)gridDim.x * kEWarps;
  pdl_wait();   // everything above is independent of the preceding kernel
  for (long long task = (long long)blockIdx.x * kEWarps + warp; task < tasks; task += tstride) {
    const long long o = task / cblocks, cb = task % cblocks;
    const long long left = inner - cb * kEPos;
    const int mtv = left >= kEPos ? kEMT : (int)((left + 7) / 8);

    // pull the next task's 2K input rows (128 bytes each) into L2 while this one runs on the tensor cores
    {
      const long long nx = task + tstride;
      if (nx < tasks) {
        const float2* nsrc = in + (nx / cblocks) * (2 * K) * inner + (nx % cblocks) * kEPos;
        for (int r = lane; r < 2 * K; r += 32) asm volatile("prefetch.global.L2 [%0];" ::"l"(nsrc + (long long)r * inner));
      }
    }

    // ---- A fragments: alpha (classes 0, 1) and beta (classes 2, 3) of this lane's position, hi / lo
    uint32_t ah[kEMT][4][4], al[kEMT][4][4];
    float2 aKv[kEMT];
#pragma unroll
    for (int mt = 0; mt < kEMT; ++mt) {
      const long long pos = cb * kEPos + 8 * mt + g8;
      const bool ok = mt < mtv && pos < inner;
      const float2* src = in + o * (2 * K) * inner + (ok ? pos : 0);
      float2 alpha[6], beta[6];
#pragma unroll
      for (int j = 0; j < 6; ++j) {
        const int g = 2 * t4 + (j % 3) + 8 * (j / 3);
        float2 v = make_float2(0.f, 0.f), u = make_float2(0.f, 0.f);
        if (ok && g < K) v = __ldcs(src + (long long)g * inner);
        if (ok && g > 0 && g <= K) u = __ldcs(src + (long long)(2 * K - g) * inner);
        const float2 r = rho[j];
        const float2 vp = make_float2(v.x * r.x + v.y * r.y, v.y * r.x - v.x * r.y);   // v * conj(rho)
        const float2 vm = make_float2(u.x * r.x - u.y * r.y, u.y * r.x + u.x * r.y);   // u * rho
        alpha[j] = make_float2(vp.x + vm.x, vp.y + vm.y);
        beta[j] = make_float2(-(vp.y - vm.y), vp.x - vm.x);                            // i (vp - vm)
      }
      {
        float2 u = make_float2(0.f, 0.f);
        if (ok) u = __ldcs(src + (long long)K * inner);                                // V_{-K}
        const float2 r = rho[6];
        aKv[mt] = make_float2(u.x * r.x - u.y * r.y, u.y * r.x + u.x * r.y);           // alpha_K = rho_K V_{-K}
      }
      // class slots t4 (h = 0) and t4 + 4 (h = 1): even cos g = 2 slot, odd g = 2 slot + 1, even sin g = 2 slot + 2
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

    float2* ob = out + o * N * inner + cb * kEPos + g8;
#pragma unroll 1
    for (int nt = 0; nt < NT; ++nt) {
      float4 bf[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) bf[c] = btab[(size_t)(nt * 4 + c) * 32 + lane];
      const int n0 = 8 * nt + 2 * t4;                      // this lane's two quadruples: n0, n0 + 1
      const float c0 = cK[n0], c1 = cK[n0 + 1];
#pragma unroll
      for (int mt = 0; mt < kEMT; ++mt) {
        if (mt < mtv) {
          float acc[4][4];
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[c][e] = 0.f;
#pragma unroll
          for (int c = 0; c < 4; ++c) mma_m16n8k8_tf32(acc[c], ah[mt][c], __float_as_uint(bf[c].x), __float_as_uint(bf[c].y));
#pragma unroll
          for (int c = 0; c < 4; ++c) mma_m16n8k8_tf32(acc[c], al[mt][c], __float_as_uint(bf[c].x), __float_as_uint(bf[c].y));
#pragma unroll
          for (int c = 0; c < 4; ++c) mma_m16n8k8_tf32(acc[c], ah[mt][c], __float_as_uint(bf[c].z), __float_as_uint(bf[c].w));
          // acc[cls] = (re, n0) (re, n0 + 1) (im, n0) (im, n0 + 1); the left-over alpha_K term joins Pe
          acc[0][0] = fmaf(aKv[mt].x, c0, acc[0][0]);
          acc[0][1] = fmaf(aKv[mt].x, c1, acc[0][1]);
          acc[0][2] = fmaf(aKv[mt].y, c0, acc[0][2]);
          acc[0][3] = fmaf(aKv[mt].y, c1, acc[0][3]);
          if (cb * kEPos + 8 * mt + g8 < inner) {
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const int n = n0 + q;
              const float per = acc[0][q], pei = acc[0][2 + q], por = acc[1][q], poi = acc[1][2 + q];
              const float qor = acc[2][q], qoi = acc[2][2 + q], qer = acc[3][q], qei = acc[3][2 + q];
              const float spr = per + por, dpr = per - por, sqr = qor + qer, dqr = qor - qer;
              const float spi = pei + poi, dpi = pei - poi, sqi = qoi + qei, dqi = qoi - qei;
              const float2 za = make_float2(spr + sqr, spi + sqi);     // z_n          = Pe+Po+Qo+Qe
              const float2 zd = make_float2(spr - sqr, spi - sqi);     // z_{N-1-n}    = Pe+Po-Qo-Qe
              const float2 zb = make_float2(dpr + dqr, dpi + dqi);     // z_{N/2-1-n}  = Pe-Po+Qo-Qe
              const float2 zc = make_float2(dpr - dqr, dpi - dqi);     // z_{N/2+n}    = Pe-Po-Qo+Qe
              float2* d = ob + 8 * mt;
              if (streaming) {   // an output far larger than L2 is not worth keeping there for the next kernel
                __stcs(d + (long long)n * inner, za);
                __stcs(d + (long long)(N / 2 - 1 - n) * inner, zb);
                __stcs(d + (long long)(N / 2 + n) * inner, zc);
                __stcs(d + (long long)(N - 1 - n) * inner, zd);
              } else {
                d[(long long)n * inner] = za;
                d[(long long)(N / 2 - 1 - n) * inner] = zb;
                d[(long long)(N / 2 + n) * inner] = zc;
                d[(long long)(N - 1 - n) * inner] = zd;
              }
            }
          }
        }
      }
    }
  }
}

template <int K>
size_t contract_smem(int N) {
  return (size_t)(N / 32) * 4 * 32 * 16 + (size_t)(N / 4) * 4 + (size_t)kCWarps * kCStages * kCStageFloats * 4;
}

template <int K>
size_t expand_smem(int N) { return (size_t)(N / 32) * 4 * 32 * 16 + (size_t)(N / 4) * 4; }

template <int K>
cudaError_t launch_mid_mma_t(bool forward, const float2* in, float2* out, long long outer, long long inner, int N,
                             float scale, cudaStream_t st) {
  const size_t smem = forward ? contract_smem<K>(N) : expand_smem<K>(N);
  const int pos = forward ? kCPos : kEPos, warps = forward ? kCWarps : kEWarps, threads = warps * 32;
  const long long tasks = outer * ((inner + pos - 1) / pos);
  const long long want = (tasks + warps - 1) / warps;
  // persistent CTAs: exactly as many as are resident at once
  auto grid_for = [&](auto kern, int* grid) -> cudaError_t {
    cudaError_t e = cudaSuccess;
    if (smem > 48 * 1024) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    const long long cap = (long long)num_sms() * per_sm;
    *grid = (int)(want < cap ? want : cap);
    return cudaSuccess;
  };
  int grid = 1;
  if (forward) {
    auto kern = mid_contract_mma_kernel<K>;
    cudaError_t e = grid_for(kern, &grid);
    if (e != cudaSuccess) return e;
    (void)launch_pdl(kern, dim3(grid), dim3(threads), smem, st, reinterpret_cast<const float*>(in), out, outer, inner, N, scale);
  } else {
    auto kern = mid_expand_mma_kernel<K>;
    cudaError_t e = grid_for(kern, &grid);
    if (e != cudaSuccess) return e;
    const int streaming = (double)outer * N * inner * 8.0 > 2.0 * 126e6 ? 1 : 0;
    (void)launch_pdl(kern, dim3(grid), dim3(threads), smem, st, in, out, outer, inner, N, scale, streaming);
  }
  return cudaGetLastError();
}

}  // namespace

bool mid_mma_supported(int N, int K, long long inner) {
  if (N % 32 != 0 || N < 32 || N > 512 || 2 * K > N) return false;
  if (!(K == 4 || K == 8 || K == 12 || K == 16)) return false;
  if (inner <= 0 || inner % 4 != 0) return false;
  // both kernels must fit the 227 KB of shared memory a CTA can opt into
  const size_t lim = 227 * 1024;
  const size_t c = contract_smem<16>(N);
  const size_t e = K == 4 ? expand_smem<4>(N) : K == 8 ? expand_smem<8>(N) : K == 12 ? expand_smem<12>(N) : expand_smem<16>(N);
  return c <= lim && e <= lim;
}

cudaError_t launch_mid_mma(bool forward, int K, const float2* in, float2* out, long long outer, long long inner,
                           int N, float scale, cudaStream_t st) {
  if (outer * inner <= 0) return cudaSuccess;
  switch (K) {
    case 4: return launch_mid_mma_t<4>(forward, in, out, outer, inner, N, scale, st);
    case 8: return launch_mid_mma_t<8>(forward, in, out, outer, inner, N, scale, st);
    case 12: return launch_mid_mma_t<12>(forward, in, out, outer, inner, N, scale, st);
    case 16: return launch_mid_mma_t<16>(forward, in, out, outer, inner, N, scale, st);
    default: return cudaErrorNotSupported;
  }
}

}  // namespace dtst
