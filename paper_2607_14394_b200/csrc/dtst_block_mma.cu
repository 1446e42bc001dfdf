// Backward pass of a point-wise linear operator on the tensor cores (the block's bypass, Section "Block Structure";
// its adjoints, Section "Backward Pass"):
//   grad_W[o][i] = sum_{b,p} g[b,o,p] x[b,i,p]          (a [C_out x points] x [points x C_in] product)
//   grad_x[b,i,p] (+)= sum_o W[o][i] g[b,o,p]           (a [C_in x C_out] x [C_out x points] product)
// in ONE pass over g and x: every grid tensor is read once, grad_x is read (when accumulated into) and written once.
// Both products run as warp-level m16n8k8 TF32 MMAs with hi/lo compensation (three MMAs per product, fp32
// accumulate): at 16 channels they are 32 multiply-adds per loaded float, which the FFMA version of this pass could
// not hide under its memory time (it ran at a third of the copy bandwidth).
//
// A CTA of four warps walks tiles of 128 points x all channels of one batch entry, staged with cp.async into
// shared memory (two buffers: the next tile is in flight while the current one is worked on); a warp owns 32 of
// the tile's points.  Rows are 132 floats apart, which makes every fragment load below conflict free:
//   weight gradient   A = g  (rows o, k = points):  g_s[o = g8 (+8)][p = t4 (+4)]      -> bank 4 g8 + t4
//                     B = x^T (k = points, n = i):  x_s[i = g8][p = t4 (+4)]            -> bank 4 g8 + t4
//   input gradient    A = W^T (rows i, k = o): constant, kept in registers as hi/lo fragments
//                     B = g  (k = o, n = points):   g_s[o = 2 t4 (+1)][p = g8]          -> bank 8 t4 + g8
//     (the MMA's k index is mapped to the channel o = 2 k for k < 4 and 2 (k - 4) + 1 otherwise; a sum does not
//      care in which order its terms are named, and with this naming the four k rows of a request are 8 banks apart)
// The weight-gradient sums live in C fragments across all tiles of the CTA; at the end the four warps' sums are
// added in warp order and the CTA's row goes to `partial`, which reduce_wb_kernel adds in ascending CTA order: the
// summation order is fixed, repeated runs give the same bits.
#include "dtst_common.cuh"
#include "dtst_mma.cuh"

namespace dtst {

namespace {

constexpr int kMTP = 128;        // points per tile
constexpr int kMSP = kMTP + 4;   // row stride in floats

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <int CI, int CO, int CIN, int CON>
// (four CTAs per SM up to 16 + 16 channels, where the fragments leave room for it: 4 % faster than three)
__global__ void __launch_bounds__(128, (CI <= 16 && CO <= 16) ? 4 : 3)
linear_backward_mma_kernel(const float* __restrict__ gz, const float* __restrict__ x, float* __restrict__ gx,
                           const float* __restrict__ Wb, float* __restrict__ partial, int B, long long P, int mode_gx,
                           int want_gw, int want_gb, int ci, int co) {
  // CI, CO: the channel counts rounded up to 16 or 32 (the 16-row MMA operand), CIN, CON rounded up to 8, 16, 24
  // or 32 (the 8-wide operands); ci, co the real ones.  The rows of the staged tiles that belong to no channel are
  // zero, as are the weights in front of them.
  static_assert(CI % 16 == 0 && CO % 16 == 0 && CI <= 32 && CO <= 32 && CIN % 8 == 0 && CON % 8 == 0 && CIN <= CI &&
                    CON <= CO, "channel counts");
  constexpr int ROWS = CO + CI;
  constexpr int MTO = CO / 16, NTI = CIN / 8;   // weight gradient: m-tiles over o, n-tiles over i
  constexpr int MTI = CI / 16, KSO = CON / 8;   // input gradient: m-tiles over i, k-steps over o
  pdl_trigger();
  extern __shared__ __align__(16) float lb_s[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;

  // W^T as A fragments (row i, column k <-> channel o = 8 ks + 2 (k % 4) + k / 4), hi/lo, for the whole kernel
  uint32_t whi[MTI][KSO][4], wlo[MTI][KSO][4];
#pragma unroll
  for (int mt = 0; mt < MTI; ++mt)
#pragma unroll
    for (int ks = 0; ks < KSO; ++ks)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int i = 16 * mt + g8 + 8 * (e & 1);
        const int o = 8 * ks + 2 * t4 + (e >> 1);
        split_tf32_rna((mode_gx && o < co && i < ci) ? Wb[o * ci + i] : 0.f, whi[mt][ks][e], wlo[mt][ks][e]);
      }
  float accW[MTO][NTI][4];
  float bs[MTO][2];
#pragma unroll
  for (int mt = 0; mt < MTO; ++mt) {
    bs[mt][0] = bs[mt][1] = 0.f;
#pragma unroll
    for (int nt = 0; nt < NTI; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) accW[mt][nt][e] = 0.f;
  }
  // rows without a channel: zero, in both buffers, once
  for (int bufz = 0; bufz < 2; ++bufz)
    for (int r = warp; r < ROWS; r += 4)
      if ((r < CO && r >= co) || (r >= CO && r - CO >= ci))
        *reinterpret_cast<float4*>(lb_s + (size_t)bufz * ROWS * kMSP + (size_t)r * kMSP + 4 * lane) =
            make_float4(0.f, 0.f, 0.f, 0.f);
  pdl_wait();

  const long long tiles_per_b = P / kMTP;
  const long long tiles = (long long)B * tiles_per_b;
  auto stage = [&](long long tile, int buf) {
    const long long b = tile / tiles_per_b, p0 = (tile % tiles_per_b) * kMTP;
    float* dstb = lb_s + (size_t)buf * ROWS * kMSP;
    for (int r = warp; r < ROWS; r += 4) {
      if (r < CO ? r >= co : r - CO >= ci) continue;
      const float* src = (r < CO ? gz + ((b * co + r) * P) : x + ((b * ci + (r - CO)) * P)) + p0 + 4 * lane;
      cp_async16(dstb + (size_t)r * kMSP + 4 * lane, src);
    }
    cp_async_commit();
  };

  long long tile = blockIdx.x;
  if (tile < tiles) stage(tile, 0);
  int buf = 0;
  for (; tile < tiles; tile += gridDim.x, buf ^= 1) {
    const long long next = tile + gridDim.x;
    if (next < tiles) {
      stage(next, buf ^ 1);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const float* g_s = lb_s + (size_t)buf * ROWS * kMSP;
    const float* x_s = g_s + (size_t)CO * kMSP;
    const long long b = tile / tiles_per_b, p0 = (tile % tiles_per_b) * kMTP;
    const int pw = 32 * warp;

    // old grad_x values of this warp's points (requested now, used after the products)
    float2 old[4][MTI][2];
    if (mode_gx == 1) {
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int mt = 0; mt < MTI; ++mt)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int i = 16 * mt + g8 + 8 * h;
            old[nt][mt][h] = i < ci ? *reinterpret_cast<const float2*>(gx + ((b * ci + i) * P) + p0 + pw + 8 * nt + 2 * t4)
                                    : make_float2(0.f, 0.f);
          }
    }

    if (want_gw) {
      // this tile's products are summed in fresh fragments and then added to the running sums with ordinary
      // fp32 additions: the tensor core's accumulate step truncates, which a chain over all tiles would show
      float tw[MTO][NTI][4];
#pragma unroll
      for (int mt = 0; mt < MTO; ++mt)
#pragma unroll
        for (int nt = 0; nt < NTI; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) tw[mt][nt][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        const int k0 = pw + 8 * ks;
        uint32_t bh[NTI][2], bl[NTI][2];
#pragma unroll
        for (int nt = 0; nt < NTI; ++nt) {
          const float* xr = x_s + (size_t)(8 * nt + g8) * kMSP + k0 + t4;
          split_tf32_round(xr[0], bh[nt][0], bl[nt][0]);
          split_tf32_round(xr[4], bh[nt][1], bl[nt][1]);
        }
#pragma unroll
        for (int mt = 0; mt < MTO; ++mt) {
          uint32_t ah[4], al[4];
          float av[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            av[e] = g_s[(size_t)(16 * mt + g8 + 8 * (e & 1)) * kMSP + k0 + t4 + 4 * (e >> 1)];
            split_tf32_round(av[e], ah[e], al[e]);
          }
          bs[mt][0] += av[0] + av[2];
          bs[mt][1] += av[1] + av[3];
#pragma unroll
          for (int nt = 0; nt < NTI; ++nt) mma3_tf32(tw[mt][nt], ah, al, bh[nt][0], bh[nt][1], bl[nt][0], bl[nt][1]);
        }
      }
#pragma unroll
      for (int mt = 0; mt < MTO; ++mt)
#pragma unroll
        for (int nt = 0; nt < NTI; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) accW[mt][nt][e] += tw[mt][nt][e];
    }

    if (mode_gx) {
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const int pc = pw + 8 * nt + g8;
        float d[MTI][4];
#pragma unroll
        for (int mt = 0; mt < MTI; ++mt) d[mt][0] = d[mt][1] = d[mt][2] = d[mt][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KSO; ++ks) {
          uint32_t bh0, bl0, bh1, bl1;
          split_tf32_round(g_s[(size_t)(8 * ks + 2 * t4) * kMSP + pc], bh0, bl0);
          split_tf32_round(g_s[(size_t)(8 * ks + 2 * t4 + 1) * kMSP + pc], bh1, bl1);
#pragma unroll
          for (int mt = 0; mt < MTI; ++mt) mma3_tf32(d[mt], whi[mt][ks], wlo[mt][ks], bh0, bh1, bl0, bl1);
        }
#pragma unroll
        for (int mt = 0; mt < MTI; ++mt)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float2 v = make_float2(d[mt][2 * h], d[mt][2 * h + 1]);
            if (mode_gx == 1) {
              v.x += old[nt][mt][h].x;
              v.y += old[nt][mt][h].y;
            }
            const int i = 16 * mt + g8 + 8 * h;
            if (i < ci) *reinterpret_cast<float2*>(gx + ((b * ci + i) * P) + p0 + pw + 8 * nt + 2 * t4) = v;
          }
      }
    }
    __syncthreads();   // every warp is done with this buffer before the tile after next is staged into it
  }

  if (want_gw) {
    // the four warps' sums, added in warp order; row layout of `partial`: [o][i] pairs, then the bias sums
    constexpr int PAIRS = CO * CI;
    float* red = lb_s;   // [4][PAIRS + CO]
    __syncthreads();
    float* mine = red + (size_t)warp * (PAIRS + CO);
#pragma unroll
    for (int mt = 0; mt < MTO; ++mt) {
#pragma unroll
      for (int nt = 0; nt < NTI; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e)
          mine[(16 * mt + g8 + 8 * (e >> 1)) * CI + 8 * nt + 2 * t4 + (e & 1)] = accW[mt][nt][e];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float s = bs[mt][h];   // this lane saw the points t4, t4 + 4 (mod 8): add the four lanes of a row group
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        if (t4 == 0) mine[PAIRS + 16 * mt + g8 + 8 * h] = s;
      }
    }
    __syncthreads();
    // the row of `partial` has the real counts: co * ci pairs [o][i], then co bias sums
    const int pairs = co * ci;
    for (int e = threadIdx.x; e < pairs + (want_gb ? co : 0); e += blockDim.x) {
      const int src = e < pairs ? (e / ci) * CI + e % ci : PAIRS + (e - pairs);
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < 4; ++w) s += red[(size_t)w * (PAIRS + CO) + src];
      partial[(long long)blockIdx.x * (pairs + co) + e] = s;
    }
  }
}

template <int CI, int CO, int CIN, int CON>
cudaError_t launch_t(const float* gz, const float* x, float* gx, int mode_gx, const float* Wb, float* partial, int B,
                     long long P, int want_gw, int want_gb, int max_ctas, int* ctas_out, int ci, int co,
                     cudaStream_t st) {
  auto kern = linear_backward_mma_kernel<CI, CO, CIN, CON>;
  size_t smem = (size_t)2 * (CO + CI) * kMSP * 4;
  const size_t red = (size_t)4 * (CO * CI + CO) * 4;
  if (smem < red) smem = red;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int per_sm = 1;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, 128, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) per_sm = 1;
  const long long tiles = (long long)B * (P / kMTP);
  long long ctas = (long long)num_sms() * per_sm;
  if (ctas > max_ctas) ctas = max_ctas;
  if (ctas > tiles) ctas = tiles;
  *ctas_out = (int)ctas;
  (void)launch_pdl(kern, dim3((unsigned)ctas), dim3(128), smem, st, gz, x, gx, Wb, partial, B, P, mode_gx, want_gw, want_gb,
                   ci, co);
  return cudaGetLastError();
}

}  // namespace

// up to 32 channels on both sides (rounded up to the MMA tiles inside), at least 20 together (below that the products
// are a few multiply-adds per value and the FFMA kernel serves), whole tiles of points
bool linear_backward_mma_supported(int Ci, int Co, long long P) {
  return Ci >= 1 && Ci <= 32 && Co >= 1 && Co <= 32 && Ci + Co >= 20 && P % kMTP == 0 && P > 0;
}

// Launches the kernel above; *ctas_out = rows of `partial` that were written (the caller reduces them).
cudaError_t launch_linear_backward_mma(const float* gz, const float* x, float* gx, int mode_gx, const float* Wb,
                                       float* partial, int B, int Ci, int Co, long long P, int want_gw, int want_gb,
                                       int max_ctas, int* ctas_out, cudaStream_t st) {
  // classes of a channel count: up to 8 -> tiles (16 | 8), up to 16 -> (16 | 16), up to 24 -> (32 | 24), up to 32 -> (32 | 32)
  auto cls = [](int c) { return c <= 8 ? 0 : (c <= 16 ? 1 : (c <= 24 ? 2 : 3)); };
  const int ki = cls(Ci), ko = cls(Co);
#define DTST_CALL(a, b, c16, d16, c8, d8) \
  if (ki == a && ko == b) \
    return launch_t<c16, d16, c8, d8>(gz, x, gx, mode_gx, Wb, partial, B, P, want_gw, want_gb, max_ctas, ctas_out, Ci, Co, st);
#define DTST_ROW(a, c16, c8)            \
  DTST_CALL(a, 0, c16, 16, c8, 8)       \
  DTST_CALL(a, 1, c16, 16, c8, 16)      \
  DTST_CALL(a, 2, c16, 32, c8, 24)      \
  DTST_CALL(a, 3, c16, 32, c8, 32)
  DTST_ROW(0, 16, 8)
  DTST_ROW(1, 16, 16)
  DTST_ROW(2, 32, 24)
  DTST_ROW(3, 32, 32)
#undef DTST_ROW
#undef DTST_CALL
  return cudaErrorNotSupported;
}

}  // namespace dtst
