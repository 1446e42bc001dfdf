// Forward pass of the block around the layer (Section "Block Structure", Algorithm 1 lines 1 and 8) with the
// bypass product on the fifth-generation tensor cores:
//     out[b, :, p] = GELU(W_bypass x[b, :, p] + y[b, :, p])        per grid point p,
// i.e. per tile of 128 points one [128 points x C_in] x [C_in x C_out] product - the one GEMM-shaped step of the
// block.  It runs as tcgen05.mma kind::tf32 with M = 128 (the points), N = C_out, K = 8 channels per instruction:
//   * x tiles arrive by TMA ([C_in channels x 32 points] boxes, 128-byte swizzle) in a four-deep ring.
//   * A operand: K-major core matrices (8 points x 4 channels of 16 bytes).  The four worker warps, one thread per
//     point, gather their point's channels from the swizzled tile (conflict-free: a warp reads 32 consecutive words
//     of one row), split every value into hi (its tf32 truncation) and lo = x - hi, and write 16-byte groups of
//     four channels into a hi tile and a lo tile.  This pass exists anyway for the hi/lo split; writing it in the
//     operand layout costs nothing extra.  (The tile as TMA delivers it is the instruction's MN-major layout, but
//     an MN-major TF32 A operand produced all-zero products on this GPU - measured with a K-major copy of the same
//     data beside it, which gave the exact result - so the K-major form is what runs.)
//   * B operand: W_bypass^T as K-major core matrices (8 output channels x 4 input channels), hi and lo, written
//     once per CTA.
//   * fp32 accuracy from three TF32 products: D = hi*Whi + hi*Wlo + lo*Whi, accumulated in fp32 in tensor memory.
//   * accumulator [128 lanes x C_out columns] in tensor memory; the four worker warps read their lane quarter with
//     tcgen05.ld (one point per thread, C_out values), add y, apply GELU and store - coalesced, since consecutive
//     lanes are consecutive points.
// One elected thread issues the TMA loads, one the MMAs; completion travels through mbarriers (tcgen05.commit for
// the tensor core).  Every wait is bounded: on expiry the kernel raises the plan's status word, drains its loads,
// frees its tensor memory and returns.  Several CTAs share an SM (about 52 KB of shared memory and 32 TMEM
// columns each at 16 channels), and inside a CTA the A operands and the accumulator are double-buffered, which is what overlaps one CTA's epilogue with another's loads.
#include <cuda.h>

#include "dtst_common.cuh"
#include "dtst_fused.cuh"
#include "dtst_sm100.cuh"

namespace dtst {

using namespace sm100;

namespace {

constexpr int kPts = 128;          // points per tile = MMA M
constexpr int kStages = 2;         // x tiles in flight per CTA (several CTAs share an SM)
constexpr int kWorkers = 4;        // worker warps (one per TMEM lane quarter)
constexpr int kThreads = (2 + kWorkers) * 32;

// Phi(z) = (1 + erf(z / sqrt 2)) / 2, the standard normal distribution function of the exact (erf) form of GELU,
// in the five-term rational form of Abramowitz & Stegun 7.1.26 / 26.2.17 (|error| <= 1.5e-7 on erf, below the
// rounding of the fp32 arithmetic around it: 8e-8 rel-L2 on GELU against 5e-8 with a correctly rounded erf),
// evaluated on the negative side as the tail itself, without cancellation.  The library erff costs about twice
// the instructions, and the passes that apply the activation are bound by exactly those.  e = exp(-z^2 / 2) is
// handed back because GELU' needs it too.
__device__ __forceinline__ float phi_f(float z, float& e) {
  const float t = __fdividef(1.0f, fmaf(0.2316418882f, fabsf(z), 1.0f));   // 0.3275911 / sqrt 2
  float poly = fmaf(1.061405429f, t, -1.453152027f);
  poly = fmaf(poly, t, 1.421413741f);
  poly = fmaf(poly, t, -0.284496736f);
  poly = fmaf(poly, t, 0.254829592f);
  e = __expf(-0.5f * z * z);
  const float q = poly * t * e;            // 2 (1 - Phi(|z|))
  return z >= 0.f ? fmaf(-0.5f, q, 1.0f) : 0.5f * q;
}

__device__ __forceinline__ float gelu_f(float v) {
  float e;
  return v * phi_f(v, e);
}

// shared-memory matrix descriptor of tcgen05.mma: start address, leading and stride byte offsets (all without
// their four low bits), descriptor version 1, swizzle mode in bits 61..63
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
  return (uint64_t)((addr >> 4) & 0x3fffu) | ((uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32) | (1ull << 46) | ((uint64_t)layout << 61);
}
constexpr uint32_t kLayoutNone = 0;

// instruction descriptor, kind::tf32: fp32 accumulator, TF32 A and B, both K-major
__host__ __device__ constexpr uint32_t instr_desc(int M, int N) {
  return (1u << 4) | (2u << 7) | (2u << 10) | (0u << 15) | (0u << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
      : "memory");
}
// the mbarrier gets one arrival when every tcgen05.mma issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 16 accumulator columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

template <int CI, int CO>
struct UmmaCfg {
  static_assert(CI % 8 == 0 && CI >= 8 && CI <= 64, "C_in: whole k-steps of 8 channels");
  static_assert(CO % 16 == 0 && CO >= 16 && CO <= 64, "C_out: MMA N with M = 128");
  static constexpr int KS = CI / 8;                       // k-steps
  static constexpr int PANEL_BYTES = CI * 128;            // [CI channels][32 points]
  static constexpr int TILE_BYTES = 4 * PANEL_BYTES;      // 128 points
  static constexpr int A_KSTEP_BYTES = kPts * 32;         // [128 points][8 channels] as core matrices
  static constexpr int B_KSTEP_BYTES = CO * 32;           // [CO][8 channels] as core matrices
  static constexpr int B_BYTES = 2 * KS * B_KSTEP_BYTES;  // hi and lo
  static constexpr int TCOLS = 2 * CO < 32 ? 32 : 2 * CO;  // TMEM columns: two accumulators (a power of two >= 32)
  static constexpr size_t SMEM = 1024 + (size_t)(kStages + 4) * TILE_BYTES + B_BYTES + 256;
};

template <int CI, int CO>
__global__ void __launch_bounds__(kThreads)
block_epilogue_umma_kernel(const __grid_constant__ CUtensorMap x_map, float* __restrict__ out, float* __restrict__ z,
                           const float* __restrict__ Wb, int B, long long P, long long tiles_per_b, int* status,
                           uint32_t poll_limit) {
  using Cfg = UmmaCfg<CI, CO>;
  pdl_trigger();
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* ring = smem;                                         // kStages x tile as TMA delivers it
  // the A operands, double-buffered: [buffer][hi | lo]; tile j uses buffer j & 1 (and accumulator j & 1), so that
  // the split of tile j + 1 overlaps the products and the epilogue of tile j
  unsigned char* a_tiles = smem + (size_t)kStages * Cfg::TILE_BYTES;
  unsigned char* bmat = a_tiles + 4 * (size_t)Cfg::TILE_BYTES;         // [hi | lo][k-step][core matrices]
  uint64_t* full = reinterpret_cast<uint64_t*>(bmat + Cfg::B_BYTES);
  uint64_t* empty = full + kStages;
  uint64_t* lo_ready = empty + kStages;     // [2]
  uint64_t* mma_done = lo_ready + 2;        // [2]
  uint64_t* tmem_free = mma_done + 2;       // [2]
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(tmem_free + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_s + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], kWorkers);
    }
    for (int k = 0; k < 2; ++k) {
      mbar_init(&lo_ready[k], kWorkers);
      mbar_init(&mma_done[k], 1);
      mbar_init(&tmem_free[k], kWorkers);
    }
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tensormap(&x_map);
  }
  if (warp == 1) {   // one warp allocates the accumulator columns and gives the permit back at once
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_s)),
                 "r"((uint32_t)Cfg::TCOLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  pdl_wait();   // W_bypass may come from the kernel before this one
  // B operand: W_bypass^T, element (n = output channel, k = input channel) of k-step ks at
  //   ks * B_KSTEP + (n / 8) * 256 + (k' / 4) * 128 + (n % 8) * 16 + (k' % 4) * 4,  k' = k - 8 ks
  for (int e = threadIdx.x; e < CO * CI; e += blockDim.x) {
    const int n = e / CI, k = e % CI;
    const float w = Wb[e];
    const float hi = __uint_as_float(__float_as_uint(w) & 0xffffe000u);
    const int ks = k / 8, kk = k % 8;
    const int off = ks * Cfg::B_KSTEP_BYTES + (n / 8) * 256 + (kk / 4) * 128 + (n % 8) * 16 + (kk % 4) * 4;
    *reinterpret_cast<float*>(bmat + off) = hi;
    *reinterpret_cast<float*>(bmat + Cfg::KS * Cfg::B_KSTEP_BYTES + off) = w - hi;
  }
  fence_proxy_async_smem();   // the tensor core reads these through the async proxy
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_s;

  const long long tiles = (long long)B * tiles_per_b;
  const long long first = blockIdx.x;
  const long long n_local = first < tiles ? (tiles - first + gridDim.x - 1) / gridDim.x : 0;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      for (long long j = 0; j < n_local; ++j) {
        const long long t = first + j * gridDim.x;
        const int s = (int)(j % kStages);
        if (!mbar_wait_bounded(&empty[s], (uint32_t)(((j / kStages) & 1) ^ 1), abort_flag, poll_limit)) break;
        const long long b = t / tiles_per_b, p0 = (t % tiles_per_b) * kPts;
        mbar_arrive_expect_tx(&full[s], (uint32_t)Cfg::TILE_BYTES);
#pragma unroll
        for (int h = 0; h < 4; ++h)   // points beyond the end of the row are filled with zeros
          tma_load_2d(ring + (size_t)s * Cfg::TILE_BYTES + (size_t)h * Cfg::PANEL_BYTES, &x_map, (int)(p0 + 32 * h),
                      (int)(b * CI), &full[s]);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(kPts, CO);
      const uint32_t b_addr = smem_u32(bmat);
      for (long long j = 0; j < n_local; ++j) {
        const int k2 = (int)(j & 1);
        const uint32_t ph = (uint32_t)((j >> 1) & 1);
        if (!mbar_wait_bounded(&lo_ready[k2], ph, abort_flag, poll_limit)) break;                // split done
        if (j >= 2 && !mbar_wait_bounded(&tmem_free[k2], ph ^ 1u, abort_flag, poll_limit)) break;  // accumulator read
        tc_fence_after();
        const uint32_t hi_addr = smem_u32(a_tiles + (size_t)(2 * k2) * Cfg::TILE_BYTES);
        const uint32_t lo_addr = hi_addr + Cfg::TILE_BYTES;
        const uint32_t d_addr = tmem_base + (uint32_t)(k2 * CO);
#pragma unroll
        for (int ks = 0; ks < Cfg::KS; ++ks) {
          // K-major, no swizzle: core matrices 128 bytes apart along K, 256 bytes apart along M / N
          const uint64_t a_hi = smem_desc(hi_addr + ks * Cfg::A_KSTEP_BYTES, 128, 256, kLayoutNone);
          const uint64_t a_lo = smem_desc(lo_addr + ks * Cfg::A_KSTEP_BYTES, 128, 256, kLayoutNone);
          const uint64_t b_hi = smem_desc(b_addr + ks * Cfg::B_KSTEP_BYTES, 128, 256, kLayoutNone);
          const uint64_t b_lo = smem_desc(b_addr + (Cfg::KS + ks) * Cfg::B_KSTEP_BYTES, 128, 256, kLayoutNone);
          umma_tf32(d_addr, a_hi, b_hi, idesc, ks > 0 ? 1u : 0u);
          umma_tf32(d_addr, a_hi, b_lo, idesc, 1u);
          umma_tf32(d_addr, a_lo, b_hi, idesc, 1u);
        }
        umma_commit(&mma_done[k2]);   // accumulator k2 is complete (and A buffer k2 may be rewritten)
      }
    }
  } else {
    // ---------------- workers: split tile j + 1, then the epilogue of tile j ----------------
    const int quarter = warp & 3;                          // the TMEM lanes this warp may read
    const int pt = quarter * 32 + lane;                    // this thread's point within a tile
    // y of this thread's point of tile j for every output channel (requested long before it is needed)
    auto load_y = [&](long long j, float (&yv)[CO]) {
      const long long t = first + j * gridDim.x;
      const long long b = t / tiles_per_b, p0 = (t % tiles_per_b) * kPts;
      const bool live = p0 + pt < P;
      const float* yb = out + (b * CO) * P + p0 + pt;
#pragma unroll
      for (int o = 0; o < CO; ++o) yv[o] = live ? yb[(long long)o * P] : 0.f;
    };
    // this thread's point of tile j: its channels from the swizzled x tile (channel c of point p sits in panel
    // p / 32, row c, 16-byte chunk ((p % 32) / 4) ^ (c % 8)), split into hi = tf32 truncation and lo = x - hi, and
    // written four channels at a time into the K-major core matrices of A buffer j & 1:
    //   k-step (c / 8): + (p / 8) * 256 + ((c % 8) / 4) * 128 + (p % 8) * 16 bytes
    auto split = [&](long long j) -> bool {
      const int s = (int)(j % kStages);
      bool ok = mbar_wait_bounded(&full[s], (uint32_t)((j / kStages) & 1), abort_flag, poll_limit);
      ok = __all_sync(0xffffffffu, ok) != 0;
      if (!ok) return false;
      unsigned char* hi_tile = a_tiles + (size_t)(2 * (j & 1)) * Cfg::TILE_BYTES;
      unsigned char* lo_tile = hi_tile + Cfg::TILE_BYTES;
      const unsigned char* srcb = ring + (size_t)s * Cfg::TILE_BYTES + (pt / 32) * Cfg::PANEL_BYTES + (pt % 4) * 4;
      const int chunk = (pt % 32) / 4;
#pragma unroll
      for (int c4 = 0; c4 < CI / 4; ++c4) {
        float v[4], h[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int c = 4 * c4 + k;
          v[k] = *reinterpret_cast<const float*>(srcb + c * 128 + ((chunk ^ (c & 7)) << 4));
          h[k] = __uint_as_float(__float_as_uint(v[k]) & 0xffffe000u);
        }
        const int off = (c4 / 2) * Cfg::A_KSTEP_BYTES + (pt / 8) * 256 + (c4 % 2) * 128 + (pt % 8) * 16;
        *reinterpret_cast<float4*>(hi_tile + off) = make_float4(h[0], h[1], h[2], h[3]);
        *reinterpret_cast<float4*>(lo_tile + off) = make_float4(v[0] - h[0], v[1] - h[1], v[2] - h[2], v[3] - h[3]);
      }
      fence_proxy_async_smem();   // the tensor core reads the A tiles through the async proxy
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&empty[s]);            // this warp has read its quarter of the x tile
        mbar_arrive(&lo_ready[j & 1]);     // and written its quarter of the A tiles
      }
      return true;
    };
    float y_cur[CO], y_next[CO];
    bool alive = n_local > 0;
    if (alive) {
      load_y(0, y_cur);
      alive = split(0);
    }
    for (long long j = 0; alive && j < n_local; ++j) {
      if (j + 1 < n_local) {
        load_y(j + 1, y_next);
        alive = split(j + 1);
        if (!alive) break;
      }
      const int k2 = (int)(j & 1);
      bool ok = mbar_wait_bounded(&mma_done[k2], (uint32_t)((j >> 1) & 1), abort_flag, poll_limit);
      ok = __all_sync(0xffffffffu, ok) != 0;
      if (!ok) break;
      tc_fence_after();
      float acc[CO];
#pragma unroll
      for (int c0 = 0; c0 < CO; c0 += 16) {
        float part[16];
        tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(k2 * CO + c0), part);
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[c0 + i] = part[i];
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_free[k2]);   // products of tile j + 2 may overwrite this accumulator
      const long long t = first + j * gridDim.x;
      const long long b = t / tiles_per_b, p0 = (t % tiles_per_b) * kPts;
      if (p0 + pt < P) {
        float* ob = out + (b * CO) * P + p0 + pt;
        float* zb = z ? z + (b * CO) * P + p0 + pt : nullptr;
#pragma unroll
        for (int o = 0; o < CO; ++o) {
          const float v = acc[o] + y_cur[o];
          if (zb) __stcs(zb + (long long)o * P, v);
          __stcs(ob + (long long)o * P, gelu_f(v));
        }
      }
#pragma unroll
      for (int o = 0; o < CO; ++o) y_cur[o] = y_next[o];
    }
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    // loads that were armed but never consumed may still be in flight
    for (int s = 0; s < kStages; ++s) mbar_wait_plain(&full[s], 0, 1u << 12), mbar_wait_plain(&full[s], 1, 1u << 12);
    atomicExch(status, 1);
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg::TCOLS) : "memory");
  }
}

template <int CI, int CO>
cudaError_t launch_umma_t(const float* x, float* out, float* z, const float* Wb, int B, long long P, int* status,
                          cudaStream_t st) {
  using Cfg = UmmaCfg<CI, CO>;
  CUtensorMap map;
  if (!make_points_map(&map, x, (long long)B * CI, P, CI)) return cudaErrorNotSupported;
  auto kern = block_epilogue_umma_kernel<CI, CO>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::SMEM);
  if (e != cudaSuccess) return e;
  int per_sm = 1;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, Cfg::SMEM);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) per_sm = 1;
  if (per_sm > 512 / Cfg::TCOLS) per_sm = 512 / Cfg::TCOLS;   // tensor memory: 512 columns per SM
  const long long tiles_per_b = (P + kPts - 1) / kPts;
  const long long tiles = (long long)B * tiles_per_b;
  long long grid = (long long)num_sms() * per_sm;
  if (grid > tiles) grid = tiles;
  (void)launch_pdl(kern, dim3((unsigned)grid), dim3(kThreads), Cfg::SMEM, st, map, out, z, Wb, B, P, tiles_per_b, status,
                   kDefaultPollLimit);
  return cudaGetLastError();
}

}  // namespace

bool block_umma_supported(int Ci, int Co, long long P, int B) {
  if (!((Ci == 8 || Ci == 16 || Ci == 32) && (Co == 16 || Co == 32))) return false;
  if (P % 4 != 0 || P >= (1ll << 31) || (long long)B * Ci >= (1ll << 31)) return false;
  return tma_encode_available();
}

cudaError_t launch_block_epilogue_umma(const float* x, float* out, float* z, const float* Wb, int B, int Ci, int Co,
                                       long long P, int* status, cudaStream_t st) {
#define DTST_UMMA_CASE(a, b) \
  if (Ci == a && Co == b) return launch_umma_t<a, b>(x, out, z, Wb, B, P, status, st);
  DTST_UMMA_CASE(8, 16)
  DTST_UMMA_CASE(16, 16)
  DTST_UMMA_CASE(32, 16)
  DTST_UMMA_CASE(8, 32)
  DTST_UMMA_CASE(16, 32)
  DTST_UMMA_CASE(32, 32)
#undef DTST_UMMA_CASE
  return cudaErrorNotSupported;
}

}  // namespace dtst
