// Row kernels: the contiguous (rfft) dimension alone, for shapes the plane kernels are not instantiated for
// (any N3 that is a multiple of 32 up to 256, any k3 <= 16).  The remaining dimensions run in dtst_mid.cu.
//
//   row_contract_kernel:  x[rows][N3] real  ->  out[rows][k3] complex   (grid read once, TMA-fed ring)
//   row_expand_kernel:    in[rows][k3] complex -> y[rows][N3] real      (grid written once, TMA stores)
//
// Both are "fold four mirrored samples, multiply by a per-parity-class basis" (see dtst_fused.cu for the
// algebra): a quadruple (j, N/2-1-j, N/2+j, N-1-j) gives uu, ud, vs, vd, which are exactly the A operands of
// four small GEMMs  [rows x quadruples] x [quadruples x <=8 frequencies]  (even-f cos, odd-f cos, odd-f sin,
// even-f sin).  With k3 = 16 every class has 8 frequencies - a full MMA n-tile - so here the contraction
// itself runs on the tensor cores (warp-level m16n8k8 TF32, hi/lo error-compensated, fp32 accumulate); the
// fragment gather from the swizzled TMA tile is bank-conflict free, and each lane ends up holding all four
// class sums of four consecutive frequencies, so the complex result is assembled and stored from registers.
#include <cuda.h>

#include "dtst_fused.cuh"
#include "dtst_sm100.cuh"

namespace dtst {

using namespace sm100;

namespace {

constexpr int kRowSmemLimit = 232448;

// fp32 -> (hi, lo) for the error-compensated TF32 product.  The tensor core reads only the upper 19 bits
// of an operand, so hi is the value with its low 13 mantissa bits cleared and lo = v - hi is exact in fp32;
// lo is passed as is (the hardware drops its low bits, an error of 2^-20 |v| at most).  One AND and one
// subtraction: the rounding conversion (cvt.rna) costs several times more issue slots, which is what
// bounded these kernels.
__device__ __forceinline__ void split_tf32_r(float v, uint32_t& hi, uint32_t& lo) {
  hi = __float_as_uint(v) & 0xffffe000u;
  lo = __float_as_uint(v - __uint_as_float(hi));
}

// (not volatile: a pure register-to-register operation the compiler may schedule freely among the loads)
__device__ __forceinline__ void mma_tf32_r(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Plain C++ accesses through a pointer into the shared array (`base` + 32-bit offset): the compiler keeps them
// on the right side of the barrier waits and arrivals (those are asm statements with a memory clobber) but is
// free to hoist the next k-step's loads above this k-step's MMAs.
struct SmemTile {
  unsigned char* base;   // generic pointer derived from the __shared__ array
  uint32_t s;            // its 32-bit shared-space address
};
__device__ __forceinline__ float lds32_s(const SmemTile& t, uint32_t addr) {
  return *reinterpret_cast<const float*>(t.base + (addr - t.s));
}
__device__ __forceinline__ void sts64_s(const SmemTile& t, uint32_t addr, float a, float b) {
  *reinterpret_cast<float2*>(t.base + (addr - t.s)) = make_float2(a, b);
}

// byte offset of element (row, col) of a [BOXR rows x N3] tile stored as N3/32 panels of [BOXR x 128 B],
// each written by TMA with the 128-byte swizzle
__device__ __forceinline__ uint32_t tile_off(int row, int col, int boxr) {
  return (uint32_t)(col >> 5) * (uint32_t)(boxr * 128) + (uint32_t)row * 128u +
         ((((uint32_t)(col & 31) >> 2) ^ ((uint32_t)row & 7u)) << 4) + (((uint32_t)col & 3u) << 2);
}

// basis table entry for (class, quadruple j, frequency slot gi): classes 0 = even-f cos, 1 = odd-f cos,
// 2 = odd-f sin, 3 = even-f sin; zero beyond k3
__device__ __forceinline__ float row_basis(int cls, int j, int gi, int N3, int K3) {
  const int f = (cls == 0 || cls == 3) ? 2 * gi : 2 * gi + 1;
  if (f >= K3) return 0.f;
  double sn, cs;
  sincospi((double)(((long long)f * (2 * j + 1)) % (2ll * N3)) / (double)N3, &sn, &cs);
  return (cls <= 1) ? (float)cs : (float)sn;
}

struct RowWait {
  volatile uint32_t* fill_seq;
  uint64_t* full;
  volatile int* abort_flag;
};

__device__ __forceinline__ bool row_wait_fill(const RowWait& w, int slot, uint32_t q) {
  for (uint32_t it = 0; w.fill_seq[slot] < q + 1u; ++it) {
    if ((it & 63u) == 63u) {
      if (*w.abort_flag) return false;
      __nanosleep(64);
    }
    if (it > (1u << 24)) {
      *w.abort_flag = 1;
      return false;
    }
  }
  return mbar_wait_bounded(&w.full[slot], q & 1u, w.abort_flag);
}

// The same wait with one verdict for the whole warp (every lane calls it): the lanes poll independently, and a
// lane whose barrier completed just as another warp raised the abort flag must not go on alone into the
// warp-synchronous MMA code.
__device__ __forceinline__ bool row_wait_fill_warp(const RowWait& w, int slot, uint32_t q) {
  return __all_sync(0xffffffffu, row_wait_fill(w, slot, q)) != 0;
}

// ---------------------------------------------------------------------------------------------
// forward: MT m-tiles of 16 rows per task; W consumer warps + one producer warp
// ---------------------------------------------------------------------------------------------
template <int MT, int W>
__global__ void __launch_bounds__((W + 1) * 32, 1)
row_contract_kernel(const __grid_constant__ CUtensorMap in_map, float2* __restrict__ out, long long rows, int N3,
                    int K3, float scale, int herm, int stages, int* __restrict__ status) {
  pdl_trigger();
  constexpr int BOXR = 16 * MT;
  const int NKS = N3 / 32;                       // k-steps of 8 quadruples
  const uint32_t slot_bytes = (uint32_t)BOXR * N3 * 4;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t ring_s = smem_u32(smem);
  const SmemTile tl_{smem, ring_s};
  // basis fragments: [cls][ks][lane] float4 = (b0 hi, b1 hi, b0 lo, b1 lo)
  float4* btab = reinterpret_cast<float4*>(smem + (size_t)stages * slot_bytes);
  uint64_t* full = reinterpret_cast<uint64_t*>(btab + (size_t)4 * NKS * 32);
  uint64_t* empty = full + 16;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(empty + 16);
  volatile uint32_t* fill_seq = reinterpret_cast<volatile uint32_t*>(empty + 16) + 4;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g8 = lane >> 2, t4 = lane & 3;

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
  for (int e = threadIdx.x; e < 4 * NKS * 32; e += blockDim.x) {
    const int l = e & 31, ks = (e >> 5) % NKS, cls = (e >> 5) / NKS;
    const int lg = l >> 2, lt = l & 3;
    const float v0 = row_basis(cls, 8 * ks + lt, lg, N3, K3);
    const float v1 = row_basis(cls, 8 * ks + lt + 4, lg, N3, K3);
    uint32_t h0, l0, h1, l1;
    split_tf32_r(v0, h0, l0);
    split_tf32_r(v1, h1, l1);
    btab[e] = make_float4(__uint_as_float(h0), __uint_as_float(h1), __uint_as_float(l0), __uint_as_float(l1));
  }
  __syncthreads();
  pdl_wait();   // everything above is independent of the preceding kernel

  const long long num_tasks = (rows + BOXR - 1) / BOXR;
  const long long first = blockIdx.x;
  const long long n_local = first < num_tasks ? (num_tasks - first + gridDim.x - 1) / gridDim.x : 0;

  if (warp == 0) {
    if (lane == 0) {
      for (long long tl = 0; tl < n_local; ++tl) {
        const long long task = first + tl * gridDim.x;
        const int slot = (int)(tl % stages);
        const uint32_t ph = (uint32_t)((tl / stages) & 1);
        if (!mbar_wait_bounded(&empty[slot], ph ^ 1u, abort_flag)) break;
        fill_seq[slot] = (uint32_t)(tl / stages) + 1u;
        mbar_arrive_expect_tx(&full[slot], slot_bytes);
        for (int h = 0; h < N3 / 32; ++h)     // rows past the end of the tensor are zero-filled by TMA
          tma_load_2d(smem + (size_t)slot * slot_bytes + (size_t)h * BOXR * 128, &in_map, h * 32,
                      (int)(task * BOXR), &full[slot]);
      }
    }
    __syncwarp();
  } else {
    const int w = warp - 1;
    const RowWait rw{fill_seq, full, abort_flag};
    // rotation (deferred half-sample phase, scale, Hermitian weight) of this lane's four frequencies
    float2 rot[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int f = 4 * t4 + i;
      double sn, cs;
      sincospi((double)f / (double)N3, &sn, &cs);
      const float wgt = scale * (herm ? herm_weight(f, N3) : 1.0f);
      rot[i] = make_float2((float)cs * wgt, (float)sn * wgt);
    }
    for (long long tl = w; tl < n_local; tl += W) {
      const long long task = first + tl * gridDim.x;
      const int slot = (int)(tl % stages);
      if (!row_wait_fill_warp(rw, slot, (uint32_t)(tl / stages))) break;
      const uint32_t st = ring_s + (uint32_t)slot * slot_bytes;
      // two accumulator sets (even / odd k-steps) halve the dependent-MMA chains; summed at the end
      float acc2[2][MT][4][4];
#pragma unroll
      for (int z = 0; z < 2; ++z)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc2[z][mt][c][e] = 0.f;

      // Gather addressing.  Element (row, j) of the swizzled tile: panel (j >> 5), 16-byte chunk ((j & 31) >> 2)
      // XOR (row & 7), word j & 3.  With j = 8 ks + t4 + 4 h the chunk is 2 (ks & 3) + h and the word is t4; the
      // mirrored column N3-1-j has chunk 7 - that and word 3 - t4, i.e. the same XOR term flipped by 0x70.  When
      // N3 is a multiple of 64 the half-row offsets N3/2 are whole panels, so everything but one XOR and the
      // panel offsets is a per-lane constant.
      const bool fastaddr = (N3 % 64) == 0;
      const uint32_t gx = (uint32_t)g8 << 4;
      const uint32_t P = (uint32_t)BOXR * 128u;
      const int NP = N3 / 32;
#pragma unroll 1
      for (int ks0 = 0; ks0 < NKS; ks0 += 4) {
        const uint32_t pa = (uint32_t)(ks0 >> 2);
        const uint32_t panA = st + pa * P, panD = st + ((uint32_t)NP - 1u - pa) * P;
        const uint32_t panC = st + ((uint32_t)(NP / 2) + pa) * P, panB = st + ((uint32_t)(NP / 2) - 1u - pa) * P;
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) {
          const int ks = ks0 + k4;
          if (ks >= NKS) break;
          float4 bf[4];
#pragma unroll
          for (int c = 0; c < 4; ++c) bf[c] = btab[(c * NKS + ks) * 32 + lane];
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            uint32_t ah[4][4], al[4][4];   // [class][fragment element]
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int row = 16 * mt + g8 + 8 * (e & 1);
              float a, b, c, d;
              if (fastaddr) {
                const uint32_t xa = ((uint32_t)((2 * k4 + (e >> 1)) << 4)) ^ gx;
                const uint32_t wa = (uint32_t)row * 128u + ((uint32_t)t4 << 2);
                const uint32_t wd = (uint32_t)row * 128u + ((uint32_t)(3 - t4) << 2);
                a = lds32_s(tl_, panA + wa + xa);
                d = lds32_s(tl_, panD + wd + (xa ^ 0x70u));
                c = lds32_s(tl_, panC + wa + xa);
                b = lds32_s(tl_, panB + wd + (xa ^ 0x70u));
              } else {
                const int j = 8 * ks + t4 + 4 * (e >> 1);
                a = lds32_s(tl_, st + tile_off(row, j, BOXR));
                b = lds32_s(tl_, st + tile_off(row, N3 / 2 - 1 - j, BOXR));
                c = lds32_s(tl_, st + tile_off(row, N3 / 2 + j, BOXR));
                d = lds32_s(tl_, st + tile_off(row, N3 - 1 - j, BOXR));
              }
              const float u = a + d, v = a - d, up = b + c, vp = b - c;
              split_tf32_r(u + up, ah[0][e], al[0][e]);   // uu: even-f cos
              split_tf32_r(u - up, ah[1][e], al[1][e]);   // ud: odd-f cos
              split_tf32_r(v + vp, ah[2][e], al[2][e]);   // vs: odd-f sin
              split_tf32_r(v - vp, ah[3][e], al[3][e]);   // vd: even-f sin
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const uint32_t bh0 = __float_as_uint(bf[c].x), bh1 = __float_as_uint(bf[c].y);
              const uint32_t bl0 = __float_as_uint(bf[c].z), bl1 = __float_as_uint(bf[c].w);
              mma_tf32_r(acc2[k4 & 1][mt][c], ah[c], bh0, bh1);
              mma_tf32_r(acc2[k4 & 1][mt][c], al[c], bh0, bh1);
              mma_tf32_r(acc2[k4 & 1][mt][c], ah[c], bl0, bl1);
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[slot]);
      float acc[MT][4][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[mt][c][e] = acc2[0][mt][c][e] + acc2[1][mt][c][e];

      // X_f = rot_f (C_f - i S_f); this lane holds f = 4 t4 .. 4 t4 + 3 of rows g8 and g8 + 8 of every m-tile
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int hrow = 0; hrow < 2; ++hrow) {
          const long long row = task * BOXR + 16 * mt + g8 + 8 * hrow;
          if (row >= rows) continue;
          float res[8];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int sl = i >> 1;                     // frequency slot 2 t4 + sl
            const bool odd = i & 1;
            const float C = odd ? acc[mt][1][2 * hrow + sl] : acc[mt][0][2 * hrow + sl];
            const float S = odd ? acc[mt][2][2 * hrow + sl] : acc[mt][3][2 * hrow + sl];
            res[2 * i] = rot[i].x * C + rot[i].y * S;
            res[2 * i + 1] = rot[i].y * C - rot[i].x * S;
          }
          float2* dst = out + row * K3 + 4 * t4;
          if (4 * t4 + 3 < K3 && (K3 & 1) == 0) {
            *reinterpret_cast<float4*>(dst) = make_float4(res[0], res[1], res[2], res[3]);
            *reinterpret_cast<float4*>(dst + 2) = make_float4(res[4], res[5], res[6], res[7]);
          } else {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              if (4 * t4 + i < K3) dst[i] = make_float2(res[2 * i], res[2 * i + 1]);
          }
        }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, 1);
}

// ---------------------------------------------------------------------------------------------
// inverse: y[row][j] from in[row][f]; W warps, each owns a task of BOXR rows and a staging tile
// ---------------------------------------------------------------------------------------------
template <int MT, int W>
__global__ void __launch_bounds__(W * 32, 1)
row_expand_kernel(const __grid_constant__ CUtensorMap out_map, const float2* __restrict__ in, long long rows, int N3,
                  int K3, float scale, int herm) {
  pdl_trigger();
  constexpr int BOXR = 16 * MT;
  const int NNT = N3 / 32;                       // n-tiles of 8 quadruples
  const uint32_t tile_bytes = (uint32_t)BOXR * N3 * 4;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g8 = lane >> 2, t4 = lane & 3;
  // two staging tiles per warp, used alternately: a tile is rewritten only after the store issued two tasks
  // ago has read it, so a store's latency hides behind a whole task of work
  unsigned char* staging0 = smem + (size_t)warp * 2 * tile_bytes;
  const SmemTile tl_{staging0, smem_u32(staging0)};
  // basis fragments as MMA B operands: k = frequency slot, n = quadruple; [cls][nt][lane] float4
  float4* btab = reinterpret_cast<float4*>(smem + (size_t)W * 2 * tile_bytes);

  if (threadIdx.x == 0) prefetch_tensormap(&out_map);
  for (int e = threadIdx.x; e < 4 * NNT * 32; e += blockDim.x) {
    const int l = e & 31, nt = (e >> 5) % NNT, cls = (e >> 5) / NNT;
    const int lg = l >> 2, lt = l & 3;
    // b0: (k = lt, n = lg), b1: (k = lt + 4, n = lg)
    const float v0 = row_basis(cls, 8 * nt + lg, lt, N3, K3);
    const float v1 = row_basis(cls, 8 * nt + lg, lt + 4, N3, K3);
    uint32_t h0, l0, h1, l1;
    split_tf32_r(v0, h0, l0);
    split_tf32_r(v1, h1, l1);
    btab[e] = make_float4(__uint_as_float(h0), __uint_as_float(h1), __uint_as_float(l0), __uint_as_float(l1));
  }
  __syncthreads();

  // conjugate rotation, scale and Hermitian weight of this lane's four frequencies 2 gi + p, gi = t4 (+4)
  float2 rotv[2][2];
#pragma unroll
  for (int hs = 0; hs < 2; ++hs)
#pragma unroll
    for (int p = 0; p < 2; ++p) {
      const int f = 2 * (t4 + 4 * hs) + p;
      double sn, cs;
      sincospi((double)f / (double)N3, &sn, &cs);
      const float wgt = scale * (herm ? herm_weight(f, N3) : 1.0f);
      rotv[hs][p] = make_float2((float)cs * wgt, -(float)sn * wgt);
    }

  const long long num_tasks = (rows + BOXR - 1) / BOXR;
  const long long tstride = (long long)gridDim.x * W;
  // raw input values of a task, fetched one task ahead: element (mt, e) needs frequencies 2 gi and 2 gi + 1,
  // which are adjacent in memory: one 16-byte load when k3 is even (every row then starts 16-byte aligned)
  float2 vin[MT][4][2];
  const bool pairload = (K3 & 1) == 0;
  pdl_wait();   // everything above is independent of the preceding kernel
  auto load_inputs = [&](long long t) {
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const long long row = t * BOXR + 16 * mt + g8 + 8 * (e & 1);
        const int f0 = 2 * (t4 + 4 * (e >> 1));
        const bool live = t < num_tasks && row < rows;
        if (pairload) {
          float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
          if (live && f0 < K3) v = __ldg(reinterpret_cast<const float4*>(in + row * K3 + f0));
          vin[mt][e][0] = make_float2(v.x, v.y);
          vin[mt][e][1] = make_float2(v.z, v.w);
        } else {
#pragma unroll
          for (int p = 0; p < 2; ++p)
            vin[mt][e][p] = (live && f0 + p < K3) ? __ldg(in + row * K3 + f0 + p) : make_float2(0.f, 0.f);
        }
      }
  };
  load_inputs((long long)blockIdx.x + (long long)warp * gridDim.x);
  int iter = 0;
  for (long long task = (long long)blockIdx.x + (long long)warp * gridDim.x; task < num_tasks; task += tstride) {
    // A fragments: z'[row][slot] = scale c_f e^{-i pi f / N3} in[row][f]; classes take Re of even f, Re of
    // odd f, Im of odd f, Im of even f.  Element (row, slot): e&1 selects row + 8, e>>1 selects slot + 4.
    uint32_t ah[MT][4][4], al[MT][4][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float re[2], im[2];
#pragma unroll
        for (int p = 0; p < 2; ++p) {
          const float2 v = vin[mt][e][p];
          const float rx = rotv[e >> 1][p].x, ry = rotv[e >> 1][p].y;
          re[p] = v.x * rx - v.y * ry;
          im[p] = v.x * ry + v.y * rx;
        }
        split_tf32_r(re[0], ah[mt][0][e], al[mt][0][e]);
        split_tf32_r(re[1], ah[mt][1][e], al[mt][1][e]);
        split_tf32_r(im[1], ah[mt][2][e], al[mt][2][e]);
        split_tf32_r(im[0], ah[mt][3][e], al[mt][3][e]);
      }
    load_inputs(task + tstride);   // the next task's values travel while this one is expanded
    // the store issued two tasks ago (same tile) must have finished reading it
    unsigned char* staging = staging0 + (size_t)(iter & 1) * tile_bytes;
    const uint32_t staging_s = tl_.s + (uint32_t)(iter & 1) * tile_bytes;
    ++iter;
    if (lane == 0) tma_store_wait_read<1>();
    __syncwarp();
    // Staging addressing, as in the contraction kernel: quadruple pair j0 = 8 nt + 2 t4 sits in panel nt >> 2,
    // chunk 2 (nt & 3) + (t4 >> 1), 8-byte slot (t4 & 1); its mirror images flip the chunk (XOR 0x70) and the slot.
    const bool fastaddr = (N3 % 64) == 0;
    const uint32_t gx = (uint32_t)g8 << 4;
    const uint32_t P = (uint32_t)BOXR * 128u;
    const int NP = N3 / 32;
#pragma unroll 1
    for (int nt0 = 0; nt0 < NNT; nt0 += 4) {
      const uint32_t pa = (uint32_t)(nt0 >> 2);
      const uint32_t panA = staging_s + pa * P, panD = staging_s + ((uint32_t)NP - 1u - pa) * P;
      const uint32_t panC = staging_s + ((uint32_t)(NP / 2) + pa) * P;
      const uint32_t panB = staging_s + ((uint32_t)(NP / 2) - 1u - pa) * P;
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        const int nt = nt0 + k4;
        if (nt >= NNT) break;
        float4 bf[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) bf[c] = btab[(c * NNT + nt) * 32 + lane];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          float acc[4][4];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[c][e] = 0.f;
            const uint32_t bh0 = __float_as_uint(bf[c].x), bh1 = __float_as_uint(bf[c].y);
            const uint32_t bl0 = __float_as_uint(bf[c].z), bl1 = __float_as_uint(bf[c].w);
            mma_tf32_r(acc[c], ah[mt][c], bh0, bh1);
            mma_tf32_r(acc[c], al[mt][c], bh0, bh1);
            mma_tf32_r(acc[c], ah[mt][c], bl0, bl1);
          }
          // C fragment elements 2h, 2h+1: row = 16 mt + g8 + 8 h, quadruples j0 = 8 nt + 2 t4 and j0 + 1:
          // their four outputs are pairwise adjacent in the row, so each pair is one 8-byte store
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int row = 16 * mt + g8 + 8 * h;
            float ya[2], yd[2], yb[2], yc[2];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const int e = 2 * h + q;
              const float Ea = acc[0][e], Oa = acc[1][e], Ob = acc[2][e], Eb = acc[3][e];
              const float sa = Ea + Oa, da = Ea - Oa, sb = Eb + Ob, db = Eb - Ob;
              ya[q] = sa - sb;   // y[j]
              yd[q] = sa + sb;   // y[N3-1-j]
              yb[q] = da + db;   // y[N3/2-1-j]
              yc[q] = da - db;   // y[N3/2+j]
            }
            if (fastaddr) {
              const uint32_t xa = ((uint32_t)((2 * k4 + (t4 >> 1)) << 4)) ^ gx;
              const uint32_t wa = (uint32_t)row * 128u + ((uint32_t)(t4 & 1) << 3);
              const uint32_t wd = (uint32_t)row * 128u + ((uint32_t)(1 - (t4 & 1)) << 3);
              sts64_s(tl_, panA + wa + xa, ya[0], ya[1]);
              sts64_s(tl_, panD + wd + (xa ^ 0x70u), yd[1], yd[0]);
              sts64_s(tl_, panB + wd + (xa ^ 0x70u), yb[1], yb[0]);
              sts64_s(tl_, panC + wa + xa, yc[0], yc[1]);
            } else {
              const int j0 = 8 * nt + 2 * t4;
              sts64_s(tl_, staging_s + tile_off(row, j0, BOXR), ya[0], ya[1]);
              sts64_s(tl_, staging_s + tile_off(row, N3 - 2 - j0, BOXR), yd[1], yd[0]);
              sts64_s(tl_, staging_s + tile_off(row, N3 / 2 - 2 - j0, BOXR), yb[1], yb[0]);
              sts64_s(tl_, staging_s + tile_off(row, N3 / 2 + j0, BOXR), yc[0], yc[1]);
            }
          }
        }
      }
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
      for (int h = 0; h < N3 / 32; ++h)    // rows past the end of the tensor are clipped by TMA
        tma_store_2d(&out_map, h * 32, (int)(task * BOXR), staging + (size_t)h * BOXR * 128);
      tma_store_commit();
    }
  }
  if (lane == 0) tma_store_wait_all<0>();
}

// 2 KB TMA load boxes (16 rows) starve the contraction kernel (3.6 instead of 5.9 TB/s at N3 = 256): it uses
// 32-row tasks; the expansion kernel keeps 16-row tiles at N3 > 128 so that two of them fit per warp.
int pick_mt(int N3) { return N3 <= 64 ? 4 : 2; }
int pick_mt_expand(int N3) { return N3 <= 64 ? 4 : (N3 <= 128 ? 2 : 1); }

template <int MT>
cudaError_t launch_row_contract_t(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm,
                                  int* status, cudaStream_t st) {
  constexpr int W = 7;
  constexpr int BOXR = 16 * MT;
  const size_t slot = (size_t)BOXR * N3 * 4;
  const size_t fixed = 1024 + (size_t)4 * (N3 / 32) * 32 * 16 + 512;
  int stages = (int)((kRowSmemLimit - fixed) / slot);
  if (stages > 16) stages = 16;
  if (stages < 3) return cudaErrorInvalidConfiguration;
  const size_t total = (size_t)stages * slot + fixed;
  CUtensorMap map;
  if (!make_rows_map(&map, x, rows, N3, BOXR)) return cudaErrorNotSupported;
  auto kern = row_contract_kernel<MT, W>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)total);
  if (e != cudaSuccess) return e;
  const long long tasks = (rows + BOXR - 1) / BOXR;
  const int grid = (int)(tasks < num_sms() ? tasks : num_sms());
  (void)launch_pdl(kern, dim3(grid), dim3((W + 1) * 32), total, st, map, out, rows, N3, K3, scale, herm, stages, status);
  return cudaGetLastError();
}

template <int MT>
cudaError_t launch_row_expand_t(const float2* in, float* y, long long rows, int N3, int K3, float scale, int herm,
                                cudaStream_t st) {
  constexpr int BOXR = 16 * MT;
  const size_t tile = (size_t)BOXR * N3 * 4;
  const size_t fixed = 1024 + (size_t)4 * (N3 / 32) * 32 * 16;
  int W = (int)((kRowSmemLimit - fixed) / (2 * tile));
  if (W > 12) W = 12;
  if (W < 2) return cudaErrorInvalidConfiguration;
  CUtensorMap map;
  if (!make_rows_map(&map, y, rows, N3, BOXR)) return cudaErrorNotSupported;
  const long long tasks = (rows + BOXR - 1) / BOXR;
  auto launch = [&](auto kern, int w) -> cudaError_t {
    const size_t total = (size_t)w * 2 * tile + fixed;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)total);
    if (e != cudaSuccess) return e;
    const long long want = (tasks + w - 1) / w;
    const int grid = (int)(want < num_sms() ? want : num_sms());
    (void)launch_pdl(kern, dim3(grid), dim3(w * 32), total, st, map, in, rows, N3, K3, scale, herm);
    return cudaGetLastError();
  };
  if (W >= 12 && MT <= 2) return launch(row_expand_kernel<MT, 12>, 12);
  if (W >= 10 && MT <= 2) return launch(row_expand_kernel<MT, 10>, 10);
  if (W >= 8) return launch(row_expand_kernel<MT, 8>, 8);
  if (W >= 6) return launch(row_expand_kernel<MT, 6>, 6);
  if (W >= 4) return launch(row_expand_kernel<MT, 4>, 4);
  return launch(row_expand_kernel<MT, 2>, 2);
}

}  // namespace

bool row_supported(int N3, int K3) {
  return N3 % 32 == 0 && N3 >= 32 && N3 <= 256 && K3 >= 1 && K3 <= 16 && 2 * (K3 - 1) < N3;
}

cudaError_t launch_row_contract(const float* x, float2* out, long long rows, int N3, int K3, float scale, int herm,
                                int* status, cudaStream_t st) {
  switch (pick_mt(N3)) {
    case 4: return launch_row_contract_t<4>(x, out, rows, N3, K3, scale, herm, status, st);
    case 2: return launch_row_contract_t<2>(x, out, rows, N3, K3, scale, herm, status, st);
    default: return launch_row_contract_t<1>(x, out, rows, N3, K3, scale, herm, status, st);
  }
}

cudaError_t launch_row_expand(const float2* in, float* y, long long rows, int N3, int K3, float scale, int herm,
                              cudaStream_t st) {
  switch (pick_mt_expand(N3)) {
    case 4: return launch_row_expand_t<4>(in, y, rows, N3, K3, scale, herm, st);
    case 2: return launch_row_expand_t<2>(in, y, rows, N3, K3, scale, herm, st);
    default: return launch_row_expand_t<1>(in, y, rows, N3, K3, scale, herm, st);
  }
}

}  // namespace dtst
