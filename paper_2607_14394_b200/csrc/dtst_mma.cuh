// Warp-level TF32 tensor-core helpers shared by the reduced-tensor kernels: the m16n8k8 MMA and the hi/lo split
// that makes three of them reproduce an fp32 product ("3xTF32": hi*hi + lo*hi + hi*lo, fp32 accumulate).
//
// Fragment coordinates of mma.m16n8k8 (g8 = lane / 4, t4 = lane % 4):
//   A (16 x 8, row):  a[e] = A[g8 + 8 (e & 1)][t4 + 4 (e >> 1)]
//   B ( 8 x 8, col):  b0 = B[t4][g8], b1 = B[t4 + 4][g8]
//   C (16 x 8):       c[e] = C[g8 + 8 (e >> 1)][2 t4 + (e & 1)]
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace dtst {

// fp32 -> (hi, lo): hi keeps the top 10 mantissa bits (exactly representable in TF32), lo = v - hi is exact in
// fp32 and is truncated to TF32 by the tensor core; hi*hi + lo*hi + hi*lo misses only lo*lo (~2^-20 relative).
__device__ __forceinline__ void split_tf32_trunc(float v, uint32_t& hi, uint32_t& lo) {
  hi = __float_as_uint(v) & 0xffffe000u;
  lo = __float_as_uint(v - __uint_as_float(hi));
}

// Same split with hi rounded to nearest (half an ulp added to the magnitude before the mask): |lo| <= 2^-11 |v|,
// unbiased, one integer add more.  For operands that are split in the inner loop.
__device__ __forceinline__ void split_tf32_round(float v, uint32_t& hi, uint32_t& lo) {
  hi = (__float_as_uint(v) + 0x1000u) & 0xffffe000u;
  lo = __float_as_uint(v - __uint_as_float(hi));
}

// Split with both parts rounded by the conversion instruction: for tables that are built once.
__device__ __forceinline__ void split_tf32_rna(float v, uint32_t& hi, uint32_t& lo) {
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(hi) : "f"(v));
  const float r = v - __uint_as_float(hi);
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(lo) : "f"(r));
}

// D += A(16x8, row) * B(8x8, col), TF32 inputs, fp32 accumulate
__device__ __forceinline__ void mma_m16n8k8_tf32(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// one compensated product: d += (ahi + alo) * (bhi + blo) without the lo*lo term
__device__ __forceinline__ void mma3_tf32(float (&d)[4], const uint32_t (&ahi)[4], const uint32_t (&alo)[4],
                                          uint32_t bh0, uint32_t bh1, uint32_t bl0, uint32_t bl1) {
  mma_m16n8k8_tf32(d, ahi, bh0, bh1);
  mma_m16n8k8_tf32(d, alo, bh0, bh1);
  mma_m16n8k8_tf32(d, ahi, bl0, bl1);
}

// cos / sin of pi * g * (2 q + 1) / N (the half-sample phase psi_g (q + 1/2), psi_g = 2 pi g / N) with the phase
// reduced exactly in integers: the basis of the folded two-sided dimensions
__device__ __forceinline__ void basis_cs(int g, int q, int N, float& cs, float& sn) {
  double s, c;
  sincospi((double)(((long long)g * (2 * q + 1)) % (2ll * N)) / (double)N, &s, &c);
  cs = (float)c;
  sn = (float)s;
}

// frequency of slot s in parity class cls (0: even cos, 1: odd cos, 2: odd sin, 3: even sin)
__device__ __forceinline__ int class_freq(int cls, int s) { return cls == 0 ? 2 * s : (cls == 3 ? 2 * s + 2 : 2 * s + 1); }

}  // namespace dtst
