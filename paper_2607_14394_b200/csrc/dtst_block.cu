// The rest of the block around the spectral layer (Section "Block Structure", Algorithm 1 lines 1 and 8):
//     out = GELU(W_bypass x + y),   y = I(M(F(x), W))  the spectral layer's output,
// and its backward pass.  W_bypass is the point-wise linear operator [C_out][C_in] (no bias), GELU the exact
// erf form z Phi(z).  Everything here is HBM-bound element-wise work over the grid: one pass that reads x and y
// and writes the activation (and, for training, the pre-activation), one pass for GELU', and one pass that adds
// W_bypass^T g_z to grad_x while it reduces grad_W_bypass.
//
// Kernels in this file serve any channel count in exact fp32 FFMA; dtst_block_umma.cu holds the tensor-core
// (tcgen05, accumulator in TMEM) version of the forward pass's bypass product for channel counts it fits.
#include "dtst_common.cuh"

namespace dtst {
namespace {

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

// d GELU / dz = Phi(z) + z phi(z)
__device__ __forceinline__ float gelu_grad_f(float v) {
  float e;
  const float Phi = phi_f(v, e);
  return fmaf(v * 0.39894228040143268f, e, Phi);
}

constexpr int kOC = 4;   // output channels per register tile of the FFMA kernels

// out[b,o,p] = GELU(sum_i Wb[o,i] x[b,i,p] + out[b,o,p]) in place (out holds y on entry); z (optional) gets the
// pre-activation.  One thread owns four consecutive points and walks the output channels four at a time; the
// input channels of its points are re-read from L1 for every group of four outputs.
// With LINEAR the same loop is a plain point-wise linear layer (the lifting and projection layers of an FNO):
// out[b,o,p] = sum_i Wb[o,i] x[b,i,p] + bias[o], `z` then carries the bias (or NULL) and out is write-only.
template <bool LINEAR>
__global__ void __launch_bounds__(256) block_epilogue_kernel(const float* __restrict__ x, float* __restrict__ out,
                                                            float* __restrict__ z, const float* __restrict__ Wb,
                                                            int B, int Ci, int Co, long long P) {
  pdl_trigger();
  extern __shared__ float wb_s[];   // [Co][Ci]
  pdl_wait();
  for (int e = threadIdx.x; e < Co * Ci; e += blockDim.x) wb_s[e] = Wb[e];
  __syncthreads();
  const long long quads = P / 4;
  const long long total = (long long)B * quads;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (long long)gridDim.x * blockDim.x) {
    const long long b = t / quads, q = t % quads;
    const float4* xb = reinterpret_cast<const float4*>(x + b * Ci * P) + q;
    float4* ob = reinterpret_cast<float4*>(out + b * Co * P) + q;
    float4* zb = (!LINEAR && z) ? reinterpret_cast<float4*>(z + b * Co * P) + q : nullptr;
    for (int o0 = 0; o0 < Co; o0 += kOC) {
      float4 acc[kOC];
#pragma unroll
      for (int k = 0; k < kOC; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int i = 0; i < Ci; ++i) {
        const float4 xv = __ldg(xb + (long long)i * quads);
#pragma unroll
        for (int k = 0; k < kOC; ++k) {
          const float w = (o0 + k < Co) ? wb_s[(o0 + k) * Ci + i] : 0.f;
          acc[k].x = fmaf(w, xv.x, acc[k].x);
          acc[k].y = fmaf(w, xv.y, acc[k].y);
          acc[k].z = fmaf(w, xv.z, acc[k].z);
          acc[k].w = fmaf(w, xv.w, acc[k].w);
        }
      }
#pragma unroll
      for (int k = 0; k < kOC; ++k) {
        if (o0 + k < Co) {
          const long long off = (long long)(o0 + k) * quads;
          if constexpr (LINEAR) {
            const float bo = z ? z[o0 + k] : 0.f;
            ob[off] = make_float4(acc[k].x + bo, acc[k].y + bo, acc[k].z + bo, acc[k].w + bo);
          } else {
            const float4 yv = ob[off];
            const float4 zv = make_float4(acc[k].x + yv.x, acc[k].y + yv.y, acc[k].z + yv.z, acc[k].w + yv.w);
            if (zb) __stcs(zb + off, zv);
            __stcs(ob + off, make_float4(gelu_f(zv.x), gelu_f(zv.y), gelu_f(zv.z), gelu_f(zv.w)));
          }
        }
      }
    }
  }
}

// The same pass with a thread's x values held in registers: all C_in loads of a thread are in flight at once (the
// loop above has one), and x is read exactly once instead of once per four output channels.  A thread owns V
// consecutive points: four up to 20 input channels, two for 32 (64 registers of x either way).
template <int V>
struct PointVec {
  float v[V];
};
template <int V>
__device__ __forceinline__ PointVec<V> ld_points(const float* p) {
  PointVec<V> r;
  if constexpr (V == 4) {
    const float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    r.v[0] = t.x; r.v[1] = t.y; r.v[2] = t.z; r.v[3] = t.w;
  } else {
    const float2 t = __ldcs(reinterpret_cast<const float2*>(p));
    r.v[0] = t.x; r.v[1] = t.y;
  }
  return r;
}
template <int V>
__device__ __forceinline__ void st_points(float* p, const PointVec<V>& r, bool streaming) {
  if constexpr (V == 4) {
    const float4 t = make_float4(r.v[0], r.v[1], r.v[2], r.v[3]);
    if (streaming) __stcs(reinterpret_cast<float4*>(p), t); else *reinterpret_cast<float4*>(p) = t;
  } else {
    const float2 t = make_float2(r.v[0], r.v[1]);
    if (streaming) __stcs(reinterpret_cast<float2*>(p), t); else *reinterpret_cast<float2*>(p) = t;
  }
}

template <bool LINEAR, int CI, int V>
__global__ void __launch_bounds__(256, 2) block_epilogue_regx_kernel(const float* __restrict__ x, float* __restrict__ out,
                                                                    float* __restrict__ z,
                                                                    const float* __restrict__ Wb, int B, int Co,
                                                                    long long P) {
  pdl_trigger();
  extern __shared__ float wb_s[];   // [Co][CI]
  pdl_wait();
  for (int e = threadIdx.x; e < Co * CI; e += blockDim.x) wb_s[e] = Wb[e];
  __syncthreads();
  const long long groups = P / V;
  const long long total = (long long)B * groups;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (long long)gridDim.x * blockDim.x) {
    const long long b = t / groups, p0 = (t % groups) * V;
    const float* xb = x + b * CI * P + p0;
    float* ob = out + b * Co * P + p0;
    float* zb = (!LINEAR && z) ? z + b * Co * P + p0 : nullptr;
    PointVec<V> xv[CI];
#pragma unroll
    for (int i = 0; i < CI; ++i) xv[i] = ld_points<V>(xb + (long long)i * P);
    for (int o0 = 0; o0 < Co; o0 += 4) {
      PointVec<V> acc[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if constexpr (LINEAR) {
          const float bo = (z && o0 + k < Co) ? z[o0 + k] : 0.f;
#pragma unroll
          for (int c = 0; c < V; ++c) acc[k].v[c] = bo;
        } else {
          if (o0 + k < Co) {
            acc[k] = ld_points<V>(ob + (long long)(o0 + k) * P);   // the layer's output: requested before the products
          } else {
#pragma unroll
            for (int c = 0; c < V; ++c) acc[k].v[c] = 0.f;
          }
        }
      }
#pragma unroll
      for (int i = 0; i < CI; ++i)
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float w = (o0 + k < Co) ? wb_s[(o0 + k) * CI + i] : 0.f;
#pragma unroll
          for (int c = 0; c < V; ++c) acc[k].v[c] = fmaf(w, xv[i].v[c], acc[k].v[c]);
        }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (o0 + k < Co) {
          const long long off = (long long)(o0 + k) * P;
          if constexpr (LINEAR) {
            st_points<V>(ob + off, acc[k], false);
          } else {
            if (zb) st_points<V>(zb + off, acc[k], true);
            PointVec<V> g;
#pragma unroll
            for (int c = 0; c < V; ++c) g.v[c] = gelu_f(acc[k].v[c]);
            st_points<V>(ob + off, g, true);
          }
        }
      }
    }
  }
}

// g_z = grad_out * GELU'(z), element-wise, 16 bytes per access (gz may alias grad_out)
__global__ void __launch_bounds__(256) gelu_backward_kernel(const float4* g, const float4* __restrict__ z,
                                                           float4* gz, long long n4) {
  pdl_trigger();
  pdl_wait();
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < n4; t += (long long)gridDim.x * blockDim.x) {
    const float4 gv = __ldcs(g + t), zv = __ldcs(z + t);
    gz[t] = make_float4(gv.x * gelu_grad_f(zv.x), gv.y * gelu_grad_f(zv.y), gv.z * gelu_grad_f(zv.z),
                        gv.w * gelu_grad_f(zv.w));
  }
}

// The bypass in the backward pass, one pass over the grid:
//   grad_x[b,i,p] += sum_o Wb[o,i] g_z[b,o,p]          (added to what the spectral layer's adjoint left there)
//   partial[cta][o][i] = sum over this CTA's points of g_z[b,o,p] x[b,i,p]
// A CTA stages tiles of kTP points of g_z (all C_out channels) and x (all C_in channels) in shared memory.
// Weight gradient: the (o, i) pairs are cut into 4 x 4 blocks; a thread owns one block for every npg-th quad of
// points (npg = 256 / blocks point groups work side by side), so that 8 shared-memory loads of 16 bytes feed 64
// multiply-adds; its 16 sums live in registers across all tiles of the CTA and are added over the point groups in
// ascending order at the end - a fixed order, so repeated runs give the same bits.  Input gradient: a thread owns
// four input channels times four points per round.
constexpr int kTP = 128;
constexpr int kTS = kTP + 4;     // row stride of the staged tiles in floats (rows shifted by 16 bytes in the banks)

__global__ void __launch_bounds__(256, 3) bypass_backward_kernel(const float* __restrict__ gz, const float* __restrict__ x,
                                                             float* __restrict__ gx, const float* __restrict__ Wb,
                                                             float* __restrict__ partial, int B, int Ci, int Co,
                                                             long long P, int want_gx, int want_gw, int want_gb) {
  pdl_trigger();
  extern __shared__ float bb_s[];
  float* wb_s = bb_s;                       // [Co][Ci]
  float* gz_s = wb_s + ((Co * Ci + 3) & ~3);   // [Co][kTP], rows kTS apart, 16-byte aligned
  float* x_s = gz_s + Co * kTS;             // [Ci][kTP], rows kTS apart
  pdl_wait();
  for (int e = threadIdx.x; e < Co * Ci; e += blockDim.x) wb_s[e] = Wb[e];
  const int ob_n = (Co + 3) / 4, ib_n = (Ci + 3) / 4;
  const int blocks = ob_n * ib_n;                       // <= 256 (C_in * C_out <= 4096)
  const int npg = 256 / blocks;                         // point groups
  const int pg = threadIdx.x / blocks, blk = threadIdx.x % blocks;
  const bool gw_thread = want_gw && pg < npg;
  const int o0 = 4 * (blk / ib_n), i0 = 4 * (blk % ib_n);
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[a][c] = 0.f;
  float bsum[4] = {0.f, 0.f, 0.f, 0.f};   // sum over points of g_z (the gradient of a bias), on the threads with i0 == 0
  const long long tiles_per_b = (P + kTP - 1) / kTP;
  const long long tiles = (long long)B * tiles_per_b;
  // Each thread stages up to kLd 16-byte pieces of a tile; the pieces of the NEXT tile are requested before the
  // current one is worked on, so that their latency hides behind the arithmetic (C_in + C_out <= 8 * kLd).
  constexpr int kLd = 8;
  const int pieces = (Co + Ci) * (kTP / 4);
  float4 nxt[kLd];
  auto fetch = [&](long long tt) {
    const long long bb = tt / tiles_per_b, pp0 = (tt % tiles_per_b) * kTP;
    const int nnp = (int)((P - pp0) < kTP ? (P - pp0) : kTP);
#pragma unroll
    for (int k = 0; k < kLd; ++k) {
      const int e = threadIdx.x + 256 * k;
      nxt[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (e < pieces) {
        const int c = e / (kTP / 4), q = e % (kTP / 4);
        if (4 * q < nnp) {
          const float* src = c < Co ? gz + (bb * Co + c) * P : x + (bb * Ci + (c - Co)) * P;
          nxt[k] = __ldcs(reinterpret_cast<const float4*>(src + pp0) + q);
        }
      }
    }
  };
  if ((long long)blockIdx.x < tiles) fetch(blockIdx.x);
  for (long long t = blockIdx.x; t < tiles; t += gridDim.x) {
    const long long b = t / tiles_per_b, p0 = (t % tiles_per_b) * kTP;
    const int np = (int)((P - p0) < kTP ? (P - p0) : kTP);   // a multiple of 4
    __syncthreads();   // the previous tile has been consumed (and wb_s is complete)
#pragma unroll
    for (int k = 0; k < kLd; ++k) {
      const int e = threadIdx.x + 256 * k;
      if (e < pieces) {
        const int c = e / (kTP / 4), q = e % (kTP / 4);
        reinterpret_cast<float4*>(c < Co ? gz_s + c * kTS : x_s + (c - Co) * kTS)[q] = nxt[k];
      }
    }
    __syncthreads();
    if (t + gridDim.x < tiles) fetch(t + gridDim.x);
    if (gw_thread) {
      for (int q = pg; q < kTP / 4; q += npg) {     // quads beyond the end of a ragged tile hold zeros
        float4 gv[4], xv[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          gv[a] = (o0 + a < Co) ? reinterpret_cast<const float4*>(gz_s + (o0 + a) * kTS)[q] : make_float4(0.f, 0.f, 0.f, 0.f);
          xv[a] = (i0 + a < Ci) ? reinterpret_cast<const float4*>(x_s + (i0 + a) * kTS)[q] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int c = 0; c < 4; ++c)
            acc[a][c] = fmaf(gv[a].x, xv[c].x, fmaf(gv[a].y, xv[c].y, fmaf(gv[a].z, xv[c].z, fmaf(gv[a].w, xv[c].w, acc[a][c]))));
        if (want_gb && i0 == 0) {
#pragma unroll
          for (int a = 0; a < 4; ++a) bsum[a] += (gv[a].x + gv[a].y) + (gv[a].z + gv[a].w);
        }
      }
    }
    if (want_gx) {
      // (pair of input channels, quad of points) per thread, as many rounds as the tile needs; what the spectral
      // layer's adjoint left in grad_x is requested first and added last, so that its latency hides behind the sums
      const int groups = (Ci + 1) / 2;
      for (int e = threadIdx.x; e < groups * (kTP / 4); e += blockDim.x) {
        const int gi = e / (kTP / 4), q = e % (kTP / 4);
        if (4 * q >= np) continue;
        const int i0g = 2 * gi;
        const bool two = i0g + 1 < Ci;
        float4* d0 = reinterpret_cast<float4*>(gx + (b * Ci + i0g) * P + p0) + q;
        float4* d1 = reinterpret_cast<float4*>(gx + (b * Ci + i0g + (two ? 1 : 0)) * P + p0) + q;
        const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
        const float4 old0 = want_gx == 1 ? *d0 : zero4;          // 1: add to what is there, 2: assign
        const float4 old1 = (two && want_gx == 1) ? *d1 : zero4;
        float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
        for (int o = 0; o < Co; ++o) {
          const float4 gv = reinterpret_cast<const float4*>(gz_s + o * kTS)[q];
          const float w0 = wb_s[o * Ci + i0g], w1 = two ? wb_s[o * Ci + i0g + 1] : 0.f;
          a0.x = fmaf(w0, gv.x, a0.x);
          a0.y = fmaf(w0, gv.y, a0.y);
          a0.z = fmaf(w0, gv.z, a0.z);
          a0.w = fmaf(w0, gv.w, a0.w);
          a1.x = fmaf(w1, gv.x, a1.x);
          a1.y = fmaf(w1, gv.y, a1.y);
          a1.z = fmaf(w1, gv.z, a1.z);
          a1.w = fmaf(w1, gv.w, a1.w);
        }
        __stcs(d0, make_float4(old0.x + a0.x, old0.y + a0.y, old0.z + a0.z, old0.w + a0.w));
        if (two) __stcs(d1, make_float4(old1.x + a1.x, old1.y + a1.y, old1.z + a1.z, old1.w + a1.w));
      }
    }
  }
  if (want_gw) {
    // add the point groups in ascending order through shared memory (the staged tiles are no longer needed)
    __syncthreads();
    float* red = gz_s;                                  // [npg][blocks][16] floats <= 256 * 16
    if (gw_thread) {
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < 4; ++c) red[(pg * blocks + blk) * 16 + 4 * a + c] = acc[a][c];
    }
    __syncthreads();
    const int pairs = Co * Ci;
    for (int pr = threadIdx.x; pr < pairs; pr += blockDim.x) {
      const int o = pr / Ci, i = pr % Ci;
      const int bk = (o / 4) * ib_n + (i / 4), el = 4 * (o % 4) + (i % 4);
      float s = 0.f;
      for (int g = 0; g < npg; ++g) s += red[(g * blocks + bk) * 16 + el];
      partial[(long long)blockIdx.x * (pairs + Co) + pr] = s;
    }
    if (want_gb) {
      __syncthreads();
      if (gw_thread && i0 == 0) {
#pragma unroll
        for (int a = 0; a < 4; ++a) red[pg * 4 * ob_n + (o0 + a)] = bsum[a];
      }
      __syncthreads();
      for (int o = threadIdx.x; o < Co; o += blockDim.x) {
        float s = 0.f;
        for (int g = 0; g < npg; ++g) s += red[g * 4 * ob_n + o];
        partial[(long long)blockIdx.x * (pairs + Co) + pairs + o] = s;
      }
    }
  }
}

// grad_Wb[pair] = sum over CTAs (ascending) of partial[cta][pair]
// (entries [pairs, pairs + n_bias) of a row are the bias gradient)
__global__ void __launch_bounds__(256) reduce_wb_kernel(const float* __restrict__ partial, float* __restrict__ gWb,
                                                       float* __restrict__ gb, int pairs, int n_bias, int ctas) {
  pdl_trigger();
  pdl_wait();
  const int pr = blockIdx.x * blockDim.x + threadIdx.x;
  const int row = pairs + n_bias;
  if (pr >= row) return;
  float s = 0.f;
  for (int c = 0; c < ctas; ++c) s += partial[(long long)c * row + pr];
  if (pr < pairs) {
    if (gWb) gWb[pr] = s;
  } else if (gb) {
    gb[pr - pairs] = s;
  }
}

}  // namespace

bool block_supported(int Ci, int Co, long long P) {
  return P % 4 == 0 && ((Ci + 3) / 4) * ((Co + 3) / 4) <= 256 && Ci + Co <= 64 && (size_t)(((Ci * Co + 3) & ~3) + (Ci + Co) * kTS) * 4 <= 200 * 1024;
}

static cudaError_t launch_epilogue_any(bool linear, const float* x, float* out, float* z, const float* Wb, int B, int Ci,
                                       int Co, long long P, cudaStream_t st) {
  const long long total = (long long)B * (P / 4);
  if (total <= 0) return cudaSuccess;
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)num_sms() * 8;
  if (blocks > cap) blocks = cap;
  const size_t smem = (size_t)Ci * Co * 4;
  cudaError_t e = cudaSuccess;
#define DTST_REGX(ci, v)                                                                                           \
  if (Ci == ci) {                                                                                                  \
    auto k2 = linear ? block_epilogue_regx_kernel<true, ci, v> : block_epilogue_regx_kernel<false, ci, v>;         \
    if (smem > 48 * 1024) e = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);    \
    if (e != cudaSuccess) return e;                                                                                \
    long long bl = ((long long)B * (P / v) + 255) / 256;                                                           \
    if (bl > cap) bl = cap;                                                                                        \
    (void)launch_pdl(k2, dim3((unsigned)bl), dim3(256), smem, st, x, out, z, Wb, B, Co, P);                        \
    return cudaGetLastError();                                                                                     \
  }
  DTST_REGX(3, 4)
  DTST_REGX(4, 4)
  DTST_REGX(5, 4)
  DTST_REGX(8, 4)
  DTST_REGX(16, 4)
  DTST_REGX(20, 4)
  DTST_REGX(32, 2)
#undef DTST_REGX
  auto kern = linear ? block_epilogue_kernel<true> : block_epilogue_kernel<false>;
  if (smem > 48 * 1024) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  (void)launch_pdl(kern, dim3((unsigned)blocks), dim3(256), smem, st, x, out, z, Wb, B, Ci, Co, P);
  return cudaGetLastError();
}

cudaError_t launch_block_epilogue(const float* x, float* out, float* z, const float* Wb, int B, int Ci, int Co,
                                  long long P, cudaStream_t st) {
  return launch_epilogue_any(false, x, out, z, Wb, B, Ci, Co, P, st);
}

cudaError_t launch_pointwise_linear(const float* x, float* out, const float* bias, const float* W, int B, int Ci,
                                    int Co, long long P, cudaStream_t st) {
  return launch_epilogue_any(true, x, out, const_cast<float*>(bias), W, B, Ci, Co, P, st);
}

cudaError_t launch_gelu_backward(const float* g, const float* z, float* gz, long long n, cudaStream_t st) {
  const long long n4 = n / 4;
  if (n4 <= 0) return cudaSuccess;
  long long blocks = (n4 + 255) / 256;
  const long long cap = (long long)num_sms() * 16;
  if (blocks > cap) blocks = cap;
  (void)launch_pdl(gelu_backward_kernel, dim3((unsigned)blocks), dim3(256), 0, st, reinterpret_cast<const float4*>(g),
                   reinterpret_cast<const float4*>(z), reinterpret_cast<float4*>(gz), n4);
  return cudaGetLastError();
}

// mode_gx: 0 = no input gradient, 1 = add it to gx, 2 = assign it.  gb (optional): the sum of gz over batch and points
// per output channel.  `partial` holds kBlockPartialRows rows of C_in * C_out + C_out floats.
cudaError_t launch_linear_backward(const float* gz, const float* x, float* gx, int mode_gx, const float* Wb, float* gWb,
                                   float* gb, float* partial, int B, int Ci, int Co, long long P, cudaStream_t st,
                                   long long* launches) {
  const long long tiles = (long long)B * ((P + kTP - 1) / kTP);
  if (tiles <= 0) return cudaSuccess;
  if (linear_backward_mma_supported(Ci, Co, P)) {
    // up to 32 channels per side, 20 or more together: both products on the tensor cores (dtst_block_mma.cu)
    const int want = (gWb != nullptr || gb != nullptr) ? 1 : 0;
    int rows = 0;
    cudaError_t em = launch_linear_backward_mma(gz, x, gx, gx != nullptr ? mode_gx : 0, Wb, partial, B, Ci, Co, P, want,
                                                gb != nullptr ? 1 : 0, kBlockPartialRows, &rows, st);
    if (em != cudaSuccess) return em;
    if (launches) ++*launches;
    if (want) {
      const int pairs = Ci * Co;
      (void)launch_pdl(reduce_wb_kernel, dim3((unsigned)((pairs + Co + 255) / 256)), dim3(256), 0, st,
                       static_cast<const float*>(partial), gWb, gb, pairs, Co, rows);
      if (launches) ++*launches;
    }
    return cudaGetLastError();
  }
  size_t smem = (size_t)(((Ci * Co + 3) & ~3) + (Ci + Co) * kTS) * 4;
  const size_t red_bytes = (size_t)(((Ci * Co + 3) & ~3) + 256 * 16) * 4;   // the final reduction's scratch
  if (smem < red_bytes) smem = red_bytes;
  cudaError_t e = cudaSuccess;
  if (smem > 48 * 1024) e = cudaFuncSetAttribute(bypass_backward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int per_sm = 1;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bypass_backward_kernel, 256, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) per_sm = 1;
  long long ctas = (long long)num_sms() * per_sm;
  if (ctas > kBlockPartialRows) ctas = kBlockPartialRows;
  if (ctas > tiles) ctas = tiles;
  const int want_gw = (gWb != nullptr || gb != nullptr) ? 1 : 0;
  (void)launch_pdl(bypass_backward_kernel, dim3((unsigned)ctas), dim3(256), smem, st, gz, x, gx, Wb, partial, B, Ci, Co, P,
                   gx != nullptr ? mode_gx : 0, want_gw, gb != nullptr ? 1 : 0);
  if (launches) ++*launches;
  if (want_gw) {
    const int pairs = Ci * Co;
    (void)launch_pdl(reduce_wb_kernel, dim3((unsigned)((pairs + Co + 255) / 256)), dim3(256), 0, st,
                     static_cast<const float*>(partial), gWb, gb, pairs, Co, (int)ctas);
    if (launches) ++*launches;
  }
  return cudaGetLastError();
}

cudaError_t launch_bypass_backward(const float* gz, const float* x, float* gx, const float* Wb, float* gWb,
                                   float* partial, int B, int Ci, int Co, long long P, cudaStream_t st,
                                   long long* launches) {
  return launch_linear_backward(gz, x, gx, 1, Wb, gWb, nullptr, partial, B, Ci, Co, P, st, launches);
}

}  // namespace dtst
