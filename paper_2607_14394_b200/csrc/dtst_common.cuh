// Shared declarations of the DTST CUDA library: the plan object, the description
// of one per-dimension contraction, and the on-device basis generator.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <stddef.h>

#include "../../include/dtst.h"

namespace dtst {

constexpr int kMaxDims = DTST_MAX_DIMS;
constexpr int kFallbackSMs = 148;            // B200; used only if the attribute query fails
constexpr size_t kStatusBytes = 256;         // head of the workspace: device status word

// One application of a (generated) complex matrix E[R x Q] along one dimension of
// a tensor viewed as [slab][outer][Q][inner] -> [slab][outer][R][inner].
//   forward (Eq. 18):  r = position in the retained list, q = local grid index,
//                      E[r][q] = w * exp(-2 pi i s(r) (offset + q) / N)
//   expand  (B^H):     r = local grid index, q = position in the retained list,
//                      E[r][q] = w * exp(+2 pi i s(q) (offset + r) / N)
// w = scale * (herm ? c(f) : 1) with c the Hermitian doubling weight of the
// one-sided dimension (1 at f = 0 and Nyquist, else 2).
struct DimOp {
  long long outer, inner;
  int Q, R;
  int N;            // global extent of this dimension
  int k;            // retained modes parameter
  int two_sided;    // 1: list [0..k-1, N-k..N-1]; 0: [0..k-1]
  int offset;       // global index of local element 0 (slab 0)
  int offset_step;  // added per slab
  int forward;      // 1: contraction grid -> modes; 0: expansion modes -> grid
  int herm;         // apply c(f) (only meaningful on the one-sided dimension)
  float scale;
  int slabs;        // blockIdx.y range
  long long in_outer_stride, out_outer_stride;   // in elements of the respective type
  long long in_slab_stride, out_slab_stride;
  int basis_in_smem;
  int es_sr, es_sq;    // shared-memory basis: entry (r, q) sits at r * es_sr + q * es_sq (set by the launcher)
};

// Number of SMs of the current device (persistent kernels launch one CTA per SM, or a multiple): queried
// once per device and cached.
inline int num_sms() {
  static int cache[64] = {};   // 0 = not yet queried; a racing first query writes the same value twice
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    (void)cudaGetLastError();
    return kFallbackSMs;
  }
  int n = cache[dev];
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
      (void)cudaGetLastError();
      n = kFallbackSMs;
    }
    cache[dev] = n;
  }
  return n;
}

// Retained DFT index at position pos of a dimension's list.
__host__ __device__ inline int mode_at(int pos, int k, int N, int two_sided) {
  return (!two_sided || pos < k) ? pos : N - 2 * k + pos;
}

// Hermitian doubling weight of one-sided frequency f.
__host__ __device__ inline float herm_weight(int f, int N) {
  return (f == 0 || 2 * f == N) ? 1.0f : 2.0f;
}

#ifdef __CUDACC__
// Programmatic dependent launch.  Every kernel of the library is launched with the programmatic-serialisation
// attribute and follows one protocol: `pdl_trigger()` first thing (the next kernel of the stream may then be
// scheduled as soon as SMs free up), then the prologue that touches nothing a predecessor produced (basis
// tables from (N, k, offset), barrier set-up, tensor-map prefetch), then `pdl_wait()` - reached by EVERY thread of
// every CTA, before its first global-memory access and before any early exit - which returns once the
// preceding kernel has completed and its writes are visible.  So a kernel's launch latency and table build hide
// behind its predecessor's tail; the data dependencies are exactly those of plain stream order.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  static const bool off = getenv("DTST_NO_PDL") != nullptr;
  cfg.numAttrs = off ? 0 : 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// exp(sign * 2 pi i * (s*n mod N) / N): the integer phase is reduced exactly before
// any floating-point operation, then evaluated in double and rounded once.
__device__ inline float2 twiddle(int s, long long n, int N, int sign) {
  long long r = ((long long)s * n) % (long long)N;
  double sn, cs;
  sincospi(2.0 * (double)r / (double)N, &sn, &cs);
  return make_float2((float)cs, (float)(sign > 0 ? sn : -sn));
}

__device__ inline float2 dimop_entry(const DimOp& p, int r, int q, int slab) {
  const long long off = (long long)p.offset + (long long)slab * p.offset_step;
  int pos = p.forward ? r : q;
  long long n = off + (p.forward ? q : r);
  int s = mode_at(pos, p.k, p.N, p.two_sided);
  float2 e = twiddle(s, n, p.N, p.forward ? -1 : +1);
  float w = p.scale * (p.herm ? herm_weight(s, p.N) : 1.0f);
  e.x *= w;
  e.y *= w;
  return e;
}
#endif

}  // namespace dtst

struct dtst_host_io;   // streams, events and staging offsets of dtst_step_host (dtst_hostio.cu)

// The plan: pure host-side configuration plus a caller-owned workspace pointer.
struct dtst_plan {
  int d;
  int B, C_in, C_out;
  long long Ng[dtst::kMaxDims];    // global extents
  long long Nl[dtst::kMaxDims];    // local extents
  long long off[dtst::kMaxDims];   // global offsets
  int kmax[dtst::kMaxDims];
  int K[dtst::kMaxDims];           // retained entries per dim
  long long M;                     // prod K
  long long points_local;          // prod Nl
  long long points_global;         // prod Ng
  int P;                           // virtual shards along dim 0
  int path_request;                // DTST_PATH_*
  int device;                      // CUDA device at creation, -1 if none
  void* ws;
  size_t ws_bytes;
  long long launches;
  int last_cuda_error;             // cudaError_t of the last failing runtime call / launch
  unsigned dbg_poll_limit;         // 0 = default budget of the bounded waits
  long long dbg_withhold_after;    // < 0 = off (the default)
  dtst_host_io* host_io;           // non-null after dtst_plan_enable_host_io
  int colfuse;                     // third dimension inside the forward plane kernel: 0 auto, 1 whenever built, -1 never
  int fast_math;                   // single-pass TF32 in the kernels for any extent (dtst_plan_set_arithmetic)
  int order_rank[dtst::kMaxDims];  // contraction order of the dimensions behind the grid-side kernel: lower = earlier
  int complex_io;                  // 1: complex fields, two-sided retained set on the last dimension too
  int block_epilogue;              // DTST_BLOCK_EPILOGUE_*
  int require_fast;                // 1: compute calls refuse to run if any stage would take the generic kernel
  int colexp_ring;                 // > 0: expand the dimension in front of the plane inside the inverse plane kernel
  // optional per-kernel event timing (benchmarks only)
  int timing_cap;
  int timing_n[DTST_KERNEL_KINDS];
  cudaEvent_t* timing_ev[DTST_KERNEL_KINDS][2];
};

namespace dtst {

// Poll budget of the bounded device-side waits and the diagnostic that makes one of them run out
// (dtst_plan_debug_ring_fault): the producer of the forward plane kernel's ring stops after `withhold_after` fills.
struct RingDebug {
  uint32_t poll_limit;        // polls before a wait gives up
  long long withhold_after;   // < 0: never withhold
};
constexpr uint32_t kDefaultPollLimit = 1u << 24;

struct WsLayout {
  size_t status, bufA, bufB, partial, gy, gx, counters, wb_partial, total;
  size_t szA, szB, szPartial, szG, szCounters, szWbPartial;
};

constexpr int kBlockPartialRows = 1024;   // most CTAs the bypass weight-gradient reduction is spread over

bool fused_eligible(const dtst_plan* p);
void host_io_release(dtst_plan* p);

// Brackets one kernel launch with events when timing is enabled (no-ops otherwise).
struct KernelTimer {
  dtst_plan* p;
  int kind, slot;
  cudaStream_t st;
  KernelTimer(dtst_plan* plan, int kind_, cudaStream_t st_, bool enabled = true)
      : p(plan), kind(kind_), slot(-1), st(st_) {
    if (enabled && p->timing_cap > 0 && p->timing_n[kind] < p->timing_cap) {
      slot = p->timing_n[kind]++;
      cudaEventRecord(p->timing_ev[kind][0][slot], st);
    }
  }
  ~KernelTimer() {
    if (slot >= 0) cudaEventRecord(p->timing_ev[kind][1][slot], st);
  }
};

WsLayout ws_layout(const dtst_plan* p);

// generic kernels (dtst_generic.cu)
cudaError_t launch_apply_dim(const DimOp& op, bool in_real, bool out_real, const void* in, void* out,
                             cudaStream_t st);
cudaError_t launch_reduce_partials(const float2* partial, float2* out, long long n, int P, cudaStream_t st);
cudaError_t launch_mix(const float2* X, const float2* W, float2* Y, int B, int Ci, int Co, long long M,
                       cudaStream_t st, long long* launches);
cudaError_t launch_mix_modes(const float2* X, const float2* W, float2* Y, int B, int Ci, int Co, long long M,
                             long long m0, long long cnt, cudaStream_t st, long long* launches);
cudaError_t launch_mix_adjoint_modes(const float2* GY, const float2* X, const float2* W, float2* GX, float2* GW,
                                     int B, int Ci, int Co, long long M, long long m0, long long cnt,
                                     cudaStream_t st, long long* launches);
cudaError_t launch_mix_adjoint(const float2* GY, const float2* X, const float2* W, float2* GX, float2* GW,
                               int B, int Ci, int Co, long long M, cudaStream_t st, long long* launches);

// the block around the layer: bypass + GELU and their backward pass (dtst_block.cu)
bool block_supported(int Ci, int Co, long long P);
cudaError_t launch_block_epilogue(const float* x, float* out, float* z, const float* Wb, int B, int Ci, int Co,
                                  long long P, cudaStream_t st);
cudaError_t launch_pointwise_linear(const float* x, float* out, const float* bias, const float* W, int B, int Ci,
                                    int Co, long long P, cudaStream_t st);
cudaError_t launch_linear_backward(const float* gz, const float* x, float* gx, int mode_gx, const float* Wb, float* gWb,
                                   float* gb, float* partial, int B, int Ci, int Co, long long P, cudaStream_t st,
                                   long long* launches);
cudaError_t launch_gelu_backward(const float* g, const float* z, float* gz, long long n, cudaStream_t st);
// Tensor-core version of the pass below for up to 32 channels per side (at least 20 together) and points % 128 == 0
// (dtst_block_mma.cu);
// *ctas_out = rows of `partial` written.
bool linear_backward_mma_supported(int Ci, int Co, long long P);
cudaError_t launch_linear_backward_mma(const float* gz, const float* x, float* gx, int mode_gx, const float* Wb,
                                       float* partial, int B, int Ci, int Co, long long P, int want_gw, int want_gb,
                                       int max_ctas, int* ctas_out, cudaStream_t st);
cudaError_t launch_bypass_backward(const float* gz, const float* x, float* gx, const float* Wb, float* gWb,
                                   float* partial, int B, int Ci, int Co, long long P, cudaStream_t st,
                                   long long* launches);

// offset / virtual-shard kernels for a two-sided middle dimension (dtst_slab.cu)
bool slab_supported(int Nl, int K);
// (fast: single-pass TF32 where the stage runs on the kernels of dtst_midg.cu; the others are not affected)
cudaError_t launch_slab(bool forward, int K, const float2* in, float2* out, long long outer, long long inner, int Nl,
                        int N, int off, int P, bool fast, cudaStream_t st);

// folded kernels for a two-sided middle dimension: tensor-core version (dtst_midmma.cu) where the shape allows,
// else the FFMA register-accumulator version (dtst_mid.cu)
bool mid_supported(int N, int K);
// tensor-core variant of the middle-dimension kernels (N % 32 == 0, inner % 4 == 0)
// folded tensor-core kernels for any extent and any mode count up to 32 (dtst_midg.cu)
bool midg_supported(int N, int K);
cudaError_t launch_midg(bool forward, int K, const float2* in, float2* out, long long outer, long long inner, int N,
                        float scale, bool fast, cudaStream_t st);
// ... for Nl local rows that start at global index `off` of an extent Ng (a rank's block; virtual slabs taken together)
bool midg_local_supported(int Nl, int K);
cudaError_t launch_midg_local(bool forward, int K, const float2* in, float2* out, long long outer, long long inner, int Nl,
                              int Ng, int off, float scale, bool fast, cudaStream_t st);
bool mid_mma_supported(int N, int K, long long inner);
cudaError_t launch_mid_mma(bool forward, int K, const float2* in, float2* out, long long outer, long long inner, int N,
                           float scale, cudaStream_t st);
cudaError_t launch_mid(bool forward, int K, const float2* in, float2* out, long long outer, long long inner, int N,
                       float scale, bool fast, cudaStream_t st);

}  // namespace dtst
