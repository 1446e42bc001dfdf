// C ABI of the DTST library: plan handling, argument validation and the
// sequencing of kernels for each call.  No arithmetic of the method lives here.
#include <cstdlib>
#include <cstring>
#include <new>

#include "dtst_common.cuh"
#include "dtst_fused.cuh"

using namespace dtst;

namespace {

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

// Records a failing CUDA call in the plan; true when the call failed.
inline bool cuda_failed(dtst_plan* p, cudaError_t e) {
  if (e == cudaSuccess) return false;
  p->last_cuda_error = (int)e;
  (void)cudaGetLastError();
  return true;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// elements of the tensor after the forward stages d-1..j have run (complex)
long long fwd_stage_elems(const dtst_plan* p, int j, int Cn) {
  long long n = (long long)p->B * Cn;
  for (int i = 0; i < j; ++i) n *= p->Nl[i];
  for (int i = j; i < p->d; ++i) n *= p->K[i];
  return n;
}

bool mul_overflows(long long a, long long b) {
  if (a == 0 || b == 0) return false;
  return a > INT64_MAX / b;
}

dtst_status create_common(dtst_plan** out, int d, const int64_t* Ng, const int64_t* Nl, const int64_t* off,
                          const int32_t* kmax, int B, int C_in, int C_out, bool complex_io = false) {
  if (out == nullptr) return DTST_ERR_INVALID_ARG;
  *out = nullptr;
  if (Ng == nullptr || kmax == nullptr || d < 1 || d > kMaxDims) return DTST_ERR_INVALID_ARG;
  if (B < 1 || C_in < 1 || C_out < 1) return DTST_ERR_INVALID_ARG;
  long long pts_l = 1, pts_g = 1, M = 1;
  for (int j = 0; j < d; ++j) {
    const long long ng = Ng[j];
    const long long nl = Nl ? Nl[j] : ng;
    const long long o = off ? off[j] : 0;
    if (ng < 1 || ng > (1ll << 30) || nl < 1 || o < 0 || o + nl > ng) return DTST_ERR_INVALID_ARG;
    const long long k = kmax[j];
    if (k < 1) return DTST_ERR_INVALID_ARG;
    if (j < d - 1 || complex_io) {
      if (2 * k > ng) return DTST_ERR_INVALID_ARG;     // the two halves of S_j must not overlap
    } else {
      if (k > ng / 2 + 1) return DTST_ERR_INVALID_ARG; // one-sided: at most up to Nyquist
    }
    const long long K = (j < d - 1 || complex_io) ? 2 * k : k;
    if (mul_overflows(pts_l, nl) || mul_overflows(pts_g, ng) || mul_overflows(M, K)) return DTST_ERR_INVALID_ARG;
    pts_l *= nl;
    pts_g *= ng;
    M *= K;
  }
  const long long cmax = C_in > C_out ? C_in : C_out;
  if (mul_overflows(pts_l, (long long)B * cmax) || pts_l * B * cmax > (1ll << 46)) return DTST_ERR_INVALID_ARG;
  if (mul_overflows(M, (long long)C_in * C_out) || M * C_in * C_out > (1ll << 46)) return DTST_ERR_INVALID_ARG;

  dtst_plan* p = new (std::nothrow) dtst_plan;
  if (p == nullptr) return DTST_ERR_ALLOC;
  std::memset(p, 0, sizeof(*p));
  p->d = d;
  p->B = B;
  p->C_in = C_in;
  p->C_out = C_out;
  for (int j = 0; j < d; ++j) {
    p->Ng[j] = Ng[j];
    p->Nl[j] = Nl ? Nl[j] : Ng[j];
    p->off[j] = off ? off[j] : 0;
    p->kmax[j] = kmax[j];
    p->K[j] = (j < d - 1 || complex_io) ? 2 * kmax[j] : kmax[j];
  }
  p->M = M;
  p->points_local = pts_l;
  p->points_global = pts_g;
  p->P = 1;
  p->path_request = DTST_PATH_AUTO;
  for (int j = 0; j < kMaxDims; ++j) p->order_rank[j] = d - 1 - j;   // default: d-2 first, dimension 0 last
  p->dbg_withhold_after = -1;
  p->complex_io = complex_io ? 1 : 0;
  p->device = -1;
  int dev = -1;
  if (cudaGetDevice(&dev) == cudaSuccess) p->device = dev;
  (void)cudaGetLastError();   // a machine without a GPU may still build plans (host logic only)
  *out = p;
  return DTST_OK;
}

// A two-sided dimension that is whole on this device, starts at global index 0 and is not cut into
// virtual slabs can use the folded middle-dimension kernels.
bool use_mid(const dtst_plan* p, int j) {
  if (p->path_request != DTST_PATH_AUTO || j >= p->d - 1) return false;
  if (p->Nl[j] != p->Ng[j] || p->off[j] != 0) return false;
  if (j == 0 && p->P > 1) return false;
  return mid_supported((int)p->Ng[j], p->kmax[j]);
}

// Expansion of such a dimension: virtual slabs change nothing here - slab p's rows are the rows [p nl, (p+1) nl) of
// the plain expansion (same global phases, no reduction between slabs), so the folded kernel serves them too.
bool use_mid_expand(const dtst_plan* p, int j) {
  if (p->path_request != DTST_PATH_AUTO || j >= p->d - 1) return false;
  if (p->Nl[j] != p->Ng[j] || p->off[j] != 0) return false;
  return mid_supported((int)p->Ng[j], p->kmax[j]);
}

// A two-sided dimension that carries a phase offset, is only partly local, or is cut into virtual slabs.
bool use_slab(const dtst_plan* p, int j) {
  if (p->path_request != DTST_PATH_AUTO || j >= p->d - 1 || use_mid(p, j)) return false;
  return slab_supported((int)p->Nl[j], p->kmax[j]);
}

// (the plane and row kernels read a REAL grid: complex plans take the generic kernel on the contiguous dimension)
bool use_fused(const dtst_plan* p) { return p->path_request == DTST_PATH_AUTO && !p->complex_io && fused_eligible(p); }

// Row kernels: the contiguous dimension alone (whole on this device, zero offset), for shapes without a
// plane kernel; the other dimensions then run on the reduced tensor.
bool use_row(const dtst_plan* p) {
  if (p->path_request != DTST_PATH_AUTO || p->complex_io || use_fused(p)) return false;
  const int a = p->d - 1;
  if (p->Nl[a] != p->Ng[a] || p->off[a] != 0) return false;
  if (p->d == 1 && p->P > 1) return false;
  long long rows = (long long)p->B * (p->C_in > p->C_out ? p->C_in : p->C_out);
  for (int i = 0; i < a; ++i) rows *= p->Nl[i];
  if (row_supported((int)p->Ng[a], p->kmax[a])) return rows < (1ll << 31);   // 32-bit TMA coordinates
  // any extent up to 512: the cp.async-fed kernels of dtst_rowg.cu; longer rows: the chunked ones of dtst_rowl.cu
  return rowg_supported((int)p->Ng[a], p->kmax[a]) || rowl_supported((int)p->Ng[a], p->kmax[a]);
}

// Row path with the second-last dimension inside the grid-side kernel (dtst_rowg.cu): for contiguous extents the
// tensor-map row kernels do not take, when that dimension is whole, carries no offset and is not cut into slabs.
bool use_planeg(const dtst_plan* p) {
  static const bool off = std::getenv("DTST_NO_PLANEG") != nullptr;   // diagnostic: keep the separate stage
  if (off || !use_row(p) || p->d < 2) return false;
  const int a = p->d - 1, b = p->d - 2;
  if (row_supported((int)p->Ng[a], p->kmax[a])) return false;
  if (p->Nl[b] != p->Ng[b] || p->off[b] != 0 || (b == 0 && p->P > 1)) return false;
  return planeg_supported((int)p->Ng[a], p->kmax[a], (int)p->Ng[b], p->kmax[b]);
}

// True when no stage of any transform of this plan falls back to the generic one-thread-per-output kernel: the
// grid-side stage runs on a plane or row kernel and every other dimension on a folded or slab kernel, in both
// directions.
bool all_streaming(const dtst_plan* p) {
  if (p->complex_io) return false;   // the contiguous dimension of a complex plan runs on the generic kernel
  int first;
  if (use_fused(p)) first = p->d - 3;
  else if (use_row(p)) first = use_planeg(p) ? p->d - 3 : p->d - 2;
  else return false;
  for (int j = first; j >= 0; --j) {
    if (!(use_slab(p, j) || use_mid(p, j))) return false;          // contraction
    if (!(use_mid_expand(p, j) || use_slab(p, j))) return false;   // expansion
  }
  return true;
}

// The dimensions 0..j_top in the order the forward transform contracts them (the expansion walks it backwards):
// ascending rank, the plan's contraction order (dtst_plan_set_contraction_order; default d-2, d-3, .., 0).
int middle_order(const dtst_plan* p, int j_top, int* out) {
  int n = 0;
  for (int j = 0; j <= j_top; ++j) out[n++] = j;
  for (int a = 1; a < n; ++a)          // insertion sort by rank
    for (int b = a; b > 0 && p->order_rank[out[b]] < p->order_rank[out[b - 1]]; --b) {
      const int t = out[b];
      out[b] = out[b - 1];
      out[b - 1] = t;
    }
  return n;
}

// The stages of a transform that starts on the grid itself, in forward order (an expansion walks it backwards).
// Real plans contract the contiguous dimension first: it carries the rfft fold and it is the stage the streaming
// kernels exist for.  Complex plans have no streaming kernel for it, so they contract it LAST - on the most reduced
// tensor, where the generic kernel that serves it touches a few percent of the bytes - and the folded kernels of the
// other dimensions stream the grid (their inner extent then contains the whole contiguous dimension: coalesced).
// Dimension 0 still closes the list when it carries virtual shards (its slab partials are summed after it).
int grid_order(const dtst_plan* p, int* out) {
  const int d = p->d;
  if (!p->complex_io) {
    out[0] = d - 1;
    return 1 + (d >= 2 ? middle_order(p, d - 2, out + 1) : 0);
  }
  int n = d >= 2 ? middle_order(p, d - 2, out) : 0;
  if (n > 0 && p->P > 1 && out[n - 1] == 0) {
    out[n - 1] = d - 1;
    out[n++] = 0;
  } else {
    out[n++] = d - 1;
  }
  return n;
}

// complex elements of a tensor in which dimension i has its retained entries (contracted[i]) or its local grid extent
long long state_elems(const dtst_plan* p, int Cn, const bool* contracted) {
  long long n = (long long)p->B * Cn;
  for (int i = 0; i < p->d; ++i) n *= contracted[i] ? p->K[i] : p->Nl[i];
  return n;
}

// One per-dimension operation on a tensor whose other dimensions are in the state `contracted` says.
DimOp make_op(const dtst_plan* p, int j, bool forward, int Cn, const bool* contracted) {
  DimOp op;
  std::memset(&op, 0, sizeof(op));
  long long outer = (long long)p->B * Cn;
  for (int i = 0; i < j; ++i) outer *= contracted[i] ? p->K[i] : p->Nl[i];
  long long inner = 1;
  for (int i = j + 1; i < p->d; ++i) inner *= contracted[i] ? p->K[i] : p->Nl[i];
  op.outer = outer;
  op.inner = inner;
  op.Q = forward ? (int)p->Nl[j] : p->K[j];
  op.R = forward ? p->K[j] : (int)p->Nl[j];
  op.N = (int)p->Ng[j];
  op.k = p->kmax[j];
  op.two_sided = (j < p->d - 1 || p->complex_io) ? 1 : 0;
  op.offset = (int)p->off[j];
  op.offset_step = 0;
  op.forward = forward ? 1 : 0;
  op.herm = 0;
  op.scale = 1.0f;
  op.slabs = 1;
  op.in_outer_stride = (long long)op.Q * inner;
  op.out_outer_stride = (long long)op.R * inner;
  op.in_slab_stride = 0;
  op.out_slab_stride = 0;
  return op;
}

// Forward stages on `cur`: the last dimension first when j_from == d-1 (then `cur` is the grid itself), then the
// dimensions 0..min(j_from, d-2) in the plan's contraction order, ping-ponging through the workspace; the result
// lands in Xhat.  scale/herm apply on the last dimension's stage only.
dtst_status forward_stages(dtst_plan* p, const void* cur, int j_from, int flip, float2* Xhat, int Cn,
                           float scale, bool herm, cudaStream_t st) {
  const WsLayout L = ws_layout(p);
  char* ws = static_cast<char*>(p->ws);
  float2* buf[2] = {reinterpret_cast<float2*>(ws + L.bufA), reinterpret_cast<float2*>(ws + L.bufB)};
  float2* partial = reinterpret_cast<float2*>(ws + L.partial);
  int list[kMaxDims + 1];
  const int n = j_from == p->d - 1 ? grid_order(p, list) : middle_order(p, j_from, list);
  bool contracted[kMaxDims];
  for (int i = 0; i < p->d; ++i) contracted[i] = i > j_from;
  bool need_reduce = false;
  for (int idx = 0; idx < n; ++idx) {
    const int j = list[idx];
    const bool last = idx == n - 1;
    DimOp op = make_op(p, j, true, Cn, contracted);
    contracted[j] = true;
    const bool in_real = (j == p->d - 1) && !p->complex_io;
    if (j == p->d - 1) {
      op.scale = scale;
      op.herm = herm ? 1 : 0;
    }
    if (!in_real && use_slab(p, j)) {
      // slabs (or a rank's block) of this dimension: partial spectra formed and summed inside one kernel
      void* sdst = last ? static_cast<void*>(Xhat) : static_cast<void*>(buf[flip]);
      if (cuda_failed(p, launch_slab(true, p->kmax[j], static_cast<const float2*>(cur), static_cast<float2*>(sdst),
                                     op.outer, op.inner, (int)p->Nl[j], op.N, (int)p->off[j], j == 0 ? p->P : 1, p->fast_math != 0, st)))
        return DTST_ERR_CUDA;
      ++p->launches;
      cur = sdst;
      flip ^= 1;
      continue;
    }
    void* dst;
    if (j == 0 && p->P > 1) {
      // slab p contracts rows [p*nl, (p+1)*nl) of dim 0 with its own phase offset (Eq. 6, Eq. 18); the P partial
      // spectra are summed afterwards, so this stage is the last one (the contraction order guarantees it)
      const int nl = (int)(p->Nl[0] / p->P);
      op.slabs = p->P;
      op.Q = nl;
      op.offset_step = nl;
      op.in_outer_stride = p->Nl[0] * op.inner;
      op.in_slab_stride = (long long)nl * op.inner;
      op.out_slab_stride = (long long)p->B * Cn * p->M;
      dst = partial;
      need_reduce = true;
    } else {
      dst = last ? static_cast<void*>(Xhat) : static_cast<void*>(buf[flip]);
    }
    if (!in_real && use_mid(p, j)) {
      if (cuda_failed(p, launch_mid(true, p->kmax[j], static_cast<const float2*>(cur), static_cast<float2*>(dst),
                                    op.outer, op.inner, op.N, 1.0f, p->fast_math != 0, st)))
        return DTST_ERR_CUDA;
    } else {
      KernelTimer kt(p, DTST_KERNEL_GRID_READ, st, in_real);
      if (cuda_failed(p, launch_apply_dim(op, in_real, false, cur, dst, st))) return DTST_ERR_CUDA;
    }
    ++p->launches;
    cur = dst;
    flip ^= 1;
  }
  if (need_reduce) {
    if (cuda_failed(p, launch_reduce_partials(partial, Xhat, (long long)p->B * Cn * p->M, p->P, st))) return DTST_ERR_CUDA;
    ++p->launches;
  }
  return DTST_OK;
}

// Generic forward-type transform: real grid tensor -> [B*Cn, M] spectrum.
dtst_status run_forward_generic(dtst_plan* p, const float* x, float2* Xhat, int Cn, float scale, bool herm,
                                cudaStream_t st) {
  return forward_stages(p, x, p->d - 1, 0, Xhat, Cn, scale, herm, st);
}

// Whether the forward plane kernel also contracts the dimension in front of the plane: that dimension must be the
// first of the middle stages in the plan's order, whole on this device, without offset and not cut into slabs.
bool use_fwd_col(const dtst_plan* p, int Cn) {
  const int d = p->d;
  if (d < 3 || !use_fused(p)) return false;
  const int c = d - 3;
  int list[kMaxDims];
  if (middle_order(p, c, list) < 1 || list[0] != c) return false;
  if (!use_mid(p, c)) return false;
  // a CTA takes whole columns: with few columns per CTA the last round is mostly idle (a rank's thin slab), and
  // the plain kernel, whose tasks are single planes, balances better than this one gains
  if (p->colfuse < 0) return false;
  if (p->colfuse == 0) {
    long long cols = (long long)p->B * Cn;
    for (int i = 0; i < c; ++i) cols *= p->Nl[i];
    const long long sms = num_sms(), rounds = (cols + sms - 1) / sms;
    if (cols * 100 < rounds * sms * 95) return false;
  }
  return fwd_plane_col_supported((int)p->Ng[d - 1], p->kmax[d - 1], (int)p->Ng[d - 2], p->kmax[d - 2], (int)p->Ng[c],
                                 p->kmax[c]);
}

// Fused forward: the plane kernel streams the grid once and contracts the last two dimensions;
// the remaining dimensions run on the reduced tensor.
dtst_status run_forward_fused(dtst_plan* p, const float* x, float2* Xhat, int Cn, float scale, bool herm,
                              cudaStream_t st) {
  const int d = p->d, a = d - 1, b = d - 2;
  const WsLayout L = ws_layout(p);
  char* ws = static_cast<char*>(p->ws);
  long long planes = (long long)p->B * Cn;
  for (int i = 0; i < b; ++i) planes *= p->Nl[i];
  float2* t1 = (d == 2) ? Xhat : reinterpret_cast<float2*>(ws + L.bufA);
  if (use_fwd_col(p, Cn)) {
    // the third dimension is contracted inside the plane kernel: no reduced tensor in HBM, one launch less
    const int c = d - 3;
    float2* dst = (d == 3) ? Xhat : t1;
    {
      KernelTimer kt(p, DTST_KERNEL_GRID_READ, st);
      const RingDebug dbg{p->dbg_poll_limit ? p->dbg_poll_limit : kDefaultPollLimit, p->dbg_withhold_after};
      if (cuda_failed(p, launch_fwd_plane_col((int)p->Ng[a], p->kmax[a], (int)p->Ng[b], p->kmax[b], (int)p->Ng[c],
                                              p->kmax[c], x, dst, planes * p->Ng[b], scale, herm ? 1 : 0,
                                              reinterpret_cast<int*>(ws + L.status), dbg, st)))
        return DTST_ERR_CUDA;
    }
    ++p->launches;
    if (d == 3) return DTST_OK;
    return forward_stages(p, t1, d - 4, 1, Xhat, Cn, 1.0f, false, st);
  }
  {
    KernelTimer kt(p, DTST_KERNEL_GRID_READ, st);
    const RingDebug dbg{p->dbg_poll_limit ? p->dbg_poll_limit : kDefaultPollLimit, p->dbg_withhold_after};
    if (cuda_failed(p, launch_fwd_plane((int)p->Ng[a], p->kmax[a], (int)p->Ng[b], p->kmax[b], x, t1, planes * p->Ng[b], scale,
                         herm ? 1 : 0, reinterpret_cast<int*>(ws + L.status), dbg, st))) return DTST_ERR_CUDA;
  }
  ++p->launches;
  if (d == 2) return DTST_OK;
  return forward_stages(p, t1, d - 3, 1, Xhat, Cn, 1.0f, false, st);
}

// One expansion stage (B^H along dimension j) from `cur` into `dst` with whichever kernel family serves it; the
// other dimensions are in the state `contracted` says.  The last dimension's stage writes the grid and carries the
// scale and the Hermitian weights.
dtst_status expand_stage(dtst_plan* p, int j, int Cn, const void* cur, void* dst, float scale, bool herm,
                         const bool* contracted, cudaStream_t st) {
  DimOp op = make_op(p, j, false, Cn, contracted);
  const bool out_real = (j == p->d - 1) && !p->complex_io;
  if (j == p->d - 1) {
    op.scale = scale;
    op.herm = herm ? 1 : 0;
  }
  const long long outer = op.outer, inner = op.inner;
  if (j == 0 && p->P > 1) {
    // slab p expands to rows [p*nl, (p+1)*nl) with the same offset phases; no reduction needed
    const int nl = (int)(p->Nl[0] / p->P);
    op.slabs = p->P;
    op.R = nl;
    op.offset_step = nl;
    op.out_outer_stride = p->Nl[0] * op.inner;
    op.out_slab_stride = (long long)nl * op.inner;
  }
  cudaError_t e;
  if (!out_real && use_mid_expand(p, j)) {
    e = launch_mid(false, p->kmax[j], static_cast<const float2*>(cur), static_cast<float2*>(dst), outer, inner,
                   (int)p->Ng[j], 1.0f, p->fast_math != 0, st);
  } else if (!out_real && use_slab(p, j)) {
    e = launch_slab(false, p->kmax[j], static_cast<const float2*>(cur), static_cast<float2*>(dst), outer, inner,
                    (int)p->Nl[j], (int)p->Ng[j], (int)p->off[j], j == 0 ? p->P : 1, p->fast_math != 0, st);
  } else {
    KernelTimer kt(p, DTST_KERNEL_GRID_WRITE, st, out_real);
    e = launch_apply_dim(op, false, out_real, cur, dst, st);
  }
  if (cuda_failed(p, e)) return DTST_ERR_CUDA;
  ++p->launches;
  return DTST_OK;
}

// Expansion of the dimensions 0..j_top (the forward contraction order walked backwards; `skip`, if >= 0, is left to
// the caller and must come last) on `cur`, ping-ponging through the workspace; returns the buffer holding the
// result through *out_buf (cur_in itself when nothing is expanded) and the number of stages through *stages.
dtst_status inverse_stages_complex(dtst_plan* p, const float2* cur_in, int j_top, int skip, int Cn,
                                   const float2** out_buf, int* stages, cudaStream_t st) {
  const WsLayout L = ws_layout(p);
  char* ws = static_cast<char*>(p->ws);
  float2* buf[2] = {reinterpret_cast<float2*>(ws + L.bufA), reinterpret_cast<float2*>(ws + L.bufB)};
  const void* cur = cur_in;
  int list[kMaxDims], n = j_top >= 0 ? middle_order(p, j_top, list) : 0;
  bool contracted[kMaxDims];
  for (int i = 0; i < p->d; ++i) contracted[i] = true;
  int flip = 0, done = 0;
  for (int idx = n - 1; idx >= 0; --idx) {
    const int j = list[idx];
    if (j == skip) continue;
    void* dst = buf[flip];
    const dtst_status s = expand_stage(p, j, Cn, cur, dst, 1.0f, false, contracted, st);
    if (s != DTST_OK) return s;
    contracted[j] = false;
    cur = dst;
    flip ^= 1;
    ++done;
  }
  *out_buf = static_cast<const float2*>(cur);
  if (stages) *stages = done;
  return DTST_OK;
}

// Generic expansion: [B*Cn, M] spectrum -> grid tensor (real, or complex for a complex plan): the stages of
// grid_order walked backwards through the ping-pong buffers, the last one writing the grid.
dtst_status run_inverse_generic(dtst_plan* p, const float2* Yhat, void* y, int Cn, float scale, bool herm,
                                cudaStream_t st) {
  const WsLayout L = ws_layout(p);
  char* ws = static_cast<char*>(p->ws);
  float2* buf[2] = {reinterpret_cast<float2*>(ws + L.bufA), reinterpret_cast<float2*>(ws + L.bufB)};
  int list[kMaxDims + 1];
  const int n = grid_order(p, list);
  bool contracted[kMaxDims];
  for (int i = 0; i < p->d; ++i) contracted[i] = true;
  const void* cur = Yhat;
  int flip = 0;
  for (int idx = n - 1; idx >= 0; --idx) {
    const int j = list[idx];
    void* dst = idx == 0 ? y : static_cast<void*>(buf[flip]);
    const dtst_status s = expand_stage(p, j, Cn, cur, dst, j == p->d - 1 ? scale : 1.0f, herm, contracted, st);
    if (s != DTST_OK) return s;
    contracted[j] = false;
    cur = dst;
    flip ^= 1;
  }
  return DTST_OK;
}

// The dimension in front of the plane can be expanded inside the inverse plane kernel by a helper warp
// (dtst_plan_set_column_expansion): when the caller asked for it, the dimension is whole on this device with zero
// offset, and the kernel is built for its shape.
bool use_colexp(const dtst_plan* p) {
  if (p->colexp_ring <= 0 || p->d < 3 || !use_fused(p)) return false;
  const int c = p->d - 3, a = p->d - 1, b = p->d - 2;
  if (!use_mid_expand(p, c)) return false;
  int list[kMaxDims];
  if (middle_order(p, c, list) < 1 || list[0] != c) return false;   // it must be the last dimension to be expanded
  return inv_plane_colexp_supported((int)p->Ng[a], p->kmax[a], (int)p->Ng[b], p->kmax[b], (int)p->Ng[c], p->kmax[c]);
}

// Fused expansion: stages for the leading dimensions on the small tensor, then the inverse plane kernel
// expands the last two dimensions and writes the grid once; where the shape allows, the dimension in front of
// them is expanded inside that kernel too.
dtst_status run_inverse_fused(dtst_plan* p, const float2* Yhat, float* y, int Cn, float scale, bool herm,
                              cudaStream_t st) {
  const int d = p->d, a = d - 1, b = d - 2;
  const bool colexp = use_colexp(p);
  const float2* src = Yhat;
  int stages = 0;
  if (d > 2) {
    dtst_status s = inverse_stages_complex(p, Yhat, d - 3, colexp ? d - 3 : -1, Cn, &src, &stages, st);
    if (s != DTST_OK) return s;
  }
  long long planes = (long long)p->B * Cn;
  for (int i = 0; i < b; ++i) planes *= p->Nl[i];
  const WsLayout L = ws_layout(p);
  char* ws = static_cast<char*>(p->ws);
  KernelTimer kt(p, DTST_KERNEL_GRID_WRITE, st);
  if (colexp) {
    const int c = d - 3;
    // the ping-pong buffer the separate expansion of dimension c would have written: its first ring_cols columns
    float2* ring = reinterpret_cast<float2*>(ws + ((stages & 1) ? L.bufB : L.bufA));
    const long long cols = planes / p->Nl[c];
    long long ring_cols = p->colexp_ring;
    if (ring_cols > cols) ring_cols = cols;
    if (cuda_failed(p, launch_inv_plane_colexp((int)p->Ng[a], p->kmax[a], (int)p->Ng[b], p->kmax[b], (int)p->Ng[c],
                                               p->kmax[c], src, ring, (int)ring_cols,
                                               reinterpret_cast<int*>(ws + L.counters), cols, y, planes * p->Ng[b],
                                               scale, herm ? 1 : 0, reinterpret_cast<int*>(ws + L.status),
                                               p->dbg_poll_limit ? p->dbg_poll_limit : kDefaultPollLimit, st)))
      return DTST_ERR_CUDA;
  } else if (2 * p->kmax[a] == p->Ng[a] && std::getenv("DTST_NO_PLANEG") == nullptr &&
             planeg_supported((int)p->Ng[a], p->kmax[a], (int)p->Ng[b], p->kmax[b])) {
    // half of the contiguous extent retained: the lane-per-row expansion of the tensor-map plane kernel is bound by its
    // multiply-adds there (1.9 TB/s on the paper's layer), the tensor-core one of dtst_rowg.cu is not
    if (cuda_failed(p, launch_planeg_expand(src, y, planes, (int)p->Ng[a], p->kmax[a], (int)p->Ng[b], p->kmax[b], scale,
                                            herm ? 1 : 0, p->fast_math != 0, st)))
      return DTST_ERR_CUDA;
  } else if (cuda_failed(p, launch_inv_plane((int)p->Ng[a], p->kmax[a], (int)p->Ng[b], p->kmax[b], src, y,
                                             planes * p->Ng[b], scale, herm ? 1 : 0, nullptr, st))) {
    return DTST_ERR_CUDA;
  }
  ++p->launches;
  return DTST_OK;
}

// Row path: the row kernel streams the grid once along its contiguous dimension; the rest runs reduced.
dtst_status run_forward_row(dtst_plan* p, const float* x, float2* Xhat, int Cn, float scale, bool herm,
                            cudaStream_t st) {
  const int d = p->d, a = d - 1;
  const WsLayout L = ws_layout(p);
  char* ws = static_cast<char*>(p->ws);
  long long rows = (long long)p->B * Cn;
  for (int i = 0; i < a; ++i) rows *= p->Nl[i];
  float2* t1 = (d == 1) ? Xhat : reinterpret_cast<float2*>(ws + L.bufA);
  if (use_planeg(p)) {
    const int b = d - 2;
    float2* dst = (d == 2) ? Xhat : t1;
    {
      KernelTimer kt(p, DTST_KERNEL_GRID_READ, st);
      if (cuda_failed(p, launch_planeg_contract(x, dst, rows / p->Ng[b], (int)p->Ng[a], p->kmax[a], (int)p->Ng[b],
                                                p->kmax[b], scale, herm ? 1 : 0, p->fast_math != 0, st)))
        return DTST_ERR_CUDA;
    }
    ++p->launches;
    if (d == 2) return DTST_OK;
    return forward_stages(p, t1, d - 3, 1, Xhat, Cn, 1.0f, false, st);
  }
  {
    KernelTimer kt(p, DTST_KERNEL_GRID_READ, st);
    const cudaError_t e = row_supported((int)p->Ng[a], p->kmax[a])
                              ? launch_row_contract(x, t1, rows, (int)p->Ng[a], p->kmax[a], scale, herm ? 1 : 0,
                                                    reinterpret_cast<int*>(ws + L.status), st)
                          : rowg_supported((int)p->Ng[a], p->kmax[a])
                              ? launch_rowg_contract(x, t1, rows, (int)p->Ng[a], p->kmax[a], scale, herm ? 1 : 0,
                                                     p->fast_math != 0, st)
                              : launch_rowl_contract(x, t1, rows, (int)p->Ng[a], p->kmax[a], scale, herm ? 1 : 0,
                                                     p->fast_math != 0, st);
    if (cuda_failed(p, e)) return DTST_ERR_CUDA;
  }
  ++p->launches;
  if (d == 1) return DTST_OK;
  return forward_stages(p, t1, d - 2, 1, Xhat, Cn, 1.0f, false, st);
}

dtst_status run_inverse_row(dtst_plan* p, const float2* Yhat, float* y, int Cn, float scale, bool herm,
                            cudaStream_t st) {
  const int d = p->d, a = d - 1;
  const float2* src = Yhat;
  const bool pg = use_planeg(p);
  if (d > (pg ? 2 : 1)) {
    dtst_status s = inverse_stages_complex(p, Yhat, pg ? d - 3 : d - 2, -1, Cn, &src, nullptr, st);
    if (s != DTST_OK) return s;
  }
  long long rows = (long long)p->B * Cn;
  for (int i = 0; i < a; ++i) rows *= p->Nl[i];
  KernelTimer kt(p, DTST_KERNEL_GRID_WRITE, st);
  if (pg) {
    const int b = d - 2;
    if (cuda_failed(p, launch_planeg_expand(src, y, rows / p->Ng[b], (int)p->Ng[a], p->kmax[a], (int)p->Ng[b], p->kmax[b],
                                            scale, herm ? 1 : 0, p->fast_math != 0, st)))
      return DTST_ERR_CUDA;
    ++p->launches;
    return DTST_OK;
  }
  const cudaError_t e = row_supported((int)p->Ng[a], p->kmax[a])
                            ? launch_row_expand(src, y, rows, (int)p->Ng[a], p->kmax[a], scale, herm ? 1 : 0, st)
                        : rowg_supported((int)p->Ng[a], p->kmax[a])
                            ? launch_rowg_expand(src, y, rows, (int)p->Ng[a], p->kmax[a], scale, herm ? 1 : 0,
                                                 p->fast_math != 0, st)
                            : launch_rowl_expand(src, y, rows, (int)p->Ng[a], p->kmax[a], scale, herm ? 1 : 0,
                                                 p->fast_math != 0, st);
  if (cuda_failed(p, e)) return DTST_ERR_CUDA;
  ++p->launches;
  return DTST_OK;
}

// A plan belongs to the device that was current when it was created: its workspace and the caller's tensors live
// there, so a compute call with another device current would launch on the wrong GPU with foreign pointers.
dtst_status check_device(const dtst_plan* p) {
  if (p == nullptr) return DTST_ERR_INVALID_ARG;
  if (p->device >= 0) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
      (void)cudaGetLastError();
      return DTST_ERR_CUDA;
    }
    if (dev != p->device) return DTST_ERR_INVALID_ARG;
  }
  return DTST_OK;
}

dtst_status check_ready(const dtst_plan* p) {
  const dtst_status sd = check_device(p);
  if (sd != DTST_OK) return sd;
  if (p->require_fast && !all_streaming(p)) return DTST_ERR_UNSUPPORTED;
  const WsLayout L = ws_layout(p);
  if (p->ws == nullptr || p->ws_bytes < L.total) return DTST_ERR_WORKSPACE;
  return DTST_OK;
}

}  // namespace

namespace dtst {

WsLayout ws_layout(const dtst_plan* p) {
  WsLayout L;
  std::memset(&L, 0, sizeof(L));
  const int Cn = p->C_in > p->C_out ? p->C_in : p->C_out;
  // Ping-pong buffers A and B: walk the stage chains of every kernel family (a plan option may switch families
  // later) in the plan's contraction order and keep the largest tensor each buffer ever receives.
  long long a = 0, b = 0;
  auto put = [&](int which, long long n) {
    if (which == 0) a = n > a ? n : a; else b = n > b ? n : b;
  };
  for (int j_from = p->d - 1; j_from >= p->d - 3 && j_from >= -1; --j_from) {
    bool contracted[kMaxDims];
    // forward: the grid-side kernel (if any) leaves its result in A, the following stages alternate from B
    for (int i = 0; i < p->d; ++i) contracted[i] = i > j_from;
    int list[kMaxDims + 1];
    const int n = j_from == p->d - 1 ? grid_order(p, list) : (j_from >= 0 ? middle_order(p, j_from, list) : 0);
    int flip = 0;
    if (j_from < p->d - 1) {
      put(0, state_elems(p, Cn, contracted));
      flip = 1;
    }
    for (int idx = 0; idx < n; ++idx) {
      contracted[list[idx]] = true;
      if (idx != n - 1) put(flip, state_elems(p, Cn, contracted));
      flip ^= 1;
    }
    // expansion: the same order backwards, every stage into a buffer, starting with A (a chain that starts on
    // the grid itself ends there: its first stage writes the caller's tensor, not a buffer)
    for (int i = 0; i < p->d; ++i) contracted[i] = true;
    flip = 0;
    for (int idx = n - 1; idx >= (j_from == p->d - 1 ? 1 : 0); --idx) {
      contracted[list[idx]] = false;
      put(flip, state_elems(p, Cn, contracted));
      flip ^= 1;
    }
  }
  L.szA = (size_t)a * sizeof(float2);
  L.szB = (size_t)b * sizeof(float2);
  L.szPartial = p->P > 1 ? (size_t)p->P * p->B * Cn * p->M * sizeof(float2) : 0;
  L.szG = (size_t)p->B * Cn * p->M * sizeof(float2);
  size_t o = 0;
  L.status = o; o += kStatusBytes;
  L.bufA = o; o += align256(L.szA);
  L.bufB = o; o += align256(L.szB);
  L.partial = o; o += align256(L.szPartial);
  L.gy = o; o += align256(L.szG);
  L.gx = o; o += align256(L.szG);
  // flow-control counters of the kernels that expand or contract a leading dimension inside a plane kernel:
  // two ints per column (a column = one index tuple of batch, channel and the dimensions in front of the last three)
  {
    long long cols = (long long)p->B * Cn;
    for (int i = 0; i + 3 < p->d; ++i) cols *= p->Nl[i];
    L.szCounters = p->d >= 3 ? (size_t)2 * cols * sizeof(int) : 0;
  }
  L.counters = o; o += align256(L.szCounters);
  // per-CTA partial sums of the bypass weight gradient (dtst_block_backward)
  L.szWbPartial = (size_t)kBlockPartialRows * ((size_t)p->C_in * p->C_out + p->C_out) * sizeof(float);
  L.wb_partial = o; o += align256(L.szWbPartial);
  L.total = o;
  return L;
}

}  // namespace dtst

extern "C" {

dtst_status dtst_plan_create(dtst_plan** out, int d, const int64_t N[], const int32_t kmax[], int B, int C_in,
                             int C_out) {
  return create_common(out, d, N, nullptr, nullptr, kmax, B, C_in, C_out);
}

dtst_status dtst_plan_create_local(dtst_plan** out, int d, const int64_t N_global[], const int64_t N_local[],
                                   const int64_t offset[], const int32_t kmax[], int B, int C_in, int C_out) {
  if (N_local == nullptr || offset == nullptr) {
    if (out) *out = nullptr;
    return DTST_ERR_INVALID_ARG;
  }
  return create_common(out, d, N_global, N_local, offset, kmax, B, C_in, C_out);
}

dtst_status dtst_plan_set_virtual_shards(dtst_plan* p, int P) {
  if (p == nullptr || P < 1 || p->Nl[0] % P != 0) return DTST_ERR_INVALID_ARG;
  if (P > 1 && p->d >= 2) {   // dimension 0 must be the last one contracted (see dtst_plan_set_contraction_order)
    int list[kMaxDims];
    const int n = middle_order(p, p->d - 2, list);
    if (list[n - 1] != 0) return DTST_ERR_INVALID_ARG;
  }
  p->P = P;
  return DTST_OK;
}

dtst_status dtst_plan_set_kernel_path(dtst_plan* p, int path) {
  if (p == nullptr || (path != DTST_PATH_AUTO && path != DTST_PATH_GENERIC)) return DTST_ERR_INVALID_ARG;
  p->path_request = path;
  return DTST_OK;
}

// bytes the stages behind the grid-side kernel move in one forward-type transform (complex64 in and out per stage)
static double middle_stage_bytes(const dtst_plan* p) {
  const int j_top = use_fused(p) ? p->d - 3 : p->d - 2;
  if (j_top < 0) return 0.0;
  int list[kMaxDims];
  const int n = middle_order(p, j_top, list);
  bool contracted[kMaxDims];
  for (int i = 0; i < p->d; ++i) contracted[i] = i > j_top;
  double bytes = 0.0;
  for (int idx = 0; idx < n; ++idx) {
    bytes += 8.0 * (double)state_elems(p, p->C_in, contracted);
    contracted[list[idx]] = true;
    bytes += 8.0 * (double)state_elems(p, p->C_in, contracted);
  }
  return bytes;
}

dtst_status dtst_plan_set_contraction_order(dtst_plan* p, const int32_t order[], int n) {
  if (p == nullptr || order == nullptr || n != p->d - 1) return DTST_ERR_INVALID_ARG;
  bool seen[kMaxDims] = {};
  for (int i = 0; i < n; ++i) {
    if (order[i] < 0 || order[i] > p->d - 2 || seen[order[i]]) return DTST_ERR_INVALID_ARG;
    seen[order[i]] = true;
  }
  // the slab partial sums of virtual shards are added after the last stage: dimension 0 then has to be that stage
  if (p->P > 1 && n > 0 && order[n - 1] != 0) return DTST_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) p->order_rank[order[i]] = i;
  return DTST_OK;
}

dtst_status dtst_plan_get_contraction_order(const dtst_plan* p, int32_t order[]) {
  if (p == nullptr || (order == nullptr && p->d > 1)) return DTST_ERR_INVALID_ARG;
  int list[kMaxDims];
  const int n = p->d >= 2 ? middle_order(p, p->d - 2, list) : 0;
  for (int i = 0; i < n; ++i) order[i] = list[i];
  return DTST_OK;
}

dtst_status dtst_plan_tune_contraction_order(dtst_plan* p, double* bytes_before, double* bytes_after) {
  if (p == nullptr) return DTST_ERR_INVALID_ARG;
  if (bytes_before) *bytes_before = middle_stage_bytes(p);
  // the most compressing dimension first: ascending K_j / n_j; ties keep the default (higher dimension first);
  // dimension 0 stays last when it carries virtual shards
  int list[kMaxDims], n = 0;
  for (int j = p->d - 2; j >= 0; --j) list[n++] = j;
  auto before = [&](int x, int y) {
    if (p->P > 1 && (x == 0 || y == 0)) return y == 0 && x != 0;
    const long long lhs = (long long)p->K[x] * p->Nl[y], rhs = (long long)p->K[y] * p->Nl[x];   // K_x/n_x < K_y/n_y
    if (lhs != rhs) return lhs < rhs;
    return x > y;
  };
  for (int a = 1; a < n; ++a)
    for (int b = a; b > 0 && before(list[b], list[b - 1]); --b) {
      const int t = list[b];
      list[b] = list[b - 1];
      list[b - 1] = t;
    }
  for (int i = 0; i < n; ++i) p->order_rank[list[i]] = i;
  if (bytes_after) *bytes_after = middle_stage_bytes(p);
  return DTST_OK;
}

dtst_status dtst_plan_set_column_contraction(dtst_plan* p, int mode) {
  if (p == nullptr || mode < -1 || mode > 1) return DTST_ERR_INVALID_ARG;
  p->colfuse = mode;
  return DTST_OK;
}

dtst_status dtst_plan_set_arithmetic(dtst_plan* p, int mode) {
  if (p == nullptr || (mode != DTST_ARITH_TF32X3 && mode != DTST_ARITH_TF32)) return DTST_ERR_INVALID_ARG;
  p->fast_math = mode == DTST_ARITH_TF32 ? 1 : 0;
  return DTST_OK;
}

dtst_status dtst_plan_set_block_epilogue(dtst_plan* p, int mode) {
  if (p == nullptr || mode < DTST_BLOCK_EPILOGUE_AUTO || mode > DTST_BLOCK_EPILOGUE_TENSOR) return DTST_ERR_INVALID_ARG;
  if (mode == DTST_BLOCK_EPILOGUE_TENSOR &&
      (p->path_request != DTST_PATH_AUTO || !block_umma_supported(p->C_in, p->C_out, p->points_local, p->B)))
    return DTST_ERR_UNSUPPORTED;
  p->block_epilogue = mode;
  return DTST_OK;
}

dtst_status dtst_plan_require_fast_path(dtst_plan* p, int required) {
  if (p == nullptr) return DTST_ERR_INVALID_ARG;
  p->require_fast = 0;
  if (!required) return DTST_OK;
  if (!all_streaming(p)) return DTST_ERR_UNSUPPORTED;
  p->require_fast = 1;
  return DTST_OK;
}

dtst_status dtst_plan_set_column_expansion(dtst_plan* p, int ring_columns) {
  if (p == nullptr || ring_columns < 0) return DTST_ERR_INVALID_ARG;
  p->colexp_ring = ring_columns;
  if (ring_columns > 0 && !use_colexp(p)) {
    p->colexp_ring = 0;
    return DTST_ERR_UNSUPPORTED;
  }
  return DTST_OK;
}

dtst_status dtst_plan_kernel_path(const dtst_plan* p, int* path) {
  if (p == nullptr || path == nullptr) return DTST_ERR_INVALID_ARG;
  *path = use_fused(p) ? DTST_PATH_AUTO : (use_row(p) ? DTST_PATH_ROW : DTST_PATH_GENERIC);
  return DTST_OK;
}

static void free_timing(dtst_plan* p) {
  for (int kind = 0; kind < DTST_KERNEL_KINDS; ++kind)
    for (int se = 0; se < 2; ++se) {
      if (p->timing_ev[kind][se] != nullptr) {
        for (int i = 0; i < p->timing_cap; ++i)
          if (p->timing_ev[kind][se][i] != nullptr) cudaEventDestroy(p->timing_ev[kind][se][i]);
        std::free(p->timing_ev[kind][se]);
        p->timing_ev[kind][se] = nullptr;
      }
    }
  p->timing_cap = 0;
  std::memset(p->timing_n, 0, sizeof(p->timing_n));
}

dtst_status dtst_plan_enable_kernel_timing(dtst_plan* p, int capacity) {
  if (p == nullptr || capacity < 0 || capacity > (1 << 16)) return DTST_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return DTST_ERR_CUDA;
  free_timing(p);
  if (capacity == 0) return DTST_OK;
  p->timing_cap = capacity;
  for (int kind = 0; kind < DTST_KERNEL_KINDS; ++kind)
    for (int se = 0; se < 2; ++se) {
      cudaEvent_t* arr = static_cast<cudaEvent_t*>(std::calloc((size_t)capacity, sizeof(cudaEvent_t)));
      if (arr == nullptr) {
        free_timing(p);
        return DTST_ERR_ALLOC;
      }
      p->timing_ev[kind][se] = arr;
      for (int i = 0; i < capacity; ++i)
        if (cudaEventCreate(&arr[i]) != cudaSuccess) {
          free_timing(p);
          return DTST_ERR_CUDA;
        }
    }
  return DTST_OK;
}

dtst_status dtst_plan_kernel_timing(dtst_plan* p, int kind, int64_t* launches, double* total_ms) {
  if (p == nullptr || kind < 0 || kind >= DTST_KERNEL_KINDS || launches == nullptr || total_ms == nullptr)
    return DTST_ERR_INVALID_ARG;
  *launches = 0;
  *total_ms = 0.0;
  if (p->timing_cap == 0) return DTST_OK;
  if (cudaDeviceSynchronize() != cudaSuccess) return DTST_ERR_CUDA;
  for (int i = 0; i < p->timing_n[kind]; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, p->timing_ev[kind][0][i], p->timing_ev[kind][1][i]) != cudaSuccess)
      return DTST_ERR_CUDA;
    *total_ms += ms;
    ++*launches;
  }
  p->timing_n[kind] = 0;
  return DTST_OK;
}

dtst_status dtst_plan_destroy(dtst_plan* p) {
  if (p == nullptr) return DTST_ERR_INVALID_ARG;
  free_timing(p);
  host_io_release(p);
  delete p;
  return DTST_OK;
}

dtst_status dtst_plan_num_modes(const dtst_plan* p, int64_t* M, int64_t K[]) {
  if (p == nullptr || M == nullptr) return DTST_ERR_INVALID_ARG;
  *M = p->M;
  if (K != nullptr)
    for (int j = 0; j < p->d; ++j) K[j] = p->K[j];
  return DTST_OK;
}

dtst_status dtst_plan_mode_indices(const dtst_plan* p, int dim, int64_t* idx) {
  if (p == nullptr || idx == nullptr || dim < 0 || dim >= p->d) return DTST_ERR_INVALID_ARG;
  for (int r = 0; r < p->K[dim]; ++r)
    idx[r] = mode_at(r, p->kmax[dim], (int)p->Ng[dim], (dim < p->d - 1 || p->complex_io) ? 1 : 0);
  return DTST_OK;
}

dtst_status dtst_plan_workspace_bytes(const dtst_plan* p, size_t* bytes) {
  if (p == nullptr || bytes == nullptr) return DTST_ERR_INVALID_ARG;
  *bytes = ws_layout(p).total;
  return DTST_OK;
}

dtst_status dtst_plan_set_workspace(dtst_plan* p, void* dev_ptr, size_t bytes) {
  if (p == nullptr || dev_ptr == nullptr || (reinterpret_cast<uintptr_t>(dev_ptr) & 255u) != 0)
    return DTST_ERR_INVALID_ARG;
  if (bytes < ws_layout(p).total) return DTST_ERR_WORKSPACE;
  if (cudaMemset(dev_ptr, 0, kStatusBytes) != cudaSuccess) {
    (void)cudaGetLastError();
    return DTST_ERR_CUDA;
  }
  p->ws = dev_ptr;
  p->ws_bytes = bytes;
  return DTST_OK;
}

dtst_status dtst_plan_create_complex(dtst_plan** out, int d, const int64_t N_global[], const int64_t N_local[],
                                     const int64_t offset[], const int32_t kmax[], int B, int C_in, int C_out) {
  return create_common(out, d, N_global, N_local, offset, kmax, B, C_in, C_out, true);
}

dtst_status dtst_forward_complex(dtst_plan* p, const void* x, void* Xhat, void* stream) {
  dtst_status s = check_ready(p);
  if (s != DTST_OK) return s;
  if (!p->complex_io || x == nullptr || Xhat == nullptr || !aligned16(x) || !aligned16(Xhat)) return DTST_ERR_INVALID_ARG;
  return run_forward_generic(p, static_cast<const float*>(x), static_cast<float2*>(Xhat), p->C_in, 1.0f, false,
                             static_cast<cudaStream_t>(stream));
}

dtst_status dtst_inverse_complex(dtst_plan* p, const void* Yhat, void* y, void* stream) {
  dtst_status s = check_ready(p);
  if (s != DTST_OK) return s;
  if (!p->complex_io || Yhat == nullptr || y == nullptr || !aligned16(Yhat) || !aligned16(y)) return DTST_ERR_INVALID_ARG;
  return run_inverse_generic(p, static_cast<const float2*>(Yhat), static_cast<float*>(y), p->C_out,
                             (float)(1.0 / (double)p->points_global), false, static_cast<cudaStream_t>(stream));
}

dtst_status dtst_backward_complex(dtst_plan* p, const void* grad_y, const void* Xhat_saved, const void* W, void* grad_x,
                                  void* grad_W, void* stream) {
  dtst_status s = check_ready(p);
  if (s != DTST_OK) return s;
  if (!p->complex_io || grad_y == nullptr || W == nullptr || (grad_x == nullptr && grad_W == nullptr) ||
      (grad_W != nullptr && Xhat_saved == nullptr))
    return DTST_ERR_INVALID_ARG;
  if (!aligned16(grad_y) || !aligned16(Xhat_saved) || !aligned16(W) || !aligned16(grad_x) || !aligned16(grad_W))
    return DTST_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const WsLayout L = ws_layout(p);
  char* ws = static_cast<char*>(p->ws);
  float2* GY = reinterpret_cast<float2*>(ws + L.gy);
  float2* GX = reinterpret_cast<float2*>(ws + L.gx);
  // adjoint of the inverse: G_Y = F(grad_y) / prod N (no Hermitian weights: nothing was doubled)
  s = run_forward_generic(p, static_cast<const float*>(grad_y), GY, p->C_out, (float)(1.0 / (double)p->points_global),
                          false, st);
  if (s != DTST_OK) return s;
  if (cuda_failed(p, launch_mix_adjoint(GY, static_cast<const float2*>(Xhat_saved), static_cast<const float2*>(W),
                                        grad_x ? GX : nullptr, static_cast<float2*>(grad_W), p->B, p->C_in, p->C_out,
                                        p->M, st, &p->launches)))
    return DTST_ERR_CUDA;
  if (grad_x != nullptr) return run_inverse_generic(p, GX, static_cast<float*>(grad_x), p->C_in, 1.0f, false, st);
  return DTST_OK;
}

dtst_status dtst_forward(dtst_plan* p, const float* x, void* Xhat, void* stream) {
  dtst_status s = check_ready(p);
  if (s != DTST_OK) return s;
  if (p->complex_io) return DTST_ERR_INVALID_ARG;   // a complex plan: dtst_forward_complex
  if (x == nullptr || Xhat == nullptr || !aligned16(x) || !aligned16(Xhat)) return DTST_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (use_fused(p)) return run_forward_fused(p, x, static_cast<float2*>(Xhat), p->C_in, 1.0f, false, st);
  if (use_row(p)) return run_forward_row(p, x, static_cast<float2*>(Xhat), p->C_in, 1.0f, false, st);
  return run_forward_generic(p, x, static_cast<float2*>(Xhat), p->C_in, 1.0f, false, st);
}

dtst_status dtst_spectral_mul(dtst_plan* p, const void* Xhat, const void* W, void* Yhat, void* stream) {
  if (check_device(p) != DTST_OK) return check_device(p);
  if (Xhat == nullptr || W == nullptr || Yhat == nullptr || !aligned16(Xhat) || !aligned16(W) ||
      !aligned16(Yhat) || Yhat == Xhat || Yhat == W)
    return DTST_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  KernelTimer kt(p, DTST_KERNEL_MIX, st);
  if (cuda_failed(p, launch_mix(static_cast<const float2*>(Xhat), static_cast<const float2*>(W), static_cast<float2*>(Yhat),
                 p->B, p->C_in, p->C_out, p->M, st, &p->launches))) return DTST_ERR_CUDA;
  return DTST_OK;
}

dtst_status dtst_inverse(dtst_plan* p, const void* Yhat, float* y, void* stream) {
  dtst_status s = check_ready(p);
  if (s != DTST_OK) return s;
  if (p->complex_io || Yhat == nullptr || y == nullptr || !aligned16(Yhat) || !aligned16(y)) return DTST_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const float scale = (float)(1.0 / (double)p->points_global);
  if (use_fused(p)) return run_inverse_fused(p, static_cast<const float2*>(Yhat), y, p->C_out, scale, true, st);
  if (use_row(p)) return run_inverse_row(p, static_cast<const float2*>(Yhat), y, p->C_out, scale, true, st);
  return run_inverse_generic(p, static_cast<const float2*>(Yhat), y, p->C_out, scale, true, st);
}

dtst_status dtst_backward(dtst_plan* p, const float* grad_y, const void* Xhat_saved, const void* W,
                          float* grad_x, void* grad_W, void* stream) {
  dtst_status s = check_ready(p);
  if (s != DTST_OK) return s;
  // Xhat_saved is read for grad_W only
  if (p->complex_io || grad_y == nullptr || W == nullptr || (grad_x == nullptr && grad_W == nullptr) ||
      (grad_W != nullptr && Xhat_saved == nullptr))
    return DTST_ERR_INVALID_ARG;
  if (!aligned16(grad_y) || !aligned16(Xhat_saved) || !aligned16(W) || !aligned16(grad_x) || !aligned16(grad_W))
    return DTST_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const WsLayout L = ws_layout(p);
  char* ws = static_cast<char*>(p->ws);
  float2* GY = reinterpret_cast<float2*>(ws + L.gy);
  float2* GX = reinterpret_cast<float2*>(ws + L.gx);
  const float scale = (float)(1.0 / (double)p->points_global);
  // adjoint of I: G_Y = (c / prod N) F(grad_y)
  s = use_fused(p) ? run_forward_fused(p, grad_y, GY, p->C_out, scale, true, st)
      : use_row(p) ? run_forward_row(p, grad_y, GY, p->C_out, scale, true, st)
                   : run_forward_generic(p, grad_y, GY, p->C_out, scale, true, st);
  if (s != DTST_OK) return s;
  // adjoint of M
  {
    KernelTimer kt(p, DTST_KERNEL_MIX_ADJOINT, st);
    if (cuda_failed(p, launch_mix_adjoint(GY, static_cast<const float2*>(Xhat_saved), static_cast<const float2*>(W),
                           grad_x ? GX : nullptr, static_cast<float2*>(grad_W), p->B, p->C_in, p->C_out, p->M,
                           st, &p->launches))) return DTST_ERR_CUDA;
  }
  // adjoint of F: plain expansion, no doubling, no 1/prod N
  if (grad_x != nullptr) {
    s = use_fused(p) ? run_inverse_fused(p, GX, grad_x, p->C_in, 1.0f, false, st)
        : use_row(p) ? run_inverse_row(p, GX, grad_x, p->C_in, 1.0f, false, st)
                     : run_inverse_generic(p, GX, grad_x, p->C_in, 1.0f, false, st);
    if (s != DTST_OK) return s;
  }
  return DTST_OK;
}

// Which kernel forms the bypass product of dtst_block_forward: the tensor-core one (tcgen05) only when asked for.
// Left to the library it is the fp32 FFMA kernel, which holds a thread's input channels in registers and is the
// faster one at every channel count measured (34 GB moved at 16 channels: 5.8 ms against 12.0 ms; 17 GB at 32
// channels: 3.9 ms against 5.7 ms - the tensor-core kernel's per-tile chain of split, product and epilogue is
// latency-bound at four CTAs per SM).
static bool use_block_tensor(const dtst_plan* p) {
  if (p->path_request != DTST_PATH_AUTO || p->block_epilogue != DTST_BLOCK_EPILOGUE_TENSOR) return false;
  return block_umma_supported(p->C_in, p->C_out, p->points_local, p->B);
}

// ---- the whole block: GELU(W_bypass x + I(M(F(x), W))) and its backward pass
dtst_status dtst_block_forward(dtst_plan* p, const float* x, const void* W, const float* W_bypass, float* out,
                               void* Xhat_saved, float* z_saved, void* stream) {
  dtst_status s = check_ready(p);
  if (s != DTST_OK) return s;
  if (x == nullptr || W == nullptr || W_bypass == nullptr || out == nullptr || Xhat_saved == nullptr)
    return DTST_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(W) || !aligned16(W_bypass) || !aligned16(out) || !aligned16(Xhat_saved) ||
      !aligned16(z_saved) || out == x || z_saved == x || (z_saved != nullptr && z_saved == out))
    return DTST_ERR_INVALID_ARG;
  if (!block_supported(p->C_in, p->C_out, p->points_local)) return DTST_ERR_UNSUPPORTED;
  const WsLayout L = ws_layout(p);
  void* Yhat = static_cast<char*>(p->ws) + L.gy;
  s = dtst_forward(p, x, Xhat_saved, stream);
  if (s != DTST_OK) return s;
  s = dtst_spectral_mul(p, Xhat_saved, W, Yhat, stream);
  if (s != DTST_OK) return s;
  s = dtst_inverse(p, Yhat, out, stream);          // out holds y; the epilogue turns it into the activation in place
  if (s != DTST_OK) return s;
  KernelTimer kt(p, DTST_KERNEL_BLOCK_EPILOGUE, static_cast<cudaStream_t>(stream));
  if (use_block_tensor(p)) {
    if (cuda_failed(p, launch_block_epilogue_umma(x, out, z_saved, W_bypass, p->B, p->C_in, p->C_out, p->points_local,
                                                  reinterpret_cast<int*>(static_cast<char*>(p->ws) + L.status),
                                                  static_cast<cudaStream_t>(stream))))
      return DTST_ERR_CUDA;
  } else if (cuda_failed(p, launch_block_epilogue(x, out, z_saved, W_bypass, p->B, p->C_in, p->C_out,
                                                  p->points_local, static_cast<cudaStream_t>(stream)))) {
    return DTST_ERR_CUDA;
  }
  ++p->launches;
  return DTST_OK;
}

dtst_status dtst_block_backward(dtst_plan* p, const float* grad_out, const float* x, const float* z_saved,
                                const void* Xhat_saved, const void* W, const float* W_bypass, float* scratch,
                                float* grad_x, void* grad_W, float* grad_W_bypass, void* stream) {
  dtst_status s = check_ready(p);
  if (s != DTST_OK) return s;
  if (grad_out == nullptr || x == nullptr || z_saved == nullptr || W == nullptr || W_bypass == nullptr ||
      scratch == nullptr || (grad_x == nullptr && grad_W == nullptr && grad_W_bypass == nullptr) ||
      (grad_W != nullptr && Xhat_saved == nullptr))
    return DTST_ERR_INVALID_ARG;
  if (!aligned16(grad_out) || !aligned16(x) || !aligned16(z_saved) || !aligned16(Xhat_saved) || !aligned16(W) ||
      !aligned16(W_bypass) || !aligned16(scratch) || !aligned16(grad_x) || !aligned16(grad_W) ||
      !aligned16(grad_W_bypass) || scratch == x || scratch == z_saved || scratch == grad_x)
    return DTST_ERR_INVALID_ARG;
  if (!block_supported(p->C_in, p->C_out, p->points_local)) return DTST_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const WsLayout L = ws_layout(p);
  // adjoint of the activation: g_z = grad_out * GELU'(z)
  {
    KernelTimer kt(p, DTST_KERNEL_GELU_BACKWARD, st);
    if (cuda_failed(p, launch_gelu_backward(grad_out, z_saved, scratch,
                                            (long long)p->B * p->C_out * p->points_local, st)))
      return DTST_ERR_CUDA;
  }
  ++p->launches;
  // adjoint of the spectral layer on g_z
  if (grad_x != nullptr || grad_W != nullptr) {
    s = dtst_backward(p, scratch, Xhat_saved, W, grad_x, grad_W, stream);
    if (s != DTST_OK) return s;
  }
  // adjoint of the bypass: grad_x += W_bypass^T g_z, grad_W_bypass = sum g_z x^T
  if (grad_x != nullptr || grad_W_bypass != nullptr) {
    KernelTimer kt(p, DTST_KERNEL_BYPASS_BACKWARD, st);
    if (cuda_failed(p, launch_bypass_backward(scratch, x, grad_x, W_bypass, grad_W_bypass,
                                              reinterpret_cast<float*>(static_cast<char*>(p->ws) + L.wb_partial), p->B,
                                              p->C_in, p->C_out, p->points_local, st, &p->launches)))
      return DTST_ERR_CUDA;
  }
  return DTST_OK;
}

// ---- point-wise linear layers (the lifting and projection layers around the blocks of an FNO)
dtst_status dtst_pointwise_linear(int B, int C_in, int C_out, int64_t points, const float* x, const float* W,
                                  const float* bias, float* out, void* stream) {
  if (B < 1 || C_in < 1 || C_out < 1 || points < 4 || points % 4 != 0 || x == nullptr || W == nullptr ||
      out == nullptr || out == x || !aligned16(x) || !aligned16(out) || !aligned16(W) ||
      (reinterpret_cast<uintptr_t>(bias) & 3u) != 0)
    return DTST_ERR_INVALID_ARG;
  if ((size_t)C_in * C_out * 4 > 200 * 1024) return DTST_ERR_UNSUPPORTED;
  if (launch_pointwise_linear(x, out, bias, W, B, C_in, C_out, points, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
    (void)cudaGetLastError();
    return DTST_ERR_CUDA;
  }
  return DTST_OK;
}

dtst_status dtst_pointwise_linear_scratch_bytes(int C_in, int C_out, size_t* bytes) {
  if (C_in < 1 || C_out < 1 || bytes == nullptr) return DTST_ERR_INVALID_ARG;
  *bytes = align256((size_t)kBlockPartialRows * ((size_t)C_in * C_out + C_out) * sizeof(float));
  return DTST_OK;
}

dtst_status dtst_pointwise_linear_backward(int B, int C_in, int C_out, int64_t points, const float* grad_out,
                                           const float* x, const float* W, float* grad_x, float* grad_W,
                                           float* grad_bias, void* scratch, size_t scratch_bytes, void* stream) {
  if (B < 1 || C_in < 1 || C_out < 1 || points < 4 || points % 4 != 0 || grad_out == nullptr || x == nullptr ||
      W == nullptr || (grad_x == nullptr && grad_W == nullptr && grad_bias == nullptr) || grad_x == grad_out ||
      grad_x == x)
    return DTST_ERR_INVALID_ARG;
  if (!aligned16(grad_out) || !aligned16(x) || !aligned16(W) || !aligned16(grad_x) || !aligned16(grad_W) ||
      (reinterpret_cast<uintptr_t>(grad_bias) & 3u) != 0 || !aligned16(scratch))
    return DTST_ERR_INVALID_ARG;
  if (!block_supported(C_in, C_out, points)) return DTST_ERR_UNSUPPORTED;
  size_t need = 0;
  dtst_pointwise_linear_scratch_bytes(C_in, C_out, &need);
  if ((grad_W != nullptr || grad_bias != nullptr) && (scratch == nullptr || scratch_bytes < need)) return DTST_ERR_WORKSPACE;
  if (launch_linear_backward(grad_out, x, grad_x, 2, W, grad_W, grad_bias, static_cast<float*>(scratch), B, C_in, C_out,
                             points, static_cast<cudaStream_t>(stream), nullptr) != cudaSuccess) {
    (void)cudaGetLastError();
    return DTST_ERR_CUDA;
  }
  return DTST_OK;
}

// ---- the steps of the layer one by one, for a caller that exchanges spectra between ranks in between them
dtst_status dtst_spectral_mul_modes(dtst_plan* p, const void* Xhat, const void* W_shard, void* Yhat_chunk,
                                    int64_t m0, int64_t count, void* stream) {
  if (check_device(p) != DTST_OK) return check_device(p);
  if (Xhat == nullptr || W_shard == nullptr || Yhat_chunk == nullptr || !aligned16(Xhat) || !aligned16(W_shard) ||
      !aligned16(Yhat_chunk) || Yhat_chunk == Xhat || Yhat_chunk == W_shard)
    return DTST_ERR_INVALID_ARG;
  if (m0 < 0 || count < 1 || m0 + count > p->M) return DTST_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cuda_failed(p, launch_mix_modes(static_cast<const float2*>(Xhat), static_cast<const float2*>(W_shard),
                                      static_cast<float2*>(Yhat_chunk), p->B, p->C_in, p->C_out, p->M, m0, count, st,
                                      &p->launches)))
    return DTST_ERR_CUDA;
  return DTST_OK;
}

dtst_status dtst_backward_spectrum(dtst_plan* p, const float* grad_y, void* GY, void* stream) {
  dtst_status s = check_ready(p);
  if (s != DTST_OK) return s;
  if (p->complex_io || grad_y == nullptr || GY == nullptr || !aligned16(grad_y) || !aligned16(GY)) return DTST_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const float scale = (float)(1.0 / (double)p->points_global);
  float2* out = static_cast<float2*>(GY);
  return use_fused(p) ? run_forward_fused(p, grad_y, out, p->C_out, scale, true, st)
         : use_row(p) ? run_forward_row(p, grad_y, out, p->C_out, scale, true, st)
                      : run_forward_generic(p, grad_y, out, p->C_out, scale, true, st);
}

dtst_status dtst_backward_mix_modes(dtst_plan* p, const void* GY, const void* Xhat_saved, const void* W_shard,
                                    void* GX_chunk, void* grad_W_shard, int64_t m0, int64_t count, void* stream) {
  if (check_device(p) != DTST_OK) return check_device(p);
  if (GY == nullptr || W_shard == nullptr || (GX_chunk == nullptr && grad_W_shard == nullptr) ||
      (grad_W_shard != nullptr && Xhat_saved == nullptr))
    return DTST_ERR_INVALID_ARG;
  if (!aligned16(GY) || !aligned16(Xhat_saved) || !aligned16(W_shard) || !aligned16(GX_chunk) ||
      !aligned16(grad_W_shard))
    return DTST_ERR_INVALID_ARG;
  if (m0 < 0 || count < 1 || m0 + count > p->M) return DTST_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cuda_failed(p, launch_mix_adjoint_modes(static_cast<const float2*>(GY), static_cast<const float2*>(Xhat_saved),
                                              static_cast<const float2*>(W_shard), static_cast<float2*>(GX_chunk),
                                              static_cast<float2*>(grad_W_shard), p->B, p->C_in, p->C_out, p->M, m0,
                                              count, st, &p->launches)))
    return DTST_ERR_CUDA;
  return DTST_OK;
}

dtst_status dtst_backward_input(dtst_plan* p, const void* GX, float* grad_x, void* stream) {
  dtst_status s = check_ready(p);
  if (s != DTST_OK) return s;
  if (p->complex_io || GX == nullptr || grad_x == nullptr || !aligned16(GX) || !aligned16(grad_x)) return DTST_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const float2* in = static_cast<const float2*>(GX);
  return use_fused(p) ? run_inverse_fused(p, in, grad_x, p->C_in, 1.0f, false, st)
         : use_row(p) ? run_inverse_row(p, in, grad_x, p->C_in, 1.0f, false, st)
                      : run_inverse_generic(p, in, grad_x, p->C_in, 1.0f, false, st);
}

dtst_status dtst_plan_status(dtst_plan* p, void* stream) {
  if (p == nullptr) return DTST_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) return DTST_ERR_CUDA;
  if (p->ws == nullptr) return DTST_OK;
  int word = 0;
  if (cudaMemcpy(&word, p->ws, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return DTST_ERR_CUDA;
  if (word != 0) {
    if (cudaMemset(p->ws, 0, kStatusBytes) != cudaSuccess) return DTST_ERR_CUDA;
    return DTST_ERR_DEVICE_TIMEOUT;
  }
  return DTST_OK;
}

dtst_status dtst_plan_debug_ring_fault(dtst_plan* p, int64_t withhold_after_fills, uint32_t poll_limit) {
  if (p == nullptr) return DTST_ERR_INVALID_ARG;
  if (withhold_after_fills >= 0 && (poll_limit == 0 || poll_limit > (1u << 16))) return DTST_ERR_INVALID_ARG;
  p->dbg_withhold_after = withhold_after_fills < 0 ? -1 : (long long)withhold_after_fills;
  p->dbg_poll_limit = withhold_after_fills < 0 ? 0u : poll_limit;
  return DTST_OK;
}

dtst_status dtst_plan_last_cuda_error(const dtst_plan* p, int* code, const char** text) {
  if (p == nullptr || code == nullptr || text == nullptr) return DTST_ERR_INVALID_ARG;
  *code = p->last_cuda_error;
  *text = cudaGetErrorString((cudaError_t)p->last_cuda_error);
  return DTST_OK;
}

dtst_status dtst_plan_launch_count(const dtst_plan* p, int64_t* launches) {
  if (p == nullptr || launches == nullptr) return DTST_ERR_INVALID_ARG;
  *launches = p->launches;
  return DTST_OK;
}

const char* dtst_status_string(dtst_status s) {
  switch (s) {
    case DTST_OK: return "ok";
    case DTST_ERR_INVALID_ARG: return "invalid argument";
    case DTST_ERR_UNSUPPORTED: return "unsupported configuration";
    case DTST_ERR_ALLOC: return "host allocation failed";
    case DTST_ERR_CUDA: return "CUDA error";
    case DTST_ERR_WORKSPACE: return "workspace missing or too small";
    case DTST_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case DTST_ERR_STATIC_LIMIT: return "intermediates exceed the fixed scratch of dtst_forward_static";
    default: return "unknown status";
  }
}

int dtst_version(void) { return 100; }

}  // extern "C"
