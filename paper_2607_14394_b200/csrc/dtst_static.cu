// dtst_forward_static: the forward partial DFT for callers that cannot allocate
// device memory.  Its intermediates live in one fixed device array that is part
// of this library's image instead of a caller-provided workspace.
#include <mutex>

#include "dtst_common.cuh"

using namespace dtst;

namespace {

// The scratch itself.  Every GPU that loads the library carries these bytes until
// the process exits.  In host code this name is only a handle for
// cudaGetSymbolAddress; it is NOT a device address and must never be handed to a
// kernel directly.
static __device__ __align__(256) unsigned char g_static_scratch[DTST_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device

// Once per device, with that device current: resolve the array's device address.
cudaError_t scratch_of_current_device(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (ptr == nullptr) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

// complex elements after forward stages d-1..j
long long stage_elems(const dtst_plan* p, int j) {
  long long n = (long long)p->B * p->C_in;
  for (int i = 0; i < j; ++i) n *= p->Nl[i];
  for (int i = j; i < p->d; ++i) n *= p->K[i];
  return n;
}

}  // namespace

extern "C" dtst_status dtst_forward_static(dtst_plan* p, const float* x, void* Xhat_, void* stream) {
  if (p == nullptr || x == nullptr || Xhat_ == nullptr || p->complex_io) return DTST_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x) & 15u) || (reinterpret_cast<uintptr_t>(Xhat_) & 15u))
    return DTST_ERR_INVALID_ARG;
  float2* Xhat = static_cast<float2*>(Xhat_);
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  // carve two ping-pong buffers and the slab partials out of the fixed array
  size_t szA = 0, szB = 0;
  int flip = 0;
  for (int j = p->d - 1; j >= 1; --j) {
    const size_t n = (size_t)stage_elems(p, j) * sizeof(float2);
    if (flip == 0) szA = n > szA ? n : szA; else szB = n > szB ? n : szB;
    flip ^= 1;
  }
  const size_t szP = p->P > 1 ? (size_t)p->P * p->B * p->C_in * p->M * sizeof(float2) : 0;
  const size_t offA = 0, offB = up256(szA), offP = offB + up256(szB), total = offP + up256(szP);
  if (total > (size_t)DTST_STATIC_SCRATCH_BYTES) return DTST_ERR_STATIC_LIMIT;

  // a failing runtime call or launch is recorded in the plan for dtst_plan_last_cuda_error
  auto failed = [p](cudaError_t e) {
    if (e == cudaSuccess) return false;
    p->last_cuda_error = (int)e;
    (void)cudaGetLastError();
    return true;
  };
  if (p->device >= 0) {
    int dev = -1;
    if (failed(cudaGetDevice(&dev))) return DTST_ERR_CUDA;
    if (dev != p->device) return DTST_ERR_INVALID_ARG;   // the plan belongs to another device
  }
  void* base = nullptr;
  if (failed(scratch_of_current_device(&base))) return DTST_ERR_CUDA;
  char* s = static_cast<char*>(base);
  float2* buf[2] = {reinterpret_cast<float2*>(s + offA), reinterpret_cast<float2*>(s + offB)};
  float2* partial = reinterpret_cast<float2*>(s + offP);

  const void* cur = x;
  flip = 0;
  for (int j = p->d - 1; j >= 0; --j) {
    DimOp op;
    memset(&op, 0, sizeof(op));
    long long outer = (long long)p->B * p->C_in;
    for (int i = 0; i < j; ++i) outer *= p->Nl[i];
    long long inner = 1;
    for (int i = j + 1; i < p->d; ++i) inner *= p->K[i];
    op.outer = outer;
    op.inner = inner;
    op.Q = (int)p->Nl[j];
    op.R = p->K[j];
    op.N = (int)p->Ng[j];
    op.k = p->kmax[j];
    op.two_sided = (j < p->d - 1) ? 1 : 0;
    op.offset = (int)p->off[j];
    op.forward = 1;
    op.scale = 1.0f;
    op.slabs = 1;
    op.in_outer_stride = (long long)op.Q * inner;
    op.out_outer_stride = (long long)op.R * inner;
    void* dst;
    if (j == 0 && p->P > 1) {
      const int nl = (int)(p->Nl[0] / p->P);
      op.slabs = p->P;
      op.Q = nl;
      op.offset_step = nl;
      op.in_outer_stride = p->Nl[0] * inner;
      op.in_slab_stride = (long long)nl * inner;
      op.out_slab_stride = (long long)p->B * p->C_in * p->M;
      dst = partial;
    } else {
      dst = (j == 0) ? static_cast<void*>(Xhat) : static_cast<void*>(buf[flip]);
    }
    if (failed(launch_apply_dim(op, j == p->d - 1, false, cur, dst, st))) return DTST_ERR_CUDA;
    ++p->launches;
    cur = dst;
    flip ^= 1;
  }
  if (p->P > 1) {
    if (failed(launch_reduce_partials(partial, Xhat, (long long)p->B * p->C_in * p->M, p->P, st)))
      return DTST_ERR_CUDA;
    ++p->launches;
  }
  return DTST_OK;
}
