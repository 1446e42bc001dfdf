// The whole step (F, M, I, B) for callers whose activations live in HOST memory: dtst_step_host copies x and grad_y
// in, runs the four calls and copies y, grad_x and grad_W out, with the transfers overlapped with the kernels and
// with each other on three internal streams (copy-in, compute, copy-out) chained by events - also across
// consecutive steps.  The streams and events are created once by dtst_plan_enable_host_io; a step allocates
// nothing.  Pinned (page-locked) host buffers give asynchronous copies; pageable ones work but serialise.
#include "dtst_common.cuh"

#include <new>

using namespace dtst;

struct dtst_host_io {
  char* dev;                 // caller-owned device staging: x, g, y, gx, Xhat, Yhat, gW
  size_t off_x, off_g, off_y, off_gx, off_X, off_Y, off_gW, total;
  cudaStream_t s_in, s_cmp, s_out;
  cudaEvent_t ev_x, ev_g, ev_fwd_read, ev_y, ev_b, ev_y_copied, ev_done;
  bool first;
};

namespace {

inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

void layout(const dtst_plan* p, dtst_host_io* h) {
  const size_t gin = (size_t)p->B * p->C_in * p->points_local * sizeof(float);
  const size_t gout = (size_t)p->B * p->C_out * p->points_local * sizeof(float);
  const size_t sin = (size_t)p->B * p->C_in * p->M * sizeof(float2), sout = (size_t)p->B * p->C_out * p->M * sizeof(float2);
  const size_t w = (size_t)p->C_in * p->C_out * p->M * sizeof(float2);
  size_t o = 0;
  h->off_x = o; o += up256(gin);
  h->off_g = o; o += up256(gout);
  h->off_y = o; o += up256(gout);
  h->off_gx = o; o += up256(gin);
  h->off_X = o; o += up256(sin);
  h->off_Y = o; o += up256(sout);
  h->off_gW = o; o += up256(w);
  h->total = o;
}

void destroy(dtst_host_io* h) {
  if (h == nullptr) return;
  cudaStream_t* ss[3] = {&h->s_in, &h->s_cmp, &h->s_out};
  for (auto s : ss) if (*s) cudaStreamDestroy(*s);
  cudaEvent_t* es[7] = {&h->ev_x, &h->ev_g, &h->ev_fwd_read, &h->ev_y, &h->ev_b, &h->ev_y_copied, &h->ev_done};
  for (auto e : es) if (*e) cudaEventDestroy(*e);
  delete h;
}

}  // namespace

namespace dtst {
void host_io_release(dtst_plan* p) {
  destroy(p->host_io);
  p->host_io = nullptr;
}
}  // namespace dtst

extern "C" {

dtst_status dtst_plan_host_io_bytes(const dtst_plan* p, size_t* bytes) {
  if (p == nullptr || bytes == nullptr || p->complex_io) return DTST_ERR_INVALID_ARG;
  dtst_host_io tmp{};
  layout(p, &tmp);
  *bytes = tmp.total;
  return DTST_OK;
}

dtst_status dtst_plan_enable_host_io(dtst_plan* p, void* dev_staging, size_t bytes) {
  if (p == nullptr || p->complex_io) return DTST_ERR_INVALID_ARG;
  host_io_release(p);
  if (dev_staging == nullptr) return DTST_OK;   // switched off
  if ((reinterpret_cast<uintptr_t>(dev_staging) & 255u) != 0) return DTST_ERR_INVALID_ARG;
  dtst_host_io* h = new (std::nothrow) dtst_host_io{};
  if (h == nullptr) return DTST_ERR_ALLOC;
  layout(p, h);
  if (bytes < h->total) {
    delete h;
    return DTST_ERR_WORKSPACE;
  }
  h->dev = static_cast<char*>(dev_staging);
  h->first = true;
  bool ok = cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&h->s_cmp, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking) == cudaSuccess;
  cudaEvent_t* es[7] = {&h->ev_x, &h->ev_g, &h->ev_fwd_read, &h->ev_y, &h->ev_b, &h->ev_y_copied, &h->ev_done};
  for (auto e : es) ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    p->last_cuda_error = (int)cudaGetLastError();
    destroy(h);
    return DTST_ERR_CUDA;
  }
  p->host_io = h;
  return DTST_OK;
}

dtst_status dtst_step_host(dtst_plan* p, const float* hx, const float* hgy, const void* dW, float* hy, float* hgx,
                           void* hgW) {
  if (p == nullptr || p->host_io == nullptr || hx == nullptr || hgy == nullptr || dW == nullptr || hy == nullptr ||
      hgx == nullptr || hgW == nullptr)
    return DTST_ERR_INVALID_ARG;
  dtst_host_io* h = p->host_io;
  const size_t gin = (size_t)p->B * p->C_in * p->points_local * sizeof(float);
  const size_t gout = (size_t)p->B * p->C_out * p->points_local * sizeof(float);
  const size_t w = (size_t)p->C_in * p->C_out * p->M * sizeof(float2);
  float* x = reinterpret_cast<float*>(h->dev + h->off_x);
  float* g = reinterpret_cast<float*>(h->dev + h->off_g);
  float* y = reinterpret_cast<float*>(h->dev + h->off_y);
  float* gx = reinterpret_cast<float*>(h->dev + h->off_gx);
  void* X = h->dev + h->off_X;
  void* Y = h->dev + h->off_Y;
  void* gW = h->dev + h->off_gW;
  auto fail = [p](cudaError_t e) {
    if (e == cudaSuccess) return false;
    p->last_cuda_error = (int)e;
    (void)cudaGetLastError();
    return true;
  };
#define DTST_TRY(call) do { if (fail(call)) return DTST_ERR_CUDA; } while (0)
  // copy-in stream
  if (!h->first) DTST_TRY(cudaStreamWaitEvent(h->s_in, h->ev_fwd_read, 0));   // the previous F has consumed x
  DTST_TRY(cudaMemcpyAsync(x, hx, gin, cudaMemcpyHostToDevice, h->s_in));
  DTST_TRY(cudaEventRecord(h->ev_x, h->s_in));
  if (!h->first) DTST_TRY(cudaStreamWaitEvent(h->s_in, h->ev_b, 0));          // the previous B has consumed grad_y
  DTST_TRY(cudaMemcpyAsync(g, hgy, gout, cudaMemcpyHostToDevice, h->s_in));
  DTST_TRY(cudaEventRecord(h->ev_g, h->s_in));
  // compute stream
  DTST_TRY(cudaStreamWaitEvent(h->s_cmp, h->ev_x, 0));
  dtst_status s = dtst_forward(p, x, X, h->s_cmp);
  if (s != DTST_OK) return s;
  DTST_TRY(cudaEventRecord(h->ev_fwd_read, h->s_cmp));
  s = dtst_spectral_mul(p, X, dW, Y, h->s_cmp);
  if (s != DTST_OK) return s;
  if (!h->first) DTST_TRY(cudaStreamWaitEvent(h->s_cmp, h->ev_y_copied, 0));  // the previous y has left the device
  s = dtst_inverse(p, Y, y, h->s_cmp);
  if (s != DTST_OK) return s;
  DTST_TRY(cudaEventRecord(h->ev_y, h->s_cmp));
  DTST_TRY(cudaStreamWaitEvent(h->s_cmp, h->ev_g, 0));
  if (!h->first) DTST_TRY(cudaStreamWaitEvent(h->s_cmp, h->ev_done, 0));      // previous grad_x / grad_W have left
  s = dtst_backward(p, g, X, dW, gx, gW, h->s_cmp);
  if (s != DTST_OK) return s;
  DTST_TRY(cudaEventRecord(h->ev_b, h->s_cmp));
  // copy-out stream
  DTST_TRY(cudaStreamWaitEvent(h->s_out, h->ev_y, 0));
  DTST_TRY(cudaMemcpyAsync(hy, y, gout, cudaMemcpyDeviceToHost, h->s_out));
  DTST_TRY(cudaEventRecord(h->ev_y_copied, h->s_out));
  DTST_TRY(cudaStreamWaitEvent(h->s_out, h->ev_b, 0));
  DTST_TRY(cudaMemcpyAsync(hgx, gx, gin, cudaMemcpyDeviceToHost, h->s_out));
  DTST_TRY(cudaMemcpyAsync(hgW, gW, w, cudaMemcpyDeviceToHost, h->s_out));
  DTST_TRY(cudaEventRecord(h->ev_done, h->s_out));
#undef DTST_TRY
  h->first = false;
  return DTST_OK;
}

dtst_status dtst_host_io_wait(dtst_plan* p) {
  if (p == nullptr || p->host_io == nullptr) return DTST_ERR_INVALID_ARG;
  if (p->host_io->first) return DTST_OK;
  if (cudaEventSynchronize(p->host_io->ev_done) != cudaSuccess) {
    p->last_cuda_error = (int)cudaGetLastError();
    return DTST_ERR_CUDA;
  }
  return DTST_OK;
}

}  // extern "C"
