// mq_w4a8_msq_linear_noalloc: the W4A8 MSQ linear for callers that have no way of
// providing a workspace.
//
// Who needs it.  mq_w4a8_msq_linear asks its caller for scratch (the int8 activation codes,
// the split-K partial sums of the small-T path and the status word).  A caller normally
// gets that buffer from cudaMalloc or from its framework's caching allocator.  Some cannot:
// a plugin that runs inside somebody else's inference loop and is handed only its input
// and output tensors; code on a latency-critical decode step where an allocation may take
// a device-wide lock or trigger a synchronising free; a process whose device memory has
// been handed over entirely to another pool, so that cudaMalloc would simply fail.  For
// them the scratch lives in a fixed array that is part of this library's device image.
//
// Cost and limit.  The array is MQ_NOALLOC_WS_BYTES (4 MiB) of global memory on EVERY
// device that loads the library, held until the process exits.  It is sized for
// decode-shaped calls: the int8 codes (T * K bytes) plus one [T, N] int32 slice per K split
// must fit, which admits e.g. K = 4096, N = 13696 up to T = 256 but K = 13696, N = 4096
// (four K splits) only up to T = 48.  Larger problems are rejected with MQ_ERR_WORKSPACE
// and must use mq_w4a8_msq_linear with a caller-owned workspace.
//
// The array's name is only a handle in host code -- it is not a device address -- so the
// address is looked up with cudaGetSymbolAddress, once per device, with that device
// current, and that pointer is what the kernels receive.
#include <mutex>

#include "mq_common.cuh"

namespace {

static __device__ __align__(256) unsigned char g_noalloc_ws[MQ_NOALLOC_WS_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_ws_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device (nullptr on failure).
void* noalloc_ws_for_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_ws_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_ws) != cudaSuccess || !p) return nullptr;
    g_ws_ptr[dev] = p;
  }
  return g_ws_ptr[dev];
}

}  // namespace

extern "C" int mq_w4a8_msq_linear_noalloc(const mq_linear_desc* d, const void* X, int64_t ldx,
                                          const mq_segments* seg, float s_vis, float s_txt,
                                          const void* W_layout, const float* s_w, const float* bias,
                                          void* Y, int64_t ldy, int32_t* acc_out, int32_t* status_out,
                                          void* stream) {
  if (!d) return MQ_ERR_INVALID_ARG;
  if (d->T < 0 || d->K <= 0 || d->N <= 0) return MQ_ERR_INVALID_ARG;
  const size_t need = mq_workspace_bytes(d);
  if (need == 0) {
    // bad descriptor: let the main entry point name the reason (it touches no memory then)
    return mq_w4a8_msq_linear(d, X, ldx, seg, s_vis, s_txt, W_layout, s_w, bias, Y, ldy, acc_out, nullptr, 0,
                              stream);
  }
  if (need > (size_t)MQ_NOALLOC_WS_BYTES) return MQ_ERR_WORKSPACE;
  void* ws = noalloc_ws_for_current_device();
  if (!ws) return MQ_ERR_CUDA;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the previous call left.  The status word is sticky, so it must
  // start from MQ_OK; the activation codes are fully rewritten, and every K split overwrites
  // its own [T, N] slice with plain stores before the finalize kernel reads it.
  if (cudaMemsetAsync(ws, 0, mq::kStatusBytes, cs) != cudaSuccess) return MQ_ERR_CUDA;
  const int rc = mq_w4a8_msq_linear(d, X, ldx, seg, s_vis, s_txt, W_layout, s_w, bias, Y, ldy, acc_out, ws,
                                    (size_t)MQ_NOALLOC_WS_BYTES, stream);
  if (rc != MQ_OK) return rc;
  if (status_out &&
      cudaMemcpyAsync(status_out, ws, 2 * sizeof(int32_t), cudaMemcpyDeviceToDevice, cs) != cudaSuccess)
    return MQ_ERR_CUDA;
  return MQ_OK;
}
