// Shared device/host helpers of the MSQ W4A8 kernels (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "mq.h"
#include "mq_device_table.h"

namespace mq {

// ---- workspace layout -------------------------------------------------------------
// [0,256)   status block: int32 status, int32 site, reserved
// [256, ..) int8 activation codes (when X arrives as bf16), then split-K accumulators
constexpr size_t kStatusBytes = 256;

struct SegTable {
  int n_seg;
  const int32_t* seg_end;
  const uint8_t* seg_mod;
};

__host__ __device__ inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Modality of row t, looked up cooperatively by one warp (all 32 lanes must call).
// Row t belongs to the first segment whose exclusive end exceeds t; text otherwise.
__device__ __forceinline__ int warp_row_modality(const SegTable& seg, int t) {
  const int lane = threadIdx.x & 31;
  for (int base = 0; base < seg.n_seg; base += 32) {
    const int i = base + lane;
    const bool hit = (i < seg.n_seg) && (t < seg.seg_end[i]);
    const unsigned m = __ballot_sync(0xffffffffu, hit);
    if (m) {
      const int first = base + __ffs(m) - 1;
      return seg.seg_mod[first] ? MQ_VISUAL : MQ_TEXT;
    }
  }
  return MQ_TEXT;
}

// Same lookup by a single thread (used where one thread owns one row / column).
__device__ __forceinline__ int thread_row_modality(const SegTable& seg, int t) {
  for (int i = 0; i < seg.n_seg; ++i)
    if (t < seg.seg_end[i]) return seg.seg_mod[i] ? MQ_VISUAL : MQ_TEXT;
  return MQ_TEXT;
}

// A failed runtime call also leaves its error in the runtime's per-thread "last error" slot, where the
// next launcher's cudaGetLastError() would find it: clear it when reporting the failure.
inline int cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return MQ_OK;
  (void)cudaGetLastError();
  return MQ_ERR_CUDA;
}

// ---- per-device host state ------------------------------------------------------------
// SM count of the CURRENT device (148 if the query fails), cached per device.
inline int sm_count() {
  static PerDeviceTable<int> table;
  int dev = -1, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) dev = -1;
  const bool ok = table.get(dev, [](int d, int* out) {
    return d >= 0 && cudaDeviceGetAttribute(out, cudaDevAttrMultiProcessorCount, d) == cudaSuccess && *out > 0;
  }, &n);
  return ok ? n : 148;
}

// Raises `kernel`'s dynamic shared-memory limit to `bytes` on the current device, once per device
// (function attributes belong to the device's context, not to the process).  `table` is the
// caller's static table for that kernel.
template <typename Kernel>
inline bool ensure_dynamic_smem(PerDeviceTable<char>& table, Kernel kernel, int bytes) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) dev = -1;
  char done = 0;
  const bool ok = table.get(dev, [&](int, char* out) {
    *out = 1;
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
  }, &done);
  if (!ok) (void)cudaGetLastError();
  return ok;
}

// ---- programmatic dependent launch ----------------------------------------------------
// The hot-path kernels follow one another on a stream, each a few tens of microseconds long,
// so the launch latency between them is a visible share of a step.  They are launched with
// programmatic stream serialization: a kernel lets its successor start launching at once
// (pdl_launch_dependents at its top), and every such kernel executes pdl_wait -- which returns
// once the preceding kernel has completed and its writes are visible -- after its private
// set-up and BEFORE it reads or writes any global memory other than its parameters.  Because
// every kernel of the chain waits before it exits, completion is transitive along the chain.
// On a launch without the attribute both instructions do nothing.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_ordered(bool programmatic, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                  cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = programmatic ? 1 : 0;  // 0: plain stream order
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
  return launch_ordered(true, kernel, grid, block, smem, st, static_cast<Args&&>(args)...);
}

// host launchers implemented in the .cu files -----------------------------------------
int launch_fwht_quant(const void* X, int T, int K, int64_t ldx, SegTable seg, float s_vis,
                      float s_txt, int rot_block, int8_t* Q, int64_t ldq, float* rotated_out,
                      cudaStream_t st, int8_t* side_out = nullptr, int side_ld = 0, int act_bits = 8);
int launch_kron_quant(const void* X, int T, int K, int64_t ldx, SegTable seg, float s_vis, float s_txt, int m,
                      const uint8_t* h_neg, int8_t* Q, int64_t ldq, float* rotated_out, cudaStream_t st);
int launch_dyn_quant(const void* X, int T, int K, int64_t ldx, int rot_block, int8_t* Q, int64_t ldq, float* s_rows,
                     cudaStream_t st);
int launch_calibrate(const void* X, int T, int K, int64_t ldx, SegTable seg, int rot_block,
                     int accumulate, uint32_t* amax_state, float* s_vis_out, float* s_txt_out,
                     cudaStream_t st, int act_bits = 8);
int launch_pack_w4(const float* W, int N, int K, int64_t ldw, uint8_t* packed, float* s_w,
                   void* layout, cudaStream_t st, int group = 0);
int launch_pack_codes(const float* W, int N, int K, int64_t ldw, const float* s_w, uint8_t* packed,
                      void* layout, int skip, cudaStream_t st, int group = 0);
int launch_pack_w8(const float* W, int N, int K, int64_t ldw, int8_t* q_out, int64_t ldq, float* s_w, void* layout,
                   cudaStream_t st);
int launch_repack_w4(const uint8_t* packed, int N, int K, void* layout, cudaStream_t st);
int launch_unpack_w4(const uint8_t* packed, const void* layout, int N, int K, int8_t* q,
                     int64_t ldq, cudaStream_t st);
int launch_aifs_reorder(const void* X, void* X_out, int L, int D, int64_t ldx, int64_t ldo,
                        const uint8_t* is_visual, const uint8_t* is_pad, int32_t* perm,
                        int32_t* inv_perm, int32_t* n_first_out, int direction, cudaStream_t st);
int launch_mask_remap(const int32_t* perm, const int32_t* pos_ids, const uint8_t* is_pad,
                      const int32_t* n_first, int L, int32_t* pos_out, int32_t* seg_end_out,
                      uint8_t* seg_mod_out, uint8_t* dense, cudaStream_t st);

// rotation magnitude suppression (mq_rms.cu)
int launch_rms_detect(const float* W, int N, int K, int64_t ldw, int nb, uint8_t* flags, int32_t* count,
                      cudaStream_t st);
int launch_rms_pack(const float* W, int N, int K, int64_t ldw, int nb, uint8_t* packed, float* s_w, void* layout,
                    int8_t* q_side, int side_k, float* s_w_side, void* side_layout, cudaStream_t st);
int launch_layout_from_codes(const int8_t* q, int64_t ldq, int N, int K, void* layout, cudaStream_t st);

struct GemmArgs {
  int T, K, N;
  const int8_t* Qx;
  int64_t ldq;
  // launch_gemv only, when Qx == nullptr: bf16 activations that the kernel rotates and quantizes itself
  const void* Xb;
  int64_t ldx;
  int rot_block;
  SegTable seg;
  float s_vis, s_txt;
  const void* W_layout;
  const float* s_w;
  const float* bias;
  void* Y;
  int64_t ldy;
  int y_is_f32;
  int32_t* acc_out;
  int32_t* status;     // device int32[2]: status, site
  int32_t* splitk_acc; // device int32 scratch of gemm_splitk_bytes (small-T path) or nullptr
  const float* row_scales;  // optional device float [T]: per-token activation scales (dynamic comparison path)
  // Split part of the rotation-magnitude-suppression linear (side_layout != nullptr selects it):
  // a second product on K = side_k with its own weights and scale, accumulated beside the main one
  // and added in the epilogue:  y = fl(acc * fl(s_a s_w)) + fl(acc_side * fl(s_a s_w_side)) (+ bias).
  const int8_t* Qs;    // activation codes of the split product [T, side_cols], pitch side_k
  int side_k;          // multiple of 32
  int side_cols;       // columns of Qs that hold codes (<= side_k); the rest is never read
  const void* side_layout;
  const float* s_w_side;
  int32_t* acc_side_out;
  // Variants: group_size = 128 selects group-wise weight scales (s_w is then [K / 128][N]; acc_out, if given,
  // receives the per-group accumulators [K / 128][T][N]); w_bits = 8 selects 8-bit weights (W_layout from
  // mq_pack_w8).  0 / 0 is the W4 per-channel hot path.
  int group_size;
  int w_bits;
};
int launch_gemm(const GemmArgs& a, cudaStream_t st);
// one to three tokens: CUDA-core GEMV (mq_gemv.cu); launch_gemm routes there when it applies
bool gemv_applies(int T, int K, int N, int side_k = 0);
int launch_gemv(const GemmArgs& a, cudaStream_t st);
size_t gemm_splitk_bytes(int T, int K, int N, bool rms = false, int group_size = 0, int w_bits = 4);

}  // namespace mq
