// C ABI of the library: host-side argument validation and dispatch to the kernel launchers.
// Nothing here allocates device memory or synchronises (except mq_last_device_status).
#include <cmath>
#include <cstring>

#include "mq_common.cuh"

namespace {

using namespace mq;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline bool good_scale(float s) { return std::isfinite(s) && s > 0.0f; }

int check_rot(int rot_block, int K) {
  if (rot_block == 0) return MQ_OK;
  if (rot_block < 0) return MQ_ERR_INVALID_ARG;
  if (rot_block & (rot_block - 1)) return MQ_ERR_INVALID_ARG;
  if (rot_block < 32 || rot_block > 1024) return MQ_ERR_UNSUPPORTED;
  if (K % rot_block) return MQ_ERR_INVALID_ARG;
  return MQ_OK;
}

int check_seg(const mq_segments* seg, SegTable* out) {
  out->n_seg = 0;
  out->seg_end = nullptr;
  out->seg_mod = nullptr;
  if (!seg) return MQ_OK;  // no table: every row is text
  if (seg->n_seg < 0) return MQ_ERR_INVALID_ARG;
  if (seg->n_seg > 0 && (!seg->seg_end || !seg->seg_mod)) return MQ_ERR_INVALID_ARG;
  out->n_seg = seg->n_seg;
  out->seg_end = seg->seg_end;
  out->seg_mod = seg->seg_mod;
  return MQ_OK;
}

int check_desc(const mq_linear_desc* d) {
  if (!d) return MQ_ERR_INVALID_ARG;
  if (d->T < 0 || d->K <= 0 || d->N <= 0) return MQ_ERR_INVALID_ARG;
  if (d->K % 32 || d->N % 16) return MQ_ERR_INVALID_ARG;
  if (d->K > 131040) return MQ_ERR_UNSUPPORTED;  // 16x accumulators must stay below 2^31
  if (d->group_size < 0) return MQ_ERR_INVALID_ARG;
  if (d->group_size != 0 && d->group_size != MQ_W_TILE_K) return MQ_ERR_UNSUPPORTED;  // a group is one K block
  if (d->group_size && d->K % MQ_W_TILE_K) return MQ_ERR_INVALID_ARG;
  if (d->flags & ~(MQ_FLAG_X_IS_INT8 | MQ_FLAG_Y_IS_F32 | MQ_FLAG_A4 | MQ_FLAG_W8)) return MQ_ERR_INVALID_ARG;
  if ((d->flags & MQ_FLAG_W8) && d->group_size) return MQ_ERR_UNSUPPORTED;
  if (d->flags & MQ_FLAG_X_IS_INT8) {
    if (d->rot_block != 0) return MQ_ERR_INVALID_ARG;
    return MQ_OK;
  }
  return check_rot(d->rot_block, d->K);
}

struct WsLayout {
  size_t qx_off, qx_bytes, splitk_off, splitk_bytes, total;
};
WsLayout ws_layout(const mq_linear_desc* d) {
  WsLayout w{};
  w.qx_off = kStatusBytes;
  w.qx_bytes = (d->flags & MQ_FLAG_X_IS_INT8) ? 0 : align_up((size_t)d->T * d->K, 256);
  w.splitk_off = w.qx_off + w.qx_bytes;
  w.splitk_bytes = align_up(gemm_splitk_bytes(d->T, d->K, d->N, false, d->group_size, (d->flags & MQ_FLAG_W8) ? 8 : 4), 256);
  w.total = w.splitk_off + w.splitk_bytes;
  return w;
}

}  // namespace

extern "C" {

int mq_version(void) { return MQ_VERSION; }

const char* mq_status_string(int status) {
  switch (status) {
    case MQ_OK: return "MQ_OK";
    case MQ_ERR_INVALID_ARG: return "MQ_ERR_INVALID_ARG";
    case MQ_ERR_UNSUPPORTED: return "MQ_ERR_UNSUPPORTED";
    case MQ_ERR_ALIGNMENT: return "MQ_ERR_ALIGNMENT";
    case MQ_ERR_CUDA: return "MQ_ERR_CUDA";
    case MQ_ERR_TIMEOUT: return "MQ_ERR_TIMEOUT";
    case MQ_ERR_WORKSPACE: return "MQ_ERR_WORKSPACE";
    default: return "MQ_ERR_UNKNOWN";
  }
}

size_t mq_workspace_bytes(const mq_linear_desc* d) {
  if (check_desc(d) != MQ_OK) return 0;
  return ws_layout(d).total;
}

size_t mq_w4_layout_bytes(int32_t N, int32_t K) {
  if (N <= 0 || K <= 0) return 0;
  const size_t tn = (N + MQ_W_TILE_N - 1) / MQ_W_TILE_N, kb = (K + MQ_W_TILE_K - 1) / MQ_W_TILE_K;
  return tn * kb * (size_t)(MQ_W_TILE_N * MQ_W_TILE_K / 2);
}

int mq_calibrate_static_scales(const void* X, int32_t T, int32_t K, int64_t ldx, const mq_segments* seg,
                               int32_t rot_block, int32_t accumulate, uint32_t* amax_state, float* s_vis_out,
                               float* s_txt_out, void* stream) {
  if (T < 0 || K <= 0 || K % 32) return MQ_ERR_INVALID_ARG;
  if (!amax_state || !s_vis_out || !s_txt_out) return MQ_ERR_INVALID_ARG;
  if (T > 0 && !X) return MQ_ERR_INVALID_ARG;
  if (ldx < K) return MQ_ERR_INVALID_ARG;
  if (!aligned16(X) || (ldx * 2) % 16) return MQ_ERR_ALIGNMENT;
  int rc = check_rot(rot_block, K);
  if (rc != MQ_OK) return rc;
  SegTable st;
  if ((rc = check_seg(seg, &st)) != MQ_OK) return rc;
  return launch_calibrate(X, T, K, ldx, st, rot_block, accumulate, amax_state, s_vis_out, s_txt_out,
                          static_cast<cudaStream_t>(stream));
}

int mq_calibrate_static_scales_bits(const void* X, int32_t T, int32_t K, int64_t ldx, const mq_segments* seg,
                                    int32_t rot_block, int32_t act_bits, int32_t accumulate, uint32_t* amax_state,
                                    float* s_vis_out, float* s_txt_out, void* stream) {
  if (act_bits != 4 && act_bits != 8) return MQ_ERR_UNSUPPORTED;
  if (T < 0 || K <= 0 || K % 32) return MQ_ERR_INVALID_ARG;
  if (!amax_state || !s_vis_out || !s_txt_out) return MQ_ERR_INVALID_ARG;
  if (T > 0 && !X) return MQ_ERR_INVALID_ARG;
  if (ldx < K) return MQ_ERR_INVALID_ARG;
  if (!aligned16(X) || (ldx * 2) % 16) return MQ_ERR_ALIGNMENT;
  int rc = check_rot(rot_block, K);
  if (rc != MQ_OK) return rc;
  SegTable st;
  if ((rc = check_seg(seg, &st)) != MQ_OK) return rc;
  return launch_calibrate(X, T, K, ldx, st, rot_block, accumulate, amax_state, s_vis_out, s_txt_out,
                          static_cast<cudaStream_t>(stream), act_bits);
}

int mq_pack_w4(const float* W, int32_t N, int32_t K, int64_t ldw, int32_t group_size, uint8_t* packed, float* s_w,
               void* gemm_layout, void* stream) {
  if (N <= 0 || K <= 0 || !W || !s_w) return MQ_ERR_INVALID_ARG;
  if (K % 32 || N % 16 || ldw < K || group_size < 0) return MQ_ERR_INVALID_ARG;
  if (group_size != 0 && group_size != MQ_W_TILE_K) return MQ_ERR_UNSUPPORTED;
  if (group_size && K % group_size) return MQ_ERR_INVALID_ARG;
  if (gemm_layout && !aligned(gemm_layout, 128)) return MQ_ERR_ALIGNMENT;
  return launch_pack_w4(W, N, K, ldw, packed, s_w, gemm_layout, static_cast<cudaStream_t>(stream), group_size);
}

size_t mq_w8_layout_bytes(int32_t N, int32_t K) { return 2 * mq_w4_layout_bytes(N, K); }

int mq_pack_w8(const float* W, int32_t N, int32_t K, int64_t ldw, int8_t* q_out, int64_t ldq, float* s_w,
               void* gemm_layout, void* stream) {
  if (N <= 0 || K <= 0 || !W || !s_w || (!q_out && !gemm_layout)) return MQ_ERR_INVALID_ARG;
  if (K % 32 || N % 16 || ldw < K || (q_out && ldq < K)) return MQ_ERR_INVALID_ARG;
  if (gemm_layout && !aligned(gemm_layout, 128)) return MQ_ERR_ALIGNMENT;
  return launch_pack_w8(W, N, K, ldw, q_out, ldq, s_w, gemm_layout, static_cast<cudaStream_t>(stream));
}

int mq_repack_w4(const uint8_t* packed, int32_t N, int32_t K, void* gemm_layout, void* stream) {
  if (N <= 0 || K <= 0 || !packed || !gemm_layout) return MQ_ERR_INVALID_ARG;
  if (K % 32 || N % 16) return MQ_ERR_INVALID_ARG;
  if (!aligned(gemm_layout, 128)) return MQ_ERR_ALIGNMENT;
  return launch_repack_w4(packed, N, K, gemm_layout, static_cast<cudaStream_t>(stream));
}

int mq_unpack_w4(const uint8_t* packed, const void* gemm_layout, int32_t N, int32_t K, int8_t* q_out, int64_t ldq,
                 void* stream) {
  if (N <= 0 || K <= 0 || !q_out || (!packed && !gemm_layout)) return MQ_ERR_INVALID_ARG;
  if (K % 32 || N % 16 || ldq < K) return MQ_ERR_INVALID_ARG;
  return launch_unpack_w4(packed, gemm_layout, N, K, q_out, ldq, static_cast<cudaStream_t>(stream));
}

int mq_aifs_reorder(const void* X, void* X_out, int32_t L, int32_t D, int64_t ldx, int64_t ldo,
                    const uint8_t* is_visual, const uint8_t* is_pad, int32_t* perm, int32_t* inv_perm,
                    int32_t* n_first_out, int32_t direction, void* stream) {
  if (L < 0 || D < 0 || (direction != 0 && direction != 1)) return MQ_ERR_INVALID_ARG;
  if ((X == nullptr) != (X_out == nullptr)) return MQ_ERR_INVALID_ARG;
  if (X && X == X_out) return MQ_ERR_INVALID_ARG;
  if (!perm && L > 0) return MQ_ERR_INVALID_ARG;
  if (direction == 0 && L > 0 && !is_visual) return MQ_ERR_INVALID_ARG;
  if (X) {
    if (D % 8) return MQ_ERR_ALIGNMENT;
    if (ldx < D || ldo < D) return MQ_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(X_out) || (ldx * 2) % 16 || (ldo * 2) % 16) return MQ_ERR_ALIGNMENT;
  }
  return launch_aifs_reorder(X, X_out, L, D, ldx, ldo, is_visual, is_pad, perm, inv_perm, n_first_out, direction,
                             static_cast<cudaStream_t>(stream));
}

int mq_attn_mask_remap(const int32_t* perm, const int32_t* pos_ids, const uint8_t* is_pad, const int32_t* n_first,
                       int32_t L, int32_t* pos_ids_out, int32_t* seg_end_out, uint8_t* seg_mod_out,
                       uint8_t* dense_mask_out, void* stream) {
  if (L < 0) return MQ_ERR_INVALID_ARG;
  if (L > 0 && !perm) return MQ_ERR_INVALID_ARG;
  if ((seg_end_out == nullptr) != (seg_mod_out == nullptr)) return MQ_ERR_INVALID_ARG;
  if (seg_end_out && !n_first) return MQ_ERR_INVALID_ARG;
  if (dense_mask_out && L > 16384) return MQ_ERR_UNSUPPORTED;
  return launch_mask_remap(perm, pos_ids, is_pad, n_first, L, pos_ids_out, seg_end_out, seg_mod_out,
                           dense_mask_out, static_cast<cudaStream_t>(stream));
}

int mq_fwht_quant_i8(const void* X, int32_t T, int32_t K, int64_t ldx, const mq_segments* seg, float s_vis,
                     float s_txt, int32_t rot_block, int8_t* Q, int64_t ldq, float* rotated_out, void* stream) {
  if (T < 0 || K <= 0 || K % 32) return MQ_ERR_INVALID_ARG;
  if (T > 0 && (!X || !Q)) return MQ_ERR_INVALID_ARG;
  if (ldx < K || ldq < K) return MQ_ERR_INVALID_ARG;
  if (!good_scale(s_vis) || !good_scale(s_txt)) return MQ_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(Q) || (ldx * 2) % 16 || ldq % 16) return MQ_ERR_ALIGNMENT;
  if (rotated_out && !aligned16(rotated_out)) return MQ_ERR_ALIGNMENT;
  int rc = check_rot(rot_block, K);
  if (rc != MQ_OK) return rc;
  SegTable st;
  if ((rc = check_seg(seg, &st)) != MQ_OK) return rc;
  return launch_fwht_quant(X, T, K, ldx, st, s_vis, s_txt, rot_block, Q, ldq, rotated_out,
                           static_cast<cudaStream_t>(stream));
}

int mq_kron_quant_i8(const void* X, int32_t T, int32_t K, int64_t ldx, const mq_segments* seg, float s_vis, float s_txt,
                     int32_t m, const uint8_t* h_neg, int8_t* Q, int64_t ldq, float* rotated_out, void* stream) {
  if (T < 0 || K <= 0 || m < 1 || m > 256 || K % m) return MQ_ERR_INVALID_ARG;
  const int n2 = K / m;
  if (n2 & (n2 - 1)) return MQ_ERR_INVALID_ARG;               // K / m must be a power of two
  if (n2 < 32 || n2 > 1024) return MQ_ERR_UNSUPPORTED;
  if ((size_t)K * sizeof(float) + (size_t)m * m > 200 * 1024) return MQ_ERR_UNSUPPORTED;  // the row lives in shared memory
  if (T > 0 && (!X || !Q || !h_neg)) return MQ_ERR_INVALID_ARG;
  if (ldx < K || ldq < K) return MQ_ERR_INVALID_ARG;
  if (!good_scale(s_vis) || !good_scale(s_txt)) return MQ_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(Q) || (ldx * 2) % 16 || ldq % 16) return MQ_ERR_ALIGNMENT;
  if (rotated_out && !aligned16(rotated_out)) return MQ_ERR_ALIGNMENT;
  SegTable st;
  const int rc = check_seg(seg, &st);
  if (rc != MQ_OK) return rc;
  return launch_kron_quant(X, T, K, ldx, st, s_vis, s_txt, m, h_neg, Q, ldq, rotated_out,
                           static_cast<cudaStream_t>(stream));
}

int mq_fwht_quant_bits(const void* X, int32_t T, int32_t K, int64_t ldx, const mq_segments* seg, float s_vis,
                       float s_txt, int32_t rot_block, int32_t act_bits, int8_t* Q, int64_t ldq, void* stream) {
  if (act_bits != 4 && act_bits != 8) return MQ_ERR_UNSUPPORTED;
  if (T < 0 || K <= 0 || K % 32) return MQ_ERR_INVALID_ARG;
  if (T > 0 && (!X || !Q)) return MQ_ERR_INVALID_ARG;
  if (ldx < K || ldq < K) return MQ_ERR_INVALID_ARG;
  if (!good_scale(s_vis) || !good_scale(s_txt)) return MQ_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(Q) || (ldx * 2) % 16 || ldq % 16) return MQ_ERR_ALIGNMENT;
  int rc = check_rot(rot_block, K);
  if (rc != MQ_OK) return rc;
  SegTable st;
  if ((rc = check_seg(seg, &st)) != MQ_OK) return rc;
  return launch_fwht_quant(X, T, K, ldx, st, s_vis, s_txt, rot_block, Q, ldq, nullptr,
                           static_cast<cudaStream_t>(stream), nullptr, 0, act_bits);
}

int mq_w4a8_msq_linear(const mq_linear_desc* d, const void* X, int64_t ldx, const mq_segments* seg, float s_vis,
                       float s_txt, const void* W_layout, const float* s_w, const float* bias, void* Y, int64_t ldy,
                       int32_t* acc_out, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_desc(d);
  if (rc != MQ_OK) return rc;
  if (!good_scale(s_vis) || !good_scale(s_txt)) return MQ_ERR_INVALID_ARG;
  SegTable st;
  if ((rc = check_seg(seg, &st)) != MQ_OK) return rc;
  if (d->T == 0) return MQ_OK;
  if (!X || !W_layout || !s_w || !Y) return MQ_ERR_INVALID_ARG;
  if (ldx < d->K || ldy < d->N) return MQ_ERR_INVALID_ARG;
  const bool x_i8 = (d->flags & MQ_FLAG_X_IS_INT8) != 0;
  const bool y_f32 = (d->flags & MQ_FLAG_Y_IS_F32) != 0;
  if (!aligned16(X) || (ldx * (x_i8 ? 1 : 2)) % 16) return MQ_ERR_ALIGNMENT;
  if (!aligned(W_layout, 128) || !aligned16(Y) || !aligned16(s_w)) return MQ_ERR_ALIGNMENT;
  if (!ws) return MQ_ERR_WORKSPACE;
  if (!aligned(ws, 256)) return MQ_ERR_ALIGNMENT;
  const WsLayout wl = ws_layout(d);
  if (ws_bytes < wl.total) return MQ_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  uint8_t* wsb = static_cast<uint8_t*>(ws);

  const int8_t* qx;
  int64_t ldq;
  const int act_bits = (d->flags & MQ_FLAG_A4) ? 4 : 8;
  const int w_bits = (d->flags & MQ_FLAG_W8) ? 8 : 4;
  const bool variant = act_bits != 8 || w_bits != 4 || d->group_size != 0;  // neighbours of the hot path
  if (!variant && !x_i8 && gemv_applies(d->T, d->K, d->N)) {
    // one to three tokens: a single kernel rotates, quantizes and multiplies (mq_gemv.cu)
    GemmArgs g{};
    g.T = d->T; g.K = d->K; g.N = d->N;
    g.Xb = X; g.ldx = ldx; g.rot_block = d->rot_block; g.seg = st; g.s_vis = s_vis; g.s_txt = s_txt;
    g.W_layout = W_layout; g.s_w = s_w; g.bias = bias; g.Y = Y; g.ldy = ldy; g.y_is_f32 = y_f32 ? 1 : 0;
    g.acc_out = acc_out;
    return launch_gemv(g, cs);
  }
  if (x_i8) {
    qx = static_cast<const int8_t*>(X);
    ldq = ldx;
  } else {
    int8_t* q = reinterpret_cast<int8_t*>(wsb + wl.qx_off);
    rc = launch_fwht_quant(X, d->T, d->K, ldx, st, s_vis, s_txt, d->rot_block, q, d->K, nullptr, cs, nullptr, 0, act_bits);
    if (rc != MQ_OK) return rc;
    qx = q;
    ldq = d->K;
  }
  GemmArgs a{};
  a.T = d->T; a.K = d->K; a.N = d->N;
  a.group_size = d->group_size; a.w_bits = w_bits;
  a.Qx = qx; a.ldq = ldq; a.seg = st; a.s_vis = s_vis; a.s_txt = s_txt;
  a.W_layout = W_layout; a.s_w = s_w; a.bias = bias; a.Y = Y; a.ldy = ldy; a.y_is_f32 = y_f32 ? 1 : 0;
  a.acc_out = acc_out;
  a.status = reinterpret_cast<int32_t*>(wsb);
  a.splitk_acc = wl.splitk_bytes ? reinterpret_cast<int32_t*>(wsb + wl.splitk_off) : nullptr;
  return launch_gemm(a, cs);
}

// ---- rotation magnitude suppression (Sec. 3.2) -------------------------------------------
namespace {
int check_rms_shape(int32_t N, int32_t K, int32_t rot_block) {
  if (N <= 0 || K <= 0 || K % 32 || N % 16) return MQ_ERR_INVALID_ARG;
  if (rot_block == 0) return MQ_ERR_INVALID_ARG;  // the split columns are defined by the rotation block
  return check_rot(rot_block, K);
}
// K of the split product: one code per rotation block, padded to the GEMM's granularity.
int rms_side_k(int32_t K, int32_t rot_block) { return (int)align_up((size_t)(K / rot_block), 32); }

struct RmsWsLayout {
  size_t qx_off, xs_off, splitk_off, splitk_bytes, total;
};
RmsWsLayout rms_ws_layout(const mq_linear_desc* d) {
  RmsWsLayout w{};
  const int sk = rms_side_k(d->K, d->rot_block);
  w.qx_off = kStatusBytes;
  w.xs_off = w.qx_off + align_up((size_t)d->T * d->K, 256);
  w.splitk_off = w.xs_off + align_up((size_t)d->T * sk, 256);
  w.splitk_bytes = align_up(gemm_splitk_bytes(d->T, d->K, d->N, true), 256);
  w.total = w.splitk_off + w.splitk_bytes;
  return w;
}
}  // namespace

size_t mq_rms_side_ld(int32_t K, int32_t rot_block) {
  if (K <= 0 || K % 32 || rot_block == 0 || check_rot(rot_block, K) != MQ_OK) return 0;
  return (size_t)rms_side_k(K, rot_block);
}

int mq_rms_detect(const float* W, int32_t N, int32_t K, int64_t ldw, int32_t rot_block, uint8_t* flags,
                  int32_t* count_out, void* stream) {
  int rc = check_rms_shape(N, K, rot_block);
  if (rc != MQ_OK) return rc;
  if (!W || ldw < K || (!flags && !count_out)) return MQ_ERR_INVALID_ARG;
  return launch_rms_detect(W, N, K, ldw, rot_block, flags, count_out, static_cast<cudaStream_t>(stream));
}

int mq_pack_w4_rms(const float* W_rot, int32_t N, int32_t K, int64_t ldw, int32_t rot_block, uint8_t* packed,
                   float* s_w, void* gemm_layout, int8_t* q_side, float* s_w_side, void* side_layout,
                   void* stream) {
  int rc = check_rms_shape(N, K, rot_block);
  if (rc != MQ_OK) return rc;
  if (!W_rot || !s_w || !q_side || !s_w_side || ldw < K) return MQ_ERR_INVALID_ARG;
  if (gemm_layout && !aligned(gemm_layout, 128)) return MQ_ERR_ALIGNMENT;
  if (side_layout && !aligned(side_layout, 128)) return MQ_ERR_ALIGNMENT;
  return launch_rms_pack(W_rot, N, K, ldw, rot_block, packed, s_w, gemm_layout, q_side, rms_side_k(K, rot_block),
                         s_w_side, side_layout, static_cast<cudaStream_t>(stream));
}

size_t mq_rms_workspace_bytes(const mq_linear_desc* d) {
  if (check_desc(d) != MQ_OK || d->rot_block == 0 || (d->flags & MQ_FLAG_X_IS_INT8)) return 0;
  return rms_ws_layout(d).total;
}

int mq_w4a8_msq_linear_rms(const mq_linear_desc* d, const void* X, int64_t ldx, const mq_segments* seg, float s_vis,
                           float s_txt, const void* W_layout, const float* s_w, const void* side_layout,
                           const float* s_w_side, const float* bias, void* Y, int64_t ldy, int32_t* acc_out,
                           int32_t* acc_side_out, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_desc(d);
  if (rc != MQ_OK) return rc;
  if (d->rot_block == 0 || (d->flags & MQ_FLAG_X_IS_INT8)) return MQ_ERR_INVALID_ARG;
  if (!good_scale(s_vis) || !good_scale(s_txt)) return MQ_ERR_INVALID_ARG;
  SegTable st;
  if ((rc = check_seg(seg, &st)) != MQ_OK) return rc;
  if (d->T == 0) return MQ_OK;
  if (!X || !W_layout || !s_w || !side_layout || !s_w_side || !Y) return MQ_ERR_INVALID_ARG;
  if (ldx < d->K || ldy < d->N) return MQ_ERR_INVALID_ARG;
  if (!aligned16(X) || (ldx * 2) % 16) return MQ_ERR_ALIGNMENT;
  if (!aligned(W_layout, 128) || !aligned(side_layout, 128) || !aligned16(Y) || !aligned16(s_w) ||
      !aligned16(s_w_side))
    return MQ_ERR_ALIGNMENT;
  if (!ws) return MQ_ERR_WORKSPACE;
  if (!aligned(ws, 256)) return MQ_ERR_ALIGNMENT;
  const RmsWsLayout wl = rms_ws_layout(d);
  if (ws_bytes < wl.total) return MQ_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  uint8_t* wsb = static_cast<uint8_t*>(ws);
  const int sk = rms_side_k(d->K, d->rot_block);
  if (gemv_applies(d->T, d->K, d->N, sk)) {
    // one to three tokens: rotation, quantizer, both products and the epilogue in one GEMV kernel
    GemmArgs g{};
    g.T = d->T; g.K = d->K; g.N = d->N;
    g.Xb = X; g.ldx = ldx; g.rot_block = d->rot_block; g.seg = st; g.s_vis = s_vis; g.s_txt = s_txt;
    g.W_layout = W_layout; g.s_w = s_w; g.bias = bias; g.Y = Y; g.ldy = ldy;
    g.y_is_f32 = (d->flags & MQ_FLAG_Y_IS_F32) ? 1 : 0;
    g.acc_out = acc_out;
    g.side_k = sk; g.side_layout = side_layout; g.s_w_side = s_w_side; g.acc_side_out = acc_side_out;
    return launch_gemv(g, cs);
  }
  int8_t* qx = reinterpret_cast<int8_t*>(wsb + wl.qx_off);
  int8_t* xs = reinterpret_cast<int8_t*>(wsb + wl.xs_off);

  // activation codes; the quantizer also writes the codes of the first channel of every
  // rotation block side by side (the split product's operand)
  rc = launch_fwht_quant(X, d->T, d->K, ldx, st, s_vis, s_txt, d->rot_block, qx, d->K, nullptr, cs, xs, sk);
  if (rc != MQ_OK) return rc;
  // one GEMM launch: every tile runs the split product into a second accumulator, then the main one
  GemmArgs a{};
  a.T = d->T; a.K = d->K; a.N = d->N;
  a.Qx = qx; a.ldq = d->K; a.seg = st; a.s_vis = s_vis; a.s_txt = s_txt;
  a.W_layout = W_layout; a.s_w = s_w; a.bias = bias; a.Y = Y; a.ldy = ldy;
  a.y_is_f32 = (d->flags & MQ_FLAG_Y_IS_F32) ? 1 : 0;
  a.acc_out = acc_out;
  a.status = reinterpret_cast<int32_t*>(wsb);
  a.splitk_acc = wl.splitk_bytes ? reinterpret_cast<int32_t*>(wsb + wl.splitk_off) : nullptr;
  a.Qs = xs; a.side_k = sk; a.side_cols = d->K / d->rot_block; a.side_layout = side_layout; a.s_w_side = s_w_side; a.acc_side_out = acc_side_out;
  return launch_gemm(a, cs);
}

// ---- per-token dynamic A8: the comparison scheme (Sec. 1, Sec. 4.3) -----------------------
int mq_dynamic_quant_i8(const void* X, int32_t T, int32_t K, int64_t ldx, int32_t rot_block, int8_t* Q,
                        int64_t ldq, float* s_rows, void* stream) {
  if (T < 0 || K <= 0 || K % 32) return MQ_ERR_INVALID_ARG;
  if (T == 0) return MQ_OK;
  if (!X || !Q || !s_rows || ldx < K || ldq < K) return MQ_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(Q) || (ldx * 2) % 16 || ldq % 16) return MQ_ERR_ALIGNMENT;
  const int rc = check_rot(rot_block, K);
  if (rc != MQ_OK) return rc;
  if (K > 32 * 1024) return MQ_ERR_UNSUPPORTED;  // one warp per 1024 channels, one CTA per row
  return launch_dyn_quant(X, T, K, ldx, rot_block, Q, ldq, s_rows, static_cast<cudaStream_t>(stream));
}

size_t mq_dynamic_workspace_bytes(const mq_linear_desc* d) {
  if (check_desc(d) != MQ_OK || (d->flags & MQ_FLAG_X_IS_INT8) || d->K > 32 * 1024) return 0;
  return ws_layout(d).total + align_up((size_t)d->T * sizeof(float), 256);
}

int mq_w4a8_dynamic_linear(const mq_linear_desc* d, const void* X, int64_t ldx, const void* W_layout,
                           const float* s_w, const float* bias, void* Y, int64_t ldy, int32_t* acc_out,
                           float* s_rows_out, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_desc(d);
  if (rc != MQ_OK) return rc;
  if (d->flags & MQ_FLAG_X_IS_INT8) return MQ_ERR_INVALID_ARG;
  if (d->K > 32 * 1024) return MQ_ERR_UNSUPPORTED;
  if (d->T == 0) return MQ_OK;
  if (!X || !W_layout || !s_w || !Y) return MQ_ERR_INVALID_ARG;
  if (ldx < d->K || ldy < d->N) return MQ_ERR_INVALID_ARG;
  if (!aligned16(X) || (ldx * 2) % 16) return MQ_ERR_ALIGNMENT;
  if (!aligned(W_layout, 128) || !aligned16(Y) || !aligned16(s_w)) return MQ_ERR_ALIGNMENT;
  if (!ws) return MQ_ERR_WORKSPACE;
  if (!aligned(ws, 256)) return MQ_ERR_ALIGNMENT;
  const WsLayout wl = ws_layout(d);
  if (ws_bytes < wl.total + align_up((size_t)d->T * sizeof(float), 256)) return MQ_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  uint8_t* wsb = static_cast<uint8_t*>(ws);
  int8_t* qx = reinterpret_cast<int8_t*>(wsb + wl.qx_off);
  float* s_rows = s_rows_out ? s_rows_out : reinterpret_cast<float*>(wsb + wl.total);
  rc = launch_dyn_quant(X, d->T, d->K, ldx, d->rot_block, qx, d->K, s_rows, cs);
  if (rc != MQ_OK) return rc;
  GemmArgs a{};
  a.T = d->T; a.K = d->K; a.N = d->N;
  a.Qx = qx; a.ldq = d->K; a.s_vis = 1.0f; a.s_txt = 1.0f; a.row_scales = s_rows;
  a.W_layout = W_layout; a.s_w = s_w; a.bias = bias; a.Y = Y; a.ldy = ldy;
  a.y_is_f32 = (d->flags & MQ_FLAG_Y_IS_F32) ? 1 : 0;
  a.acc_out = acc_out;
  a.status = reinterpret_cast<int32_t*>(wsb);
  a.splitk_acc = wl.splitk_bytes ? reinterpret_cast<int32_t*>(wsb + wl.splitk_off) : nullptr;
  return launch_gemm(a, cs);
}

int mq_last_device_status(void* ws, void* stream, int32_t* site_out) {
  if (!ws) return MQ_ERR_INVALID_ARG;
  int32_t host[2] = {0, 0};
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(host, ws, sizeof(host), cudaMemcpyDeviceToHost, cs) != cudaSuccess) return MQ_ERR_CUDA;
  if (cudaStreamSynchronize(cs) != cudaSuccess) return MQ_ERR_CUDA;
  if (site_out) *site_out = host[1];
  return host[0];
}

int mq_reset_device_status(void* ws, void* stream) {
  if (!ws) return MQ_ERR_INVALID_ARG;
  return cuda_status(cudaMemsetAsync(ws, 0, kStatusBytes, static_cast<cudaStream_t>(stream)));
}

}  // extern "C"
