// K1: fused online block-Hadamard rotation + modality-specific static int8 quantizer,
// and the calibration reduce that shares its front end.
//
// Method: Fig. 4(a) (online fast Hadamard transform in front of the down-projection
// quantizer), App. A.3 (H_2 and the Kronecker recursion), Eq. 2 / Eq. 3 (static
// per-modality scale, round-to-nearest, clamp).
//
// Mapping.  A warp owns 1024 consecutive channels of one row per pass.  A rotation block
// of n = 32 * TPB channels is held by TPB adjacent lanes, each lane keeping four 16-byte
// chunks (8 bf16 each): chunk c = i * TPB + j for lane-in-block j and i = 0..3.  With the
// element index written as  e = r + 8 * (j + TPB * i)  the butterfly strides 1,2,4 act on
// r (registers), strides 8 .. 4n/32 act on j (warp shuffles) and the last two strides act
// on i (registers), so the stages run in increasing stride order -- the same rounding
// sequence as a textbook in-place transform -- with only log2(TPB) shuffle stages.
// Every global access is a full 16-byte (load) or 8-byte (store) vector and every 32-byte
// sector touched is used completely; the kernel is bounded by HBM traffic of 3 bytes per
// element (2 read + 1 written).
#include "mq_common.cuh"
#include "mq_fwht_warp.cuh"

namespace mq {
namespace {

constexpr int kWarpsPerCta = 8;
constexpr int kWarpTile = kFwhtWarpTile;  // channels per warp pass

// kQuantSide: also writes the code of the first channel of every rotation block to
// side_out[row, block] -- the activation operand of the split product of rotation
// magnitude suppression (Sec. 3.2), K-contiguous for the GEMM's tensor map.
// kQuant4: 4-bit codes (clamp to [-8, 7]) for the W4A4 setting.
enum Mode { kQuant = 0, kQuantDump = 1, kAbsMax = 2, kQuantSide = 3, kQuant4 = 4 };

template <int LOG_TPB, bool ROT, int MODE>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
fwht_quant_kernel(const uint16_t* __restrict__ X, int T, int K, int64_t ldx, SegTable seg,
                  float inv_vis, float inv_txt, float c_n, int8_t* __restrict__ Q, int64_t ldq,
                  float* __restrict__ rotated_out, uint32_t* __restrict__ amax_state,
                  int tiles_per_row, unsigned n_warp_tiles, int8_t* __restrict__ side_out, int side_ld) {
  constexpr int TPB = 1 << LOG_TPB;
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const unsigned wt = blockIdx.x * (unsigned)kWarpsPerCta + (unsigned)warp;  // 32-bit: a 64-bit division
  if (wt >= n_warp_tiles) return;                                            // here costs ~10 % of the kernel
  const int row = (int)(wt / (unsigned)tiles_per_row);
  const int tile = (int)(wt - (unsigned)row * (unsigned)tiles_per_row);
  const int j = lane & (TPB - 1);
  const int blk = lane >> LOG_TPB;
  const int blk_start = tile * kWarpTile + blk * (32 * TPB);

  float v[4][8];
  fwht_warp_tile<LOG_TPB, ROT>(X + (int64_t)row * ldx, K, blk_start, j, c_n, v);

  const int mod = warp_row_modality(seg, row);

  if (MODE == kAbsMax) {
    float m = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int r = 0; r < 8; ++r) m = fmaxf(m, fabsf(v[i][r]));  // fmaxf drops NaN
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0 && m > 0.0f) atomicMax(&amax_state[mod], __float_as_uint(m));
    return;
  }

  const float inv = (mod == MQ_VISUAL) ? inv_vis : inv_txt;
  int8_t* qrow = Q + (int64_t)row * ldq;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int off = blk_start + (i * TPB + j) * 8;
    if (off >= K) continue;
    if (MODE == kQuantDump) {
      float4* dst = reinterpret_cast<float4*>(rotated_out + (int64_t)row * K + off);
      dst[0] = make_float4(v[i][0], v[i][1], v[i][2], v[i][3]);
      dst[1] = make_float4(v[i][4], v[i][5], v[i][6], v[i][7]);
    }
    const uint2 o = MODE == kQuant4 ? quant_chunk_s4(v[i], inv) : quant_chunk_s8(v[i], inv);
    *reinterpret_cast<uint2*>(qrow + off) = o;
    if (MODE == kQuantSide && i == 0 && j == 0)  // element 0 of the block is in chunk 0 of lane-in-block 0
      side_out[(int64_t)row * side_ld + (blk_start >> (5 + LOG_TPB))] = (int8_t)(o.x & 0xffu);
  }
}

__global__ void calib_reset_kernel(uint32_t* amax_state) {
  if (threadIdx.x < 2) amax_state[threadIdx.x] = 0u;
}

__global__ void calib_finalize_kernel(const uint32_t* amax_state, float* s_vis_out, float* s_txt_out, float qmax) {
  if (threadIdx.x == 0) {
    const float mt = __uint_as_float(amax_state[MQ_TEXT]);
    const float mv = __uint_as_float(amax_state[MQ_VISUAL]);
    *s_txt_out = mt > 0.0f ? __fdiv_rn(mt, qmax) : 1.0f;
    *s_vis_out = mv > 0.0f ? __fdiv_rn(mv, qmax) : 1.0f;
  }
}

template <int MODE>
int dispatch(const void* X, int T, int K, int64_t ldx, SegTable seg, float inv_vis, float inv_txt,
             int rot_block, int8_t* Q, int64_t ldq, float* rotated_out, uint32_t* amax_state,
             cudaStream_t st, int8_t* side_out = nullptr, int side_ld = 0) {
  if (T == 0 || K == 0) return MQ_OK;
  const int tiles_per_row = (K + kWarpTile - 1) / kWarpTile;
  const long long n_warp_tiles = (long long)T * tiles_per_row;
  const long long ctas = (n_warp_tiles + kWarpsPerCta - 1) / kWarpsPerCta;
  if (n_warp_tiles > 0xfffffff0LL) return MQ_ERR_UNSUPPORTED;
  const dim3 grid((unsigned)ctas), block(kWarpsPerCta * 32);
  const float c_n = rot_block ? (float)(1.0 / sqrt((double)rot_block)) : 1.0f;
  const uint16_t* x = static_cast<const uint16_t*>(X);
#define MQ_LAUNCH(LOG_TPB, ROT)                                                              \
  launch_pdl(fwht_quant_kernel<LOG_TPB, ROT, MODE>, grid, block, 0, st, x, T, K, ldx, seg, inv_vis, inv_txt, c_n, \
             Q, ldq, rotated_out, amax_state, tiles_per_row, (unsigned)n_warp_tiles, side_out, side_ld)
  switch (rot_block) {
    case 0: MQ_LAUNCH(2, false); break;
    case 32: MQ_LAUNCH(0, true); break;
    case 64: MQ_LAUNCH(1, true); break;
    case 128: MQ_LAUNCH(2, true); break;
    case 256: MQ_LAUNCH(3, true); break;
    case 512: MQ_LAUNCH(4, true); break;
    case 1024: MQ_LAUNCH(5, true); break;
    default: return MQ_ERR_UNSUPPORTED;
  }
#undef MQ_LAUNCH
  return cuda_status(cudaGetLastError());
}

}  // namespace

int launch_fwht_quant(const void* X, int T, int K, int64_t ldx, SegTable seg, float s_vis,
                      float s_txt, int rot_block, int8_t* Q, int64_t ldq, float* rotated_out,
                      cudaStream_t st, int8_t* side_out, int side_ld, int act_bits) {
  const float inv_vis = 1.0f / s_vis, inv_txt = 1.0f / s_txt;
  if (act_bits == 4) {
    if (side_out || rotated_out) return MQ_ERR_UNSUPPORTED;
    return dispatch<kQuant4>(X, T, K, ldx, seg, inv_vis, inv_txt, rot_block, Q, ldq, nullptr, nullptr, st);
  }
  if (side_out) {
    if (!rot_block || rotated_out) return MQ_ERR_INVALID_ARG;
    return dispatch<kQuantSide>(X, T, K, ldx, seg, inv_vis, inv_txt, rot_block, Q, ldq, nullptr, nullptr, st,
                                side_out, side_ld);
  }
  if (rotated_out)
    return dispatch<kQuantDump>(X, T, K, ldx, seg, inv_vis, inv_txt, rot_block, Q, ldq, rotated_out,
                                nullptr, st);
  return dispatch<kQuant>(X, T, K, ldx, seg, inv_vis, inv_txt, rot_block, Q, ldq, nullptr, nullptr, st);
}

int launch_calibrate(const void* X, int T, int K, int64_t ldx, SegTable seg, int rot_block,
                     int accumulate, uint32_t* amax_state, float* s_vis_out, float* s_txt_out,
                     cudaStream_t st, int act_bits) {
  if (!accumulate) calib_reset_kernel<<<1, 32, 0, st>>>(amax_state);
  int rc = dispatch<kAbsMax>(X, T, K, ldx, seg, 1.0f, 1.0f, rot_block, nullptr, 0, nullptr, amax_state, st);
  if (rc != MQ_OK) return rc;
  calib_finalize_kernel<<<1, 32, 0, st>>>(amax_state, s_vis_out, s_txt_out, act_bits == 4 ? 7.0f : 127.0f);
  return cuda_status(cudaGetLastError());
}

}  // namespace mq
