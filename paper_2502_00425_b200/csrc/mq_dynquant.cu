// Comparison kernel: online block-Hadamard rotation + PER-TOKEN DYNAMIC int8 quantizer.
//
// Method: the activation scheme that MSQ replaces (Sec. 1; the "per-token dynamic" column of
// the latency comparison in Sec. 4.3): every token row gets its own Eq. 2 scale
// s_t = max_k |r[t,k]| / 127 from the row the quantizer is about to see (after the rotation),
// and is quantized with it.  It exists so that the static-versus-dynamic gap can be measured
// on this hardware with otherwise identical kernels; it is not part of the MSQ path.
//
// Mapping.  One CTA per row, one warp per 1024 channels (the quantizer kernel's warp routine),
// so the whole rotated row stays in registers between the abs-max reduction and the rounding:
// one pass over the input.  Rows of up to 32 * 1024 channels.
#include "mq_common.cuh"
#include "mq_fwht_warp.cuh"

namespace mq {
namespace {

template <int LOG_TPB, bool ROT>
__global__ void __launch_bounds__(1024)
dyn_quant_kernel(const uint16_t* __restrict__ X, int K, int64_t ldx, float c_n, int8_t* __restrict__ Q, int64_t ldq,
                 float* __restrict__ s_rows) {
  constexpr int TPB = 1 << LOG_TPB;
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float red[32];
  __shared__ float s_inv;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
  const int row = blockIdx.x;
  const int j = lane & (TPB - 1);
  const int blk_start = warp * kFwhtWarpTile + (lane >> LOG_TPB) * (32 * TPB);
  float v[4][8];
  fwht_warp_tile<LOG_TPB, ROT>(X + (int64_t)row * ldx, K, blk_start, j, c_n, v);  // zeros past K
  float m = 0.0f;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int r = 0; r < 8; ++r) m = fmaxf(m, fabsf(v[i][r]));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) red[warp] = m;
  __syncthreads();
  if (warp == 0) {
    m = lane < warps ? red[lane] : 0.0f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) {
      const float s = m > 0.0f ? __fdiv_rn(m, 127.0f) : 1.0f;  // Eq. 2; an all-zero row keeps s = 1
      s_rows[row] = s;
      s_inv = __fdiv_rn(1.0f, s);
    }
  }
  __syncthreads();
  const float inv = s_inv;
  int8_t* qrow = Q + (int64_t)row * ldq;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int off = blk_start + (i * TPB + j) * 8;
    if (off < K) *reinterpret_cast<uint2*>(qrow + off) = quant_chunk_s8(v[i], inv);
  }
}

}  // namespace

int launch_dyn_quant(const void* X, int T, int K, int64_t ldx, int rot_block, int8_t* Q, int64_t ldq, float* s_rows,
                     cudaStream_t st) {
  if (T == 0 || K == 0) return MQ_OK;
  const int warps = (K + kFwhtWarpTile - 1) / kFwhtWarpTile;
  if (warps > 32) return MQ_ERR_UNSUPPORTED;
  const dim3 grid((unsigned)T), block(warps * 32);
  const float c_n = rot_block ? (float)(1.0 / sqrt((double)rot_block)) : 1.0f;
  const uint16_t* x = static_cast<const uint16_t*>(X);
  cudaError_t e;
#define MQ_LAUNCH(LOG_TPB, ROT) e = launch_pdl(dyn_quant_kernel<LOG_TPB, ROT>, grid, block, 0, st, x, K, ldx, c_n, Q, ldq, s_rows)
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
  return cuda_status(e);
}

}  // namespace mq
