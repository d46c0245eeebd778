// Full-width online rotation for K = m * 2^k fused with the MSQ quantizer.
//
// Method: the paper's online transform in front of the down-projection (Fig. 4(a)) is a Hadamard rotation; App. A.3
// defines H_{2^n} only, and K = 14336 or 18944 is not a power of two.  The usual completion is the Kronecker
// form H_K = H_m (x) H_{2^k} with a Hadamard matrix of a small non-power-of-two order m (14336 = 28 * 512,
// 18944 = 148 * 128).  The library takes H_m from the caller as a sign table (it constructs none); the
// quantizer is the one of Eq. 2 / Eq. 3.
//
// With the channels of a row read as an m x n2 array X (channel = i * n2 + j):
//   U = X . H_n2            butterflies in increasing stride order on every run of n2 channels, un-normalised
//   Y[a, j] = sum_i H_m[i, a] * U[i, j]      added one term at a time for i = 0, 1, ..., m - 1 in float32
//   r = Y * float32(1 / sqrt(K)),   q = sat_int8(round_half_even(r * (1 / s_mod(row))))
// One CTA per row: its warps transform the 1024-channel tiles into a float32 copy of the row in shared
// memory, then every thread takes one column j and a strip of eight outputs a, reads U[i, j] once per i
// and adds it, signed, into its eight sums.  m * K additions per row make this far more expensive than the
// block rotation (148 or 28 times the additions of the second stage alone); it is the exact, simple form.
#include <cmath>

#include "mq_common.cuh"
#include "mq_fwht_warp.cuh"

namespace mq {
namespace {

constexpr int kKronThreads = 256;
constexpr int kStrip = 8;  // outputs per thread and column

template <int LOG_TPB>
__global__ void __launch_bounds__(kKronThreads)
kron_quant_kernel(const uint16_t* __restrict__ X, int K, int64_t ldx, SegTable seg, float inv_vis, float inv_txt,
                  float c_k, int m, int n2, const uint8_t* __restrict__ h_neg, int8_t* __restrict__ Q, int64_t ldq,
                  float* __restrict__ rotated_out) {
  constexpr int TPB = 1 << LOG_TPB;
  extern __shared__ __align__(16) uint8_t smem_raw[];
  float* U = reinterpret_cast<float*>(smem_raw);                 // [K]
  uint8_t* neg = smem_raw + (size_t)K * sizeof(float);           // [m][m]: 1 where H_m[i, a] = -1
  pdl_launch_dependents();
  pdl_wait();
  const int row = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint16_t* xrow = X + (int64_t)row * ldx;

  for (int i = threadIdx.x; i < m * m; i += blockDim.x) neg[i] = h_neg[i];
  // stage 1: un-normalised transform of every run of n2 channels (c_n = 1 multiplies exactly)
  const int tiles = (K + kFwhtWarpTile - 1) / kFwhtWarpTile;
  const int j = lane & (TPB - 1), blk = lane >> LOG_TPB;
  for (int tile = warp; tile < tiles; tile += kKronThreads / 32) {
    const int blk_start = tile * kFwhtWarpTile + blk * (32 * TPB);
    float v[4][8];
    fwht_warp_tile<LOG_TPB, true>(xrow, K, blk_start, j, 1.0f, v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int off = blk_start + (i * TPB + j) * 8;
      if (off < K) {
        float4* dst = reinterpret_cast<float4*>(U + off);
        dst[0] = make_float4(v[i][0], v[i][1], v[i][2], v[i][3]);
        dst[1] = make_float4(v[i][4], v[i][5], v[i][6], v[i][7]);
      }
    }
  }
  __syncthreads();

  // stage 2 + quantizer
  const float inv = thread_row_modality(seg, row) == MQ_VISUAL ? inv_vis : inv_txt;
  const int strips = (m + kStrip - 1) / kStrip;
  for (int unit = threadIdx.x; unit < strips * n2; unit += blockDim.x) {
    const int col = unit % n2;      // consecutive threads take consecutive columns: conflict-free reads
    const int a0 = (unit / n2) * kStrip;
    float acc[kStrip];
#pragma unroll
    for (int r = 0; r < kStrip; ++r) acc[r] = 0.0f;
    for (int i = 0; i < m; ++i) {
      const float u = U[(size_t)i * n2 + col];
      const uint8_t* nrow = neg + i * m + a0;
#pragma unroll
      for (int r = 0; r < kStrip; ++r) {
        const bool minus = a0 + r < m && nrow[r] != 0;
        acc[r] = __fadd_rn(acc[r], minus ? -u : u);
      }
    }
#pragma unroll
    for (int r = 0; r < kStrip; ++r) {
      if (a0 + r < m) {
        const float y = __fmul_rn(acc[r], c_k);
        const int64_t k = (int64_t)(a0 + r) * n2 + col;
        if (rotated_out) rotated_out[(int64_t)row * K + k] = y;
        const int qv = __float2int_rn(__fmul_rn(y, inv));
        Q[(int64_t)row * ldq + k] = (int8_t)max(-128, min(127, qv));
      }
    }
  }
}

}  // namespace

int launch_kron_quant(const void* X, int T, int K, int64_t ldx, SegTable seg, float s_vis, float s_txt, int m,
                      const uint8_t* h_neg, int8_t* Q, int64_t ldq, float* rotated_out, cudaStream_t st) {
  if (T == 0) return MQ_OK;
  const int n2 = K / m;
  const size_t smem = (size_t)K * sizeof(float) + (size_t)m * m + 16;
  const float c_k = (float)(1.0 / sqrt((double)K));
  const float inv_vis = 1.0f / s_vis, inv_txt = 1.0f / s_txt;
  const uint16_t* x = static_cast<const uint16_t*>(X);
#define MQ_KRON(LOG_TPB, SLOT)                                                                                      \
  {                                                                                                                 \
    static PerDeviceTable<char> attr;                                                                               \
    if (!ensure_dynamic_smem(attr, kron_quant_kernel<LOG_TPB>, 200 * 1024)) return MQ_ERR_CUDA;                      \
    return cuda_status(launch_pdl(kron_quant_kernel<LOG_TPB>, dim3((unsigned)T), dim3(kKronThreads), smem, st, x, K, \
                                  ldx, seg, inv_vis, inv_txt, c_k, m, n2, h_neg, Q, ldq, rotated_out));              \
  }
  switch (n2) {
    case 32: MQ_KRON(0, 0)
    case 64: MQ_KRON(1, 1)
    case 128: MQ_KRON(2, 2)
    case 256: MQ_KRON(3, 3)
    case 512: MQ_KRON(4, 4)
    case 1024: MQ_KRON(5, 5)
    default: return MQ_ERR_UNSUPPORTED;
  }
#undef MQ_KRON
}

}  // namespace mq
