// Rotation Magnitude Suppression (Sec. 3.2, Eq. 9): the down-projection whose input is
// rotated online by I (x) H_n.
//
// The online Hadamard turns a non-zero channel mean of a weight block into one large entry:
// the first input channel of every rotated block carries sqrt(n) * mean(w) (the relation
// stated between Eq. 7 and Eq. 9).  Eq. 9 flags an (output channel, block) pair when that
// entry exceeds the block's largest original weight.  The remedy has three steps: split the
// first input channel of every block off the rotated weight, zero it in the main matrix,
// and add the split part's product back to the main GEMM's output.
//
// Here:
//   rms_detect_kernel   Eq. 9 on the UNROTATED weight (offline; flags + count).
//   rms_scale_kernel    per-output-channel int4 scales of the main part (split columns
//                       excluded) and of the split part (only the split columns).
//   rms_side_quant      int4 codes of the split part, one int8 per code, rows padded to a
//                       multiple of four codes so the combine kernel reads 32-bit words.
//   rms_combine_kernel  acc_side[t, n] = sum_b qx[t, b*n_rot] * q_side[n, b] and
//                       y = main + float(acc_side) * (s_a * s_w_side[n]) + bias.
// The main matrix goes through the ordinary W4A8 GEMM with the split columns packed as
// code 0, so that kernel is unchanged.
#include <cuda_bf16.h>

#include "mq_common.cuh"

namespace mq {
namespace {

__device__ __forceinline__ int rtn_int4(float w, float s) {
  int q = __float2int_rn(__fdiv_rn(w, s));
  return max(-8, min(7, q));
}

// One thread per (output channel, block).  Double precision: the decision is an inequality
// between two derived quantities and must not depend on the summation order in practice.
__global__ void rms_detect_kernel(const float* __restrict__ W, int N, int KBn, int64_t ldw, int nb,
                                  uint8_t* __restrict__ flags, int32_t* __restrict__ count) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int hit = 0;
  if (idx < (int64_t)N * KBn) {
    const int n = (int)(idx / KBn), b = (int)(idx % KBn);
    const float* w = W + (int64_t)n * ldw + (int64_t)b * nb;
    double sum = 0.0, mx = -1.0 / 0.0;
    for (int k = 0; k < nb; ++k) {
      const double v = (double)w[k];
      sum += v;
      mx = fmax(mx, v);
    }
    hit = sqrt((double)nb) * (sum / (double)nb) > mx;
    if (flags) flags[idx] = (uint8_t)hit;
  }
  const unsigned m = __ballot_sync(0xffffffffu, hit);
  if (count && (threadIdx.x & 31) == 0 && m) atomicAdd(count, __popc(m));
}

// One CTA per output channel: abs-max over the main columns (k % nb != 0) and over the split
// columns (k % nb == 0), each turned into an Eq. 2 int4 scale.
__global__ void rms_scale_kernel(const float* __restrict__ W, int N, int K, int64_t ldw, int nb,
                                 float* __restrict__ s_w, float* __restrict__ s_side) {
  const int n = blockIdx.x;
  if (n >= N) return;
  float m_main = 0.0f, m_side = 0.0f;
  for (int k = threadIdx.x; k < K; k += blockDim.x) {
    const float a = fabsf(W[(int64_t)n * ldw + k]);
    if (k % nb == 0) m_side = fmaxf(m_side, a);
    else m_main = fmaxf(m_main, a);
  }
  __shared__ float red[2][32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    m_main = fmaxf(m_main, __shfl_xor_sync(0xffffffffu, m_main, o));
    m_side = fmaxf(m_side, __shfl_xor_sync(0xffffffffu, m_side, o));
  }
  if ((threadIdx.x & 31) == 0) {
    red[0][threadIdx.x >> 5] = m_main;
    red[1][threadIdx.x >> 5] = m_side;
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    const bool live = threadIdx.x < (blockDim.x >> 5);
    m_main = live ? red[0][threadIdx.x] : 0.0f;
    m_side = live ? red[1][threadIdx.x] : 0.0f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      m_main = fmaxf(m_main, __shfl_xor_sync(0xffffffffu, m_main, o));
      m_side = fmaxf(m_side, __shfl_xor_sync(0xffffffffu, m_side, o));
    }
    if (threadIdx.x == 0) {
      s_w[n] = m_main > 0.0f ? __fdiv_rn(m_main, 7.0f) : 1.0f;
      s_side[n] = m_side > 0.0f ? __fdiv_rn(m_side, 7.0f) : 1.0f;
    }
  }
}

// One thread per (output channel, padded block index); the padding codes are 0.
__global__ void rms_side_quant_kernel(const float* __restrict__ W, int N, int KBn, int64_t ldw, int nb,
                                      const float* __restrict__ s_side, int8_t* __restrict__ q_side,
                                      int side_ld) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)N * side_ld) return;
  const int n = (int)(idx / side_ld), b = (int)(idx % side_ld);
  q_side[idx] = b < KBn ? (int8_t)rtn_int4(W[(int64_t)n * ldw + (int64_t)b * nb], s_side[n]) : (int8_t)0;
}

// ------------------------------------------------------------------------------ combine
// Step 3 of the remedy: the split part's product is added back.  A CTA owns kTok tokens and
// kCombineThreads output channels.  The tokens' codes at the first channel of every block are
// gathered into shared memory once (stride n_rot in the code matrix); a thread then walks
// its channel's row of q_side four codes at a time with dp4a.  Arithmetic of the fp32 result:
//   y = fadd(y_main, fmul(float(acc_side), fmul(s_a, s_w_side[n]))), then fadd(bias[n]).
constexpr int kTok = 8;
constexpr int kCombineThreads = 256;

__global__ void __launch_bounds__(kCombineThreads)
rms_combine_kernel(const float* __restrict__ y_main, const int8_t* __restrict__ qx, int64_t ldq, int T, int N, int nb,
                   int KBn, SegTable seg, float s_vis, float s_txt, const int8_t* __restrict__ q_side, int side_ld,
                   const float* __restrict__ s_w_side, const float* __restrict__ bias, void* __restrict__ Y,
                   int64_t ldy, int y_is_f32, int32_t* __restrict__ acc_side_out) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  int32_t* xs = reinterpret_cast<int32_t*>(smem_raw);  // [kTok][side_ld / 4] words
  __shared__ float s_tok[kTok];
  const int t0 = blockIdx.y * kTok;
  const int words = side_ld >> 2;
  int8_t* xb = reinterpret_cast<int8_t*>(xs);
  for (int i = threadIdx.x; i < kTok * side_ld; i += blockDim.x) {
    const int tt = i / side_ld, b = i % side_ld;
    const int t = t0 + tt;
    xb[i] = (t < T && b < KBn) ? qx[(int64_t)t * ldq + (int64_t)b * nb] : (int8_t)0;
  }
  if (threadIdx.x < kTok) {
    const int t = t0 + threadIdx.x;
    s_tok[threadIdx.x] = (t < T && thread_row_modality(seg, t) == MQ_VISUAL) ? s_vis : s_txt;
  }
  __syncthreads();
  const int n = blockIdx.x * kCombineThreads + threadIdx.x;
  if (n >= N) return;
  int acc[kTok];
#pragma unroll
  for (int j = 0; j < kTok; ++j) acc[j] = 0;
  const int32_t* qrow = reinterpret_cast<const int32_t*>(q_side + (int64_t)n * side_ld);
  for (int w = 0; w < words; ++w) {
    const int q = __ldg(qrow + w);
#pragma unroll
    for (int j = 0; j < kTok; ++j) acc[j] = __dp4a(xs[j * words + w], q, acc[j]);
  }
  const float sw = s_w_side[n];
  const float bs = bias ? bias[n] : 0.0f;
#pragma unroll
  for (int j = 0; j < kTok; ++j) {
    const int t = t0 + j;
    if (t >= T) break;
    float y = __fadd_rn(y_main[(int64_t)t * N + n], __fmul_rn((float)acc[j], __fmul_rn(s_tok[j], sw)));
    if (bias) y = __fadd_rn(y, bs);
    if (y_is_f32) static_cast<float*>(Y)[(int64_t)t * ldy + n] = y;
    else static_cast<__nv_bfloat16*>(Y)[(int64_t)t * ldy + n] = __float2bfloat16_rn(y);
    if (acc_side_out) acc_side_out[(int64_t)t * N + n] = acc[j];
  }
}

}  // namespace

int launch_rms_detect(const float* W, int N, int K, int64_t ldw, int nb, uint8_t* flags, int32_t* count,
                      cudaStream_t st) {
  if (count && cudaMemsetAsync(count, 0, sizeof(int32_t), st) != cudaSuccess) return MQ_ERR_CUDA;
  const int KBn = K / nb;
  const int64_t n = (int64_t)N * KBn;
  if (n == 0) return MQ_OK;
  rms_detect_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(W, N, KBn, ldw, nb, flags, count);
  return cuda_status(cudaGetLastError());
}

int launch_rms_pack(const float* W, int N, int K, int64_t ldw, int nb, uint8_t* packed, float* s_w, void* layout,
                    int8_t* q_side, int side_ld, float* s_w_side, cudaStream_t st) {
  if (N == 0 || K == 0) return MQ_OK;
  rms_scale_kernel<<<N, 256, 0, st>>>(W, N, K, ldw, nb, s_w, s_w_side);
  const int64_t n = (int64_t)N * side_ld;
  rms_side_quant_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(W, N, K / nb, ldw, nb, s_w_side, q_side,
                                                                       side_ld);
  if (cudaGetLastError() != cudaSuccess) return MQ_ERR_CUDA;
  return launch_pack_codes(W, N, K, ldw, s_w, packed, layout, nb, st);
}

int launch_rms_combine(const float* y_main, const int8_t* qx, int64_t ldq, int T, int K, int N, int nb, SegTable seg,
                       float s_vis, float s_txt, const int8_t* q_side, int side_ld, const float* s_w_side,
                       const float* bias, void* Y, int64_t ldy, int y_is_f32, int32_t* acc_side_out,
                       cudaStream_t st) {
  if (T == 0 || N == 0) return MQ_OK;
  const size_t smem = (size_t)kTok * side_ld;
  if (smem > 48 * 1024) return MQ_ERR_UNSUPPORTED;
  dim3 grid((N + kCombineThreads - 1) / kCombineThreads, (T + kTok - 1) / kTok);
  rms_combine_kernel<<<grid, kCombineThreads, smem, st>>>(y_main, qx, ldq, T, N, nb, K / nb, seg, s_vis, s_txt,
                                                          q_side, side_ld, s_w_side, bias, Y, ldy, y_is_f32,
                                                          acc_side_out);
  return cuda_status(cudaGetLastError());
}

}  // namespace mq
