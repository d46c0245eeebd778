// Glue of a decoder block between the library's linears (layer mode): RMSNorm, rotary embedding, SwiGLU and the
// residual add as single-pass bf16 kernels with float32 arithmetic.  They exist so that a block can run end to
// end without float32 temporaries in HBM; none of them is part of the quantized path and none is tuned beyond
// "one read and one write of every tensor".
//   RMSNorm: y = x / sqrt(mean(x^2) + eps) * gain                       (App. A.14)
//   rotary:  channel pairs (2i, 2i+1) of every head rotated by pos * base^(-2i/D); positions are the ORIGINAL
//            token indices carried through the AIFS reorder             (App. A.2)
//   SwiGLU:  y = gate / (1 + exp(-gate)) * up, the input of the down-projection
#include <cuda_bf16.h>

#include "mq_common.cuh"

namespace mq {
namespace {

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

// One CTA per row; every thread keeps its 8-element chunks in registers between the two passes.
template <int kChunks>
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const uint16_t* __restrict__ X, int64_t ldx, const float* __restrict__ gain, float eps, int D,
               __nv_bfloat16* __restrict__ Y, int64_t ldy) {
  const int row = blockIdx.x;
  const uint16_t* x = X + (int64_t)row * ldx;
  float v[kChunks][8];
  float ss = 0.0f;
#pragma unroll
  for (int c = 0; c < kChunks; ++c) {
    const int off = (c * 256 + threadIdx.x) * 8;
    uint4 w = make_uint4(0u, 0u, 0u, 0u);
    if (off < D) w = *reinterpret_cast<const uint4*>(x + off);
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      v[c][2 * p] = __uint_as_float(ww[p] << 16);
      v[c][2 * p + 1] = __uint_as_float(ww[p] & 0xffff0000u);
      ss = fmaf(v[c][2 * p], v[c][2 * p], ss);
      ss = fmaf(v[c][2 * p + 1], v[c][2 * p + 1], ss);
    }
  }
  __shared__ float red[8];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.0f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  const float r = rsqrtf(tot / (float)D + eps);
#pragma unroll
  for (int c = 0; c < kChunks; ++c) {
    const int off = (c * 256 + threadIdx.x) * 8;
    if (off >= D) continue;
    const float4 g0 = *reinterpret_cast<const float4*>(gain + off), g1 = *reinterpret_cast<const float4*>(gain + off + 4);
    const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
    __nv_bfloat162 o[4];
#pragma unroll
    for (int p = 0; p < 4; ++p) o[p] = __floats2bfloat162_rn(v[c][2 * p] * r * g[2 * p], v[c][2 * p + 1] * r * g[2 * p + 1]);
    *reinterpret_cast<uint4*>(Y + (int64_t)row * ldy + off) = *reinterpret_cast<const uint4*>(o);
  }
}

// One thread per channel pair.
__global__ void rope_kernel(const __nv_bfloat16* __restrict__ X, int64_t ldx, const int32_t* __restrict__ pos, int L,
                            int n_heads, int D, float log2_base, __nv_bfloat16* __restrict__ Y, int64_t ldy) {
  const int half = D / 2;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t per_row = (int64_t)n_heads * half;
  if (idx >= (int64_t)L * per_row) return;
  const int t = (int)(idx / per_row);
  const int rem = (int)(idx % per_row);
  const int h = rem / half, i = rem % half;
  const float theta = exp2f(-2.0f * (float)i / (float)D * log2_base);
  float s, c;
  sincosf((float)pos[t] * theta, &s, &c);
  const int64_t col = (int64_t)h * D + 2 * i;
  const __nv_bfloat162 xv = *reinterpret_cast<const __nv_bfloat162*>(X + (int64_t)t * ldx + col);
  const float x0 = __low2float(xv), x1 = __high2float(xv);
  *reinterpret_cast<__nv_bfloat162*>(Y + (int64_t)t * ldy + col) = __floats2bfloat162_rn(x0 * c - x1 * s, x0 * s + x1 * c);
}

// Eight channels per thread.
__global__ void swiglu_kernel(const uint16_t* __restrict__ G, int64_t ldg, const uint16_t* __restrict__ U, int64_t ldu,
                              int T, int M, __nv_bfloat16* __restrict__ Y, int64_t ldy) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int per_row = M / 8;
  if (idx >= (int64_t)T * per_row) return;
  const int t = (int)(idx / per_row), off = (int)(idx % per_row) * 8;
  const uint4 g = *reinterpret_cast<const uint4*>(G + (int64_t)t * ldg + off);
  const uint4 u = *reinterpret_cast<const uint4*>(U + (int64_t)t * ldu + off);
  const uint32_t gw[4] = {g.x, g.y, g.z, g.w}, uw[4] = {u.x, u.y, u.z, u.w};
  __nv_bfloat162 o[4];
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    const float g0 = __uint_as_float(gw[p] << 16), g1 = __uint_as_float(gw[p] & 0xffff0000u);
    const float u0 = __uint_as_float(uw[p] << 16), u1 = __uint_as_float(uw[p] & 0xffff0000u);
    o[p] = __floats2bfloat162_rn(g0 / (1.0f + expf(-g0)) * u0, g1 / (1.0f + expf(-g1)) * u1);
  }
  *reinterpret_cast<uint4*>(Y + (int64_t)t * ldy + off) = *reinterpret_cast<const uint4*>(o);
}

__global__ void residual_add_kernel(const uint16_t* __restrict__ A, int64_t lda, const uint16_t* __restrict__ Bm, int64_t ldb,
                                    int T, int D, __nv_bfloat16* __restrict__ Y, int64_t ldy) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int per_row = D / 8;
  if (idx >= (int64_t)T * per_row) return;
  const int t = (int)(idx / per_row), off = (int)(idx % per_row) * 8;
  const uint4 a = *reinterpret_cast<const uint4*>(A + (int64_t)t * lda + off);
  const uint4 b = *reinterpret_cast<const uint4*>(Bm + (int64_t)t * ldb + off);
  const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
  __nv_bfloat162 o[4];
#pragma unroll
  for (int p = 0; p < 4; ++p)
    o[p] = __floats2bfloat162_rn(__uint_as_float(aw[p] << 16) + __uint_as_float(bw[p] << 16),
                                 __uint_as_float(aw[p] & 0xffff0000u) + __uint_as_float(bw[p] & 0xffff0000u));
  *reinterpret_cast<uint4*>(Y + (int64_t)t * ldy + off) = *reinterpret_cast<const uint4*>(o);
}

inline bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace
}  // namespace mq

using namespace mq;

extern "C" int mq_glue_rmsnorm(const void* X, int32_t T, int32_t D, int64_t ldx, const float* gain, float eps, void* Y,
                               int64_t ldy, void* stream) {
  if (T < 0 || D <= 0 || D % 8 || ldx < D || ldy < D || !(eps >= 0.0f)) return MQ_ERR_INVALID_ARG;
  if (T == 0) return MQ_OK;
  if (!X || !Y || !gain) return MQ_ERR_INVALID_ARG;
  if (!al16(X) || !al16(Y) || !al16(gain) || (ldx * 2) % 16 || (ldy * 2) % 16) return MQ_ERR_ALIGNMENT;
  if (D > 8 * 2048) return MQ_ERR_UNSUPPORTED;  // a row is held in the registers of one 256-thread CTA
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const uint16_t* x = static_cast<const uint16_t*>(X);
  __nv_bfloat16* y = static_cast<__nv_bfloat16*>(Y);
  const int chunks = (D + 2047) / 2048;
  switch (chunks) {
    case 1: rmsnorm_kernel<1><<<T, 256, 0, st>>>(x, ldx, gain, eps, D, y, ldy); break;
    case 2: rmsnorm_kernel<2><<<T, 256, 0, st>>>(x, ldx, gain, eps, D, y, ldy); break;
    case 3: rmsnorm_kernel<3><<<T, 256, 0, st>>>(x, ldx, gain, eps, D, y, ldy); break;
    case 4: rmsnorm_kernel<4><<<T, 256, 0, st>>>(x, ldx, gain, eps, D, y, ldy); break;
    default: rmsnorm_kernel<8><<<T, 256, 0, st>>>(x, ldx, gain, eps, D, y, ldy); break;
  }
  return cuda_status(cudaGetLastError());
}

extern "C" int mq_glue_rope(const void* X, int32_t L, int32_t n_heads, int32_t head_dim, int64_t ldx, const int32_t* pos,
                            float base, void* Y, int64_t ldy, void* stream) {
  if (L < 0 || n_heads <= 0 || head_dim <= 0 || head_dim % 2 || !(base > 1.0f)) return MQ_ERR_INVALID_ARG;
  const int64_t width = (int64_t)n_heads * head_dim;
  if (ldx < width || ldy < width) return MQ_ERR_INVALID_ARG;
  if (L == 0) return MQ_OK;
  if (!X || !Y || !pos) return MQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(X) & 3u) || (reinterpret_cast<uintptr_t>(Y) & 3u) || ldx % 2 || ldy % 2) return MQ_ERR_ALIGNMENT;
  const int64_t n = (int64_t)L * n_heads * (head_dim / 2);
  rope_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(X), ldx, pos, L, n_heads, head_dim, log2f(base), static_cast<__nv_bfloat16*>(Y), ldy);
  return cuda_status(cudaGetLastError());
}

extern "C" int mq_glue_swiglu(const void* G, int64_t ldg, const void* U, int64_t ldu, int32_t T, int32_t M, void* Y,
                              int64_t ldy, void* stream) {
  if (T < 0 || M <= 0 || M % 8 || ldg < M || ldu < M || ldy < M) return MQ_ERR_INVALID_ARG;
  if (T == 0) return MQ_OK;
  if (!G || !U || !Y) return MQ_ERR_INVALID_ARG;
  if (!al16(G) || !al16(U) || !al16(Y) || (ldg * 2) % 16 || (ldu * 2) % 16 || (ldy * 2) % 16) return MQ_ERR_ALIGNMENT;
  const int64_t n = (int64_t)T * (M / 8);
  swiglu_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint16_t*>(G), ldg, static_cast<const uint16_t*>(U), ldu, T, M, static_cast<__nv_bfloat16*>(Y), ldy);
  return cuda_status(cudaGetLastError());
}

extern "C" int mq_glue_residual_add(const void* A, int64_t lda, const void* Bm, int64_t ldb, int32_t T, int32_t D, void* Y,
                                    int64_t ldy, void* stream) {
  if (T < 0 || D <= 0 || D % 8 || lda < D || ldb < D || ldy < D) return MQ_ERR_INVALID_ARG;
  if (T == 0) return MQ_OK;
  if (!A || !Bm || !Y) return MQ_ERR_INVALID_ARG;
  if (!al16(A) || !al16(Bm) || !al16(Y) || (lda * 2) % 16 || (ldb * 2) % 16 || (ldy * 2) % 16) return MQ_ERR_ALIGNMENT;
  const int64_t n = (int64_t)T * (D / 8);
  residual_add_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint16_t*>(A), lda, static_cast<const uint16_t*>(Bm), ldb, T, D, static_cast<__nv_bfloat16*>(Y), ldy);
  return cuda_status(cudaGetLastError());
}
