// K0b: per-output-channel symmetric int4 round-to-nearest weight quantizer and the two
// storage layouts (offline, untimed).
//
// Method: Eq. 2 with b = 4 and zero-point 0; Algorithm 1 lists per-channel weight scales
// among the outputs.  s_w[n] = max_k |W[n,k]| / 7, q = clamp(rne(W / s_w), -8, 7).
//
// GEMM weight layout.  W is cut into tiles of 128 output channels x 128 input channels
// (zero-padded at the edges).  Tile (tn, kb) is one contiguous 8 KB block at
// ((tn * KB + kb) * 8192); inside it, 16-byte piece (jj, r) at (jj * 128 + r) * 16 holds
// the 32 codes k = kb*128 + jj*32 .. +31 of channel tn*128 + r: 32-bit word i of the piece
// carries codes k0 = jj*32 + i*8 .. +7 with code k0+b in the LOW nibble of byte b and code
// k0+4+b in the HIGH nibble of byte b.  A thread of the GEMM that owns channel r then reads
// its four pieces with conflict-free 16-byte shared-memory loads and turns one word into
// eight consecutive int8 values with two logic operations (see mq_gemm.cu).
#include "mq_common.cuh"

namespace mq {
namespace {

__device__ __forceinline__ int rtn_int4(float w, float s) {
  int q = __float2int_rn(__fdiv_rn(w, s));
  return max(-8, min(7, q));
}

__global__ void row_scale_kernel(const float* __restrict__ W, int N, int K, int64_t ldw,
                                 float* __restrict__ s_w, float qmax) {
  const int n = blockIdx.x;
  if (n >= N) return;
  float m = 0.0f;
  for (int k = threadIdx.x; k < K; k += blockDim.x) m = fmaxf(m, fabsf(W[(int64_t)n * ldw + k]));
  __shared__ float red[32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.0f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (threadIdx.x == 0) s_w[n] = m > 0.0f ? __fdiv_rn(m, qmax) : 1.0f;
  }
}

// Group-wise scales (App. A.12: g = 128): one warp per (output channel n, group g) takes the abs-max of the
// group's input channels; s_wg[g * N + n] = max / 7 (1 for an all-zero group).  Group-major so that the GEMM's
// epilogue lanes, which own consecutive channels, read consecutive floats.
__global__ void group_scale_kernel(const float* __restrict__ W, int N, int K, int64_t ldw, int group,
                                   float* __restrict__ s_wg) {
  const int64_t wid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const int G = K / group;
  if (wid >= (int64_t)N * G) return;
  const int n = (int)(wid / G), g = (int)(wid % G);
  float m = 0.0f;
  for (int k = lane; k < group; k += 32) m = fmaxf(m, fabsf(W[(int64_t)n * ldw + (int64_t)g * group + k]));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) s_wg[(int64_t)g * N + n] = m > 0.0f ? __fdiv_rn(m, 7.0f) : 1.0f;
}

// The scale of weight (n, k): per output channel, or per (group of input channels, output channel).
__device__ __forceinline__ float weight_scale(const float* s_w, int N, int n, int k, int group) {
  return group ? s_w[(int64_t)(k / group) * N + n] : s_w[n];
}

// skip != 0: input channels k with k % skip == 0 are written as code 0 (they were split off the
// main matrix, see mq_rms.cu).
__device__ __forceinline__ int rtn_int4_masked(const float* W, int64_t idx, int k, float s, int skip) {
  return (skip && k % skip == 0) ? 0 : rtn_int4(W[idx], s);
}

__global__ void pack_canonical_kernel(const float* __restrict__ W, int N, int K, int64_t ldw,
                                      const float* __restrict__ s_w, uint8_t* __restrict__ packed, int skip,
                                      int group) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int half = K / 2;
  if (idx >= (int64_t)N * half) return;
  const int n = (int)(idx / half), j = (int)(idx % half);
  const float s = weight_scale(s_w, N, n, 2 * j, group);  // 2j and 2j + 1 share a group (group is even)
  const int q0 = rtn_int4_masked(W, (int64_t)n * ldw + 2 * j, 2 * j, s, skip);
  const int q1 = rtn_int4_masked(W, (int64_t)n * ldw + 2 * j + 1, 2 * j + 1, s, skip);
  packed[idx] = (uint8_t)((q0 & 15) | ((q1 & 15) << 4));
}

// One thread per 32-bit word of the GEMM layout.
struct WordCoord {
  int n, k0;
};
__device__ __forceinline__ WordCoord layout_word_coord(int64_t word, int KB) {
  // word index = ((tn * KB + kb) * 4 + jj) * 512 + r * 4 + i
  const int i = (int)(word & 3);
  const int r = (int)((word >> 2) & 127);
  const int64_t rest = word >> 9;
  const int jj = (int)(rest & 3);
  const int64_t tile = rest >> 2;
  const int kb = (int)(tile % KB);
  const int tn = (int)(tile / KB);
  return {tn * MQ_W_TILE_N + r, kb * MQ_W_TILE_K + jj * 32 + i * 8};
}

__global__ void pack_layout_kernel(const float* __restrict__ W, int N, int K, int64_t ldw,
                                   const float* __restrict__ s_w, uint32_t* __restrict__ layout,
                                   int KB, int64_t n_words, int skip, int group) {
  const int64_t word = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (word >= n_words) return;
  const WordCoord c = layout_word_coord(word, KB);
  uint32_t out = 0;
  if (c.n < N) {
    const float s = weight_scale(s_w, N, c.n, min(c.k0, K - 1), group);  // the word's eight codes share a group
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int klo = c.k0 + b, khi = c.k0 + 4 + b;
      const int qlo = klo < K ? rtn_int4_masked(W, (int64_t)c.n * ldw + klo, klo, s, skip) : 0;
      const int qhi = khi < K ? rtn_int4_masked(W, (int64_t)c.n * ldw + khi, khi, s, skip) : 0;
      out |= (uint32_t)((qlo & 15) | ((qhi & 15) << 4)) << (8 * b);
    }
  }
  layout[word] = out;
}

__device__ __forceinline__ int canon_nibble(const uint8_t* packed, int half, int n, int k) {
  return (packed[(int64_t)n * half + (k >> 1)] >> (4 * (k & 1))) & 15;
}

__global__ void repack_kernel(const uint8_t* __restrict__ packed, int N, int K,
                              uint32_t* __restrict__ layout, int KB, int64_t n_words) {
  const int64_t word = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (word >= n_words) return;
  const WordCoord c = layout_word_coord(word, KB);
  uint32_t out = 0;
  if (c.n < N) {
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int klo = c.k0 + b, khi = c.k0 + 4 + b;
      const int qlo = klo < K ? canon_nibble(packed, K / 2, c.n, klo) : 0;
      const int qhi = khi < K ? canon_nibble(packed, K / 2, c.n, khi) : 0;
      out |= (uint32_t)(qlo | (qhi << 4)) << (8 * b);
    }
  }
  layout[word] = out;
}

// GEMM layout from int4 codes stored one per byte (q [N, K], pitch ldq).
__global__ void layout_from_codes_kernel(const int8_t* __restrict__ q, int64_t ldq, int N, int K,
                                         uint32_t* __restrict__ layout, int KB, int64_t n_words) {
  const int64_t word = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (word >= n_words) return;
  const WordCoord c = layout_word_coord(word, KB);
  uint32_t out = 0;
  if (c.n < N) {
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int klo = c.k0 + b, khi = c.k0 + 4 + b;
      const int qlo = klo < K ? q[(int64_t)c.n * ldq + klo] & 15 : 0;
      const int qhi = khi < K ? q[(int64_t)c.n * ldq + khi] & 15 : 0;
      out |= (uint32_t)(qlo | (qhi << 4)) << (8 * b);
    }
  }
  layout[word] = out;
}

__global__ void unpack_kernel(const uint8_t* __restrict__ packed, const uint8_t* __restrict__ layout,
                              int N, int K, int KB, int8_t* __restrict__ q, int64_t ldq) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)N * K) return;
  const int n = (int)(idx / K), k = (int)(idx % K);
  int nib;
  if (packed) {
    nib = canon_nibble(packed, K / 2, n, k);
  } else {
    const int tn = n / MQ_W_TILE_N, r = n % MQ_W_TILE_N, kb = k / MQ_W_TILE_K, kk = k % MQ_W_TILE_K;
    const int jj = kk / 32, c = kk % 32, i = c / 8, e = c % 8;
    const int64_t byte = (((int64_t)tn * KB + kb) * 4 + jj) * 2048 + r * 16 + i * 4 + (e & 3);
    nib = (layout[byte] >> (e >= 4 ? 4 : 0)) & 15;
  }
  q[(int64_t)n * ldq + k] = (int8_t)(nib >= 8 ? nib - 16 : nib);
}

inline int64_t layout_words(int N, int K) {
  const int64_t TN = (N + MQ_W_TILE_N - 1) / MQ_W_TILE_N, KB = (K + MQ_W_TILE_K - 1) / MQ_W_TILE_K;
  return TN * KB * 2048;
}

}  // namespace

// Codes and layouts from scales that are already in s_w (skip: see pack_canonical_kernel).
int launch_pack_codes(const float* W, int N, int K, int64_t ldw, const float* s_w, uint8_t* packed,
                      void* layout, int skip, cudaStream_t st, int group) {
  if (N == 0 || K == 0) return MQ_OK;
  if (packed) {
    const int64_t n = (int64_t)N * (K / 2);
    pack_canonical_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(W, N, K, ldw, s_w, packed, skip, group);
  }
  if (layout) {
    const int64_t nw = layout_words(N, K);
    pack_layout_kernel<<<(unsigned)((nw + 255) / 256), 256, 0, st>>>(
        W, N, K, ldw, s_w, static_cast<uint32_t*>(layout), (K + MQ_W_TILE_K - 1) / MQ_W_TILE_K, nw, skip, group);
  }
  return cuda_status(cudaGetLastError());
}

int launch_layout_from_codes(const int8_t* q, int64_t ldq, int N, int K, void* layout, cudaStream_t st) {
  if (N == 0 || K == 0) return MQ_OK;
  const int64_t nw = layout_words(N, K);
  layout_from_codes_kernel<<<(unsigned)((nw + 255) / 256), 256, 0, st>>>(
      q, ldq, N, K, static_cast<uint32_t*>(layout), (K + MQ_W_TILE_K - 1) / MQ_W_TILE_K, nw);
  return cuda_status(cudaGetLastError());
}

int launch_pack_w4(const float* W, int N, int K, int64_t ldw, uint8_t* packed, float* s_w,
                   void* layout, cudaStream_t st, int group) {
  if (N == 0 || K == 0) return MQ_OK;
  if (group) {
    const int64_t warps = (int64_t)N * (K / group);
    group_scale_kernel<<<(unsigned)((warps * 32 + 255) / 256), 256, 0, st>>>(W, N, K, ldw, group, s_w);
  } else {
    row_scale_kernel<<<N, 256, 0, st>>>(W, N, K, ldw, s_w, 7.0f);
  }
  return launch_pack_codes(W, N, K, ldw, s_w, packed, layout, 0, st, group);
}

// ---- 8-bit weights (the W8A8 setting, Sec. 4.1): s_w[n] = max_k |W[n,k]| / 127, codes clamp to [-128, 127].
// GEMM layout: tiles of 128 x 128 codes, 16 KB each at ((tn * KB + kb) * 16384); inside, 16-byte piece (c, r) at
// (c * 128 + r) * 16 holds the codes k = kb*128 + 16 c .. + 15 of channel tn*128 + r (zero-padded at the edges).
namespace {
__device__ __forceinline__ int rtn_int8(float w, float s) {
  const int q = __float2int_rn(__fdiv_rn(w, s));
  return max(-128, min(127, q));
}
__global__ void pack8_layout_kernel(const float* __restrict__ W, int N, int K, int64_t ldw, const float* __restrict__ s_w,
                                    uint32_t* __restrict__ layout, int8_t* __restrict__ q_out, int64_t ldq, int KB,
                                    int64_t n_words) {
  const int64_t word = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (word >= n_words) return;
  // word index = (tile * 8 + c) * 512 + r * 4 + i
  const int i = (int)(word & 3);
  const int r = (int)((word >> 2) & 127);
  const int64_t rest = word >> 9;
  const int c = (int)(rest & 7);
  const int64_t tile = rest >> 3;
  const int kb = (int)(tile % KB), tn = (int)(tile / KB);
  const int n = tn * MQ_W_TILE_N + r, k0 = kb * MQ_W_TILE_K + c * 16 + i * 4;
  uint32_t out = 0;
  if (n < N) {
    const float s = s_w[n];
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int k = k0 + b;
      if (k < K) {
        const int q = rtn_int8(W[(int64_t)n * ldw + k], s);
        out |= (uint32_t)(q & 255) << (8 * b);
        if (q_out) q_out[(int64_t)n * ldq + k] = (int8_t)q;
      }
    }
  }
  if (layout) layout[word] = out;
}
}  // namespace

int launch_pack_w8(const float* W, int N, int K, int64_t ldw, int8_t* q_out, int64_t ldq, float* s_w, void* layout,
                   cudaStream_t st) {
  if (N == 0 || K == 0) return MQ_OK;
  row_scale_kernel<<<N, 256, 0, st>>>(W, N, K, ldw, s_w, 127.0f);
  const int64_t TNs = (N + MQ_W_TILE_N - 1) / MQ_W_TILE_N, KB = (K + MQ_W_TILE_K - 1) / MQ_W_TILE_K;
  const int64_t nw = TNs * KB * 4096;
  pack8_layout_kernel<<<(unsigned)((nw + 255) / 256), 256, 0, st>>>(W, N, K, ldw, s_w, static_cast<uint32_t*>(layout),
                                                                   q_out, ldq, (int)KB, nw);
  return cuda_status(cudaGetLastError());
}

int launch_repack_w4(const uint8_t* packed, int N, int K, void* layout, cudaStream_t st) {
  if (N == 0 || K == 0) return MQ_OK;
  const int64_t nw = layout_words(N, K);
  repack_kernel<<<(unsigned)((nw + 255) / 256), 256, 0, st>>>(
      packed, N, K, static_cast<uint32_t*>(layout), (K + MQ_W_TILE_K - 1) / MQ_W_TILE_K, nw);
  return cuda_status(cudaGetLastError());
}

int launch_unpack_w4(const uint8_t* packed, const void* layout, int N, int K, int8_t* q,
                     int64_t ldq, cudaStream_t st) {
  if (N == 0 || K == 0) return MQ_OK;
  const int64_t n = (int64_t)N * K;
  unpack_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(
      packed, static_cast<const uint8_t*>(layout), N, K, (K + MQ_W_TILE_K - 1) / MQ_W_TILE_K, q, ldq);
  return cuda_status(cudaGetLastError());
}

}  // namespace mq
