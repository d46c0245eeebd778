// Warp-level front end shared by the quantizer kernel and the few-token GEMV: load 1024
// consecutive bf16 channels of one row, apply the online block-Hadamard rotation, quantize.
//
// Method: Fig. 4(a), App. A.3 (H_2 and the Kronecker recursion), Eq. 2 / Eq. 3.
// Mapping: see mq_fwht_quant.cu.  A rotation block of n = 32 * TPB channels is held by TPB
// adjacent lanes (lane-in-block j), each lane keeping four 16-byte chunks; chunk i of the lane
// covers the channels blk_start + (i * TPB + j) * 8 .. + 7.
#pragma once
#include <cstdint>

namespace mq {

constexpr int kFwhtWarpTile = 1024;  // channels per warp pass

__device__ __forceinline__ uint32_t pack_sat_s8x4(int q0, int q1, int q2, int q3) {
  // cvt.pack.sat.s8.s32.b32 d, a, b, c : d = { c[15:0], sat8(a), sat8(b) } (b in the low byte)
  uint32_t hi, out;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q3), "r"(q2), "r"(0));
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(out) : "r"(q1), "r"(q0), "r"(hi));
  return out;
}

// Loads this lane's four chunks of the row (zeros past K) and, if ROT, transforms them:
// butterflies in increasing stride order, one float32 rounding each, then x c_n = 1/sqrt(n).
// Must be called by all 32 lanes (warp shuffles).
template <int LOG_TPB, bool ROT>
__device__ __forceinline__ void fwht_warp_tile(const uint16_t* __restrict__ xrow, int K, int blk_start, int j,
                                               float c_n, float (&v)[4][8]) {
  constexpr int TPB = 1 << LOG_TPB;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int off = blk_start + (i * TPB + j) * 8;
    uint4 w = make_uint4(0u, 0u, 0u, 0u);
    if (off < K) w = __ldg(reinterpret_cast<const uint4*>(xrow + off));
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      v[i][2 * p] = __uint_as_float(ww[p] << 16);
      v[i][2 * p + 1] = __uint_as_float(ww[p] & 0xffff0000u);
    }
  }

  if (ROT) {
    // strides 1, 2, 4: inside each 8-element chunk
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
      for (int h = 1; h < 8; h <<= 1) {
#pragma unroll
        for (int r = 0; r < 8; ++r) {
          if ((r & h) == 0) {
            const float a = v[i][r], b = v[i][r + h];
            v[i][r] = __fadd_rn(a, b);
            v[i][r + h] = __fsub_rn(a, b);
          }
        }
      }
    }
    // strides 8 * 2^b for b < log2(TPB): partner lane j ^ 2^b
#pragma unroll
    for (int b = 0; b < LOG_TPB; ++b) {
      const float sgn = ((j >> b) & 1) ? -1.0f : 1.0f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int r = 0; r < 8; ++r) {
          const float p = __shfl_xor_sync(0xffffffffu, v[i][r], 1 << b);
          // lower element: own + partner; upper element: partner - own (one rounding)
          v[i][r] = __fmaf_rn(v[i][r], sgn, p);
        }
      }
    }
    // strides 8 * TPB and 16 * TPB: across the four chunks of this lane
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      float a0 = v[0][r], a1 = v[1][r], a2 = v[2][r], a3 = v[3][r];
      float b0 = __fadd_rn(a0, a1), b1 = __fsub_rn(a0, a1);
      float b2 = __fadd_rn(a2, a3), b3 = __fsub_rn(a2, a3);
      v[0][r] = __fmul_rn(__fadd_rn(b0, b2), c_n);
      v[1][r] = __fmul_rn(__fadd_rn(b1, b3), c_n);
      v[2][r] = __fmul_rn(__fsub_rn(b0, b2), c_n);
      v[3][r] = __fmul_rn(__fsub_rn(b1, b3), c_n);
    }
  }
}

// Eq. 2 with a reciprocal scale: round-to-nearest-even of v * inv, saturated to int8 (NaN -> 0).
__device__ __forceinline__ uint2 quant_chunk_s8(const float (&v)[8], float inv) {
  int q[8];
#pragma unroll
  for (int r = 0; r < 8; ++r) q[r] = __float2int_rn(__fmul_rn(v[r], inv));
  uint2 o;
  o.x = pack_sat_s8x4(q[0], q[1], q[2], q[3]);
  o.y = pack_sat_s8x4(q[4], q[5], q[6], q[7]);
  return o;
}

// The same with 4-bit codes (the activation side of W4A4, Sec. 4.1): clamp to [-8, 7]; the codes still
// occupy one byte each.
__device__ __forceinline__ uint2 quant_chunk_s4(const float (&v)[8], float inv) {
  int q[8];
#pragma unroll
  for (int r = 0; r < 8; ++r) q[r] = max(-8, min(7, __float2int_rn(__fmul_rn(v[r], inv))));
  uint2 o;
  o.x = pack_sat_s8x4(q[0], q[1], q[2], q[3]);
  o.y = pack_sat_s8x4(q[4], q[5], q[6], q[7]);
  return o;
}

}  // namespace mq
