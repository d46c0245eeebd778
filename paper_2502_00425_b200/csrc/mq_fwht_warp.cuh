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
// The loads alone: this lane's four 16-byte chunks of the tile (zeros past K), so that a caller can have the
// loads of a second tile in flight while it transforms the first.
template <int LOG_TPB>
__device__ __forceinline__ void fwht_warp_load(const uint16_t* __restrict__ xrow, int K, int blk_start, int j,
                                               uint4 (&raw)[4]) {
  constexpr int TPB = 1 << LOG_TPB;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int off = blk_start + (i * TPB + j) * 8;
    raw[i] = make_uint4(0u, 0u, 0u, 0u);
    if (off < K) raw[i] = __ldg(reinterpret_cast<const uint4*>(xrow + off));
  }
}

template <int LOG_TPB, bool ROT>
__device__ __forceinline__ void fwht_warp_compute(const uint4 (&raw)[4], int j, float c_n, float (&v)[4][8]);

template <int LOG_TPB, bool ROT>
__device__ __forceinline__ void fwht_warp_tile(const uint16_t* __restrict__ xrow, int K, int blk_start, int j,
                                               float c_n, float (&v)[4][8]) {
  uint4 raw[4];
  fwht_warp_load<LOG_TPB>(xrow, K, blk_start, j, raw);
  fwht_warp_compute<LOG_TPB, ROT>(raw, j, c_n, v);
}

// bf16 -> float32 and, if ROT, the transform of one tile from its loaded chunks.
template <int LOG_TPB, bool ROT>
__device__ __forceinline__ void fwht_warp_compute(const uint4 (&raw)[4], int j, float c_n, float (&v)[4][8]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t ww[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      v[i][2 * p] = __uint_as_float(ww[p] << 16);
      v[i][2 * p + 1] = __uint_as_float(ww[p] & 0xffff0000u);
    }
  }

  if (ROT) {
    // The butterflies run on pairs of float32 values (add / fma .f32x2: two IEEE round-to-nearest results per
    // instruction, bit-identical to the scalar ones).  A pair holds the same element r of two chunks that
    // no stage but the last combines: (chunk 0, chunk 2) in pa, (chunk 1, chunk 3) in pb.
    const float2 minus1 = make_float2(-1.0f, -1.0f);
    float2 pa[8], pb[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      pa[r] = make_float2(v[0][r], v[2][r]);
      pb[r] = make_float2(v[1][r], v[3][r]);
    }
    // strides 1, 2, 4: inside each 8-element chunk
#pragma unroll
    for (int h = 1; h < 8; h <<= 1) {
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        if ((r & h) == 0) {
          const float2 a0 = pa[r], b0 = pa[r + h], a1 = pb[r], b1 = pb[r + h];
          pa[r] = __fadd2_rn(a0, b0);
          pa[r + h] = __ffma2_rn(b0, minus1, a0);  // a - b, one rounding
          pb[r] = __fadd2_rn(a1, b1);
          pb[r + h] = __ffma2_rn(b1, minus1, a1);
        }
      }
    }
    // strides 8 * 2^b for b < log2(TPB): partner lane j ^ 2^b
#pragma unroll
    for (int b = 0; b < LOG_TPB; ++b) {
      const float sg = ((j >> b) & 1) ? -1.0f : 1.0f;
      const float2 sgn = make_float2(sg, sg);
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        float2 qa, qb;
        qa.x = __shfl_xor_sync(0xffffffffu, pa[r].x, 1 << b);
        qa.y = __shfl_xor_sync(0xffffffffu, pa[r].y, 1 << b);
        qb.x = __shfl_xor_sync(0xffffffffu, pb[r].x, 1 << b);
        qb.y = __shfl_xor_sync(0xffffffffu, pb[r].y, 1 << b);
        // lower element: own + partner; upper element: partner - own (one rounding)
        pa[r] = __ffma2_rn(pa[r], sgn, qa);
        pb[r] = __ffma2_rn(pb[r], sgn, qb);
      }
    }
    // strides 8 * TPB and 16 * TPB: across the four chunks of this lane
    const float2 cn2 = make_float2(c_n, c_n);
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      const float2 s02 = __fadd2_rn(pa[r], pb[r]);          // (c0 + c1, c2 + c3)
      const float2 d02 = __ffma2_rn(pb[r], minus1, pa[r]);  // (c0 - c1, c2 - c3)
      const float2 o02 = __fmul2_rn(make_float2(__fadd_rn(s02.x, s02.y), __fsub_rn(s02.x, s02.y)), cn2);
      const float2 o13 = __fmul2_rn(make_float2(__fadd_rn(d02.x, d02.y), __fsub_rn(d02.x, d02.y)), cn2);
      v[0][r] = o02.x;
      v[2][r] = o02.y;
      v[1][r] = o13.x;
      v[3][r] = o13.y;
    }
  }
}

// Eq. 2 with a reciprocal scale: round-to-nearest-even of v * inv, saturated to int8 (NaN -> 0).
__device__ __forceinline__ uint2 quant_chunk_s8(const float (&v)[8], float inv) {
  int q[8];
  const float2 inv2 = make_float2(inv, inv);
#pragma unroll
  for (int r = 0; r < 8; r += 2) {
    const float2 y = __fmul2_rn(make_float2(v[r], v[r + 1]), inv2);  // two IEEE products per instruction
    q[r] = __float2int_rn(y.x);
    q[r + 1] = __float2int_rn(y.y);
  }
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
