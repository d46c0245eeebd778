// K2v: the W4A8 linear for one to three tokens (single-sequence decode) as a GEMV on the
// CUDA cores, with rotation and quantizer in the same kernel.
//
// Method: the same arithmetic as the quantizer + GEMM pair (Fig. 4(a), App. A.3, Eq. 2, Eq. 3):
// codes Qx = Q_int8(FWHT(x)), acc[t,n] = sum_k Qx[t,k] q_w[n,k] in int32,
// Y = float(acc) * (s_mod(t) * s_w[n]) (+ bias).  The paper measures its decode speed with a
// dedicated W4A8 GEMV kernel (Sec. 4.3, decode table); this is that case.
//
// Why not the tensor-core kernel.  With a handful of tokens the product is one pass over the
// int4 weights, i.e. bounded by HBM, and a launch lasts only a few microseconds.  The tensor-core
// kernel's CTA takes a whole SM (512 threads, 226 KB of shared memory), so the next launch cannot
// be resident and prefetching while it runs, and its fixed parts (tensor-memory allocation,
// pipeline fill, epilogue, the boundary to the next launch) weigh as much as the stream itself;
// measured, it stays below 3 TB/s on these shapes.  For very few tokens the integer dot-product
// instruction (dp4a) needs a fraction of the issue slots at the HBM rate, so the CUDA cores are
// enough, nothing has to be staged, and small CTAs of consecutive launches overlap.
//
// Mapping.  A CTA owns 32 consecutive output channels (one quarter of a 128-channel layout
// tile) and ALL of K; warp w takes the K blocks w, w + W, w + 2W, ...  A lane owns one channel:
// its 32 codes of a K = 32 piece are one 16-byte load, and the 32 lanes of a warp read 512
// contiguous bytes of the layout tile.  The weights of the next K block are in flight while
// the current one is multiplied.  The int8 activation codes of the (up to three) tokens sit
// in shared memory; every lane reads the same address (broadcast).  With bf16 input every
// CTA rotates and quantizes the few rows for itself (the quantizer kernel's own warp routine),
// which removes one kernel boundary -- about 2 us, as much as the weights of a 4096 x 13696
// linear take to stream -- from every linear.  The warps' partial sums are added through
// shared memory and the first warp runs the dequant epilogue.
//
// Overlap between consecutive launches.  The kernel is launched with programmatic stream
// serialization.  Before it waits for its predecessor it asks L2 for its slice of the weights
// (a prefetch hint only, see below), so HBM streams the next linear's weights while the current
// one computes; it releases its own dependents only after its wait, so exactly one later
// launch runs ahead like this, not a chain of them.  W (warps per CTA) is chosen for about 24
// warps per SM over the launch, which leaves room for the CTAs of that next launch.
#include <cmath>
#include <cuda_bf16.h>

#include "mq_common.cuh"
#include "mq_fwht_warp.cuh"

namespace mq {
namespace {

constexpr int kGemvMaxT = 3;   // at four tokens the tensor-core kernel is faster (measured: 31.8 vs 34.1 us per MLP pass)
constexpr int kGemvMaxWarps = 32;
constexpr int kGemvWarpsPerSm = 24;
constexpr int kGemvSmemLimit = 200 * 1024;

struct GemvParams {
  int T, K, N;
  int kb_total;   // K blocks of 128
  int kpad;       // kb_total * 128: row pitch of the activation codes in shared memory
  const int8_t* Qx;   // int8 activation codes [T, K] (pitch ldq), or nullptr: quantize Xb here
  int64_t ldq;
  const uint16_t* Xb; // bf16 activations [T, K] (pitch ldx), used when Qx == nullptr
  int64_t ldx;
  int rot_block;      // 0 or the Hadamard block (power of two, 32..1024) applied to Xb
  float inv_vis, inv_txt, c_n;  // reciprocal activation scales, 1 / sqrt(rot_block)
  SegTable seg;
  float s_vis, s_txt;
  const uint8_t* W_layout;
  const float* s_w;
  const float* bias;
  void* Y;
  int64_t ldy;
  int y_is_f32;
  int32_t* acc_out;
  const float* row_scales;  // optional [T]: per-token activation scales (int8 input only)
  // split part of the rotation-magnitude-suppression linear (Sec. 3.2), bf16 input only: the codes of
  // the first channel of every rotation block times side_kb extra weight tiles per channel tile,
  // with their own scale, added before the bias
  const uint8_t* side_layout;  // nullptr: none
  const float* s_w_side;
  int side_kb;                 // K blocks (of 128 split codes) per channel tile
  int side_cols;               // K / rot_block: split codes per row
  int32_t* acc_side_out;
};

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
  uint4 v;
  // the weights are read exactly once: keep them out of L1
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// Rotates and quantizes the rows of Xb into the shared-memory code array (row pitch kpad).
template <int LOG_TPB, bool ROT>
__device__ __forceinline__ void stage_rows(const GemvParams& p, uint8_t* xs, int warp, int lane, int warps) {
  constexpr int TPB = 1 << LOG_TPB;
  const int tiles_per_row = (p.K + kFwhtWarpTile - 1) / kFwhtWarpTile;
  const int j = lane & (TPB - 1);
  const int blk = lane >> LOG_TPB;
  for (int wt = warp; wt < p.T * tiles_per_row; wt += warps) {  // warp-uniform trip count
    // every CTA stages the same rows: start each CTA at a different tile so that the CTAs of the
    // launch do not all ask L2 for the same lines at the same moment
    const int row = wt / tiles_per_row;
    const int tile = (wt - row * tiles_per_row + (int)blockIdx.x) % tiles_per_row;
    const int blk_start = tile * kFwhtWarpTile + blk * (32 * TPB);
    float v[4][8];
    fwht_warp_tile<LOG_TPB, ROT>(p.Xb + (int64_t)row * p.ldx, p.K, blk_start, j, p.c_n, v);
    const float inv = thread_row_modality(p.seg, row) == MQ_VISUAL ? p.inv_vis : p.inv_txt;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int off = blk_start + (i * TPB + j) * 8;
      if (off < p.K) *reinterpret_cast<uint2*>(xs + (size_t)row * p.kpad + off) = quant_chunk_s8(v[i], inv);
    }
  }
}

// One 16-byte piece of packed weights (32 codes of this lane's channel) against the 32 activation
// codes at xp (two 16-byte broadcast reads) of one token.
__device__ __forceinline__ int dot_piece(const uint4& w, const uint4* xp, int acc) {
  const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
  const uint4 xa = xp[0], xb = xp[1];
  const uint32_t xw[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int lo = (int)((ww[i] << 4) & 0xF0F0F0F0u);  // codes k0 .. k0+3, each x16
    const int hi = (int)(ww[i] & 0xF0F0F0F0u);         // codes k0+4 .. k0+7, each x16
    acc = __dp4a(lo, (int)xw[2 * i], acc);
    acc = __dp4a(hi, (int)xw[2 * i + 1], acc);
  }
  return acc;
}

template <int TT>
__global__ void __launch_bounds__(kGemvMaxWarps * 32)
w4a8_gemv_kernel(const GemvParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  uint4* xs = reinterpret_cast<uint4*>(smem_raw);                                  // [TT][kpad] int8
  int32_t* red = reinterpret_cast<int32_t*>(smem_raw + (size_t)TT * p.kpad);       // [warps][TT][32]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int warps = blockDim.x >> 5;
  const int tn = blockIdx.x >> 2, quarter = blockIdx.x & 3;
  const int r = quarter * 32 + lane;
  const int n = tn * MQ_W_TILE_N + r;
  const bool live = tn * MQ_W_TILE_N + quarter * 32 < p.N;  // false: a quarter past the last channel (whole CTA)
  if (live) {
    // The weights do not depend on the kernel running in front of this one: ask L2 for this CTA's
    // whole slice now, 512 contiguous bytes per (K block, piece), so that HBM streams while that
    // kernel finishes.  Only a hint: the loads below run after pdl_wait and go through L2, the
    // point of coherence.  (Issuing the requests from a few CTAs for everybody was measured and
    // is far slower: the bulk-prefetch rate of one SM is the limit then.)
    const uint8_t* slice = p.W_layout + (size_t)tn * p.kb_total * 8192 + quarter * 512;
    for (int c = threadIdx.x; c < p.kb_total * 4; c += blockDim.x)
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], 512;" ::"l"(slice + (size_t)c * 2048) : "memory");
  }
  pdl_wait();  // the activations come from the kernel launched just before
  // Dependents may start only now: exactly one later launch is then resident ahead of its turn
  // (prefetching its weights while this one computes), not an unbounded chain of them.
  pdl_launch_dependents();
  if (!live) return;

  // activation codes -> shared memory, zero-padded to whole K blocks
  const int chunks = p.kpad >> 4;
  if (p.Qx) {
    for (int i = threadIdx.x; i < TT * chunks; i += blockDim.x) {
      const int t = i / chunks, c = i - t * chunks;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (t < p.T && c * 16 < p.K) v = __ldg(reinterpret_cast<const uint4*>(p.Qx + (int64_t)t * p.ldq + c * 16));
      xs[i] = v;
    }
  } else {
    uint32_t* xs32 = reinterpret_cast<uint32_t*>(xs);
    const int words = p.kpad >> 2;
    // zero what the passes below do not write: channels K .. kpad of every row, and rows >= T
    for (int t = 0; t < TT; ++t) {
      const int first = t < p.T ? (p.K >> 2) : 0;
      for (int c = first + threadIdx.x; c < words; c += blockDim.x) xs32[t * words + c] = 0u;
    }
    switch (p.rot_block) {
#define MQ_STAGE(LOG_TPB, ROT) stage_rows<LOG_TPB, ROT>(p, reinterpret_cast<uint8_t*>(xs), warp, lane, warps); break;
      case 0: MQ_STAGE(2, false)
      case 32: MQ_STAGE(0, true)
      case 64: MQ_STAGE(1, true)
      case 128: MQ_STAGE(2, true)
      case 256: MQ_STAGE(3, true)
      case 512: MQ_STAGE(4, true)
      default: MQ_STAGE(5, true)
#undef MQ_STAGE
    }
  }
  // the activations' own loads went out first: they are few and everything waits for them
  const uint4* wsrc = reinterpret_cast<const uint4*>(p.W_layout + (size_t)tn * p.kb_total * 8192) + r;
  // One token: two K blocks of this warp are in flight at any time (buffers A and B are refilled
  // as soon as they have been multiplied).  More tokens: the multiplication of a block is long
  // enough to cover one load, and the second buffer is fetched while the first is multiplied
  // (measured: the deeper scheme costs registers there and is slower).
  constexpr bool kTwoInFlight = TT == 1;
  uint4 wa[4], wb[4];
  int kb = warp;
  auto fetch = [&](uint4 (&dst)[4], int k) {
    if (k < p.kb_total) {
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) dst[jj] = ldg_stream(wsrc + ((size_t)k * 4 + jj) * 128);
    }
  };
  fetch(wa, kb);
  if (kTwoInFlight) fetch(wb, kb + warps);
  __syncthreads();

  int acc[TT];
#pragma unroll
  for (int t = 0; t < TT; ++t) acc[t] = 0;
  auto multiply = [&](const uint4 (&w)[4], int k) {
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
#pragma unroll
      for (int t = 0; t < TT; ++t) acc[t] = dot_piece(w[jj], xs + (size_t)t * chunks + k * 8 + jj * 2, acc[t]);
    }
  };
  if (kTwoInFlight) {
    for (; kb < p.kb_total; kb += 2 * warps) {
      multiply(wa, kb);
      fetch(wa, kb + 2 * warps);
      if (kb + warps < p.kb_total) {
        multiply(wb, kb + warps);
        fetch(wb, kb + 3 * warps);
      }
    }
  } else {
    for (; kb < p.kb_total; kb += warps) {
      fetch(wb, kb + warps);
      multiply(wa, kb);
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) wa[jj] = wb[jj];
    }
  }

#pragma unroll
  for (int t = 0; t < TT; ++t) red[(warp * TT + t) * 32 + lane] = acc[t];
  // split part: its activation codes are those at the first channel of every rotation block;
  // gather them side by side (zero-padded to whole K blocks) behind the partial sums
  uint4* xside = reinterpret_cast<uint4*>(red + warps * TT * 32);
  const int side_pad = p.side_kb * MQ_W_TILE_K;
  if (p.side_layout) {
    const int8_t* xb8 = reinterpret_cast<const int8_t*>(xs);
    int8_t* dst = reinterpret_cast<int8_t*>(xside);
    for (int i = threadIdx.x; i < TT * side_pad; i += blockDim.x) {
      const int t = i / side_pad, b = i - t * side_pad;
      dst[i] = b < p.side_cols ? xb8[(size_t)t * p.kpad + (size_t)b * p.rot_block] : (int8_t)0;
    }
  }
  __syncthreads();
  if (warp != 0 || n >= p.N) return;
  int acc_s[TT];
#pragma unroll
  for (int t = 0; t < TT; ++t) acc_s[t] = 0;
  float sws = 0.0f;
  if (p.side_layout) {
    // a few hundred multiply-adds per channel: the first warp does them on its way out
    const uint4* ssrc = reinterpret_cast<const uint4*>(p.side_layout + (size_t)tn * p.side_kb * 8192) + r;
    for (int c = 0; c < p.side_kb * 4; ++c) {
      const uint4 w = ldg_stream(ssrc + (size_t)c * 128);
#pragma unroll
      for (int t = 0; t < TT; ++t) acc_s[t] = dot_piece(w, xside + (size_t)t * (side_pad >> 4) + c * 2, acc_s[t]);
    }
    sws = p.s_w_side[n];
  }
  const float sw = p.s_w[n];
  const float bs = p.bias ? p.bias[n] : 0.0f;
#pragma unroll
  for (int t = 0; t < TT; ++t) {
    if (t >= p.T) break;
    int a = 0;
    for (int w = 0; w < warps; ++w) a += red[(w * TT + t) * 32 + lane];
    a >>= 4;  // every product carried the factor 16 of the nibble placement: exact
    if (p.acc_out) p.acc_out[(size_t)t * p.N + n] = a;
    const float st = p.row_scales ? p.row_scales[t]
                                  : (thread_row_modality(p.seg, t) == MQ_VISUAL ? p.s_vis : p.s_txt);
    float y = __fmul_rn((float)a, __fmul_rn(st, sw));
    if (p.side_layout) {
      const int as = acc_s[t] >> 4;
      if (p.acc_side_out) p.acc_side_out[(size_t)t * p.N + n] = as;
      y = __fadd_rn(y, __fmul_rn((float)as, __fmul_rn(st, sws)));
    }
    if (p.bias) y = __fadd_rn(y, bs);
    if (p.y_is_f32) static_cast<float*>(p.Y)[(size_t)t * p.ldy + n] = y;
    else static_cast<__nv_bfloat16*>(p.Y)[(size_t)t * p.ldy + n] = __float2bfloat16_rn(y);
  }
}

size_t gemv_smem(int T, int K, int warps, int side_k = 0) {
  const int tt = T <= 1 ? 1 : (T <= 2 ? 2 : 3);
  const size_t kpad = (size_t)((K + MQ_W_TILE_K - 1) / MQ_W_TILE_K) * MQ_W_TILE_K;
  const size_t side_pad = (size_t)((side_k + MQ_W_TILE_K - 1) / MQ_W_TILE_K) * MQ_W_TILE_K;
  return (size_t)tt * kpad + (size_t)warps * tt * 32 * sizeof(int32_t) + (size_t)tt * side_pad;
}

}  // namespace

bool gemv_applies(int T, int K, int N, int side_k) {
  if (T < 1 || T > kGemvMaxT || K <= 0 || N <= 0) return false;
  return gemv_smem(T, K, kGemvMaxWarps, side_k) <= (size_t)kGemvSmemLimit;
}

int launch_gemv(const GemmArgs& a, cudaStream_t st) {
  GemvParams p{};
  p.T = a.T; p.K = a.K; p.N = a.N;
  p.kb_total = (a.K + MQ_W_TILE_K - 1) / MQ_W_TILE_K;
  p.kpad = p.kb_total * MQ_W_TILE_K;
  p.Qx = a.Qx; p.ldq = a.ldq; p.seg = a.seg; p.s_vis = a.s_vis; p.s_txt = a.s_txt;
  if (!a.Qx) {
    if (!a.Xb) return MQ_ERR_INVALID_ARG;
    p.Xb = static_cast<const uint16_t*>(a.Xb); p.ldx = a.ldx; p.rot_block = a.rot_block;
    p.inv_vis = 1.0f / a.s_vis; p.inv_txt = 1.0f / a.s_txt;
    p.c_n = a.rot_block ? (float)(1.0 / sqrt((double)a.rot_block)) : 1.0f;
  }
  p.W_layout = static_cast<const uint8_t*>(a.W_layout);
  p.s_w = a.s_w; p.bias = a.bias; p.Y = a.Y; p.ldy = a.ldy; p.y_is_f32 = a.y_is_f32; p.acc_out = a.acc_out;
  p.row_scales = a.row_scales;
  if (a.side_layout) {
    if (a.Qx || !a.rot_block) return MQ_ERR_INVALID_ARG;
    p.side_layout = static_cast<const uint8_t*>(a.side_layout);
    p.s_w_side = a.s_w_side;
    p.side_kb = (a.side_k + MQ_W_TILE_K - 1) / MQ_W_TILE_K;
    p.side_cols = a.K / a.rot_block;
    p.acc_side_out = a.acc_side_out;
  }
  const int n_tn = (a.N + MQ_W_TILE_N - 1) / MQ_W_TILE_N;
  const int ctas = n_tn * 4;
  int warps = (sm_count() * kGemvWarpsPerSm + ctas - 1) / ctas;
  if (warps > kGemvMaxWarps) warps = kGemvMaxWarps;
  if (warps > p.kb_total) warps = p.kb_total;
  if (warps < 1) warps = 1;
  const size_t smem = gemv_smem(a.T, a.K, warps, a.side_layout ? a.side_k : 0);
  auto kernel = a.T <= 1 ? w4a8_gemv_kernel<1> : (a.T <= 2 ? w4a8_gemv_kernel<2> : w4a8_gemv_kernel<3>);
  static PerDeviceTable<char> attr_set[3];
  const int ki = a.T <= 1 ? 0 : (a.T <= 2 ? 1 : 2);
  if (!ensure_dynamic_smem(attr_set[ki], kernel, kGemvSmemLimit)) return MQ_ERR_CUDA;
  return cuda_status(launch_pdl(kernel, dim3(ctas), dim3(warps * 32), smem, st, p));
}

}  // namespace mq
