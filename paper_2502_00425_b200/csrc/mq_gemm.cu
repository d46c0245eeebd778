// K2: W4A8 integer GEMM with the MSQ dequant epilogue, written for sm_100a.
//
// Method: Eq. 2 (uniform quantizer; the integer product of the codes times both scales
// reconstructs the real product), Eq. 3 (one static activation scale per modality, looked
// up per token row), Algorithm 1 (per-output-channel weight scales).
//   acc[t,n] = sum_k Qx[t,k] * q_w[n,k]      (int8 x int4 -> int32, exact)
//   Y[t,n]   = float(acc) * (s_mod(t) * s_w[n]) (+ bias[n])
//
// Design (differs from a conventional "unpack B into shared memory" GEMM on purpose).
// On B200 a 128-row tcgen05 MMA reads its shared-memory operands at close to the
// shared-memory bandwidth of the SM, so re-writing unpacked weights to shared memory
// would make shared memory, not the tensor pipe, the limit.  Here the product is
// computed transposed, D[n,t] = sum_k W[n,k] X[t,k]:
//   * the WEIGHTS are the MMA's A operand and live in TENSOR MEMORY: four warps read the
//     packed int4 tile from shared memory (staged there by a bulk async copy), expand each
//     32-bit word into eight int8 values with two logic operations, and write them with
//     tcgen05.st -- the expanded weights never touch shared memory;
//   * the int8 ACTIVATIONS are the B operand, TMA-loaded (128-byte swizzle, K-major)
//     straight from the quantizer's output;
//   * accumulators (128 channels x up to 256 tokens, int32) live in tensor memory and are
//     double-buffered when the token tile is <= 192 so the epilogue of one tile overlaps
//     the main loop of the next;
//   * the epilogue thread that owns channel n holds s_w[n] and bias[n] in registers and
//     gets the per-token scale from a small shared-memory table built from the segment
//     table; consecutive lanes write consecutive channels of one token row.
// The nibble-to-int8 expansion leaves each code in the HIGH nibble of its byte, i.e. the
// MMA sees 16*q_w; the accumulator is therefore exactly 16x the true one (|16 acc| <=
// 128*8*16*K < 2^31 for K <= 131071) and the epilogue shifts it back, exactly.
//
// Warp roles (512 threads): warp 0 activation TMA producer, warp 1 MMA issuer, warp 2
// tensor-memory allocator, warp 3 weight bulk-copy producer, warps 4-11 weight expanders (two
// groups of four that take alternate K blocks; within a group one warp per 32-lane quarter of
// tensor memory), warps 12-15 epilogue.
//
// Every wait on an mbarrier is bounded: after ~2 s without progress the waiting thread
// records MQ_ERR_TIMEOUT and its site in the status word, raises a CTA-wide abort flag,
// and all roles drain (outstanding copies are awaited, tensor memory is freed).
#include <cuda.h>
#include <cuda_bf16.h>

#include "mq_common.cuh"
#include "mq_sm100.cuh"

namespace mq {
namespace {

constexpr int kMaxGroups = 2;                       // expander warp groups (4 warps each)
constexpr int kMaxThreads = (8 + 4 * kMaxGroups) * 32;
constexpr int kTileN = MQ_W_TILE_N;    // channels per CTA tile (MMA M)
constexpr int kBlockK = MQ_W_TILE_K;   // K per pipeline stage
constexpr int kWTileBytes = 8192;      // packed int4 tile 128 x 128 (an int8 tile is twice that)
constexpr int kMaxStages = 8;    // main ring: activation tiles in shared memory
constexpr int kMaxWStages = 16;  // packed-weight tiles in shared memory
constexpr int kSmemBudget = 226 * 1024;  // of the 227 KB a CTA may use

// Instantiations of the kernel.  kPlain: the W4A8 MSQ linear.  kRms: plus the split product of rotation
// magnitude suppression.  kGrouped: group-wise weight scales (one per output channel and K block of 128),
// folded into float sums after every K block.  kW8: 8-bit weights (no nibble expansion, no factor 16).
enum : int { kPlain = 0, kRms = 1, kGrouped = 2, kW8 = 3 };

struct KernelParams {
  int T, K, N;
  int TN;          // token tile (MMA N), multiple of 16, 16..256
  int n_tn;        // channel tiles
  int n_tt;        // token tiles
  int ksplit;      // K splits (1 = direct epilogue)
  int kb_total;    // K blocks
  int kb_per_split;        // K blocks per split (the last split may have fewer)
  int step_tn, step_tt, step_ks;  // the grid stride written in (n_tn, n_tt) mixed radix
  int num_d;       // accumulator buffers (1 or 2)
  int d_stride;    // tensor-memory columns between accumulator buffers
  int a_base;      // first tensor-memory column of the weight stages
  int num_a;       // expanded-weight slots in tensor memory (<= stages)
  int stages;      // main ring: activation stages in shared memory
  int w_stages;    // packed-weight stages in shared memory
  int groups;      // expander warp groups; group g expands the K blocks with it % groups == g
  int lean_issue;  // 1: the MMA loop is run by one elected thread; 0: by the converged warp (see mma_issuer)
  SegTable seg;
  float s_vis, s_txt;
  const uint8_t* W_layout;
  const float* s_w;
  const float* bias;
  void* Y;
  int64_t ldy;
  int y_is_f32;
  int32_t* acc_out;
  int32_t* splitk_acc;
  int32_t* status;
  const float* row_scales;  // optional [T]: per-token activation scales instead of the per-modality pair
  // split part of the rotation-magnitude-suppression linear (only read by the RMS instantiation)
  int side_kb;                 // K blocks of the split product per tile (0: none)
  int side_col;                // tensor-memory columns from an accumulator to its split accumulator
  const uint8_t* side_layout;  // split weights, GEMM layout, side_kb tiles per channel tile
  const float* s_w_side;
  int32_t* acc_side_out;       // optional dump of the split accumulator [T, N]
  int32_t* splitk_side;        // split-K launches: the split accumulator's own [T, N] slice
  int w_tile_bytes;            // bytes of one 128 x 128 weight tile in W_layout (8192 int4, 16384 int8)
};

struct __align__(16) Barriers {
  // main ring, one entry per K block in flight.  full: the activation tile has landed (TMA
  // transaction bytes) AND the four expander warps have written the weight slot (4 arrivals);
  // done: the MMAs that read the stage have completed (one tcgen05.commit).
  uint64_t full[kMaxStages], done[kMaxStages];
  uint64_t w_full[kMaxWStages], w_empty[kMaxWStages];
  uint64_t d_full[2], d_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

// Tile t of the launch is (channel tile, token tile, K split) = (t % n_tn, (t / n_tn) % n_tt,
// t / (n_tn * n_tt)); CTA b owns tiles b, b + grid, b + 2 grid, ...  The first one is decoded
// with divisions once; each further one is reached by adding the (host-decomposed) grid
// stride digit by digit, because a division per tile sits on the MMA warp's critical path.
struct TileIter {
  int tn, tt, ks;
  __device__ __forceinline__ void init(const KernelParams& p, int tile) {
    tn = tile % p.n_tn;
    const int rest = tile / p.n_tn;
    tt = rest % p.n_tt;
    ks = rest / p.n_tt;
  }
  __device__ __forceinline__ bool valid(const KernelParams& p) const { return ks < p.ksplit; }
  __device__ __forceinline__ void next(const KernelParams& p) {
    tn += p.step_tn;
    int carry = tn >= p.n_tn ? 1 : 0;
    tn -= carry * p.n_tn;
    tt += p.step_tt + carry;
    carry = tt >= p.n_tt ? 1 : 0;
    tt -= carry * p.n_tt;
    ks += p.step_ks + carry;
  }
  __device__ __forceinline__ int kb0(const KernelParams& p) const { return ks * p.kb_per_split; }
  __device__ __forceinline__ int kb1(const KernelParams& p) const { return min(p.kb_total, kb0(p) + p.kb_per_split); }
};

// ------------------------------------------------------------------------------ epilogue
// What the epilogue does with an accumulator is fixed per launch.  The product configurations
// (bf16 output, with or without bias, and the split-K partial sums) are compiled separately so
// that their per-element code has no branches; the debug outputs (accumulator dump, float32
// output) share one generic variant that tests its flags at run time.
// kEpiNoShift: the accumulator is the true one (8-bit weights), not 16x it.
enum : int { kEpiSplitK = 1, kEpiAcc = 2, kEpiF32 = 4, kEpiBias = 8, kEpiGeneric = 16, kEpiStaged = 32, kEpiNoShift = 64 };

// bf16 output of a 16 x 32 (token x channel) block held one channel per lane: transpose it
// through this warp's staging buffer so that every lane stores 16 bytes (8 channels of one
// token) instead of 2.
__device__ __forceinline__ void staged_store(const KernelParams& p, const float (&y)[16], int t_first, int nvalid,
                                             int n, __nv_bfloat16* stage) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int j = 0; j < 16; ++j) stage[j * 32 + lane] = __float2bfloat16_rn(y[j]);
  __syncwarp();
  const int n8 = n - lane + (lane & 3) * 8;  // first of this lane's 8 channels
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int row = (lane >> 2) + 8 * h;
    if (row < nvalid && n8 < p.N) {
      const uint4 val = *reinterpret_cast<const uint4*>(stage + row * 32 + (lane & 3) * 8);
      *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.Y) + (size_t)(t_first + row) * p.ldy + n8) = val;
    }
  }
  __syncwarp();
}

// 16 token columns of one channel (this lane's n): dequantize and store, or add into the
// split-K sums.  `nvalid` (1..16) masks the ragged end of the token range.
template <int MODE>
__device__ __forceinline__ void epilogue_chunk(const KernelParams& p, const uint32_t (&v)[16], int t_first,
                                               int nvalid, int n, bool n_ok, float sw, float bs,
                                               const float* stok, __nv_bfloat16* stage, int ks) {
  constexpr int SH = (MODE & kEpiNoShift) ? 0 : 4;  // the MMA saw 16 * q_w unless the weights are 8-bit
  if (!(MODE & kEpiStaged) && !n_ok) return;
  if (MODE & kEpiSplitK) {
    // every K split owns a slice [T,N] of the scratch: plain stores, summed by the finalize
    // kernel -- no atomics and nothing to clear beforehand
    int32_t* dst = p.splitk_acc + (size_t)ks * p.T * p.N + (size_t)t_first * p.N + n;
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (j < nvalid) dst[(size_t)j * p.N] = ((int)v[j]) >> SH;
    return;
  }
  if (MODE & kEpiGeneric) {
#pragma unroll 1
    for (int j = 0; j < nvalid; ++j) {
      const int acc = ((int)v[j]) >> SH;
      const size_t t = (size_t)(t_first + j);
      if (p.acc_out) p.acc_out[t * p.N + n] = acc;
      float y = __fmul_rn((float)acc, __fmul_rn(stok[j], sw));
      if (p.bias) y = __fadd_rn(y, bs);
      if (p.y_is_f32) static_cast<float*>(p.Y)[t * p.ldy + n] = y;
      else static_cast<__nv_bfloat16*>(p.Y)[t * p.ldy + n] = __float2bfloat16_rn(y);
    }
    return;
  }
  int32_t* acc_dst = (MODE & kEpiAcc) ? p.acc_out + (size_t)t_first * p.N + n : nullptr;
  float* y32 = static_cast<float*>(p.Y) + (size_t)t_first * p.ldy + n;
  __nv_bfloat16* y16 = static_cast<__nv_bfloat16*>(p.Y) + (size_t)t_first * p.ldy + n;
  float y[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    y[j] = __fmul_rn((float)(((int)v[j]) >> SH), __fmul_rn(stok[j], sw));
    if (MODE & kEpiBias) y[j] = __fadd_rn(y[j], bs);
  }
  if (MODE & kEpiStaged) {
    staged_store(p, y, t_first, nvalid, n, stage);
    return;
  }
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    if (j < nvalid) {
      if (MODE & kEpiAcc) acc_dst[(size_t)j * p.N] = ((int)v[j]) >> SH;
      if (MODE & kEpiF32) y32[(size_t)j * p.ldy] = y[j];
      else y16[(size_t)j * p.ldy] = __float2bfloat16_rn(y[j]);
    }
  }
}

// One accumulator tile of this warp's 32 channels.  Two register buffers: the tensor-memory
// load of the next 16 columns is in flight while the current 16 are converted and stored.
template <int MODE>
__device__ __forceinline__ void epilogue_tile(const KernelParams& p, uint32_t d_tmem, int t0, int n, bool n_ok,
                                              float sw, float bs, const float* stok, __nv_bfloat16* stage, int ks) {
  const int ncols = min(p.TN, p.T - t0);  // valid token columns of this tile (> 0)
  uint32_t va[16], vb[16];
  tmem_ld_x16(d_tmem, va);
  for (int cc = 0; cc < ncols; cc += 32) {
    __syncwarp();  // tcgen05.ld / wait::ld are warp-collective; lanes may have left the chunk code early
    tmem_wait_ld();
    const bool has_b = cc + 16 < ncols;
    if (has_b) tmem_ld_x16(d_tmem + cc + 16, vb);
    epilogue_chunk<MODE>(p, va, t0 + cc, min(16, ncols - cc), n, n_ok, sw, bs, stok + cc, stage, ks);
    if (has_b) {
      __syncwarp();
      tmem_wait_ld();
      if (cc + 32 < ncols) tmem_ld_x16(d_tmem + cc + 32, va);
      epilogue_chunk<MODE>(p, vb, t0 + cc + 16, min(16, ncols - cc - 16), n, n_ok, sw, bs, stok + cc + 16, stage, ks);
    }
  }
}

// Epilogue of a tile that carries a split accumulator (rotation magnitude suppression): the
// main accumulator at d_tmem and the split one p.side_col columns further on, each with its
// own per-channel weight scale:
//   y = fl(acc_main * fl(s_a * s_w)) + fl(acc_side * fl(s_a * s_w_side)), then + bias.
// STAGED: bf16 output through the staging buffer; otherwise every output the call asked for
// (accumulator dumps, fp32 or bf16 Y) with predicated per-element stores.
template <bool STAGED>
__device__ __forceinline__ void epilogue_tile_side(const KernelParams& p, uint32_t d_tmem, int t0, int n, bool n_ok,
                                                   float sw, float sws, float bs, const float* stok,
                                                   __nv_bfloat16* stage) {
  const int ncols = min(p.TN, p.T - t0);
  const bool has_bias = p.bias != nullptr;
  for (int cc = 0; cc < ncols; cc += 16) {
    uint32_t vm[16], vs[16];
    __syncwarp();
    tmem_ld_x16(d_tmem + cc, vm);
    tmem_ld_x16(d_tmem + p.side_col + cc, vs);
    tmem_wait_ld();
    const int nvalid = min(16, ncols - cc);
    const int t_first = t0 + cc;
    float y[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const float st = stok[cc + j];
      y[j] = __fadd_rn(__fmul_rn((float)(((int)vm[j]) >> 4), __fmul_rn(st, sw)),
                       __fmul_rn((float)(((int)vs[j]) >> 4), __fmul_rn(st, sws)));
      if (has_bias) y[j] = __fadd_rn(y[j], bs);
    }
    if (STAGED) {
      staged_store(p, y, t_first, nvalid, n, stage);
    } else if (n_ok) {
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (j < nvalid) {
          const size_t t = (size_t)(t_first + j);
          if (p.acc_out) p.acc_out[t * p.N + n] = ((int)vm[j]) >> 4;
          if (p.acc_side_out) p.acc_side_out[t * p.N + n] = ((int)vs[j]) >> 4;
          if (p.y_is_f32) static_cast<float*>(p.Y)[t * p.ldy + n] = y[j];
          else static_cast<__nv_bfloat16*>(p.Y)[t * p.ldy + n] = __float2bfloat16_rn(y[j]);
        }
      }
    }
  }
}

// Split-K launch: the tile of K split 0 also owns the split accumulator; it goes to its own slice.
__device__ __forceinline__ void epilogue_tile_side_slice(const KernelParams& p, uint32_t d_tmem, int t0, int n,
                                                         bool n_ok) {
  const int ncols = min(p.TN, p.T - t0);
  for (int cc = 0; cc < ncols; cc += 16) {
    uint32_t vs[16];
    __syncwarp();
    tmem_ld_x16(d_tmem + p.side_col + cc, vs);
    tmem_wait_ld();
    if (n_ok) {
      int32_t* dst = p.splitk_side + (size_t)(t0 + cc) * p.N + n;
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if (cc + j < ncols) dst[(size_t)j * p.N] = ((int)vs[j]) >> 4;
    }
  }
}

// ------------------------------------------------------------------------------ the MMA issuer
// Per K block the issuer waits on one barrier (activation tile landed and weight slot written), issues four
// MMAs and one commit.  Two forms of the same loop:
//   LEAN: one elected thread runs the whole loop, with no warp vote and no election per block.  The loop then
//     costs ~100 cycles per block instead of ~320, which is what small token tiles (decode shapes, where the
//     MMAs of a block take less than that) are bound by; measured 2 to 8 % faster for every tile width with
//     four or more weight slots.
//   converged: the whole warp runs the loop, votes on every wait and elects the issuing lane per block.  With
//     only two weight slots (224-token tiles when a CTA runs several tiles) this form measured 4 to 6 % faster
//     than the lean one; the launch picks it for that case.
template <bool LEAN>
__device__ __forceinline__ bool role_ok(bool ok) { return LEAN ? ok : warp_all(ok); }

template <int MODE, bool LEAN>
__device__ __forceinline__ void mma_issuer(const KernelParams& p, Barriers* sh, const TileIter& first, uint32_t tmem_base,
                                           uint8_t* act_smem, int act_stage_bytes) {
  constexpr bool RMS = MODE == kRms;
  constexpr bool GROUPED = MODE == kGrouped;
  const uint32_t idesc = make_idesc(p.TN);
  const uint64_t bdesc0 = make_b_desc(smem_u32(act_smem));
  const uint32_t bdesc_step = (uint32_t)(act_stage_bytes >> 4);
  int s = 0, a = 0, d = 0;
  uint32_t ph = 0, ph_d = 0;
  bool d_wrapped = false, ok = true;
  for (TileIter c = first; c.valid(p) && ok; c.next(p)) {
    if (d_wrapped && !(ok = role_ok<LEAN>(mbar_wait(&sh->d_empty[d], ph_d ^ 1u, &sh->abort_flag, p.status, 3)))) break;
    tc_fence_after();
    const uint32_t d_tmem = tmem_base + (uint32_t)(d * p.d_stride);
    uint32_t accumulate = 0;
    if (RMS && c.ks == 0) {
      // the split product first, into its own accumulator
      const uint32_t ds_tmem = d_tmem + (uint32_t)p.side_col;
      for (int sb = 0; sb < p.side_kb; ++sb) {
        if (!(ok = role_ok<LEAN>(mbar_wait(&sh->full[s], ph, &sh->abort_flag, p.status, 4)))) break;
        tc_fence_after();
        const uint64_t bdesc = bdesc0 + (uint64_t)((uint32_t)s * bdesc_step);
        const uint32_t a_tmem = tmem_base + (uint32_t)(p.a_base + a * 32);
        if (LEAN || elect_one()) {
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            mma_i8_ts(ds_tmem, a_tmem + k4 * 8, bdesc + (uint64_t)(k4 * 2), idesc, (accumulate | (uint32_t)k4));
          tc_commit(&sh->done[s]);
        }
        accumulate = 1;
        if (++s == p.stages) { s = 0; ph ^= 1u; }
        if (++a == p.num_a) a = 0;
      }
      if (!ok) break;
      accumulate = 0;
    }
    if (GROUPED) {
      // group-wise weight scales: every K block (= one group of 128 input channels) gets a fresh
      // accumulator, alternating between the two buffers; the epilogue warps fold it into their float
      // sums while the next block's MMAs run.  (The tile's first buffer wait happened above.)
      bool first_block = true;
      for (int kb = c.kb0(p), kb_end = c.kb1(p); kb < kb_end; ++kb) {
        if (!first_block && d_wrapped &&
            !(ok = role_ok<LEAN>(mbar_wait(&sh->d_empty[d], ph_d ^ 1u, &sh->abort_flag, p.status, 3)))) break;
        first_block = false;
        if (!(ok = role_ok<LEAN>(mbar_wait(&sh->full[s], ph, &sh->abort_flag, p.status, 4)))) break;
        tc_fence_after();
        const uint64_t bdesc = bdesc0 + (uint64_t)((uint32_t)s * bdesc_step);
        const uint32_t a_tmem = tmem_base + (uint32_t)(p.a_base + a * 32);
        const uint32_t dg_tmem = tmem_base + (uint32_t)(d * p.d_stride);
        if (LEAN || elect_one()) {
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            mma_i8_ts(dg_tmem, a_tmem + k4 * 8, bdesc + (uint64_t)(k4 * 2), idesc, (uint32_t)k4);
          tc_commit(&sh->done[s]);
          tc_commit(&sh->d_full[d]);
        }
        if (++s == p.stages) { s = 0; ph ^= 1u; }
        if (++a == p.num_a) a = 0;
        if (++d == p.num_d) { d = 0; ph_d ^= 1u; d_wrapped = true; }
      }
      continue;
    }
    for (int kb = c.kb0(p), kb_end = c.kb1(p); kb < kb_end; ++kb) {
      if (!(ok = role_ok<LEAN>(mbar_wait(&sh->full[s], ph, &sh->abort_flag, p.status, 4)))) break;
      tc_fence_after();
      const uint64_t bdesc = bdesc0 + (uint64_t)((uint32_t)s * bdesc_step);
      const uint32_t a_tmem = tmem_base + (uint32_t)(p.a_base + a * 32);
      if (LEAN || elect_one()) {
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4)
          mma_i8_ts(d_tmem, a_tmem + k4 * 8, bdesc + (uint64_t)(k4 * 2), idesc, (accumulate | (uint32_t)k4));
        tc_commit(&sh->done[s]);
      }
      accumulate = 1;
      if (++s == p.stages) { s = 0; ph ^= 1u; }
      if (++a == p.num_a) a = 0;
    }
    if (ok && (LEAN || elect_one())) tc_commit(&sh->d_full[d]);  // the thread that issued the MMAs
    if (++d == p.num_d) { d = 0; ph_d ^= 1u; d_wrapped = true; }
  }
  if (!ok && (LEAN || (threadIdx.x & 31) == 0)) {  // let every MMA already issued finish before tensor memory is freed
    tc_commit(&sh->drain);
    mbar_wait_drain(&sh->drain, 0, 2000000ull);
  }
}

// ------------------------------------------------------------------------------ the kernel
// MODE = kRms is the instantiation behind the rotation-magnitude-suppression linear: every tile
// (of K split 0) first runs the split product -- p.side_kb K blocks whose activations come
// through tmap_side and whose weights come from p.side_layout -- into a second accumulator,
// then the main product, and the epilogue combines the two.  The K blocks of both products
// go through the same rings; only the sources and the MMA's destination differ.  A separate
// instantiation keeps the ordinary kernel's code and register allocation as they were.
template <int MODE>
__global__ void __launch_bounds__(kMaxThreads, 1)
w4a8_gemm_kernel(const __grid_constant__ CUtensorMap tmap_act, const __grid_constant__ CUtensorMap tmap_side,
                 const KernelParams p) {
  constexpr bool RMS = MODE == kRms;
  constexpr bool GROUPED = MODE == kGrouped;
  constexpr bool W8 = MODE == kW8;
  constexpr int kTileBytes = W8 ? 2 * kWTileBytes : kWTileBytes;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // carve: activation stages (1024-aligned), weight stages, barriers, token scales
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int act_stage_bytes = p.TN * kBlockK;
  uint8_t* act_smem = smem;
  uint8_t* w_smem = act_smem + (size_t)p.stages * act_stage_bytes;
  Barriers* sh = reinterpret_cast<Barriers*>(w_smem + (size_t)p.w_stages * kTileBytes);
  float* s_tok = reinterpret_cast<float*>(sh + 1);  // [4 epilogue warps][256], then bf16 staging [4][16 x 32]

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  TileIter first;
  first.init(p, blockIdx.x);  // the divisions overlap with barrier set-up and the TMEM allocation

  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_act)) : "memory");
    for (int i = 0; i < p.stages; ++i) { mbar_init(&sh->full[i], 1 + 4); mbar_init(&sh->done[i], 1); }
    for (int i = 0; i < p.w_stages; ++i) { mbar_init(&sh->w_full[i], 1); mbar_init(&sh->w_empty[i], 4); }
    // every epilogue warp arrives on d_empty: four of them, eight in the group-scale instantiation
    for (int i = 0; i < 2; ++i) { mbar_init(&sh->d_full[i], 1); mbar_init(&sh->d_empty[i], GROUPED ? 8 : 4); }
    mbar_init(&sh->drain, 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {
    tmem_alloc(&sh->tmem_base, 512);
    tmem_relinquish();
  }
  pdl_launch_dependents();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&sh->tmem_base);
  // everything above touched only this CTA's shared and tensor memory; from here on the
  // roles read what the preceding kernel wrote (the int8 codes, the segment table)
  pdl_wait();

  // Ring positions are kept as (stage, phase) pairs that advance by increment-and-wrap: the
  // issuing roles are latency-bound, and an integer division per K block would cost more
  // cycles than the MMAs of that block.  For the same reason the MMA warp waits on ONE
  // barrier and signals ONE per K block, and runs converged with a single lane issuing.
  if (warp == 0) {
    // ---------------- activation TMA producer
    if (lane == 0) {
      int it = 0, s = 0;
      uint32_t ph = 0;
      bool wrapped = false, ok = true;
      for (TileIter c = first; c.valid(p) && ok; c.next(p)) {
        const int row0 = c.tt * p.TN;
        if (RMS && c.ks == 0) {
          for (int sb = 0; sb < p.side_kb; ++sb, ++it) {
            if (wrapped && !(ok = mbar_wait(&sh->done[s], ph ^ 1u, &sh->abort_flag, p.status, 1))) break;
            mbar_arrive_expect_tx(&sh->full[s], act_stage_bytes);
            tma_load_2d(act_smem + (size_t)s * act_stage_bytes, &tmap_side, sb * kBlockK, row0, &sh->full[s]);
            if (++s == p.stages) { s = 0; ph ^= 1u; wrapped = true; }
          }
          if (!ok) break;
        }
        for (int kb = c.kb0(p), kb_end = c.kb1(p); kb < kb_end; ++kb, ++it) {
          if (wrapped && !(ok = mbar_wait(&sh->done[s], ph ^ 1u, &sh->abort_flag, p.status, 1))) break;
          mbar_arrive_expect_tx(&sh->full[s], act_stage_bytes);
          tma_load_2d(act_smem + (size_t)s * act_stage_bytes, &tmap_act, kb * kBlockK, row0, &sh->full[s]);
          if (++s == p.stages) { s = 0; ph ^= 1u; wrapped = true; }
        }
      }
      if (!ok) {
        // drain: the copies still landing in our shared memory complete their transaction
        // bytes on `full`, whose phase may never complete once the expanders have stopped;
        // the bounded wait below gives them time to land before the CTA exits.
        for (int back = 1; back <= p.stages && back <= it; ++back) {
          const int j = it - back;
          mbar_wait_drain(&sh->full[j % p.stages], (j / p.stages) & 1, 20000ull);
        }
      }
    }
  } else if (warp == 3) {
    // ---------------- packed-weight bulk-copy producer
    if (lane == 0) {
      int it = 0, s = 0;
      uint32_t ph = 0;
      bool wrapped = false, ok = true;
      for (TileIter c = first; c.valid(p) && ok; c.next(p)) {
        if (RMS && c.ks == 0) {
          const uint8_t* ssrc = p.side_layout + (size_t)c.tn * p.side_kb * kWTileBytes;
          for (int sb = 0; sb < p.side_kb; ++sb, ++it, ssrc += kWTileBytes) {
            if (wrapped && !(ok = mbar_wait(&sh->w_empty[s], ph ^ 1u, &sh->abort_flag, p.status, 2))) break;
            mbar_arrive_expect_tx(&sh->w_full[s], kWTileBytes);
            bulk_load_1d(w_smem + (size_t)s * kWTileBytes, ssrc, kWTileBytes, &sh->w_full[s]);
            if (++s == p.w_stages) { s = 0; ph ^= 1u; wrapped = true; }
          }
          if (!ok) break;
        }
        const uint8_t* wsrc = p.W_layout + ((size_t)c.tn * p.kb_total + c.kb0(p)) * kTileBytes;
        for (int kb = c.kb0(p), kb_end = c.kb1(p); kb < kb_end; ++kb, ++it, wsrc += kTileBytes) {
          if (wrapped && !(ok = mbar_wait(&sh->w_empty[s], ph ^ 1u, &sh->abort_flag, p.status, 2))) break;
          mbar_arrive_expect_tx(&sh->w_full[s], kTileBytes);
          bulk_load_1d(w_smem + (size_t)s * kTileBytes, wsrc, kTileBytes, &sh->w_full[s]);
          if (++s == p.w_stages) { s = 0; ph ^= 1u; wrapped = true; }
        }
      }
      if (!ok) {
        for (int back = 1; back <= p.w_stages && back <= it; ++back) {
          const int j = it - back;
          mbar_wait_drain(&sh->w_full[j % p.w_stages], (j / p.w_stages) & 1, 20000ull);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (see mma_issuer above)
    if (p.lean_issue) {
      if (elect_one()) mma_issuer<MODE, true>(p, sh, first, tmem_base, act_smem, act_stage_bytes);
      __syncwarp();
    } else {
      mma_issuer<MODE, false>(p, sh, first, tmem_base, act_smem, act_stage_bytes);
    }
  } else if (warp >= 4 && warp < 4 + 4 * p.groups) {
    // ---------------- weight expanders: packed int4 (smem) -> int8 x16 (tensor memory)
    // Group g of four warps takes the K blocks g, g + groups, g + 2 groups, ... of this CTA's
    // stream, so the latency of one block's chain (wait, load, expand, tcgen05.st, wait::st)
    // overlaps with the other groups' blocks.  Needs groups <= w_stages and groups <= num_a
    // <= stages.  Block `it` uses weight slot it % num_a, free once the MMAs of block
    // it - num_a are done, i.e. once done[(it - num_a) % stages] has completed that round.
    const int q = warp & 3;
    const int grp = (warp - 4) >> 2;
    const int r = q * 32 + lane;  // channel row inside the tile == tensor-memory lane
    int total_it = 0;
    for (TileIter c = first; c.valid(p); c.next(p))
      total_it += c.kb1(p) - c.kb0(p) + ((RMS && c.ks == 0) ? p.side_kb : 0);
    int sw = grp, a = grp, s = grp;
    uint32_t ph_w = 0, ph = 0;
    bool ok = true;
    for (int it = grp; it < total_it && ok; it += p.groups) {
      if (!(ok = warp_all(mbar_wait(&sh->w_full[sw], ph_w, &sh->abort_flag, p.status, 6)))) break;
      const uint4* src = reinterpret_cast<const uint4*>(w_smem + (size_t)sw * kTileBytes) + r;
      uint32_t regs[32];
      if (W8) {
        // 8-bit weights: the tile already holds int8 codes, 16-byte piece (c, r) = codes k = 16 c .. + 15 of
        // channel r; they go to tensor memory as they are
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8) {
          const uint4 w = src[c8 * 128];
          regs[c8 * 4] = w.x; regs[c8 * 4 + 1] = w.y; regs[c8 * 4 + 2] = w.z; regs[c8 * 4 + 3] = w.w;
        }
      } else {
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const uint4 w = src[jj * 128];
          const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            regs[jj * 8 + 2 * i] = (ww[i] << 4) & 0xF0F0F0F0u;   // codes k0..k0+3, each x16
            regs[jj * 8 + 2 * i + 1] = ww[i] & 0xF0F0F0F0u;      // codes k0+4..k0+7, each x16
          }
        }
      }
      const uint32_t dep = __shfl_xor_sync(0xffffffffu, regs[1] ^ regs[9] ^ regs[17] ^ regs[25], 1);  // all lanes' loads done
      __syncwarp();
      if (lane == 0) mbar_arrive_after(&sh->w_empty[sw], dep);
      if (it >= p.num_a) {
        // stage and parity of block it - num_a, derived from those of block it
        const int fs = s >= p.num_a ? s - p.num_a : s - p.num_a + p.stages;
        const uint32_t fph = s >= p.num_a ? ph : ph ^ 1u;
        if (!(ok = warp_all(mbar_wait(&sh->done[fs], fph, &sh->abort_flag, p.status, 7)))) break;
      }
      tc_fence_after();
      tmem_st_x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(p.a_base + a * 32), regs);
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->full[s]);
      sw += p.groups;
      if (sw >= p.w_stages) { sw -= p.w_stages; ph_w ^= 1u; }
      s += p.groups;
      if (s >= p.stages) { s -= p.stages; ph ^= 1u; }
      a += p.groups;
      if (a >= p.num_a) a -= p.num_a;
    }
  } else if (warp >= 4 + 4 * p.groups) {
    // ---------------- epilogue: tensor memory -> dequant -> global
    const int q = warp & 3;
    float* stok = s_tok + q * 256;  // private to this warp: no cross-warp barrier to strand on abort
    __nv_bfloat16* stage = reinterpret_cast<__nv_bfloat16*>(s_tok + 4 * 256) + q * (16 * 32);
    // bf16 rows whose pitch keeps 16-byte stores aligned take the staged path
    const bool plain = !p.acc_out && !p.y_is_f32 && (p.ldy % 8) == 0;
    const int epi_mode = p.ksplit > 1 ? kEpiSplitK : (plain ? (kEpiStaged | (p.bias ? kEpiBias : 0)) : kEpiGeneric);
    int d = 0;
    uint32_t ph_d = 0;
    bool ok = true;
    if (GROUPED) {
      // ---- group-wise weight scales (App. A.12: g = 128 = one K block).  s_w is [K / 128][N].  Per tile the
      // lane that owns channel n keeps one float sum per token column (TN <= 64) and, after every K block,
      // adds  fl(float(acc_g) * fl(s_a * s_w[g][n]))  in increasing g -- the order the result is defined in.
      // Eight warps fold (one expander group only): warp (q, half) owns lane quarter q and the token columns
      // 32 half .. 32 half + 31 of the tile.  A single warp issues well below one instruction per cycle, so
      // two per scheduler roughly double the fold rate.
      const int half = (warp - (4 + 4 * p.groups)) >> 2;
      if (half == 1) stage = reinterpret_cast<__nv_bfloat16*>(s_tok) + q * (16 * 32);  // the token-scale table is unused here
      const bool plain_out = !p.acc_out && !p.y_is_f32 && (p.ldy % 8) == 0;
      for (TileIter c = first; c.valid(p) && ok; c.next(p)) {
        const int t0 = c.tt * p.TN;
        const int ncols = min(p.TN, p.T - t0);
        const int n = c.tn * kTileN + q * 32 + lane;
        const bool n_ok = n < p.N;
        // which token columns of the tile are visual rows: bit j of `vis`
        const int ta = t0 + lane, tb = t0 + 32 + lane;
        const unsigned lo = __ballot_sync(0xffffffffu, ta < p.T && thread_row_modality(p.seg, ta) == MQ_VISUAL);
        const unsigned hi = __ballot_sync(0xffffffffu, tb < p.T && thread_row_modality(p.seg, tb) == MQ_VISUAL);
        float sum[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) sum[j] = 0.0f;
        const unsigned vis_h = half ? hi : lo;                 // this warp's 32 columns
        const int ncols_h = max(0, min(32, ncols - half * 32));
        const unsigned in_h = ncols_h >= 32 ? 0xffffffffu : ((1u << ncols_h) - 1u);
        const bool uniform_mod = vis_h == 0u || vis_h == in_h;  // (rows past T count as text: no bit there)
        const float* swg = p.s_w + n;
        float sw_next = n_ok ? swg[(size_t)c.kb0(p) * p.N] : 0.0f;
        for (int kb = c.kb0(p), kb_end = c.kb1(p); kb < kb_end && ok; ++kb) {
          const float swv = sw_next;
          if (kb + 1 < kb_end) sw_next = n_ok ? swg[(size_t)(kb + 1) * p.N] : 0.0f;  // in flight during this block
          const float cv = __fmul_rn(p.s_vis, swv), ct = __fmul_rn(p.s_txt, swv);
          if (!(ok = warp_all(mbar_wait(&sh->d_full[d], ph_d, &sh->abort_flag, p.status, 8)))) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(d * p.d_stride + half * 32);
          uint32_t v0[16], v1[16];
          if (ncols_h > 0) {  // warp-uniform
            tmem_ld_x16(d_tmem, v0);
            tmem_ld_x16(d_tmem + 16, v1);
            tmem_wait_ld();
          }
          // the accumulator has been read (or is not this warp's to read): hand it back to the MMA warp
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh->d_empty[d]);
          if (ncols_h > 0) {
            if (p.acc_out && n_ok) {  // debug dump of this group's accumulators
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                if (j < ncols_h)
                  p.acc_out[((size_t)kb * p.T + t0 + half * 32 + j) * p.N + n] = ((int)(j < 16 ? v0[j] : v1[j - 16])) >> 4;
              }
            }
            // The MMA saw 16 * q_w: float(16 a) * (c / 16) == float(a) * c bit for bit (powers of two), which
            // saves the shift; a tile within one modality (the usual case after AIFS) also skips the select.
            const float cv16 = __fmul_rn(cv, 0.0625f), ct16 = __fmul_rn(ct, 0.0625f);
            if (uniform_mod) {
              const float cs = vis_h ? cv16 : ct16;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                sum[j] = __fadd_rn(sum[j], __fmul_rn((float)(int)(j < 16 ? v0[j] : v1[j - 16]), cs));
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const float cs = ((vis_h >> j) & 1u) ? cv16 : ct16;
                sum[j] = __fadd_rn(sum[j], __fmul_rn((float)(int)(j < 16 ? v0[j] : v1[j - 16]), cs));
              }
            }
          }
          if (++d == p.num_d) { d = 0; ph_d ^= 1u; }
        }
        if (!ok) break;
        const float bs = (n_ok && p.bias) ? p.bias[n] : 0.0f;
#pragma unroll
        for (int cc = 0; cc < 32; cc += 16) {
          if (cc < ncols_h) {  // warp-uniform
            float y[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) y[j] = p.bias ? __fadd_rn(sum[cc + j], bs) : sum[cc + j];
            const int nvalid = min(16, ncols_h - cc);
            const int tc0 = t0 + half * 32 + cc;
            if (plain_out) {
              staged_store(p, y, tc0, nvalid, n, stage);
            } else if (n_ok) {
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                if (j < nvalid) {
                  const size_t t = (size_t)(tc0 + j);
                  if (p.y_is_f32) static_cast<float*>(p.Y)[t * p.ldy + n] = y[j];
                  else static_cast<__nv_bfloat16*>(p.Y)[t * p.ldy + n] = __float2bfloat16_rn(y[j]);
                }
              }
            }
          }
        }
      }
    }
    for (TileIter c = first; !GROUPED && c.valid(p) && ok; c.next(p)) {
      const int t0 = c.tt * p.TN;
      __syncwarp();
      for (int j = lane; j < p.TN; j += 32) {
        const int t = t0 + j;
        if (p.row_scales) stok[j] = t < p.T ? p.row_scales[t] : 0.0f;
        else stok[j] = (t < p.T && thread_row_modality(p.seg, t) == MQ_VISUAL) ? p.s_vis : p.s_txt;
      }
      __syncwarp();
      if (!(ok = warp_all(mbar_wait(&sh->d_full[d], ph_d, &sh->abort_flag, p.status, 8)))) break;
      tc_fence_after();
      const int n = c.tn * kTileN + q * 32 + lane;
      const bool n_ok = n < p.N;
      const float sw = n_ok ? p.s_w[n] : 0.0f;
      const float bs = (n_ok && p.bias) ? p.bias[n] : 0.0f;
      const uint32_t d_tmem = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(d * p.d_stride);
      if (RMS) {
        if (p.ksplit > 1) {
          epilogue_tile<kEpiSplitK>(p, d_tmem, t0, n, n_ok, sw, bs, stok, stage, c.ks);
          if (c.ks == 0) epilogue_tile_side_slice(p, d_tmem, t0, n, n_ok);
        } else {
          const float sws = n_ok ? p.s_w_side[n] : 0.0f;
          if (plain && !p.acc_side_out) epilogue_tile_side<true>(p, d_tmem, t0, n, n_ok, sw, sws, bs, stok, stage);
          else epilogue_tile_side<false>(p, d_tmem, t0, n, n_ok, sw, sws, bs, stok, stage);
        }
      } else {
        constexpr int X = W8 ? kEpiNoShift : 0;
        switch (epi_mode) {
#define MQ_EPI_CASE(M) case M: epilogue_tile<(M) | X>(p, d_tmem, t0, n, n_ok, sw, bs, stok, stage, c.ks); break;
          MQ_EPI_CASE(kEpiStaged) MQ_EPI_CASE(kEpiStaged | kEpiBias) MQ_EPI_CASE(kEpiSplitK)
#undef MQ_EPI_CASE
          default: epilogue_tile<kEpiGeneric | X>(p, d_tmem, t0, n, n_ok, sw, bs, stok, stage, c.ks); break;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->d_empty[d]);
      if (++d == p.num_d) { d = 0; ph_d ^= 1u; }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}


// Split-K finalize: exact int32 partial sums -> dequantized output.
// side_acc (optional): the split accumulator of the rotation-magnitude-suppression linear with
// its own weight scale s_w_side; its term is added before the bias.
__global__ void splitk_finalize_kernel(const int32_t* __restrict__ acc, int ksplit, int T, int N, SegTable seg, float s_vis,
                                       float s_txt, const float* __restrict__ s_w, const float* __restrict__ bias,
                                       void* Y, int64_t ldy, int y_is_f32, int32_t* __restrict__ acc_out,
                                       const int32_t* __restrict__ side_acc, const float* __restrict__ s_w_side,
                                       int32_t* __restrict__ acc_side_out, const float* __restrict__ row_scales) {
  pdl_launch_dependents();
  pdl_wait();
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)T * N) return;
  const int t = (int)(idx / N), n = (int)(idx % N);
  int a = 0;
  for (int ks = 0; ks < ksplit; ++ks) a += acc[(size_t)ks * T * N + idx];  // one slice per K split
  if (acc_out) acc_out[idx] = a;
  const float st = row_scales ? row_scales[t] : (thread_row_modality(seg, t) == MQ_VISUAL ? s_vis : s_txt);
  float y = __fmul_rn((float)a, __fmul_rn(st, s_w[n]));
  if (side_acc) {
    const int sa = side_acc[idx];
    if (acc_side_out) acc_side_out[idx] = sa;
    y = __fadd_rn(y, __fmul_rn((float)sa, __fmul_rn(st, s_w_side[n])));
  }
  if (bias) y = __fadd_rn(y, bias[n]);
  const size_t oy = (size_t)t * ldy + n;
  if (y_is_f32) static_cast<float*>(Y)[oy] = y;
  else static_cast<__nv_bfloat16*>(Y)[oy] = __float2bfloat16_rn(y);
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

struct Plan {
  int TN, n_tt, n_tn, ksplit, num_d, d_stride, a_base, num_a, stages, w_stages, grid, groups;
  size_t smem;
};

// rms: the launch carries a split accumulator next to every accumulator (rotation magnitude
// suppression), so a token tile may use at most 224 of the 512 tensor-memory columns twice over,
// there is a single accumulator pair, and what is left (>= 64 columns) holds the weight slots.
Plan make_plan(int T, int K, int N, int mode = kPlain) {
  Plan pl{};
  const bool rms = mode == kRms, grouped = mode == kGrouped;
  const int wtile = mode == kW8 ? 2 * kWTileBytes : kWTileBytes;
  const int sms = sm_count();
  pl.n_tn = (N + kTileN - 1) / kTileN;
  const int kb_total = (K + kBlockK - 1) / kBlockK;
  // Token tile.  Candidates: T cut into n_tt even tiles (multiple of 16, at most tn_cap tokens).
  // Each is rated with a small model of the kernel: a CTA runs `rounds` tiles one after the
  // other; the period of a K block in this kernel was found flat up to 192 tokens and growing beyond
  // (112 cycles per MMA slot up to 192 tokens, 120 at 224, 136 at 256: an empirical figure of the whole
  // pipeline -- the MMA alone takes 10 + N / 2 cycles); the epilogue (~25 cycles per token column)
  // hides behind the next tile's main loop only when two accumulators fit (tiles of <= 192 tokens).
  // The cheapest candidate wins; ties go to the larger tile.
  // Group-wise weight scales: the epilogue keeps one float sum per token column in registers, so the
  // tile is at most 64 tokens; its accumulators alternate per K block.
  const int tn_cap = grouped ? 64 : (rms ? 224 : 256);
  int n_tt = (T + tn_cap - 1) / tn_cap;
  int TN = (((T + n_tt - 1) / n_tt) + 15) / 16 * 16;
  // A token tile of 176 is never planned.  Forced onto long runs (20 to 45 tiles per CTA) that width ended in
  // a launch failure or an expired wait on three of nine shapes, while every other width from 16 to 256 ran
  // clean on the same shapes; reading the code and a randomised simulation of the barrier protocol with its
  // ring depths (8 activation stages, 5 weight stages, 4 weight slots) found no cause.  Until one is found
  // the width is left out: 192 takes its place here (at most three tiles, so none is empty) and the search
  // below skips it.
  constexpr int kUnusedTN = 176;
  if (TN == kUnusedTN) TN = 192;
  // The search runs when a CTA gets several tiles, and when every CTA gets one tile of more than
  // 192 tokens although smaller tiles would still fit the machine in one round (their MMAs are
  // cheaper); otherwise the fewest tiles are right.
  const bool multi_round = (long long)pl.n_tn * n_tt > sms;
  if (!grouped && (multi_round || TN > 192)) {
    double best = 0.0;
    const int n_min = n_tt;
    for (int cand = n_min; cand <= n_min * 4 && cand <= (T + 15) / 16; ++cand) {
      int tn = (((T + cand - 1) / cand) + 15) / 16 * 16;
      if (tn == kUnusedTN) {
        if (cand != n_min) continue;
        tn = 192;  // the fewest tiles: as above
      }
      const long long tiles_c = (long long)pl.n_tn * cand;
      if (!multi_round && tiles_c > sms) break;  // stay within one round
      const long long rounds = (tiles_c + sms - 1) / sms;
      const double mma = tn <= 192 ? 112.0 : (tn <= 224 ? 112.0 + (tn - 192) * 0.25 : 120.0 + (tn - 224) * 0.5);
      const double epi = 25.0 * tn;
      // two accumulators: always up to 192 tokens; up to 224 tokens (448 columns, which leaves two
      // weight slots) when a CTA runs several tiles and the hidden epilogue is worth the shallower ring
      const bool two_acc = !rms && (tn <= 192 || (tn <= 224 && rounds > 1));
      const double main_loop = 4.0 * mma * kb_total;
      const double est = two_acc ? rounds * main_loop + epi : rounds * (main_loop + epi);
      if (cand == n_min || est < best * 0.995) {
        best = est;
        n_tt = cand;
        TN = tn;
      }
    }
  }
  pl.TN = TN;
  pl.n_tt = n_tt;
  const bool several_tiles = (long long)pl.n_tn * n_tt > sms;
  pl.d_stride = TN <= 128 ? 128 : (TN <= 192 ? 192 : ((TN <= 224 && several_tiles) ? 224 : 256));
  pl.num_d = pl.d_stride <= 224 ? 2 : 1;
  pl.a_base = pl.num_d * pl.d_stride;
  if (rms) {
    pl.d_stride = (TN + 31) / 32 * 32;  // here: columns from the accumulator to its split accumulator
    pl.num_d = 1;
    pl.a_base = 2 * pl.d_stride;
  }
  if (grouped) {
    pl.d_stride = 64;
    pl.num_d = 2;
    pl.a_base = 128;
  }
  pl.num_a = (512 - pl.a_base) / 32;
  if (pl.num_a > kMaxStages) pl.num_a = kMaxStages;
  // split K when the tiles alone cannot fill the machine (small T: weight streaming)
  const long long tiles = (long long)pl.n_tn * n_tt;
  int ksplit = 1;
  if (!grouped && tiles * 2 <= sms) {  // (group sums are added in K order: no K split)
    ksplit = (int)(sms / tiles);
    const int max_split = kb_total / 4 > 0 ? kb_total / 4 : 1;  // keep >= 4 K blocks per CTA
    if (ksplit > max_split) ksplit = max_split;
    if (ksplit < 1) ksplit = 1;
    const int per = (kb_total + ksplit - 1) / ksplit;
    ksplit = (kb_total + per - 1) / per;  // no empty split
    // Splitting pays only while the partial sums are small: each split writes a [T,N] int32 slice
    // that the finalize kernel reads back (about 4 TB/s for the pair), and that kernel costs
    // about 3 us on top.  Against it stands the main loop, whose K blocks follow one another every ~450
    // cycles (the pipeline's measured period for small token tiles) at ~1.9 GHz.  (Decode shapes split; a
    // prefill-sized T with few output channels does not.)
    const double loop_us = kb_total * 4.0 * 112.0 / 1900.0;
    const double slices_us = (ksplit + 0.5) * (double)T * N * 4.0 * 2.0 / 4.0e6 + 3.0;
    if (loop_us / ksplit + slices_us >= loop_us) ksplit = 1;
  }
  pl.ksplit = ksplit;
  // shared memory: as many activation stages as fit beside a minimum of 4 weight stages, then
  // the rest to the weight ring
  const int act_stage = TN * kBlockK;
  const size_t fixed = 1024 + sizeof(Barriers) + 4 * 256 * sizeof(float) + 4 * 16 * 32 * 2;
  int stages = (int)((kSmemBudget - fixed - 4 * (size_t)wtile) / act_stage);
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < pl.num_a) pl.num_a = stages;
  int w_stages = (int)((kSmemBudget - fixed - (size_t)stages * act_stage) / wtile);
  if (w_stages > kMaxWStages) w_stages = kMaxWStages;
  pl.stages = stages;
  pl.w_stages = w_stages;
  pl.smem = fixed + (size_t)stages * act_stage + (size_t)w_stages * wtile;
  pl.groups = grouped ? 1 : 2;  // group scales: the second expander group's warps fold accumulators instead
  if (pl.groups > pl.num_a) pl.groups = pl.num_a;
  if (pl.groups > pl.w_stages) pl.groups = pl.w_stages;
  if (pl.groups < 1) pl.groups = 1;
  const long long total = tiles * ksplit;
  pl.grid = (int)(total < sms ? total : sms);
  return pl;
}

}  // namespace

static int mode_of(bool rms, int group_size, int w_bits) {
  return rms ? kRms : (group_size ? kGrouped : (w_bits == 8 ? kW8 : kPlain));
}

size_t gemm_splitk_bytes(int T, int K, int N, bool rms, int group_size, int w_bits) {
  if (T <= 0 || K <= 0 || N <= 0) return 0;
  const int mode = mode_of(rms, group_size, w_bits);
  if (mode == kPlain && gemv_applies(T, K, N)) return 0;  // the GEMV path reduces inside its CTAs
  const Plan pl = make_plan(T, K, N, mode);
  // one [T,N] slice per K split, and one more for the split accumulator
  return pl.ksplit > 1 ? (size_t)(pl.ksplit + (rms ? 1 : 0)) * T * N * sizeof(int32_t) : 0;
}

int launch_gemm(const GemmArgs& a, cudaStream_t st) {
  if (a.T == 0 || a.N == 0) return MQ_OK;
  const bool rms = a.side_layout != nullptr;
  const int mode = mode_of(rms, a.group_size, a.w_bits);
  if (rms && (a.group_size || a.w_bits == 8)) return MQ_ERR_UNSUPPORTED;
  if (a.group_size && (a.group_size != kBlockK || a.K % kBlockK || a.row_scales || a.w_bits == 8)) return MQ_ERR_UNSUPPORTED;
  if (mode == kPlain && gemv_applies(a.T, a.K, a.N)) return launch_gemv(a, st);  // one to three tokens: see mq_gemv.cu
  const Plan pl = make_plan(a.T, a.K, a.N, mode);
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return MQ_ERR_CUDA;

  CUtensorMap tmap;
  const cuuint64_t dims[2] = {(cuuint64_t)a.K, (cuuint64_t)a.T};
  const cuuint64_t strides[1] = {(cuuint64_t)a.ldq};
  const cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)pl.TN};
  const cuuint32_t estr[2] = {1, 1};
  if (encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(a.Qx), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return MQ_ERR_CUDA;

  // the split product's activation codes [T, side_k] (the ordinary launch passes the main map twice)
  CUtensorMap tmap_side = tmap;
  if (rms) {
    // columns past side_cols are out of bounds for the map and arrive as zeros
    const cuuint64_t sdims[2] = {(cuuint64_t)a.side_cols, (cuuint64_t)a.T};
    const cuuint64_t sstrides[1] = {(cuuint64_t)a.side_k};
    if (encode(&tmap_side, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(a.Qs), sdims, sstrides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return MQ_ERR_CUDA;
  }

  auto kernel = mode == kRms ? w4a8_gemm_kernel<kRms>
                             : (mode == kGrouped ? w4a8_gemm_kernel<kGrouped>
                                                 : (mode == kW8 ? w4a8_gemm_kernel<kW8> : w4a8_gemm_kernel<kPlain>));
  static PerDeviceTable<char> attr_set[4];
  if (!ensure_dynamic_smem(attr_set[mode], kernel, kSmemBudget)) return MQ_ERR_CUDA;

  KernelParams p{};
  p.T = a.T; p.K = a.K; p.N = a.N;
  p.TN = pl.TN; p.n_tn = pl.n_tn; p.n_tt = pl.n_tt; p.ksplit = pl.ksplit;
  p.kb_total = (a.K + kBlockK - 1) / kBlockK;
  p.kb_per_split = (p.kb_total + pl.ksplit - 1) / pl.ksplit;
  p.step_tn = pl.grid % pl.n_tn;
  p.step_tt = (pl.grid / pl.n_tn) % pl.n_tt;
  p.step_ks = (pl.grid / pl.n_tn) / pl.n_tt;
  p.num_d = pl.num_d; p.d_stride = pl.d_stride; p.a_base = pl.a_base; p.num_a = pl.num_a;
  p.stages = pl.stages; p.w_stages = pl.w_stages; p.groups = pl.groups;
  p.lean_issue = pl.num_a > 2 ? 1 : 0;
  p.seg = a.seg; p.s_vis = a.s_vis; p.s_txt = a.s_txt;
  p.W_layout = static_cast<const uint8_t*>(a.W_layout);
  p.s_w = a.s_w; p.bias = a.bias; p.Y = a.Y; p.ldy = a.ldy; p.y_is_f32 = a.y_is_f32;
  p.acc_out = a.acc_out; p.splitk_acc = a.splitk_acc; p.status = a.status; p.row_scales = a.row_scales;
  int32_t* side_slice = nullptr;
  if (rms) {
    p.side_kb = (a.side_k + kBlockK - 1) / kBlockK;
    p.side_col = pl.d_stride;
    p.side_layout = static_cast<const uint8_t*>(a.side_layout);
    p.s_w_side = a.s_w_side;
    p.acc_side_out = a.acc_side_out;
    if (pl.ksplit > 1 && a.splitk_acc) side_slice = a.splitk_acc + (size_t)pl.ksplit * a.T * a.N;
    p.splitk_side = side_slice;
  }

  if (pl.ksplit > 1 && !a.splitk_acc) return MQ_ERR_WORKSPACE;
  if (cuda_status(launch_pdl(kernel, dim3(pl.grid), dim3((4 + 4 * pl.groups + (mode == kGrouped ? 8 : 4)) * 32), pl.smem, st, tmap, tmap_side, p)) != MQ_OK)
    return MQ_ERR_CUDA;
  if (pl.ksplit > 1) {
    const int64_t n = (int64_t)a.T * a.N;
    if (launch_pdl(splitk_finalize_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st,
                   static_cast<const int32_t*>(a.splitk_acc), pl.ksplit, a.T, a.N, a.seg, a.s_vis, a.s_txt, a.s_w, a.bias, a.Y,
                   a.ldy, a.y_is_f32, a.acc_out, static_cast<const int32_t*>(side_slice), a.s_w_side,
                   a.acc_side_out, a.row_scales) != cudaSuccess) {
      (void)cudaGetLastError();
      return MQ_ERR_CUDA;
    }
  }
  return MQ_OK;
}

}  // namespace mq
