// Attention under the unified causal mask of AIFS (Sec. 3.1, Eq. 4 - Eq. 5), written for sm_100a.
//
// After AIFS the rows of a sequence stand in the order [visual (and pad) block][text block]; row i is the
// original token perm[i].  Row i may attend row j iff the original token of j does not come after that of
// i, perm[j] <= perm[i], and j is not a padded token (App. A.4); a padded row keeps its own diagonal so that
// its (discarded) softmax stays defined.  With that rule the output equals causal attention in the original
// order, which is what makes the reordering free (Eq. 5; "numerically the same").
//
//   S = Q K^T / sqrt(D);  P = softmax over the allowed columns;  O = P V     per head, grouped-query heads
//
// One CTA per (128-row query tile, query head).  Both products run on the tensor cores (tcgen05.mma
// kind::f16 on bf16 operands from shared memory, float32 accumulators in tensor memory):
//   * Q, K tiles and V^T tiles arrive by TMA (128-byte swizzle).  V is transposed once per call by a small
//     prep kernel so that the second product's B operand is K-major like every other operand here;
//   * two groups of four softmax warps share every key tile: group 0 takes its keys 0 .. 63, group 1 its keys
//     64 .. 127.  Each group has two score buffers (128 x 64) and its own output accumulator in tensor memory
//     and runs a complete online softmax over its keys; the two partial results are merged at the end (as
//     for a split over the keys).  With two buffers a group's scores for the next tile are computed while
//     its softmax works on the current one;
//   * a softmax thread owns one query row: it reads its 64 scores from tensor memory once, applies the
//     mask, takes the maximum and writes P = exp2(...) as bf16 over the scores it has read, where the second
//     product takes it as its A operand: the probabilities never touch shared memory;
//   * O_g += P V accumulates in tensor memory.  The exponents are taken relative to a reference maximum
//     that may lag the true running maximum by up to 8 powers of two; only when a row outgrows it are the
//     accumulated output and sum rescaled, so the softmax warps normally never touch O until the end;
//   * key tiles no row of the query tile may see are skipped, and tiles every row may see in full skip the
//     mask: the prep kernel stores, per 128-row tile, the smallest and largest original index.
// Every wait on an mbarrier is bounded (see mq_sm100.cuh); an expired wait raises the CTA's abort flag, all
// roles leave their loops at the next tile, and the status word carries MQ_ERR_TIMEOUT and the site.
#include <cuda.h>
#include <cuda_bf16.h>

#include <climits>

#include "mq_common.cuh"
#include "mq_device_table.h"
#include "mq_sm100.cuh"

namespace mq {
namespace {

constexpr int kD = 128;           // head dimension
constexpr int kTile = 128;        // query rows per CTA, keys per step
constexpr int kHalfBytes = 64 * kTile * 2;   // one 128-row x 64-element swizzled block
constexpr int kTileBytes = 2 * kHalfBytes;   // a 128 x 128 bf16 operand tile
constexpr int kThreads = 12 * 32;            // producer, MMA issuer, allocator, spare, 8 softmax warps
constexpr int kSoftmaxThreads = 8 * 32;
constexpr int kMaxTiles = 1024;              // 128-row tiles per sequence (the CTA's tile list lives in shared memory)

constexpr int kStages = 2;                   // K tiles and V^T tiles in flight (each ring)

struct AttnBarriers {
  uint64_t q_full;
  uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  // per softmax group and score buffer ([2 g + b]): the scores are written (MMA commit); P has replaced them (the
  // group's four warps); the product of that P into the group's accumulator is complete (MMA commit)
  uint64_t s_full[4], p_full[4], pv_done[4];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
  int n_list;     // entries of the CTA's tile list
};

struct AttnParams {
  int L, n_tiles, n_q_heads, group;  // group = query heads per key/value head
  const int32_t* perm;
  const uint8_t* pad_u;
  const int32_t* kmin;    // per key tile: smallest original index among its attendable (in range, not padded) rows
  const int32_t* kmaxc;   // largest one if the tile is clean (all rows in range, none padded), else INT_MAX
  const int32_t* qmin;    // per query tile: smallest / largest original index over its rows in range
  const int32_t* qmax;
  __nv_bfloat16* O;
  int64_t ldo;
  float scale_log2;       // log2(e) / sqrt(D)
  int32_t* status;
};

// Classes of a key tile for a query tile: 0: no row of the query tile may attend any row of the key tile (it is
// skipped); 1: some may (masked); 2: all may attend all (no mask needed).

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float fast_rcp(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// ---------------------------------------------------------------------------------------- prep
// V [L, n_kv_heads * D] -> Vt [n_kv_heads * D, Lp] (keys contiguous, zero beyond L), and the per-tile bounds
// of the original indices.  Grid (key tiles, kv heads); the blocks of head 0 also write the bounds.
__global__ void __launch_bounds__(256)
attn_prep_kernel(const uint16_t* __restrict__ V, int64_t ldv, int L, int Lp, const int32_t* __restrict__ perm,
                 const uint8_t* __restrict__ pad_u, uint16_t* __restrict__ Vt, int32_t* __restrict__ kmin,
                 int32_t* __restrict__ kmaxc, int32_t* __restrict__ qmin, int32_t* __restrict__ qmax) {
  __shared__ uint16_t tile[kTile][kD + 8];
  __shared__ int red[4][4];
  const int kt = blockIdx.x, g = blockIdx.y, j0 = kt * kTile;
  for (int c = threadIdx.x; c < kTile * (kD / 8); c += 256) {
    const int row = c / (kD / 8), piece = c % (kD / 8);
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (j0 + row < L) v = *reinterpret_cast<const uint4*>(V + (size_t)(j0 + row) * ldv + (size_t)g * kD + piece * 8);
    *reinterpret_cast<uint4*>(&tile[row][piece * 8]) = v;
  }
  __syncthreads();
  for (int c = threadIdx.x; c < kD * (kTile / 8); c += 256) {
    const int d = c / (kTile / 8), piece = c % (kTile / 8);
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e)
      w[e] = (uint32_t)tile[piece * 8 + 2 * e][d] | ((uint32_t)tile[piece * 8 + 2 * e + 1][d] << 16);
    *reinterpret_cast<uint4*>(Vt + ((size_t)g * kD + d) * Lp + j0 + piece * 8) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  if (g != 0) return;
  int a_min = INT_MAX, a_max = -1, r_min = INT_MAX, r_max = -1, dirty = 0;
  if (threadIdx.x < kTile) {
    const int j = j0 + threadIdx.x;
    if (j < L) {
      const int pj = perm[j];
      r_min = r_max = pj;
      if (pad_u && pad_u[j]) dirty = 1;
      else a_min = a_max = pj;
    } else {
      dirty = 1;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    a_min = min(a_min, __shfl_xor_sync(0xffffffffu, a_min, o));
    a_max = max(a_max, __shfl_xor_sync(0xffffffffu, a_max, o));
    r_min = min(r_min, __shfl_xor_sync(0xffffffffu, r_min, o));
    r_max = max(r_max, __shfl_xor_sync(0xffffffffu, r_max, o));
    dirty |= __shfl_xor_sync(0xffffffffu, dirty, o);
  }
  const int warp = threadIdx.x >> 5;
  if (warp < 4 && (threadIdx.x & 31) == 0) {
    red[warp][0] = a_min; red[warp][1] = dirty ? INT_MAX : a_max; red[warp][2] = r_min; red[warp][3] = r_max;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    kmin[kt] = min(min(red[0][0], red[1][0]), min(red[2][0], red[3][0]));
    kmaxc[kt] = max(max(red[0][1], red[1][1]), max(red[2][1], red[3][1]));
    qmin[kt] = min(min(red[0][2], red[1][2]), min(red[2][2], red[3][2]));
    qmax[kt] = max(max(red[0][3], red[1][3]), max(red[2][3], red[3][3]));
  }
}

// ---------------------------------------------------------------------------------------- softmax pieces
// A softmax thread works on one query row and the 64 key columns of its group's half of a key tile.  Both
// 32-column loads of the scores are in flight together and the scores stay in registers for the maximum and
// the exponentials (one read of tensor memory per tile).
//
// Loads the 64 scores at s_addr, masks them (-inf where the row may not attend the key), returns the maximum.
template <bool MASKED>
__device__ __forceinline__ float scores_load_max(uint32_t s_addr, uint32_t allowed_lo, uint32_t allowed_hi, uint32_t (&sv)[64]) {
  tmem_ld_x32(s_addr, *reinterpret_cast<uint32_t (*)[32]>(&sv[0]));
  tmem_ld_x32(s_addr + 32u, *reinterpret_cast<uint32_t (*)[32]>(&sv[32]));
  tmem_wait_ld();
  // four independent partial maxima (one chain of dependent max operations would cost more than the exponentials)
  float mx[4] = {-1.0e30f, -1.0e30f, -1.0e30f, -1.0e30f};
#pragma unroll
  for (int e = 0; e < 64; ++e) {
    if (MASKED && !(((e < 32 ? allowed_lo : allowed_hi) >> (e & 31)) & 1u)) sv[e] = 0xff800000u;  // -inf: its exponential is 0
    mx[e & 3] = fmaxf(mx[e & 3], __uint_as_float(sv[e]));
  }
  return fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
}

// P = exp2(scale * (s - m_used)) of the 64 scores as 32 bf16 pairs over the first 32 columns of the score buffer
// (all of whose scores are in registers by now).  Returns the sum of the probabilities.
__device__ __forceinline__ float probs_store(uint32_t s_addr, const uint32_t (&sv)[64], float scale_log2, float m_used) {
  const float2 scale2 = make_float2(scale_log2, scale_log2);
  const float bias = -m_used * scale_log2;
  const float2 bias2 = make_float2(bias, bias);
  float2 sum2[2] = {make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f)};
  uint32_t pk[32];
#pragma unroll
  for (int e = 0; e < 64; e += 2) {
    const float2 x = __ffma2_rn(make_float2(__uint_as_float(sv[e]), __uint_as_float(sv[e + 1])), scale2, bias2);
    const float2 pr = make_float2(fast_exp2(x.x), fast_exp2(x.y));
    sum2[(e >> 1) & 1] = __fadd2_rn(sum2[(e >> 1) & 1], pr);
    pk[e >> 1] = pack_bf16x2(pr.x, pr.y);
  }
  tmem_st_x32(s_addr, pk);
  tmem_wait_st();
  return (sum2[0].x + sum2[0].y) + (sum2[1].x + sum2[1].y);
}

// Bit j of (lo, hi): may this thread's row attend key column j of its group's half tile (kp: the 64 keys'
// original indices, INT_MAX for padded or out-of-range keys; self_col: the diagonal column of a padded row, or -1).
__device__ __forceinline__ void allowed_bits(const int32_t* kp, int perm_i, int self_col, uint32_t& lo, uint32_t& hi) {
  lo = 0; hi = 0;
#pragma unroll 8
  for (int b = 0; b < 32; ++b) lo |= (uint32_t)(kp[b] <= perm_i) << b;
#pragma unroll 8
  for (int b = 0; b < 32; ++b) hi |= (uint32_t)(kp[32 + b] <= perm_i) << b;
  if (self_col >= 0) {
    if (self_col < 32) lo |= 1u << self_col;
    else hi |= 1u << (self_col - 32);
  }
}

// ---------------------------------------------------------------------------------------- the kernel
// Tensor-memory columns: group g (0: keys 0 .. 63 of every key tile, 1: keys 64 .. 127) has two score buffers of
// 64 columns at 128 g and 128 g + 64 -- the first 32 columns of a buffer are overwritten in place by P (bf16
// pairs) once its scores have been read -- and its output accumulator at 256 + 128 g.
constexpr uint32_t kColO = 256;
// The exponent's reference maximum may lag the true running maximum by this many powers of two before the
// accumulated output is rescaled (probabilities then reach at most 2^8, harmless in float32 / bf16).
constexpr float kLagLog2 = 8.0f;

__global__ void __launch_bounds__(kThreads, 1)
aifs_attention_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                      const __grid_constant__ CUtensorMap tmap_vt, const AttnParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_smem = smem;                       // 32 KB
  uint8_t* k_smem = q_smem + kTileBytes;        // kStages x 32 KB
  uint8_t* v_smem = k_smem + kStages * kTileBytes;
  AttnBarriers* sh = reinterpret_cast<AttnBarriers*>(v_smem + kStages * kTileBytes);
  float* xch = reinterpret_cast<float*>(sh + 1);                     // [2 groups][128 rows][m, l] for the final merge
  int32_t* kp_all = reinterpret_cast<int32_t*>(xch + 2 * kTile * 2);  // [8 warps][128] keys' original indices
  int32_t* tile_list = kp_all + 8 * kTile;   // [kMaxTiles] the key tiles this query tile processes: index | class << 16

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // heavy query tiles (late rows see the most keys) first; the heads of one key/value group side by side
  const int head = blockIdx.x % p.n_q_heads;
  const int qt = p.n_tiles - 1 - blockIdx.x / p.n_q_heads;
  const int g = head / p.group;
  const int q0 = qt * kTile;

  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_q)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_k)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_vt)) : "memory");
    mbar_init(&sh->q_full, 1);
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&sh->k_full[i], 1); mbar_init(&sh->k_empty[i], 1);
      mbar_init(&sh->v_full[i], 1); mbar_init(&sh->v_empty[i], 1);
    }
    for (int i = 0; i < 4; ++i) {   // [group][buffer]
      mbar_init(&sh->s_full[i], 1); mbar_init(&sh->p_full[i], 4); mbar_init(&sh->pv_done[i], 1);
    }
    mbar_init(&sh->drain, 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {
    tmem_alloc(&sh->tmem_base, 512);
    tmem_relinquish();
  }
  if (warp == 1) {
    // The key tiles to process, in order, once per CTA: every role walks this list instead of classifying
    // all tiles itself (four dependent global loads per tile, also for the skipped ones, were most of a short
    // CTA's life).  32 tiles are classified per step, one per lane.
    const int q_lo = p.qmin[qt], q_hi = p.qmax[qt];
    int count = 0;
    for (int base = 0; base < p.n_tiles; base += 32) {
      const int kt = base + lane;
      int cls = 0;
      if (kt < p.n_tiles) cls = (kt != qt && p.kmin[kt] > q_hi) ? 0 : (p.kmaxc[kt] <= q_lo ? 2 : 1);
      const unsigned take = __ballot_sync(0xffffffffu, cls != 0);
      if (cls != 0) tile_list[count + __popc(take & ((1u << lane) - 1u))] = kt | (cls << 16);
      count += __popc(take);
    }
    if (lane == 0) sh->n_list = count;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&sh->tmem_base);
  const int n_list = *reinterpret_cast<volatile int*>(&sh->n_list);

  if (warp == 0) {
    // ---------------- TMA producer: Q once, then K and V^T tiles of every key tile that is not skipped
    if (lane == 0) {
      mbar_arrive_expect_tx(&sh->q_full, kTileBytes);
      tma_load_2d(q_smem, &tmap_q, head * kD, q0, &sh->q_full);
      tma_load_2d(q_smem + kHalfBytes, &tmap_q, head * kD + 64, q0, &sh->q_full);
      int t = 0, s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int idx = 0; idx < n_list && ok; ++idx) {
        const int kt = tile_list[idx] & 0xffff;
        if (t >= kStages && !(ok = mbar_wait(&sh->k_empty[s], ph ^ 1u, &sh->abort_flag, p.status, 21))) break;
        mbar_arrive_expect_tx(&sh->k_full[s], kTileBytes);
        tma_load_2d(k_smem + s * kTileBytes, &tmap_k, g * kD, kt * kTile, &sh->k_full[s]);
        tma_load_2d(k_smem + s * kTileBytes + kHalfBytes, &tmap_k, g * kD + 64, kt * kTile, &sh->k_full[s]);
        if (t >= kStages && !(ok = mbar_wait(&sh->v_empty[s], ph ^ 1u, &sh->abort_flag, p.status, 22))) {
          mbar_wait_drain(&sh->k_full[s], ph, 20000ull);
          break;
        }
        mbar_arrive_expect_tx(&sh->v_full[s], kTileBytes);
        tma_load_2d(v_smem + s * kTileBytes, &tmap_vt, kt * kTile, g * kD, &sh->v_full[s]);
        tma_load_2d(v_smem + s * kTileBytes + kHalfBytes, &tmap_vt, kt * kTile + 64, g * kD, &sh->v_full[s]);
        ++t;
        if (++s == kStages) { s = 0; ph ^= 1u; }
      }
      if (!ok) {
        // copies still landing in this CTA's shared memory get time to finish before it exits
        mbar_wait_drain(&sh->q_full, 0, 20000ull);
        for (int back = 1; back <= kStages && back <= t; ++back) {
          const int u = t - back;
          mbar_wait_drain(&sh->k_full[u % kStages], (uint32_t)(u / kStages) & 1u, 20000ull);
          mbar_wait_drain(&sh->v_full[u % kStages], (uint32_t)(u / kStages) & 1u, 20000ull);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer.  Per key tile t: the scores of both groups (S_g = Q K_g^T, 128 x 64, into the
    // group's buffer t & 1), then the products of tile t - 1 (O_g += P_g V_g).  A group's scores for tile t + 1
    // are therefore computed while its softmax works on tile t.  S_g(t) overwrites the buffer P_g(t - 2) is read
    // from by a product issued before it: the MMAs of one thread execute in the order they were issued, so no
    // wait is needed between the two.
    if (elect_one()) {
      const uint32_t idesc_s = make_idesc_bf16(64);      // 128 rows x 64 keys
      const uint32_t idesc_o = make_idesc_bf16(kTile);   // 128 rows x 128 head channels
      const uint64_t qdesc = make_b_desc(smem_u32(q_smem));
      bool ok = mbar_wait(&sh->q_full, 0, &sh->abort_flag, p.status, 23);
      int ks = 0, vs = 0;       // ring positions of the next K and the next V tile
      uint32_t kph = 0, vph = 0;
      auto issue_pv = [&](int u) -> bool {
        const int b = u & 1;
        const uint32_t par = (uint32_t)(u >> 1) & 1u;
        if (!mbar_wait(&sh->v_full[vs], vph, &sh->abort_flag, p.status, 24)) return false;
        const uint64_t vdesc = make_b_desc(smem_u32(v_smem + vs * kTileBytes));
#pragma unroll
        for (int grp = 0; grp < 2; ++grp) {
          if (!mbar_wait(&sh->p_full[2 * grp + b], par, &sh->abort_flag, p.status, 25)) return false;
          tc_fence_after();
          const uint32_t p_tmem = tmem_base + (uint32_t)(grp * kTile + b * 64);
          const uint32_t o_tmem = tmem_base + kColO + (uint32_t)(grp * kTile);
#pragma unroll
          for (int k = 0; k < 4; ++k)   // the group's 64 keys: key block grp of the V^T tile
            mma_bf16_ts(o_tmem, p_tmem + (uint32_t)(k * 8), vdesc + (uint64_t)(grp * (kHalfBytes >> 4) + k * 2), idesc_o,
                        (u > 0 || k > 0) ? 1u : 0u);
          tc_commit(&sh->pv_done[2 * grp + b]);
        }
        tc_commit(&sh->v_empty[vs]);
        if (++vs == kStages) { vs = 0; vph ^= 1u; }
        return true;
      };
      for (int t = 0; t < n_list && ok; ++t) {
        const int b = t & 1;
        if (!(ok = mbar_wait(&sh->k_full[ks], kph, &sh->abort_flag, p.status, 27))) break;
        tc_fence_after();
        const uint64_t kdesc = make_b_desc(smem_u32(k_smem + ks * kTileBytes));
#pragma unroll
        for (int grp = 0; grp < 2; ++grp) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {   // head channels 16 k ..: channel block k >> 2; key rows 64 grp .. of the K tile
            const uint64_t off = (uint64_t)((k >> 2) * (kHalfBytes >> 4) + (k & 3) * 2);
            mma_bf16_ss(tmem_base + (uint32_t)(grp * kTile + b * 64), qdesc + off, kdesc + off + (uint64_t)(grp * (64 * 128 >> 4)),
                        idesc_s, k ? 1u : 0u);
          }
          tc_commit(&sh->s_full[2 * grp + b]);
        }
        tc_commit(&sh->k_empty[ks]);
        if (++ks == kStages) { ks = 0; kph ^= 1u; }
        if (t >= 1 && !(ok = issue_pv(t - 1))) break;
      }
      if (ok && n_list >= 1) ok = issue_pv(n_list - 1);
      if (!ok) {  // let every MMA already issued finish before tensor memory is freed
        tc_commit(&sh->drain);
        mbar_wait_drain(&sh->drain, 0, 2000000ull);
      }
    }
    __syncwarp();
  } else if (warp >= 4) {
    // ---------------- softmax warps.  Group grp = warps 4 + 4 grp .. 7 + 4 grp takes keys 64 grp .. 64 grp + 63 of
    // every processed key tile; its thread `row` owns query row q0 + row and keeps that row's reference maximum and
    // sum over the group's keys.  A warp depends on no other softmax warp until the two groups' partial results are
    // merged at the end.
    const int quarter = warp & 3, grp = (warp - 4) >> 2;
    const int row = quarter * 32 + lane;
    const int i = q0 + row;
    const int perm_i = i < p.L ? p.perm[i] : -1;
    const bool pad_i = i < p.L && p.pad_u && p.pad_u[i];
    const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t o_addr = lane_base + kColO + (uint32_t)(grp * kTile);
    int32_t* kp = kp_all + (warp - 4) * kTile;       // this warp's copy of its 64 keys' original indices
    const float lag_raw = kLagLog2 * fast_rcp(p.scale_log2);   // the lag in units of the raw scores
    float m_used = -1.0e30f, l_run = 0.0f;           // reference maximum of the exponents; sum relative to it
    bool ok = true;
    for (int t = 0; t < n_list && ok; ++t) {
      const int kt = tile_list[t] & 0xffff;
      const bool masked = (tile_list[t] >> 16) == 1;
      const int b = t & 1;
      const uint32_t par = (uint32_t)(t >> 1) & 1u;
      uint32_t allowed_lo = ~0u, allowed_hi = ~0u;
      if (masked) {
        __syncwarp();
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const int j = kt * kTile + grp * 64 + c * 32 + lane;
          kp[c * 32 + lane] = (j < p.L && !(p.pad_u && p.pad_u[j])) ? p.perm[j] : INT_MAX;
        }
        __syncwarp();
        // a padded row attends itself: the column of the diagonal, if it lies in this group's half of the diagonal tile
        const int self_col = (pad_i && kt == qt && (row >> 6) == grp) ? (row & 63) : -1;
        allowed_bits(kp, perm_i, self_col, allowed_lo, allowed_hi);
      }
      if (!(ok = warp_all(mbar_wait(&sh->s_full[2 * grp + b], par, &sh->abort_flag, p.status, 29)))) break;
      tc_fence_after();
      const uint32_t s_addr = lane_base + (uint32_t)(grp * kTile + b * 64);
      uint32_t sv[64];
      const float mx = masked ? scores_load_max<true>(s_addr, allowed_lo, allowed_hi, sv)
                              : scores_load_max<false>(s_addr, allowed_lo, allowed_hi, sv);
      const float m_new = fmaxf(m_used, mx);
      // move the reference maximum only when some row of this warp has outgrown it; then the accumulated output
      // and sum of the warp's rows are rescaled
      if (__any_sync(0xffffffffu, m_new > m_used + lag_raw)) {
        if (t >= 1) {
          // the product of the previous tile (and with it every earlier one) must have landed in the accumulator
          if (!(ok = warp_all(mbar_wait(&sh->pv_done[2 * grp + ((t - 1) & 1)], (uint32_t)((t - 1) >> 1) & 1u, &sh->abort_flag,
                                        p.status, 30)))) break;
          tc_fence_after();
          const float f = fast_exp2((m_used - m_new) * p.scale_log2);
#pragma unroll
          for (int cb = 0; cb < kD; cb += 16) {
            uint32_t v[16];
            tmem_ld_x16(o_addr + (uint32_t)cb, v);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * f);
            tmem_st_x16(o_addr + (uint32_t)cb, v);
          }
          tmem_wait_st();
          l_run *= f;
        }
        m_used = m_new;
      }
      // P = exp2(scale * (S - m_used)) replaces the scores
      l_run += probs_store(s_addr, sv, p.scale_log2, m_used);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->p_full[2 * grp + b]);
    }
    const int n = n_list;   // both groups work on every processed tile
    // this group's last product must have landed before its accumulator is read
    if (ok && n >= 1)
      ok = warp_all(mbar_wait(&sh->pv_done[2 * grp + ((n - 1) & 1)], (uint32_t)((n - 1) >> 1) & 1u, &sh->abort_flag, p.status, 32));
    tc_fence_after();
    // merge the two groups: each is a softmax over its own key tiles with its own reference maximum
    xch[(grp * kTile + row) * 2] = m_used;
    xch[(grp * kTile + row) * 2 + 1] = l_run;
    tc_fence_before();
    const bool all_ok = !named_bar_or(1, kSoftmaxThreads, !ok);
    tc_fence_after();
    if (all_ok) {
      // (the diagonal tile is never skipped, so both groups have worked on at least one tile)
      constexpr bool two = true;
      const float m0 = xch[row * 2], l0 = xch[row * 2 + 1];
      const float m1 = two ? xch[(kTile + row) * 2] : -1.0e30f, l1 = two ? xch[(kTile + row) * 2 + 1] : 0.0f;
      const float m = fmaxf(m0, m1);
      const float f0 = fast_exp2((m0 - m) * p.scale_log2), f1 = two ? fast_exp2((m1 - m) * p.scale_log2) : 0.0f;
      const float inv = fast_rcp(l0 * f0 + l1 * f1);  // (an IEEE division would compile to a subroutine call)
      // this thread writes head channels 64 grp .. 64 grp + 63 of its row
      const float w0 = f0 * inv, w1 = f1 * inv;
      __nv_bfloat16* dst = p.O + (size_t)i * p.ldo + (size_t)head * kD + grp * 64;
#pragma unroll
      for (int cb = 0; cb < 64; cb += 32) {
        uint32_t a0[32], a1[32];
        tmem_ld_x32(lane_base + kColO + (uint32_t)(grp * 64 + cb), a0);
        if (two) tmem_ld_x32(lane_base + kColO + (uint32_t)(kTile + grp * 64 + cb), a1);
        tmem_wait_ld();
        if (i < p.L) {
#pragma unroll
          for (int c8 = 0; c8 < 4; ++c8) {
            uint32_t w[4];
#pragma unroll
            for (int e2 = 0; e2 < 4; ++e2) {
              const int e = c8 * 8 + 2 * e2;
              float x0 = __uint_as_float(a0[e]) * w0, x1 = __uint_as_float(a0[e + 1]) * w0;
              if (two) {
                x0 = fmaf(__uint_as_float(a1[e]), w1, x0);
                x1 = fmaf(__uint_as_float(a1[e + 1]), w1, x1);
              }
              w[e2] = pack_bf16x2(x0, x1);
            }
            *reinterpret_cast<uint4*>(dst + cb + c8 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

constexpr size_t kAttnSmem = 1024 + (1 + 2 * kStages) * (size_t)kTileBytes + sizeof(AttnBarriers) + 2 * kTile * 2 * sizeof(float) +
                             8 * kTile * sizeof(int32_t) + kMaxTiles * sizeof(int32_t);

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn attn_encode_fn() {
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

// bf16 matrix [rows, cols] with a row pitch in elements, read in boxes of 128 rows x 64 elements (128 bytes)
bool encode_bf16_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t pitch) {
  EncodeTiledFn encode = attn_encode_fn();
  if (!encode) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)pitch * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)kTile};
  const cuuint32_t estr[2] = {1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline size_t round_up_256(size_t v) { return (v + 255) / 256 * 256; }
inline bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace
}  // namespace mq

using namespace mq;

extern "C" size_t mq_aifs_attention_workspace_bytes(int32_t L, int32_t n_kv_heads, int32_t head_dim) {
  if (L <= 0 || n_kv_heads <= 0 || head_dim != kD) return 0;
  const size_t n_tiles = ((size_t)L + kTile - 1) / kTile;
  return round_up_256((size_t)n_kv_heads * kD * n_tiles * kTile * 2) + round_up_256(4 * n_tiles * sizeof(int32_t));
}

extern "C" int mq_aifs_attention(const void* Q, int64_t ldq, const void* K, int64_t ldk, const void* V, int64_t ldv,
                                 const int32_t* perm, const uint8_t* pad_u, int32_t L, int32_t n_q_heads,
                                 int32_t n_kv_heads, int32_t head_dim, void* O, int64_t ldo, void* ws, size_t ws_bytes,
                                 int32_t* status, void* stream) {
  if (L < 0 || n_q_heads <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads) return MQ_ERR_INVALID_ARG;
  if (head_dim != kD || L > kMaxTiles * kTile) return MQ_ERR_UNSUPPORTED;
  if (ldq < (int64_t)n_q_heads * kD || ldo < (int64_t)n_q_heads * kD || ldk < (int64_t)n_kv_heads * kD ||
      ldv < (int64_t)n_kv_heads * kD)
    return MQ_ERR_INVALID_ARG;
  if (L == 0) return MQ_OK;
  if (!Q || !K || !V || !O || !perm || !ws || !status) return MQ_ERR_INVALID_ARG;
  if (!al16(Q) || !al16(K) || !al16(V) || !al16(O) || !al16(ws) || (ldq * 2) % 16 || (ldk * 2) % 16 || (ldv * 2) % 16 ||
      (ldo * 2) % 16)
    return MQ_ERR_ALIGNMENT;
  if (ws_bytes < mq_aifs_attention_workspace_bytes(L, n_kv_heads, head_dim)) return MQ_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int n_tiles = (L + kTile - 1) / kTile;
  const int Lp = n_tiles * kTile;
  uint16_t* Vt = static_cast<uint16_t*>(ws);
  int32_t* bounds = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(ws) + round_up_256((size_t)n_kv_heads * kD * Lp * 2));
  attn_prep_kernel<<<dim3(n_tiles, n_kv_heads), 256, 0, st>>>(static_cast<const uint16_t*>(V), ldv, L, Lp, perm, pad_u, Vt,
                                                              bounds, bounds + n_tiles, bounds + 2 * n_tiles,
                                                              bounds + 3 * n_tiles);
  if (cuda_status(cudaGetLastError()) != MQ_OK) return MQ_ERR_CUDA;

  CUtensorMap mq_, mk, mv;
  if (!encode_bf16_map(&mq_, Q, L, (int64_t)n_q_heads * kD, ldq) || !encode_bf16_map(&mk, K, L, (int64_t)n_kv_heads * kD, ldk) ||
      !encode_bf16_map(&mv, Vt, (int64_t)n_kv_heads * kD, Lp, Lp))
    return MQ_ERR_CUDA;
  static PerDeviceTable<char> attr_set;
  if (!ensure_dynamic_smem(attr_set, aifs_attention_kernel, (int)kAttnSmem)) return MQ_ERR_CUDA;
  AttnParams p{};
  p.L = L; p.n_tiles = n_tiles; p.n_q_heads = n_q_heads; p.group = n_q_heads / n_kv_heads;
  p.perm = perm; p.pad_u = pad_u;
  p.kmin = bounds; p.kmaxc = bounds + n_tiles; p.qmin = bounds + 2 * n_tiles; p.qmax = bounds + 3 * n_tiles;
  p.O = static_cast<__nv_bfloat16*>(O); p.ldo = ldo;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)kD);
  p.status = status;
  aifs_attention_kernel<<<dim3((unsigned)n_tiles * (unsigned)n_q_heads), kThreads, kAttnSmem, st>>>(mq_, mk, mv, p);
  return cuda_status(cudaGetLastError());
}
