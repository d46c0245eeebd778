// K3: Attention-Invariant Flexible Switching -- token reorder (stable partition: visual and
// pad tokens first, then text), row gather / scatter, position-id and causal-mask remap.
//
// Method: Sec. 3.1 (reorder so that all visual tokens come first; the unified mask M^u of
// Eq. 5 keeps the original autoregressive relation), App. A.2 (index map
// AIFS(1..L) = (m..n, 1..m-1, n+1..L); rotary embeddings use the original index),
// App. A.4 (left pads travel with the image block and are never attended).
//
// The index build is one CTA (a sequence has at most a few 10^5 tokens; the scan is a
// few microseconds and runs once per sequence); the row copy is a plain 16-byte-vector
// gather bounded by HBM traffic of 2 * L * D * 2 bytes.
#include "mq_common.cuh"

namespace mq {
namespace {

constexpr int kScanThreads = 1024;

__device__ __forceinline__ int block_exclusive_scan(int flag, int* warp_sums, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned b = __ballot_sync(0xffffffffu, flag);
  const int in_warp = __popc(b & ((1u << lane) - 1u));
  if (lane == 0) warp_sums[warp] = __popc(b);
  __syncthreads();
  if (warp == 0) {
    int s = warp_sums[lane];
    int incl = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    warp_sums[lane] = incl - s;
    if (lane == 31) *total = incl;
  }
  __syncthreads();
  const int r = warp_sums[warp] + in_warp;
  return r;
}

__global__ void __launch_bounds__(kScanThreads)
aifs_perm_kernel(const uint8_t* __restrict__ is_visual, const uint8_t* __restrict__ is_pad, int L,
                 int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm,
                 int32_t* __restrict__ n_first_out) {
  __shared__ int warp_sums[32];
  __shared__ int total;
  __shared__ int n_first_s;
  // pass 1: size of the first (visual + pad) block
  int cnt = 0;
  for (int i = threadIdx.x; i < L; i += kScanThreads)
    cnt += (is_visual[i] != 0) || (is_pad && is_pad[i] != 0);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = cnt;
  __syncthreads();
  if (threadIdx.x == 0) {
    int s = 0;
    for (int w = 0; w < kScanThreads / 32; ++w) s += warp_sums[w];
    n_first_s = s;
    if (n_first_out) *n_first_out = s;
  }
  __syncthreads();
  const int n_first = n_first_s;
  // pass 2: stable positions
  int first_before = 0;  // first-block tokens before this chunk
  for (int base = 0; base < L; base += kScanThreads) {
    const int i = base + threadIdx.x;
    const int f = (i < L) && ((is_visual[i] != 0) || (is_pad && is_pad[i] != 0));
    __syncthreads();  // warp_sums / total reuse
    const int excl = block_exclusive_scan(f, warp_sums, &total);
    if (i < L) {
      const int fb = first_before + excl;
      const int pos = f ? fb : n_first + (i - fb);
      perm[pos] = i;
      if (inv_perm) inv_perm[i] = pos;
    }
    first_before += total;
  }
}

// dir 0: out[i] = in[perm[i]];  dir 1: out[perm[i]] = in[i].  One 16-byte vector per thread.
__global__ void row_move_kernel(const uint4* __restrict__ X, uint4* __restrict__ Y, int L, int vec_per_row,
                                int64_t ldx_vec, int64_t ldo_vec, const int32_t* __restrict__ perm,
                                int direction) {
  pdl_launch_dependents();
  pdl_wait();
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)L * vec_per_row) return;
  const int i = (int)(idx / vec_per_row), c = (int)(idx % vec_per_row);
  const int p = perm[i];
  const int src = direction == 0 ? p : i;
  const int dst = direction == 0 ? i : p;
  Y[(int64_t)dst * ldo_vec + c] = __ldg(&X[(int64_t)src * ldx_vec + c]);
}

// Index build and row gather in one launch, for sequences short enough that every CTA can
// afford to count the modality flags itself (L bytes from L2 per CTA).  A CTA owns the source
// rows [r0, r1): it counts the first-block tokens before r0 and in the whole sequence, which
// fixes the destination of each of its rows (stable partition), writes perm / inv_perm for
// them and copies the rows with 16-byte vectors.
constexpr int kFusedThreads = 256;
constexpr int kFusedMaxL = 16384;

__global__ void __launch_bounds__(kFusedThreads)
aifs_fused_gather_kernel(const uint4* __restrict__ X, uint4* __restrict__ Y, int L, int vec_per_row,
                         int64_t ldx_vec, int64_t ldo_vec, const uint8_t* __restrict__ is_visual,
                         const uint8_t* __restrict__ is_pad, int32_t* __restrict__ perm,
                         int32_t* __restrict__ inv_perm, int32_t* __restrict__ n_first_out, int rows_per_cta) {
  __shared__ int red_before[kFusedThreads / 32], red_total[kFusedThreads / 32];
  __shared__ int s_dst[64];
  pdl_launch_dependents();
  pdl_wait();
  const int r0 = blockIdx.x * rows_per_cta;
  const int r1 = min(L, r0 + rows_per_cta);
  int before = 0, total = 0;
  for (int i = threadIdx.x; i < L; i += kFusedThreads) {
    const int f = (is_visual[i] != 0) || (is_pad && is_pad[i] != 0);
    total += f;
    before += (i < r0) ? f : 0;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    before += __shfl_xor_sync(0xffffffffu, before, o);
    total += __shfl_xor_sync(0xffffffffu, total, o);
  }
  if ((threadIdx.x & 31) == 0) {
    red_before[threadIdx.x >> 5] = before;
    red_total[threadIdx.x >> 5] = total;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int b = 0, t = 0;
    for (int w = 0; w < kFusedThreads / 32; ++w) { b += red_before[w]; t += red_total[w]; }
    // destinations of this CTA's rows (rows_per_cta <= 64): sequential, a handful of rows
    int fb = b;
    for (int i = r0; i < r1; ++i) {
      const int f = (is_visual[i] != 0) || (is_pad && is_pad[i] != 0);
      const int pos = f ? fb : t + (i - fb);
      s_dst[i - r0] = pos;
      perm[pos] = i;
      if (inv_perm) inv_perm[i] = pos;
      fb += f;
    }
    if (blockIdx.x == 0 && n_first_out) *n_first_out = t;
  }
  __syncthreads();
  if (X == nullptr) return;
  const int n_vec = (r1 - r0) * vec_per_row;
  for (int v = threadIdx.x; v < n_vec; v += kFusedThreads) {
    const int rr = v / vec_per_row, c = v - rr * vec_per_row;
    Y[(int64_t)s_dst[rr] * ldo_vec + c] = __ldg(&X[(int64_t)(r0 + rr) * ldx_vec + c]);
  }
}

__global__ void remap_small_kernel(const int32_t* __restrict__ perm, const int32_t* __restrict__ pos_ids,
                                   const int32_t* __restrict__ n_first, int L,
                                   int32_t* __restrict__ pos_out, int32_t* __restrict__ seg_end_out,
                                   uint8_t* __restrict__ seg_mod_out) {
  pdl_launch_dependents();
  pdl_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (pos_out && i < L) {
    const int p = perm[i];
    pos_out[i] = pos_ids ? pos_ids[p] : p;
  }
  if (i == 0 && seg_end_out && seg_mod_out) {
    seg_end_out[0] = *n_first;
    seg_end_out[1] = L;
    seg_mod_out[0] = MQ_VISUAL;
    seg_mod_out[1] = MQ_TEXT;
  }
}

// allowed(i,j) = perm[j] <= perm[i] and not pad[perm[j]]; a pad row keeps its diagonal.
__global__ void dense_mask_kernel(const int32_t* __restrict__ perm, const uint8_t* __restrict__ is_pad,
                                  int L, uint8_t* __restrict__ mask) {
  const int i = blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= L) return;
  const int pi = perm[i], pj = perm[j];
  const bool pad_j = is_pad && is_pad[pj];
  const bool pad_i = is_pad && is_pad[pi];
  bool ok = (pj <= pi) && !pad_j;
  if (pad_i && i == j) ok = true;
  mask[(int64_t)i * L + j] = ok ? 1 : 0;
}

}  // namespace

int launch_aifs_reorder(const void* X, void* X_out, int L, int D, int64_t ldx, int64_t ldo,
                        const uint8_t* is_visual, const uint8_t* is_pad, int32_t* perm,
                        int32_t* inv_perm, int32_t* n_first_out, int direction, cudaStream_t st) {
  if (L == 0) {
    if (direction == 0 && n_first_out) cudaMemsetAsync(n_first_out, 0, sizeof(int32_t), st);
    return cuda_status(cudaGetLastError());
  }
  if (direction == 0 && L <= kFusedMaxL) {
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int rows_per_cta = (L + 4 * sms - 1) / (4 * sms);
    if (rows_per_cta > 64) rows_per_cta = 64;
    const int ctas = (L + rows_per_cta - 1) / rows_per_cta;
    const bool move = X && D > 0;
    return cuda_status(launch_pdl(aifs_fused_gather_kernel, dim3(ctas), dim3(kFusedThreads), 0, st,
                                  move ? static_cast<const uint4*>(X) : nullptr, static_cast<uint4*>(X_out), L,
                                  move ? D / 8 : 0, ldx / 8, ldo / 8, is_visual, is_pad, perm, inv_perm,
                                  n_first_out, rows_per_cta));
  }
  if (direction == 0)
    aifs_perm_kernel<<<1, kScanThreads, 0, st>>>(is_visual, is_pad, L, perm, inv_perm, n_first_out);
  if (X && D > 0) {
    const int vec = D / 8;
    const int64_t n = (int64_t)L * vec;
    if (launch_pdl(row_move_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st,
                   static_cast<const uint4*>(X), static_cast<uint4*>(X_out), L, vec, ldx / 8, ldo / 8,
                   static_cast<const int32_t*>(perm), direction) != cudaSuccess)
      return MQ_ERR_CUDA;
  }
  return cuda_status(cudaGetLastError());
}

int launch_mask_remap(const int32_t* perm, const int32_t* pos_ids, const uint8_t* is_pad,
                      const int32_t* n_first, int L, int32_t* pos_out, int32_t* seg_end_out,
                      uint8_t* seg_mod_out, uint8_t* dense, cudaStream_t st) {
  const int blocks = L > 0 ? (L + 255) / 256 : 1;
  if (launch_pdl(remap_small_kernel, dim3(blocks), dim3(256), 0, st, perm, pos_ids, n_first, L, pos_out, seg_end_out,
                 seg_mod_out) != cudaSuccess)
    return MQ_ERR_CUDA;
  if (dense && L > 0) {
    dim3 grid((L + 255) / 256, L);
    dense_mask_kernel<<<grid, 256, 0, st>>>(perm, is_pad, L, dense);
  }
  return cuda_status(cudaGetLastError());
}

}  // namespace mq
