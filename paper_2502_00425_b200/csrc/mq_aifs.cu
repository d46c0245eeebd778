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
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)L * vec_per_row) return;
  const int i = (int)(idx / vec_per_row), c = (int)(idx % vec_per_row);
  const int p = perm[i];
  const int src = direction == 0 ? p : i;
  const int dst = direction == 0 ? i : p;
  Y[(int64_t)dst * ldo_vec + c] = __ldg(&X[(int64_t)src * ldx_vec + c]);
}

__global__ void remap_small_kernel(const int32_t* __restrict__ perm, const int32_t* __restrict__ pos_ids,
                                   const int32_t* __restrict__ n_first, int L,
                                   int32_t* __restrict__ pos_out, int32_t* __restrict__ seg_end_out,
                                   uint8_t* __restrict__ seg_mod_out) {
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
  if (direction == 0)
    aifs_perm_kernel<<<1, kScanThreads, 0, st>>>(is_visual, is_pad, L, perm, inv_perm, n_first_out);
  if (X && D > 0) {
    const int vec = D / 8;
    const int64_t n = (int64_t)L * vec;
    row_move_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(
        static_cast<const uint4*>(X), static_cast<uint4*>(X_out), L, vec, ldx / 8, ldo / 8, perm, direction);
  }
  return cuda_status(cudaGetLastError());
}

int launch_mask_remap(const int32_t* perm, const int32_t* pos_ids, const uint8_t* is_pad,
                      const int32_t* n_first, int L, int32_t* pos_out, int32_t* seg_end_out,
                      uint8_t* seg_mod_out, uint8_t* dense, cudaStream_t st) {
  const int blocks = L > 0 ? (L + 255) / 256 : 1;
  remap_small_kernel<<<blocks, 256, 0, st>>>(perm, pos_ids, n_first, L, pos_out, seg_end_out, seg_mod_out);
  if (dense && L > 0) {
    dim3 grid((L + 255) / 256, L);
    dense_mask_kernel<<<grid, 256, 0, st>>>(perm, is_pad, L, dense);
  }
  return cuda_status(cudaGetLastError());
}

}  // namespace mq
