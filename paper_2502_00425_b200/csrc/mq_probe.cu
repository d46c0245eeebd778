// Measurement and self-test aids (no counterpart in the paper).
//
// 1. mq_ubench_mma_i8: the issue rate of tcgen05.mma kind::i8 with fixed operands and no loads.
//    It gives the tensor-pipe denominator of the GEMM's roofline on the machine at hand (cycles
//    per 128 x N x 32 MMA, hence int8 operations per clock and SM) and shows how the duration of
//    an MMA depends on the token-tile width N, on where the A operand lives (tensor memory or
//    shared memory) and on how many independent accumulators the MMAs rotate over.
// 2. mq_selftest_bounded_wait: runs the kernels' bounded mbarrier wait on a barrier that nothing
//    ever arrives at, with a caller-chosen limit, so that the give-up path (status word, site,
//    abort flag, orderly return) is exercised without starving a barrier inside a real kernel.
#include "mq_common.cuh"
#include "mq_sm100.cuh"

namespace mq {
namespace {

struct ProbeShared {
  uint64_t done;
  uint64_t tick;  // receives the intermediate commits of the microbenchmark (nobody waits on it)
  uint32_t tmem_base;
  int abort_flag;
};

// One CTA per block index; 128 threads.  Warp 0 issues n_mma MMAs (lane elected once, whole warp
// converged), rotating over n_acc accumulators of n_tok columns each; every MMA multiplies the same
// zero-filled operands (the tensor pipe does not look at values).  cycles_out[block] = clock64 ticks
// from the first issue to the arrival of the commit that follows the last MMA.
__global__ void __launch_bounds__(128, 1)
ubench_mma_i8_kernel(int n_tok, int n_mma, int n_acc, int a_from_smem, int commit_every,
                     unsigned long long* cycles_out, int32_t* status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* b_smem = smem;                    // 256 rows x 128 B, K-major, 128-byte swizzle atoms
  uint8_t* a_smem = smem + 256 * 128;        // 128 rows x 128 B
  ProbeShared* sh = reinterpret_cast<ProbeShared*>(a_smem + 128 * 128);
  const int warp = threadIdx.x >> 5;

  for (int i = threadIdx.x; i < (256 * 128 + 128 * 128) / 16; i += blockDim.x)
    reinterpret_cast<uint4*>(smem)[i] = make_uint4(0u, 0u, 0u, 0u);
  if (threadIdx.x == 0) {
    mbar_init(&sh->done, 1);
    mbar_init(&sh->tick, 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the zero fill is read by the tensor pipe
  if (warp == 0) {
    tmem_alloc(&sh->tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&sh->tmem_base);

  // zero the A slot (32 columns: 128 lanes x 128 int8) and the accumulators: defined inputs
  {
    uint32_t z[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) z[i] = 0u;
    const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
    for (int c = 0; c < 512; c += 32) tmem_st_x32(lane_base + (uint32_t)c, z);
    tmem_wait_st();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  if (warp == 0) {
    const uint32_t idesc = make_idesc(n_tok);
    const uint64_t bdesc = make_b_desc(smem_u32(b_smem));
    const uint64_t adesc = make_b_desc(smem_u32(a_smem));
    const uint32_t a_tmem = tmem_base + 480u;  // last 32 columns; accumulators use [0, n_acc * n_tok) <= 480
    long long t0 = 0, t1 = 0;
    const bool leader = elect_one();
    __syncwarp();
    t0 = clock64();
    if (leader) {
      int acc = 0, since = 0;
      for (int i = 0; i < n_mma; ++i) {
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * n_tok);
        const int k4 = i & 3;
        if (a_from_smem) {
          asm volatile(
              "{\n\t.reg .pred p;\n\t"
              "setp.ne.b32 p, %4, 0;\n\t"
              "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
              ::"r"(d_tmem), "l"(adesc + (uint64_t)(k4 * 2)), "l"(bdesc + (uint64_t)(k4 * 2)), "r"(idesc), "r"(1u)
              : "memory");
        } else {
          mma_i8_ts(d_tmem, a_tmem + (uint32_t)(k4 * 8), bdesc + (uint64_t)(k4 * 2), idesc, 1u);
        }
        if (++acc == n_acc) acc = 0;
        // the GEMM commits once per K block (four MMAs): what that costs the issuing thread
        if (++since == commit_every) {  // (a counter: an integer modulo per MMA would cost more than the MMA)
          since = 0;
          if (i + 1 < n_mma) tc_commit(&sh->tick);
        }
      }
      tc_commit(&sh->done);
    }
    __syncwarp();
    const bool ok = warp_all(mbar_wait(&sh->done, 0, &sh->abort_flag, status, 1));
    t1 = clock64();
    if (threadIdx.x == 0) cycles_out[blockIdx.x] = ok ? (unsigned long long)(t1 - t0) : 0ull;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}


// Cost of the weight expanders' inner step, without any barrier: `warps` warps (4 or 8; warp w owns
// tensor-memory lanes 32 (w % 4) ..) each run n_iter rounds of
//   mode 0: tcgen05.st x32 (32 registers -> 32 columns) + tcgen05.wait::st
//   mode 1: four 16-byte shared-memory loads + the 32 logic operations of the nibble expansion + the same store
//   mode 2: as mode 1 without waiting for the store before the next round's loads (wait once at the end)
// cycles_out[warp] = clock64 ticks for the n_iter rounds.
__global__ void __launch_bounds__(256, 1)
ubench_expand_kernel(int n_iter, int mode, unsigned long long* cycles_out) {
  __shared__ __align__(16) uint8_t tile[2][8192];
  __shared__ uint32_t tmem_slot;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < 2 * 8192 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(tile)[i] = 0x9e3779b9u * (i + 1);
  if (warp == 0) {
    tmem_alloc(&tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  const int q = warp & 3, grp = warp >> 2;
  const int r = q * 32 + lane;
  uint32_t regs[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) regs[i] = (uint32_t)(i * 0x01010101u);
  uint32_t sink = 0;
  __syncthreads();
  const long long t0 = clock64();
  for (int it = 0; it < n_iter; ++it) {
    if (mode >= 1) {
      const uint4* src = reinterpret_cast<const uint4*>(tile[it & 1]) + r;
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const uint4 w = src[jj * 128];
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          regs[jj * 8 + 2 * i] = (ww[i] << 4) & 0xF0F0F0F0u;
          regs[jj * 8 + 2 * i + 1] = ww[i] & 0xF0F0F0F0u;
        }
      }
      sink ^= regs[1] ^ regs[9];
    }
    const uint32_t slot = (uint32_t)(((it * 2 + grp) & 7) * 32);
    tmem_st_x32(tmem_base + ((uint32_t)(q * 32) << 16) + slot, regs);
    if (mode <= 1) tmem_wait_st();
  }
  tmem_wait_st();
  const long long t1 = clock64();
  if (lane == 0) cycles_out[warp] = (unsigned long long)(t1 - t0) + (sink == 0x12345u ? 1ull : 0ull);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// One warp waits (bounded by limit_ns) on a barrier that has no arriver.  The wait gives up, records
// MQ_ERR_TIMEOUT and `site`, raises the abort flag; a second wait in another warp then returns at once
// because the flag is up.  waited_ns_out[0] = how long the first wait lasted.
__global__ void selftest_bounded_wait_kernel(unsigned long long limit_ns, int site, int32_t* status,
                                             unsigned long long* waited_ns_out) {
  __shared__ ProbeShared sh;
  if (threadIdx.x == 0) {
    mbar_init(&sh.done, 1);
    sh.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5;
  if (warp == 0) {
    const unsigned long long t0 = globaltimer_ns();
    const bool ok = warp_all(mbar_wait(&sh.done, 0, &sh.abort_flag, status, site, limit_ns));
    const unsigned long long t1 = globaltimer_ns();
    if (threadIdx.x == 0) {
      waited_ns_out[0] = t1 - t0;
      waited_ns_out[1] = ok ? 1ull : 0ull;
    }
  }
  __syncthreads();
  if (warp == 1) {
    // the CTA is aborting: this wait must not run its own clock down
    const unsigned long long t0 = globaltimer_ns();
    const bool ok = warp_all(mbar_wait(&sh.done, 0, &sh.abort_flag, status, site + 1, 1000000000ull));
    const unsigned long long t1 = globaltimer_ns();
    if ((threadIdx.x & 31) == 0) {
      waited_ns_out[2] = t1 - t0;
      waited_ns_out[3] = ok ? 1ull : 0ull;
    }
  }
}

}  // namespace
}  // namespace mq

extern "C" int mq_ubench_mma_i8(int32_t n_tok, int32_t n_mma, int32_t n_acc, int32_t a_from_smem, int32_t commit_every,
                                int32_t ctas, uint64_t* cycles_out, int32_t* status, void* stream) {
  using namespace mq;
  if (n_tok < 16 || n_tok > 256 || n_tok % 16 || n_mma < 1 || n_mma > (1 << 20) || n_acc < 1 || commit_every < 0 || ctas < 1 ||
      ctas > 4096 || !cycles_out || !status)
    return MQ_ERR_INVALID_ARG;
  if (n_acc * n_tok > 480) return MQ_ERR_INVALID_ARG;  // accumulators share tensor memory with the A slot
  const size_t smem = 1024 + 256 * 128 + 128 * 128 + sizeof(ProbeShared);
  static PerDeviceTable<char> attr_set;
  if (!ensure_dynamic_smem(attr_set, ubench_mma_i8_kernel, (int)smem)) return MQ_ERR_CUDA;
  ubench_mma_i8_kernel<<<ctas, 128, smem, static_cast<cudaStream_t>(stream)>>>(
      n_tok, n_mma, n_acc, a_from_smem, commit_every, reinterpret_cast<unsigned long long*>(cycles_out), status);
  return cuda_status(cudaGetLastError());
}

extern "C" int mq_selftest_bounded_wait(uint64_t limit_ns, int32_t site, int32_t* status, uint64_t* waited_ns_out,
                                        void* stream) {
  using namespace mq;
  if (!status || !waited_ns_out || limit_ns == 0 || limit_ns > 1000000000ull) return MQ_ERR_INVALID_ARG;
  selftest_bounded_wait_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(
      limit_ns, site, status, reinterpret_cast<unsigned long long*>(waited_ns_out));
  return cuda_status(cudaGetLastError());
}

extern "C" int mq_ubench_expand(int32_t n_iter, int32_t warps, int32_t mode, uint64_t* cycles_out, void* stream) {
  using namespace mq;
  if (n_iter < 1 || n_iter > (1 << 20) || (warps != 4 && warps != 8) || mode < 0 || mode > 2 || !cycles_out)
    return MQ_ERR_INVALID_ARG;
  ubench_expand_kernel<<<1, warps * 32, 0, static_cast<cudaStream_t>(stream)>>>(
      n_iter, mode, reinterpret_cast<unsigned long long*>(cycles_out));
  return cuda_status(cudaGetLastError());
}
