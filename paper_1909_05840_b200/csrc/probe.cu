// qb_probe_i8_mma: measures what the tensor cores sustain for tcgen05.mma kind::i8 (s8 x s8 -> s32,
// 128 x N x 32 per instruction) with both operands resident in shared memory and no global traffic.
// It is the denominator against which qb_gemm's tensor-bound shapes are read: the GEMM cannot beat
// the rate at which the instruction itself retires.
#include "common.cuh"
#include "mbar_wait.cuh"
#include "ptx.cuh"

namespace qb {

static __device__ unsigned long long g_probe_cycles[256];

__device__ __forceinline__ uint64_t probe_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

template <int TOKENS>
__global__ void __launch_bounds__(128, 1) probe_i8_kernel(int k_blocks) {
  extern __shared__ __align__(1024) uint8_t smem[];  // A: 128 x 128 B, B: TOKENS x 128 B, then barriers
  const uint32_t base = ptx::smem_u32(smem);
  const uint32_t a_addr = base, b_addr = base + 128 * 128;
  const uint32_t bar0 = base + 128 * 128 + TOKENS * 128;  // 4 barriers
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 128 * 128 + TOKENS * 128 + 64);
  for (int i = threadIdx.x; i < (128 * 128 + TOKENS * 128) / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(smem)[i] = 0x01010101u * (i & 3);
  if (threadIdx.x == 0) {
    for (int i = 0; i < 4; ++i) ptx::mbar_init(bar0 + 8 * i, 1);
    ptx::fence_mbar_init();
  }
  if (threadIdx.x < 32) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), 2 * TOKENS);
    ptx::tmem_relinquish_alloc_permit();
  }
  ptx::fence_proxy_async_smem();
  ptx::tcgen05_fence_before_sync();
  __syncthreads();
  ptx::tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) {
    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TOKENS >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    const uint64_t a_desc = probe_desc(a_addr), b_desc = probe_desc(b_addr);
    const long long t0 = clock64();
    bool ok = true;
    for (int kb = 0; kb < k_blocks && ok; ++kb) {
      if (kb >= 4) {  // at most four K blocks in flight, as in a four-stage ring
        const uint32_t bar = bar0 + 8 * (kb & 3), parity = (uint32_t)((kb >> 2) - 1) & 1u;
        long long spins = 0;
        while (!ptx::mbar_try_wait(bar, parity))
          if (++spins > (1ll << 26)) { ok = false; break; }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
        ptx::mma_i8_ss(tmem_base + (uint32_t)((kb & 1) * TOKENS), a_desc + 2u * j, b_desc + 2u * j, idesc, j != 0);
      ptx::mma_commit(bar0 + 8 * (kb & 3));
    }
    // drain: the last commit covers every MMA issued before it
    if (ok && k_blocks > 0) {
      const int kb = k_blocks - 1;
      const uint32_t bar = bar0 + 8 * (kb & 3), parity = (uint32_t)(kb >> 2) & 1u;
      long long spins = 0;
      while (!ptx::mbar_try_wait(bar, parity))
        if (++spins > (1ll << 26)) { ok = false; break; }
    }
    const long long t1 = clock64();
    if (blockIdx.x < 256) g_probe_cycles[blockIdx.x] = ok ? (unsigned long long)(t1 - t0) : 0ull;
  }
  ptx::tcgen05_fence_before_sync();
  __syncthreads();
  if (threadIdx.x < 32) {
    ptx::tcgen05_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, 2 * TOKENS);
  }
}

}  // namespace qb

extern "C" qb_status qb_probe_i8_mma(int32_t tokens, int32_t k_blocks, double* tops_out, double* cycles_per_kblock_out) {
  if ((tokens != 128 && tokens != 256) || k_blocks < 8 || k_blocks > (1 << 22) || !tops_out) {
    qb::set_last_error("qb_probe_i8_mma: tokens must be 128 or 256, 8 <= k_blocks <= 2^22");
    return QB_ERR_INVALID;
  }
  int sms = 0;
  qb_status st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  const int smem_bytes = 128 * 128 + tokens * 128 + 128;
  cudaEvent_t e0, e1;
  QB_CUDA_TRY(cudaEventCreate(&e0));
  QB_CUDA_TRY(cudaEventCreate(&e1));
  float ms = 0.f;
  for (int rep = 0; rep < 3; ++rep) {  // the last repetition is the one reported
    QB_CUDA_TRY(cudaEventRecord(e0, 0));
    if (tokens == 256) {
      QB_CUDA_TRY(cudaFuncSetAttribute(qb::probe_i8_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
      qb::probe_i8_kernel<256><<<sms, 128, smem_bytes>>>(k_blocks);
    } else {
      QB_CUDA_TRY(cudaFuncSetAttribute(qb::probe_i8_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
      qb::probe_i8_kernel<128><<<sms, 128, smem_bytes>>>(k_blocks);
    }
    QB_CUDA_TRY(cudaGetLastError());
    QB_CUDA_TRY(cudaEventRecord(e1, 0));
    QB_CUDA_TRY(cudaEventSynchronize(e1));
    QB_CUDA_TRY(cudaEventElapsedTime(&ms, e0, e1));
  }
  unsigned long long cyc[256];
  QB_CUDA_TRY(cudaMemcpyFromSymbol(cyc, qb::g_probe_cycles, sizeof(cyc)));
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  unsigned long long worst = 0;
  for (int i = 0; i < sms && i < 256; ++i) {
    if (cyc[i] == 0) {
      qb::set_last_error("qb_probe_i8_mma: a bounded wait expired on SM slot %d", i);
      return QB_ERR_TIMEOUT;
    }
    if (cyc[i] > worst) worst = cyc[i];
  }
  const double ops = 2.0 * 128.0 * tokens * 128.0 * (double)k_blocks * sms;
  *tops_out = ops / (ms * 1e-3) / 1e12;
  if (cycles_per_kblock_out) *cycles_per_kblock_out = (double)worst / k_blocks;
  return QB_OK;
}

// qb_probe_wait_limit: the self-test of the bounded waits.  One CTA initialises an mbarrier that nothing
// ever arrives at and waits on it with the GEMM's own wait helpers (the single-thread form and the
// whole-warp form) under a short limit.  The waits must give up after `limit_cycles`, record
// QB_ERR_TIMEOUT in the workspace's status word exactly as the GEMM roles do, and the kernel must leave
// through its normal exit.  Nothing here can hang: the wait is the bounded one under test, and its
// loop ends on the cycle count alone.
namespace qb {
__global__ void __launch_bounds__(64, 1) probe_wait_limit_kernel(void* ws, long long limit_cycles,
                                                                 unsigned long long* waited_out) {
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ int abort_flag;
  const uint32_t bar = ptx::smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    ptx::mbar_init(bar, 1);  // one arrival expected; none will come
    abort_flag = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();
  const long long t0 = clock64();
  bool ok;
  if (threadIdx.x < 32) {
    ok = true;
    if (threadIdx.x == 0) ok = wait_barrier(bar, 0, &abort_flag, limit_cycles);  // the MMA issuer's form
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
  } else {
    ok = wait_barrier_warp(bar, 0, &abort_flag, limit_cycles);                    // the other roles' form
  }
  const long long waited = clock64() - t0;
  if (!ok && (threadIdx.x & 31) == 0) {
    report_status(ws, QB_ERR_TIMEOUT, (9 << 16) | (int)(threadIdx.x >> 5));
    if (waited_out) waited_out[threadIdx.x >> 5] = (unsigned long long)waited;
  }
}
}  // namespace qb

extern "C" qb_status qb_probe_wait_limit(void* ws, size_t ws_bytes, int64_t limit_cycles, uint64_t* waited_cycles_out,
                                         void* cuda_stream) {
  if (!ws || ws_bytes < qb::kWsMinBytes) {
    qb::set_last_error("qb_probe_wait_limit: workspace null or too small");
    return QB_ERR_WORKSPACE;
  }
  if (limit_cycles < 1000 || limit_cycles > 2000000000ll) {
    qb::set_last_error("qb_probe_wait_limit: limit_cycles must be in [1e3, 2e9]");
    return QB_ERR_INVALID;
  }
  int sms = 0;
  qb_status st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  qb::probe_wait_limit_kernel<<<1, 64, 0, (cudaStream_t)cuda_stream>>>(ws, (long long)limit_cycles,
                                                                       reinterpret_cast<unsigned long long*>(waited_cycles_out));
  QB_CUDA_TRY(cudaGetLastError());
  return QB_OK;
}
