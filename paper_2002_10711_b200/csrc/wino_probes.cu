// Debug probes.
//
// Tensor-pipe probe: how many int8 multiply-accumulates per second the tcgen05
// kind::i8 MMA sustains on this device when nothing else is in the way.  One CTA
// per SM, operands resident in shared memory (zeros), one thread issues a long
// run of 128x256x32 MMAs alternating between two tensor-memory accumulators.
// Used by the benchmark as a measured reference beside the nominal int8 peak.
#include "wino_launch.h"
#include "wino_ptx.cuh"

namespace wino {

__global__ void __launch_bounds__(128, 1)
k_mma_peak(int iters, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = base;                      // 128 x 128 B
  const uint32_t sB = base + 128u * 128u;        // 256 x 128 B
  const uint32_t bar = sB + 256u * 128u;
  const uint32_t tmem_slot = bar + 8u;
  const uint32_t abort_slot = tmem_slot + 4u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gen + (tmem_slot - base));
  volatile uint32_t* abort_p = reinterpret_cast<volatile uint32_t*>(gen + (abort_slot - base));
  for (uint32_t i = threadIdx.x; i < (128u + 256u) * 128u / 4u; i += blockDim.x)
    reinterpret_cast<uint32_t*>(gen)[i] = 0u;
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    *abort_p = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  fence_async_smem();
  if (threadIdx.x < 32) tmem_alloc(tmem_slot, 512u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_p;
  if (threadIdx.x == 0) {
    const uint32_t idesc = make_idesc_i8(128, 256);
    const uint64_t da = make_desc_sw128(sA), db = make_desc_sw128(sB);
    for (int i = 0; i < iters; ++i)
      mma_i8(tmem_base + (uint32_t)((i & 1) * 256), da + (uint64_t)((i & 3) * 2),
             db + (uint64_t)((i & 3) * 2), idesc, i >= 2 ? 1u : 0u);
    mma_commit(bar);
    if (!mbar_wait(bar, 0u, abort_p)) atomicExch(status, -6);   // WINO_ERR_TIMEOUT
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512u);
  }
}

int launch_mma_peak(int iters, int num_sms, int device, int* status, cudaStream_t st) {
  const size_t smem = 1024 + (128 + 256) * 128 + 64;
  static DeviceOnce once;
  if (int rc = set_max_smem(once, device, k_mma_peak, smem)) return rc;
  return launch_kernel(k_mma_peak, dim3((unsigned)num_sms), dim3(128), smem, st, false, iters, status);
}

// Bounded-wait probe: what a production kernel does when a barrier it waits for
// never completes, without making a production kernel fail.  One block, nothing
// in flight, no tensor memory held: thread 0 waits (same mbar_wait as every
// kernel, with the caller's cycle limit) on a barrier nobody arrives at, records
// WINO_ERR_TIMEOUT and the block leaves by its normal exit.
__global__ void __launch_bounds__(32)
k_wait_probe(long long limit_cycles, int* __restrict__ status) {
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ uint32_t abort_flag;
  const uint32_t bar = smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    if (!mbar_wait(bar, 0u, &abort_flag, limit_cycles)) {
      abort_flag = 1u;
      atomicExch(status, -6);   // WINO_ERR_TIMEOUT
    }
  }
  __syncwarp();
}

int launch_wait_probe(long long limit_cycles, int* status, cudaStream_t st) {
  return launch_kernel(k_wait_probe, dim3(1), dim3(32), 0, st, false, limit_cycles, status);
}

}  // namespace wino
