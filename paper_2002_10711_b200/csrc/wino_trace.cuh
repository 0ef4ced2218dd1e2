// Optional device time stamps for the staged kernels (only in builds with -DWINO_TRACE; the
// product build compiles every macro below to nothing).  Each block counts its own launches
// and files its stamps under (launch number mod kTraceSteps, block, slot), so a run of
// chained steps can be read back step by step.  One table per translation unit.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#ifdef WINO_TRACE
namespace wino {
constexpr int kTraceSteps = 32, kTraceBlocks = 2368, kTraceSlots = 16;
struct TraceTable {
  unsigned long long t[kTraceSteps][kTraceBlocks][kTraceSlots];
  unsigned int launches[kTraceBlocks];
};
__device__ __forceinline__ unsigned long long trace_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
}  // namespace wino
// `tab` is a `static __device__ TraceTable`; `step` an `int` the kernel keeps.
#define WINO_ST_BEGIN(tab, step) \
  do { if (blockIdx.x < wino::kTraceBlocks) (step) = (int)(atomicAdd(&(tab).launches[blockIdx.x], 1u) % wino::kTraceSteps); } while (0)
#define WINO_ST(tab, step, slot) \
  do { if (blockIdx.x < wino::kTraceBlocks) (tab).t[(step)][blockIdx.x][(slot)] = wino::trace_now(); } while (0)
#define WINO_ST_READER(name, tab)                                                         \
  extern "C" int name(void* host_out, int reset) {                                        \
    if (reset) {                                                                           \
      void* d = nullptr;                                                                   \
      if (cudaGetSymbolAddress(&d, tab) != cudaSuccess) return -5;                         \
      return cudaMemset(d, 0, sizeof(wino::TraceTable)) == cudaSuccess ? 0 : -5;           \
    }                                                                                      \
    return cudaMemcpyFromSymbol(host_out, tab, sizeof(wino::TraceTable)) == cudaSuccess ? 0 : -5; \
  }
#else
#define WINO_ST_BEGIN(tab, step) ((void)0)
#define WINO_ST(tab, step, slot) ((void)0)
#define WINO_ST_READER(name, tab)
#endif
