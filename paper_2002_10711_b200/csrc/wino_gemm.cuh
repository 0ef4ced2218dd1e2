// Hadamard stage of the Winograd-aware layer as t*t independent int8 GEMMs over
// channels with int32 accumulation (paper: Sections 1 and 5.3, "element-wise
// GEMM stage"):   M[xi][tau][k] = sum_c V_q[xi][tau][c] * U_q[xi][k][c]
// followed by the quantizer of the Hadamard output (paper: Fig. 2).
//
//   k_gemm_tc   : tcgen05 int8 MMA (kind::i8), operands staged in shared memory
//                 by TMA (128-byte swizzle), int32 accumulators in tensor memory.
//   k_gemm_dp4a : the same contraction with 4-way integer dot products on the
//                 ALUs; fallback for channel counts the TMA path cannot take.
#pragma once
#include <cuda.h>
#include "wino_common.cuh"

namespace wino {

// Output modes of the GEMM epilogue.
enum { kOutMq = 0, kOutI32 = 1 };

// ---------------------------------------------------------------------------
// ALU fallback.  Thread = (xi, tau, 4 consecutive k).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
k_gemm_dp4a(const __grid_constant__ Params p, const int8_t* __restrict__ Vq,
            const int8_t* __restrict__ Uq, void* __restrict__ out, int out_mode,
            unsigned* __restrict__ absmaxM) {
  const int C4 = p.C >> 2, K4 = p.K >> 2;
  const int xi = blockIdx.z;
  const long idx = blockIdx.x * (long)blockDim.x + threadIdx.x;
  float vmax = 0.0f;
  if (idx < (long)p.T * K4) {
    const int k4 = (int)(idx % K4);
    const int tau = (int)(idx / K4);
    const int* v = reinterpret_cast<const int*>(Vq) + ((long)xi * p.T + tau) * C4;
    const int* u = reinterpret_cast<const int*>(Uq) + ((long)xi * p.K + k4 * 4) * C4;
    int acc[4] = {0, 0, 0, 0};
    for (int c4 = 0; c4 < C4; ++c4) {
      const int vv = __ldg(v + c4);
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[j] = __dp4a(vv, __ldg(u + (long)j * C4 + c4), acc[j]);
    }
    const long o = ((long)xi * p.T + tau) * p.K + k4 * 4;
    if (out_mode == kOutI32) {
      *reinterpret_cast<int4*>(reinterpret_cast<int*>(out) + o) = make_int4(acc[0], acc[1], acc[2], acc[3]);
    } else {
      uint32_t wv = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float r = quant_magic(__int2float_rn(acc[j]), p.mult_M, p.lo_M, p.hi_M);
        wv |= (__float_as_uint(r) & 0xFFu) << (8 * j);
      }
      *reinterpret_cast<uint32_t*>(reinterpret_cast<int8_t*>(out) + o) = wv;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) vmax = fmaxf(vmax, fabsf(__int2float_rn(acc[j])));
  }
  if (absmaxM != nullptr) atomic_absmax(absmaxM, vmax);
}

// ---------------------------------------------------------------------------
// PTX wrappers (sm_100a).
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* ptr) {
  return (uint32_t)__cvta_generic_to_shared(ptr);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.b32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls and reports failure; the
// caller then records WINO_ERR_TIMEOUT and unwinds without touching the data.
constexpr uint32_t kSpinLimit = 1u << 22;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem),
               "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void mma_i8(uint32_t taddr, uint64_t adesc, uint64_t bdesc,
                                       uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n"
      "}\n"
      ::"r"(taddr), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor for a K-major operand tile stored as rows of
// 128 bytes with the 128-byte swizzle (what TMA writes with SWIZZLE_128B):
// start address / 16, leading offset (unused for swizzled K-major) = 1,
// stride between 8-row groups = 1024 bytes, descriptor version 1, layout 2.
__device__ __forceinline__ uint64_t make_desc_sw128(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) |
         (2ull << 61);
}
// Instruction descriptor: D = int32, A = B = signed 8-bit, both K-major, M x N.
__host__ __device__ constexpr uint32_t make_idesc_i8(int M, int N) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ---------------------------------------------------------------------------
// tcgen05 GEMM.  One CTA computes a 128 (tau) x BN (k) block of one xi.
//   warp 0 lane 0 : TMA producer         warp 1 : TMEM owner, lane 0 issues MMAs
//   all 4 warps   : epilogue (warp w reads TMEM lanes 32w .. 32w+31)
// A stage holds 128 bytes of the channel axis: A tile 128 x 128 B (16 KB),
// B tile BN x 128 B.  One MMA consumes 32 channels.
// ---------------------------------------------------------------------------
constexpr int kBM = 128;
constexpr int kStageK = 128;  // bytes (= int8 channels) per stage

struct GemmTcArgs {
  int BN;           // multiple of 16, <= 256
  int stages;       // >= 1
  int tmem_cols;    // power of two >= 32, >= BN
  int out_mode;     // kOutMq / kOutI32
};

__global__ void __launch_bounds__(128)
k_gemm_tc(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap mapV,
          const __grid_constant__ CUtensorMap mapU, const GemmTcArgs a, void* __restrict__ out,
          unsigned* __restrict__ absmaxM, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  // tiles need 1024-byte alignment for the 128-byte swizzle
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t a_bytes = kBM * kStageK, b_bytes = (uint32_t)a.BN * kStageK;
  const uint32_t tiles_end = base + (uint32_t)a.stages * (a_bytes + b_bytes);
  const uint32_t bar_full = tiles_end;                 // stages x 8 B
  const uint32_t bar_empty = bar_full + 8u * a.stages; // stages x 8 B
  const uint32_t bar_accum = bar_empty + 8u * a.stages;
  const uint32_t tmem_slot = bar_accum + 8u;
  const uint32_t abort_slot = tmem_slot + 4u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gen + (tmem_slot - base));
  volatile uint32_t* abort_p = reinterpret_cast<volatile uint32_t*>(gen + (abort_slot - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * kBM, n0 = blockIdx.y * a.BN, xi = blockIdx.z;
  const int KB = (p.C + kStageK - 1) / kStageK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      mbar_init(bar_full + 8u * s, 1);
      mbar_init(bar_empty + 8u * s, 1);
    }
    mbar_init(bar_accum, 1);
    *abort_p = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(tmem_slot, (uint32_t)a.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_p;

  if (warp == 0 && lane == 0) {
    // producer
    for (int kb = 0; kb < KB; ++kb) {
      const int s = kb % a.stages;
      const uint32_t ph = (uint32_t)(kb / a.stages) & 1u;
      if (!mbar_wait(bar_empty + 8u * s, ph ^ 1u)) { *abort_p = 1u; break; }
      const uint32_t sa = base + (uint32_t)s * (a_bytes + b_bytes);
      mbar_expect_tx(bar_full + 8u * s, a_bytes + b_bytes);
      tma_load_3d(sa, &mapV, bar_full + 8u * s, kb * kStageK, m0, xi);
      tma_load_3d(sa + a_bytes, &mapU, bar_full + 8u * s, kb * kStageK, n0, xi);
    }
  } else if (warp == 1 && lane == 0) {
    // MMA issuer
    const uint32_t idesc = make_idesc_i8(kBM, a.BN);
    bool ok = true;
    for (int kb = 0; kb < KB && ok; ++kb) {
      const int s = kb % a.stages;
      const uint32_t ph = (uint32_t)(kb / a.stages) & 1u;
      if (!mbar_wait(bar_full + 8u * s, ph)) { *abort_p = 1u; ok = false; break; }
      tc_fence_after();
      const uint32_t sa = base + (uint32_t)s * (a_bytes + b_bytes);
      const uint64_t da = make_desc_sw128(sa), db = make_desc_sw128(sa + a_bytes);
      const int rem = p.C - kb * kStageK;
      const int ksteps = rem >= kStageK ? 4 : (rem + 31) / 32;
      for (int k = 0; k < ksteps; ++k)
        mma_i8(tmem_base, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc,
               (kb | k) != 0 ? 1u : 0u);
      mma_commit(bar_empty + 8u * s);   // frees the stage when these MMAs retire
    }
    if (ok) mma_commit(bar_accum);      // accumulator complete
  }
  __syncwarp();

  // epilogue: all four warps
  bool ready = mbar_wait(bar_accum, 0u);
  if (!ready) *abort_p = 1u;
  tc_fence_after();
  __syncthreads();
  const bool aborted = (*abort_p != 0u);
  float vmax = 0.0f;
  if (!aborted) {
    const int tau = m0 + warp * 32 + lane;
    const bool row_ok = tau < p.T;
    for (int col = 0; col < a.BN; col += 32) {
      uint32_t r[32];
      tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)col, r);
      const int k0 = n0 + col;
      if (absmaxM != nullptr && row_ok) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (k0 + j < p.K) vmax = fmaxf(vmax, fabsf(__int2float_rn((int)r[j])));
      }
      if (!row_ok) continue;
      const long o = ((long)xi * p.T + tau) * p.K + k0;
      if (a.out_mode == kOutI32) {
        int4* dst = reinterpret_cast<int4*>(reinterpret_cast<int*>(out) + o);
#pragma unroll
        for (int q = 0; q < 8; ++q)
          if (k0 + q * 4 < p.K) dst[q] = make_int4((int)r[4 * q], (int)r[4 * q + 1], (int)r[4 * q + 2], (int)r[4 * q + 3]);
      } else {
        uint32_t w[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          uint32_t wv = 0;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            float f = quant_magic(__int2float_rn((int)r[4 * q + j]), p.mult_M, p.lo_M, p.hi_M);
            wv |= (__float_as_uint(f) & 0xFFu) << (8 * j);
          }
          w[q] = wv;
        }
        uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<int8_t*>(out) + o);
        if (k0 < p.K) dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
        if (k0 + 16 < p.K) dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
      }
    }
  } else if (threadIdx.x == 0) {
    atomicExch(status, -6);  // WINO_ERR_TIMEOUT
  }
  if (absmaxM != nullptr) atomic_absmax(absmaxM, vmax);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)a.tmem_cols);
}

}  // namespace wino
