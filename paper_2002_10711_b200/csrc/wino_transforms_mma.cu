// Input and output transforms of the Winograd-aware layer on the tensor cores
// (paper: Eq. 1, stages 1 and 4 of Fig. 2), for the Cook-Toom matrices of F2 and
// F4 with 128-channel chunks.
//
// B^T d B and A^T m A are linear maps of the patch, so per channel they are one
// matrix-vector product with the Kronecker matrix:
//     V[xi] = sum_ab (B^T (x) B^T)[xi][ab] d[ab],   Y[pq] = sum_xi (A^T (x) A^T)[pq][xi] m[xi].
// On integer codes with the Cook-Toom matrices every value is an integer far
// below 2^24 (|V| <= 12700, |Y| <= 45847 for F4), so the int32 result of an int8
// tensor-core product has the same bits as the fp32 chains of the arithmetic
// contract.  Per unit = (tile, 128 channels):
//   A operand  the patch itself as TMA delivers it: t*t rows (one per patch
//              position) of 128 channel bytes, 128-byte swizzle.  Channels are the
//              MMA's M dimension, the rows its K dimension: an "MN-major" operand.
//              K is padded to a multiple of 32 with whatever follows in shared
//              memory; the Kronecker matrix has zero columns there.
//   B operand  the Kronecker matrix, [N = xi or pq][K = ab or xi] K-major int8,
//              computed on the host when the plan is made, copied once per block
//              into shared memory (64-byte swizzle).
//   D          128 lanes (channels) x N columns of int32 in tensor memory.
// Epilogue: lane = channel; tcgen05.ld, int -> float, the one-FMA quantizer, a
// byte per code into a staging tile, one TMA store per unit.
#include <cstring>

#include "wino_launch.h"
#include "wino_ptx.cuh"

namespace wino {

namespace {

constexpr int kTmThreads = 160;   // warp 0: TMA + MMA issue; warps 1-4: epilogue
constexpr int kInSlots = 4;       // units in flight per block

// K-major tile of 64-byte rows with the 64-byte swizzle (8-row groups of 512 B).
__device__ __forceinline__ uint64_t desc_kmajor_sw64(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (32ull << 32) | (1ull << 46) |
         (4ull << 61);
}
__device__ __forceinline__ uint32_t sw64_off(int row, int byte) {
  const int chunk = (byte >> 4) ^ ((row >> 1) & 3);
  return (uint32_t)(row * 64 + chunk * 16 + (byte & 15));
}
// MN-major tile: rows of 128 bytes along M (one row per K index), 128-byte swizzle,
// 8-row groups of 1024 B along K.  M = 128 int8 elements is exactly one row, so the
// leading-dimension offset is not used.
__device__ __forceinline__ uint64_t desc_mnmajor_sw128(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (64ull << 16) | (64ull << 32) | (1ull << 46) |
         (2ull << 61);
}
// Instruction descriptor: D int32, A and B signed 8-bit, A MN-major (bit 15), B K-major.
__host__ __device__ constexpr uint32_t idesc_i8_a_mn(int M, int N) {
  return (2u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}

template <int N>
__device__ __forceinline__ void bulk_wait_read_n() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t (&r)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr)
               : "memory");
}

// Shared pipeline skeleton of both kernels.  Layout of dynamic shared memory
// (1024-byte aligned): kInSlots input slots of KROWS x 128 B, the Kronecker matrix
// (NB rows x 64 B), two output staging tiles, barriers.
template <int KROWS, int NB, int OUT_BYTES>
struct TmSmem {
  static constexpr uint32_t kInSlot = KROWS * 128;
  static constexpr uint32_t kB = NB * 64;
  static constexpr uint32_t kOut = (OUT_BYTES + 127) / 128 * 128;
  static constexpr uint32_t kTotal = kInSlots * kInSlot + kB + 2 * kOut + 128;
  uint32_t in, b, out, bar_full, bar_in_empty, bar_acc_full, bar_acc_empty, tmem_slot, abort_slot;
  __device__ explicit TmSmem(uint32_t base) {
    in = base;
    b = in + kInSlots * kInSlot;
    out = b + kB;
    bar_full = out + 2 * kOut;               // kInSlots x 8
    bar_in_empty = bar_full + 8 * kInSlots;  // kInSlots x 8
    bar_acc_full = bar_in_empty + 8 * kInSlots;   // 2 x 8
    bar_acc_empty = bar_acc_full + 16;            // 2 x 8
    tmem_slot = bar_acc_empty + 16;
    abort_slot = tmem_slot + 4;
  }
};

}  // namespace

// ---------------------------------------------------------------------------
// Input transform.  x [N][H][W][C] -> V_q [t*t][T][C].  Unit u = tau * (C/128) + chunk.
// ---------------------------------------------------------------------------
template <int M>
__global__ void __launch_bounds__(kTmThreads)
k_input_transform_mma(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap mapX,
                      const __grid_constant__ CUtensorMap mapV, const uint4* __restrict__ kron,
                      int* __restrict__ status) {
  constexpr int T_ = M + 2, T2 = T_ * T_;
  constexpr int KROWS = (T2 + 31) / 32 * 32;      // MMA K: 32 (F2) or 64 (F4)
  constexpr int NB = (T2 + 15) / 16 * 16;         // MMA N: 16 (F2) or 48 (F4)
  constexpr int ACC = 64;                          // tensor-memory columns per accumulator
  using L = TmSmem<KROWS, NB, T2 * 128>;
  static_assert(L::kTotal + 1024 <= 56 * 1024, "shared-memory request too small");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const L s(base);
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gen + (s.tmem_slot - base));
  volatile uint32_t* abort_p = reinterpret_cast<volatile uint32_t*>(gen + (s.abort_slot - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cchunks = p.C >> 7;
  const int units = p.T * cchunks;
  const int n_my = blockIdx.x < units ? (units - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

  griddep_launch();
  if (threadIdx.x == 0) {
    for (int i = 0; i < kInSlots; ++i) {
      mbar_init(s.bar_full + 8u * i, 1);
      mbar_init(s.bar_in_empty + 8u * i, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(s.bar_acc_full + 8u * b, 1);
      mbar_init(s.bar_acc_empty + 8u * b, 4);
    }
    *abort_p = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Kronecker matrix (B^T (x) B^T)[xi][ab] (rows of 64 bytes, zero padded; a constant of
  // the plan, never written by a kernel) -> K-major tile with the 64-byte swizzle
  for (int idx = threadIdx.x; idx < NB * 4; idx += kTmThreads)
    *reinterpret_cast<uint4*>(gen + (s.b - base) + sw64_off(idx >> 2, (idx & 3) * 16)) = __ldg(kron + idx);
  fence_async_smem();
  if (warp == 0) tmem_alloc(s.tmem_slot, 2 * ACC);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_p;

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_map(&mapX);
      tma_prefetch_map(&mapV);
      griddep_wait();   // x may be the previous kernel's output; V_q may still be read by it
      auto issue = [&](int i) {
        const int u = blockIdx.x + i * gridDim.x;
        const int tau = u / cchunks, c0 = (u - tau * cchunks) << 7;
        const int tw = tau % p.TW;
        const int th = (tau / p.TW) % p.TH;
        const int n = tau / (p.TW * p.TH);
        const uint32_t sl = (uint32_t)(i % kInSlots);
        mbar_expect_tx(s.bar_full + 8u * sl, (uint32_t)T2 * 128u);
        tma_load_4d(s.in + sl * L::kInSlot, &mapX, s.bar_full + 8u * sl, c0, tw * M - 1, th * M - 1, n);
      };
      for (int i = 0; i < n_my && i < kInSlots; ++i) issue(i);
      const uint32_t idesc = idesc_i8_a_mn(128, NB);
      const uint64_t db = desc_kmajor_sw64(s.b);
      bool ok = true;
      for (int i = 0; i < n_my; ++i) {
        // refill the slot of unit i-1 once its MMAs have read it
        if (i >= 1 && i - 1 + kInSlots < n_my) {
          const uint32_t sl = (uint32_t)((i - 1) % kInSlots);
          if (!mbar_wait<false>(s.bar_in_empty + 8u * sl, (uint32_t)((i - 1) / kInSlots) & 1u, abort_p)) { ok = false; break; }
          issue(i - 1 + kInSlots);
        }
        const uint32_t sl = (uint32_t)(i % kInSlots);
        if (!mbar_wait<false>(s.bar_full + 8u * sl, (uint32_t)(i / kInSlots) & 1u, abort_p)) { ok = false; break; }
        const int b = i & 1;
        if (!mbar_wait<false>(s.bar_acc_empty + 8u * b, ((uint32_t)(i >> 1) & 1u) ^ 1u, abort_p)) { ok = false; break; }
        tc_fence_after();
        const uint64_t da = desc_mnmajor_sw128(s.in + sl * L::kInSlot);
#pragma unroll
        for (int ks = 0; ks < KROWS / 32; ++ks)
          mma_i8(tmem_base + (uint32_t)(b * ACC), da + (uint64_t)(ks * 256), db + (uint64_t)(ks * 2),
                 idesc, ks != 0 ? 1u : 0u);
        mma_commit(s.bar_in_empty + 8u * sl);
        mma_commit(s.bar_acc_full + 8u * b);
      }
      if (!ok) *abort_p = 1u;
    }
  } else {
    const int et = threadIdx.x - 32;            // 0..127 within the epilogue group
    const int quad = warp & 3;                  // tensor-memory lane quadrant of this warp
    const int c = quad * 32 + lane;             // channel within the chunk
    const float lo = __fadd_rn(p.lo_V, kMagic), hi = __fadd_rn(p.hi_V, kMagic);
    for (int i = 0; i < n_my; ++i) {
      const int u = blockIdx.x + i * gridDim.x;
      const int tau = u / cchunks, c0 = (u - tau * cchunks) << 7;
      const int b = i & 1;
      if (et == 0) {
        if (!mbar_wait<false>(s.bar_acc_full + 8u * b, (uint32_t)(i >> 1) & 1u, abort_p)) *abort_p = 1u;
        bulk_wait_read_n<1>();                  // the store that last read staging tile b is done
      }
      epi_barrier();
      if (*abort_p != 0u) break;
      (void)mbar_try_wait(s.bar_acc_full + 8u * b, (uint32_t)(i >> 1) & 1u);
      tc_fence_after();
      const uint32_t tacc = tmem_base + (uint32_t)(b * ACC) + ((uint32_t)(quad * 32) << 16);
      uint32_t v[NB >= 32 ? 36 : 16];
      if constexpr (M == 4) {
        uint32_t r0[32], r1[4];
        tmem_ld32(tacc, r0);
        tmem_ld4(tacc + 32u, r1);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = r0[j];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[32 + j] = r1[j];
      } else {
        uint32_t r0[16];
        tmem_ld16(tacc, r0);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = r0[j];
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s.bar_acc_empty + 8u * b);
      const uint32_t wr = s.out + (uint32_t)b * L::kOut + (uint32_t)c;
      // all codes first (independent chains the compiler can interleave), then the stores
#pragma unroll
      for (int xi = 0; xi < T2; ++xi)
        v[xi] = __float_as_uint(fminf(fmaxf(__fmaf_rn(__int2float_rn((int)v[xi]), p.mult_V, kMagic), lo), hi));
      uint8_t* sp = gen + (wr - base);
#pragma unroll
      for (int xi = 0; xi < T2; ++xi) sp[xi * 128] = (uint8_t)v[xi];
      fence_async_smem();
      epi_barrier();
      if (et == 0) {
        tma_store_3d(&mapV, s.out + (uint32_t)b * L::kOut, c0, tau, 0);
        bulk_commit();
      }
    }
    if (et == 0) bulk_wait_all();
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_p != 0u && threadIdx.x == 0) atomicExch(status, -6);  // WINO_ERR_TIMEOUT
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 2 * ACC);
  }
}

// ---------------------------------------------------------------------------
// Output transform.  m_q [t*t][T][K] -> y int8 [N][H][W][K].  A block keeps one
// 128-channel chunk (its bias values stay in registers) and walks over tiles.
// ---------------------------------------------------------------------------
template <int M>
__global__ void __launch_bounds__(kTmThreads)
k_output_transform_mma(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap mapM,
                       const __grid_constant__ CUtensorMap mapY, const uint4* __restrict__ kron,
                       const float* __restrict__ bias, float s_Y, int* __restrict__ status) {
  constexpr int T_ = M + 2, T2 = T_ * T_, MM = M * M;
  constexpr int KROWS = (T2 + 31) / 32 * 32;
  constexpr int NB = 16;                           // MMA N: m*m = 4 or 16 outputs, padded to 16
  constexpr int ACC = 32;
  using L = TmSmem<KROWS, NB, MM * 128>;
  static_assert(L::kTotal + 1024 <= 56 * 1024, "shared-memory request too small");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const L s(base);
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gen + (s.tmem_slot - base));
  volatile uint32_t* abort_p = reinterpret_cast<volatile uint32_t*>(gen + (s.abort_slot - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kchunks = p.K >> 7;
  // gridDim.x is a multiple of kchunks: block -> (chunk, first tile), tiles strided
  const int kc = blockIdx.x % kchunks;
  const int t0 = blockIdx.x / kchunks, tstride = gridDim.x / kchunks;
  const int n_my = t0 < p.T ? (p.T - 1 - t0) / tstride + 1 : 0;
  const int k0 = kc << 7;

  griddep_launch();
  if (threadIdx.x == 0) {
    for (int i = 0; i < kInSlots; ++i) {
      mbar_init(s.bar_full + 8u * i, 1);
      mbar_init(s.bar_in_empty + 8u * i, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(s.bar_acc_full + 8u * b, 1);
      mbar_init(s.bar_acc_empty + 8u * b, 4);
    }
    *abort_p = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Kronecker matrix (A^T (x) A^T)[pq][xi] -> K-major tile with the 64-byte swizzle
  for (int idx = threadIdx.x; idx < NB * 4; idx += kTmThreads)
    *reinterpret_cast<uint4*>(gen + (s.b - base) + sw64_off(idx >> 2, (idx & 3) * 16)) = __ldg(kron + idx);
  fence_async_smem();
  if (warp == 0) tmem_alloc(s.tmem_slot, 2 * ACC);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_p;

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_map(&mapM);
      tma_prefetch_map(&mapY);
      griddep_wait();
      auto issue = [&](int i) {
        const int tau = t0 + i * tstride;
        const uint32_t sl = (uint32_t)(i % kInSlots);
        mbar_expect_tx(s.bar_full + 8u * sl, (uint32_t)T2 * 128u);
        tma_load_3d(s.in + sl * L::kInSlot, &mapM, s.bar_full + 8u * sl, k0, tau, 0);
      };
      for (int i = 0; i < n_my && i < kInSlots; ++i) issue(i);
      const uint32_t idesc = idesc_i8_a_mn(128, NB);
      const uint64_t db = desc_kmajor_sw64(s.b);
      bool ok = true;
      for (int i = 0; i < n_my; ++i) {
        if (i >= 1 && i - 1 + kInSlots < n_my) {
          const uint32_t sl = (uint32_t)((i - 1) % kInSlots);
          if (!mbar_wait<false>(s.bar_in_empty + 8u * sl, (uint32_t)((i - 1) / kInSlots) & 1u, abort_p)) { ok = false; break; }
          issue(i - 1 + kInSlots);
        }
        const uint32_t sl = (uint32_t)(i % kInSlots);
        if (!mbar_wait<false>(s.bar_full + 8u * sl, (uint32_t)(i / kInSlots) & 1u, abort_p)) { ok = false; break; }
        const int b = i & 1;
        if (!mbar_wait<false>(s.bar_acc_empty + 8u * b, ((uint32_t)(i >> 1) & 1u) ^ 1u, abort_p)) { ok = false; break; }
        tc_fence_after();
        const uint64_t da = desc_mnmajor_sw128(s.in + sl * L::kInSlot);
#pragma unroll
        for (int ks = 0; ks < KROWS / 32; ++ks)
          mma_i8(tmem_base + (uint32_t)(b * ACC), da + (uint64_t)(ks * 256), db + (uint64_t)(ks * 2),
                 idesc, ks != 0 ? 1u : 0u);
        mma_commit(s.bar_in_empty + 8u * sl);
        mma_commit(s.bar_acc_full + 8u * b);
      }
      if (!ok) *abort_p = 1u;
    }
  } else {
    const int et = threadIdx.x - 32;
    const int quad = warp & 3;
    const int kl = quad * 32 + lane;            // channel within the chunk
    float b_scaled = 0.0f;
    if (bias != nullptr) b_scaled = (float)((double)__ldg(bias + k0 + kl) / (double)s_Y);
    for (int i = 0; i < n_my; ++i) {
      const int tau = t0 + i * tstride;
      const int b = i & 1;
      if (et == 0) {
        if (!mbar_wait<false>(s.bar_acc_full + 8u * b, (uint32_t)(i >> 1) & 1u, abort_p)) *abort_p = 1u;
        bulk_wait_read_n<1>();
      }
      epi_barrier();
      if (*abort_p != 0u) break;
      (void)mbar_try_wait(s.bar_acc_full + 8u * b, (uint32_t)(i >> 1) & 1u);
      tc_fence_after();
      const uint32_t tacc = tmem_base + (uint32_t)(b * ACC) + ((uint32_t)(quad * 32) << 16);
      uint32_t v[16];
      tmem_ld16(tacc, v);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s.bar_acc_empty + 8u * b);
      const uint32_t wr = s.out + (uint32_t)b * L::kOut + (uint32_t)kl;
#pragma unroll
      for (int q = 0; q < MM; ++q) {
        const float yf = __fmaf_rn(__int2float_rn((int)v[q]), p.mult_Y, b_scaled);
        const float r = __fadd_rn(fminf(fmaxf(yf, p.lo_Y), p.hi_Y), kMagic);
        v[q] = (uint32_t)(magic_to_int(r) + p.z_Y);
      }
      uint8_t* sp = gen + (wr - base);
#pragma unroll
      for (int q = 0; q < MM; ++q) sp[q * 128] = (uint8_t)v[q];
      fence_async_smem();
      epi_barrier();
      if (et == 0) {
        const int tw = tau % p.TW;
        const int th = (tau / p.TW) % p.TH;
        const int n = tau / (p.TW * p.TH);
        tma_store_4d(&mapY, s.out + (uint32_t)b * L::kOut, k0, tw * M, th * M, n);
        bulk_commit();
      }
    }
    if (et == 0) bulk_wait_all();
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_p != 0u && threadIdx.x == 0) atomicExch(status, -6);  // WINO_ERR_TIMEOUT
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 2 * ACC);
  }
}

// ---------------------------------------------------------------------------
// Launchers.  Four blocks per SM (their tensor-memory allocations, 4 x 128 or
// 4 x 64 columns, fit the 512 columns of an SM; the shared-memory request keeps
// a fifth block out).
// ---------------------------------------------------------------------------
namespace {
constexpr size_t kTmSmemRequest = 56 * 1024;   // > 227 KB / 5

template <int M>
int input_mma_launch(const Params& p, const LaunchOpt& o, const CUtensorMap& mapX,
                     const CUtensorMap& mapV, const void* kron, int num_sms, int* status,
                     cudaStream_t st) {
  static DeviceOnce once;
  if (int rc = set_max_smem(once, o.device, k_input_transform_mma<M>, kTmSmemRequest)) return rc;
  const int units = p.T * (p.C >> 7);
  int grid = 4 * num_sms;
  if (grid > units) grid = units;
  return launch_kernel(k_input_transform_mma<M>, dim3((unsigned)grid), dim3(kTmThreads),
                       kTmSmemRequest, st, o.pdl, p, mapX, mapV,
                       reinterpret_cast<const uint4*>(kron), status);
}
template <int M>
int output_mma_launch(const Params& p, const LaunchOpt& o, const CUtensorMap& mapM,
                      const CUtensorMap& mapY, const void* kron, const float* bias, float s_Y,
                      int num_sms, int* status, cudaStream_t st) {
  static DeviceOnce once;
  if (int rc = set_max_smem(once, o.device, k_output_transform_mma<M>, kTmSmemRequest)) return rc;
  const int kchunks = p.K >> 7;
  int per_chunk = (4 * num_sms) / kchunks;
  if (per_chunk > p.T) per_chunk = p.T;
  if (per_chunk < 1) per_chunk = 1;
  return launch_kernel(k_output_transform_mma<M>, dim3((unsigned)(per_chunk * kchunks)),
                       dim3(kTmThreads), kTmSmemRequest, st, o.pdl, p, mapM, mapY,
                       reinterpret_cast<const uint4*>(kron), bias, s_Y, status);
}
}  // namespace

bool transform_mma_supported(const Params& p, bool std_mats, int channels) {
  return std_mats && (p.m == 2 || p.m == 4) && channels % 128 == 0;
}

// Host side: the two Kronecker matrices of the plan's tile size as int8 rows of 64 bytes
// (kKronInRows rows for the input side, then kKronOutRows for the output side).
void fill_kronecker_tables(int m, int8_t* dst) {
  std::memset(dst, 0, kKronBytes);
  const int t = m + 2, t2 = t * t, mm = m * m;
  auto bt = [&](int i, int k) { return m == 2 ? (int)std_bt<2>(i, k) : (int)std_bt<4>(i, k); };
  auto at = [&](int i, int k) { return m == 2 ? (int)std_at<2>(i, k) : (int)std_at<4>(i, k); };
  for (int xi = 0; xi < t2; ++xi)
    for (int ab = 0; ab < t2; ++ab)
      dst[xi * 64 + ab] = (int8_t)(bt(xi / t, ab / t) * bt(xi % t, ab % t));
  int8_t* out = dst + kKronInRows * 64;
  for (int pq = 0; pq < mm; ++pq)
    for (int xi = 0; xi < t2; ++xi)
      out[pq * 64 + xi] = (int8_t)(at(pq / m, xi / t) * at(pq % m, xi % t));
}

int launch_input_transform_mma(const Params& p, const LaunchOpt& o, const CUtensorMap& mapX,
                               const CUtensorMap& mapV, const void* kron, int num_sms, int* status,
                               cudaStream_t st) {
  return p.m == 2 ? input_mma_launch<2>(p, o, mapX, mapV, kron, num_sms, status, st)
                  : input_mma_launch<4>(p, o, mapX, mapV, kron, num_sms, status, st);
}
int launch_output_transform_mma(const Params& p, const LaunchOpt& o, const CUtensorMap& mapM,
                                const CUtensorMap& mapY, const void* kron, const float* bias,
                                float s_Y, int num_sms, int* status, cudaStream_t st) {
  const void* kout = reinterpret_cast<const uint8_t*>(kron) + kKronInRows * 64;
  return p.m == 2 ? output_mma_launch<2>(p, o, mapM, mapY, kout, bias, s_Y, num_sms, status, st)
                  : output_mma_launch<4>(p, o, mapM, mapY, kout, bias, s_Y, num_sms, status, st);
}

}  // namespace wino
