// The whole Winograd-aware layer (paper: Eq. 1 with the quantizers of Fig. 2) in
// ONE persistent launch, for the Cook-Toom matrices of F2 and F4 with channel
// counts that are multiples of 128:
//
//   phase A  input transform on the tensor cores (patch x Kronecker matrix, see
//            wino_transforms_mma.cu), Q_V, V_q -> workspace (stays in L2);
//   phase B  the t*t Hadamard-stage GEMMs over channels (tcgen05 kind::i8, TMA
//            operands, int32 accumulators in tensor memory), Q_M, m_q -> workspace;
//   phase C  output transform on the tensor cores, bias, Q_Y, y.
//
// One CTA per SM, every CTA runs A, then B, then C on its share of the units /
// items.  The phases of different CTAs are tied together by counters in global
// memory, one pair per block of 128 tiles ("m-block"):
//   cnt_in[mb]  input-transform units of the m-block whose V_q is stored and visible;
//   cnt_m[mb]   epilogue warps that have stored their share of an item of the m-block.
// A GEMM item waits for cnt_in of its m-block, an output unit for cnt_m of its
// m-block; nothing in phase A waits for another CTA, so the dependency graph has
// no cycle as long as every CTA is resident (the grid is at most one CTA per SM).
// Every wait is bounded; on expiry the kernel records WINO_ERR_TIMEOUT and unwinds.
// The last CTA to finish clears the counters for the next launch.
//
// Warp roles (640 threads):
//   warp 0   TMA loads of the transform units (x patches, later m_q blocks)
//   warp 1   transform MMAs (one lane)
//   warp 2   TMA loads of the GEMM operands (U_q, V_q)
//   warp 3   GEMM MMAs (one lane); owns the tensor-memory allocation
//   warps 4-19  four worker groups of four warps (one per tensor-memory lane
//            quadrant): epilogues of A, B and C, in that order.
// While the workers are still quantizing phase A, warps 2 and 3 already run the
// first GEMM item of the CTA into tensor-memory columns 0..255; the transform
// accumulators live in columns 256..511 until phase A is done.
#include "wino_launch.h"
#include "wino_ptx.cuh"

namespace wino {

namespace {

constexpr int kFlThreads = 640;
constexpr int kSlots = 6;            // transform units in flight per CTA
constexpr long long kFlagWaitCycles = 600000000ll;   // ~0.3 s

__device__ __forceinline__ uint64_t fl_desc_kmajor_sw64(uint32_t a) {
  return (uint64_t)((a & 0x3FFFFu) >> 4) | (1ull << 16) | (32ull << 32) | (1ull << 46) | (4ull << 61);
}
__device__ __forceinline__ uint32_t fl_sw64_off(int row, int byte) {
  const int chunk = (byte >> 4) ^ ((row >> 1) & 3);
  return (uint32_t)(row * 64 + chunk * 16 + (byte & 15));
}
__device__ __forceinline__ uint64_t fl_desc_mnmajor_sw128(uint32_t a) {
  return (uint64_t)((a & 0x3FFFFu) >> 4) | (64ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
__host__ __device__ constexpr uint32_t fl_idesc_a_mn(int M, int N) {
  return (2u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void fl_tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void fl_tmem_ld4(uint32_t taddr, uint32_t (&r)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr)
               : "memory");
}
template <int N>
__device__ __forceinline__ void fl_bulk_wait_n() {       // all but the N newest groups complete
  asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void fl_bulk_wait_read_n() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void group_barrier(int g) {
  asm volatile("bar.sync %0, 128;" ::"r"(g + 1) : "memory");
}
__device__ __forceinline__ void fence_async_global() {
  asm volatile("fence.proxy.async.global;" ::: "memory");
}
__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Publish: everything this thread has observed as complete becomes visible to a
// thread that reads the counter with acquire semantics.
__device__ __forceinline__ void flag_add(unsigned* p) {
  fence_async_global();
  asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}
// Bounded wait for *p >= target; then order the acquire before later TMA reads.
__device__ __forceinline__ bool flag_wait(const unsigned* p, unsigned target,
                                          volatile uint32_t* abort_flag) {
  if (ld_acquire(p) < target) {
    const long long t0 = clock64();
    for (uint32_t i = 1;; ++i) {
      if (ld_acquire(p) >= target) break;
      __nanosleep(i > 16u ? 200u : 40u);
      if ((i & 63u) == 0u) {
        if (*abort_flag != 0u) return false;
        if (clock64() - t0 > kFlagWaitCycles) return false;
      }
    }
  }
  fence_async_global();
  return true;
}

struct FusedArgs {
  int BN;             // GEMM block width (128 or 256)
  int stages;         // GEMM ring stages
  int n_mblk, n_nblk, n_items;
  int units_a, units_c;   // T * C/128, T * K/128
  unsigned* cnt_in;   // [n_mblk]
  unsigned* cnt_m;    // [n_mblk]
  unsigned* ticket;   // CTAs that have finished
};

}  // namespace

template <int M>
__global__ void __launch_bounds__(kFlThreads, 1)
k_layer_fused(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap mapX,
              const __grid_constant__ CUtensorMap mapVst, const __grid_constant__ CUtensorMap mapV,
              const __grid_constant__ CUtensorMap mapU, const __grid_constant__ CUtensorMap mapMld,
              const __grid_constant__ CUtensorMap mapY, const FusedArgs a,
              const uint4* __restrict__ kron, int8_t* __restrict__ mq, const float* __restrict__ bias,
              float s_Y, int* __restrict__ status) {
  constexpr int T_ = M + 2, T2 = T_ * T_, MM = M * M;
  constexpr int KROWS = (T2 + 31) / 32 * 32;          // transform MMA K: 32 (F2) or 64 (F4)
  constexpr int NB_IN = (T2 + 15) / 16 * 16;          // transform MMA N, input side: 16 or 48
  constexpr int NB_OUT = 16;
  constexpr uint32_t kSlotBytes = KROWS * 128;
  constexpr uint32_t kStageOut = T2 * 128;             // staging tile (input side is the larger)
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  // ---- shared-memory map ----
  const uint32_t a_bytes = kBM * kStageK, b_bytes = (uint32_t)a.BN * kStageK;
  const uint32_t stage_bytes = a_bytes + b_bytes;
  const uint32_t s_ring = base;
  const uint32_t s_slots = s_ring + (uint32_t)a.stages * stage_bytes;   // kSlots x kSlotBytes
  const uint32_t s_kron = s_slots + kSlots * kSlotBytes;                // 64 rows x 64 B
  const uint32_t s_stage = s_kron + 4096u;                              // 4 groups x 2 x kStageOut
  const uint32_t s_bias = s_stage + 8u * kStageOut;                     // K floats (<= 1040)
  const uint32_t s_bar = s_bias + 4224u;
  const uint32_t bar_full = s_bar;                        // stages (<= 8)
  const uint32_t bar_empty = bar_full + 64u;
  const uint32_t bar_acc_full = bar_empty + 64u;          // 2
  const uint32_t bar_acc_empty = bar_acc_full + 16u;      // 2
  const uint32_t bar_tin_full = bar_acc_empty + 16u;      // kSlots
  const uint32_t bar_tin_empty = bar_tin_full + 8u * kSlots;
  const uint32_t bar_tacc_full = bar_tin_empty + 8u * kSlots;   // 4
  const uint32_t bar_tacc_empty = bar_tacc_full + 32u;          // 4
  const uint32_t bar_tr_done = bar_tacc_empty + 32u;            // 1
  const uint32_t bar_gemm_done = bar_tr_done + 8u;              // 1
  const uint32_t tmem_slot = bar_gemm_done + 8u;
  const uint32_t abort_slot = tmem_slot + 4u;
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gen + (tmem_slot - base));
  volatile uint32_t* abort_p = reinterpret_cast<volatile uint32_t*>(gen + (abort_slot - base));
  float* bias_s = reinterpret_cast<float*>(gen + (s_bias - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grid = (int)gridDim.x, cta = (int)blockIdx.x;
  const int cchunks = p.C >> 7, kchunks = p.K >> 7;
  const int KB = p.C >> 7;                              // GEMM k-stages per item
  const int nA = cta < a.units_a ? (a.units_a - 1 - cta) / grid + 1 : 0;
  const int nC = cta < a.units_c ? (a.units_c - 1 - cta) / grid + 1 : 0;
  const int nI = cta < a.n_items ? (a.n_items - 1 - cta) / grid + 1 : 0;
  const int per_mb = T2 * a.n_nblk;                     // items per m-block
  const int cbuf = nI & 1;                              // GEMM accumulator buffer phase C borrows

  griddep_launch();
  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      mbar_init(bar_full + 8u * s, 1);
      mbar_init(bar_empty + 8u * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_acc_full + 8u * b, 1);
      mbar_init(bar_acc_empty + 8u * b, 16);
    }
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(bar_tin_full + 8u * s, 1);
      mbar_init(bar_tin_empty + 8u * s, 1);
    }
    for (int g = 0; g < 4; ++g) {
      mbar_init(bar_tacc_full + 8u * g, 1);
      mbar_init(bar_tacc_empty + 8u * g, 4);
    }
    mbar_init(bar_tr_done, 16);
    mbar_init(bar_gemm_done, 16);
    *abort_p = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Kronecker tables (plan constants): rows 0..47 input side, 48..63 output side
  for (int idx = threadIdx.x; idx < 64 * 4; idx += kFlThreads)
    *reinterpret_cast<uint4*>(gen + (s_kron - base) + fl_sw64_off(idx >> 2, (idx & 3) * 16)) =
        __ldg(kron + idx);
  fence_async_smem();
  if (warp == 3) tmem_alloc(tmem_slot, 512u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_p;

  if (warp == 0) {
    // =============== transform loads: x patches (A), then m_q blocks (C) ===============
    if (lane == 0) {
      tma_prefetch_map(&mapX);
      tma_prefetch_map(&mapMld);
      griddep_wait();
      bool ok = true;
      for (int jj = 0; jj < nA + nC && ok; ++jj) {
        const uint32_t sl = (uint32_t)(jj % kSlots);
        if (jj >= kSlots &&
            !mbar_wait(bar_tin_empty + 8u * sl, (uint32_t)(jj / kSlots - 1) & 1u, abort_p)) { ok = false; break; }
        mbar_expect_tx(bar_tin_full + 8u * sl, (uint32_t)T2 * 128u);
        if (jj < nA) {
          const int u = cta + jj * grid;
          const int tau = u / cchunks, c0 = (u - tau * cchunks) << 7;
          const int tw = tau % p.TW;
          const int th = (tau / p.TW) % p.TH;
          const int n = tau / (p.TW * p.TH);
          tma_load_4d(s_slots + sl * kSlotBytes, &mapX, bar_tin_full + 8u * sl, c0, tw * M - 1, th * M - 1, n);
        } else {
          const int u = cta + (jj - nA) * grid;
          const int tau = u / kchunks, k0 = (u - tau * kchunks) << 7;
          const int mb = tau >> 7;
          if (!flag_wait(a.cnt_m + mb, (unsigned)(per_mb * 16), abort_p)) { ok = false; break; }
          tma_load_3d(s_slots + sl * kSlotBytes, &mapMld, bar_tin_full + 8u * sl, k0, tau, 0);
        }
      }
      if (!ok) *abort_p = 1u;
    }
  } else if (warp == 1) {
    // =============== transform MMAs ===============
    if (lane == 0) {
      const uint32_t idesc_in = fl_idesc_a_mn(128, NB_IN), idesc_out = fl_idesc_a_mn(128, NB_OUT);
      const uint64_t db_in = fl_desc_kmajor_sw64(s_kron);
      const uint64_t db_out = fl_desc_kmajor_sw64(s_kron + 48u * 64u);
      bool ok = true;
      for (int jj = 0; jj < nA + nC && ok; ++jj) {
        const bool ph_c = jj >= nA;
        if (jj == nA && nI > 0) {
          // phase C borrows the columns of a GEMM accumulator buffer: every item of this
          // CTA must have been drained first.  (A parity wait on bar_acc_empty would not
          // do: this thread gets here long before the items, more than one phase ahead.)
          if (!mbar_wait(bar_gemm_done, 0u, abort_p)) { ok = false; break; }
        }
        const uint32_t sl = (uint32_t)(jj % kSlots);
        const int jl = ph_c ? jj - nA : jj;
        const int g = jl & 3;
        // how often group g's accumulator has been used before this unit
        const uint32_t use = (uint32_t)(jl >> 2) + (ph_c && nA > g ? (uint32_t)((nA - g + 3) >> 2) : 0u);
        if (!mbar_wait(bar_tin_full + 8u * sl, (uint32_t)(jj / kSlots) & 1u, abort_p)) { ok = false; break; }
        if (!mbar_wait(bar_tacc_empty + 8u * g, (use & 1u) ^ 1u, abort_p)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tcol = tmem_base + (uint32_t)((ph_c ? cbuf : 1) * 256 + g * 64);
        const uint64_t da = fl_desc_mnmajor_sw128(s_slots + sl * kSlotBytes);
#pragma unroll
        for (int ks = 0; ks < KROWS / 32; ++ks)
          mma_i8(tcol, da + (uint64_t)(ks * 256), (ph_c ? db_out : db_in) + (uint64_t)(ks * 2),
                 ph_c ? idesc_out : idesc_in, ks != 0 ? 1u : 0u);
        mma_commit(bar_tin_empty + 8u * sl);
        mma_commit(bar_tacc_full + 8u * g);
      }
      if (!ok) *abort_p = 1u;
    }
  } else if (warp == 2) {
    // =============== GEMM operand loads ===============
    if (lane == 0) {
      tma_prefetch_map(&mapV);
      tma_prefetch_map(&mapU);
      bool ok = true;
      int s = 0; uint32_t ph = 0;
      // U_q is a constant of the layer: the first item's weight tiles are fetched before the
      // wait on the preceding kernel; the V_q halves of the same stages follow the counter
      int pre = 0;
      if (nI > 0) {
        const int it = cta;
        const int rem = it % per_mb, xi = rem / a.n_nblk, nb = rem % a.n_nblk;
        pre = KB < a.stages ? KB : a.stages;
        for (int kb = 0; kb < pre; ++kb) {
          mbar_expect_tx(bar_full + 8u * kb, stage_bytes);
          tma_load_3d(s_ring + (uint32_t)kb * stage_bytes + a_bytes, &mapU, bar_full + 8u * kb,
                      kb * kStageK, nb * a.BN, xi);
        }
      }
      griddep_wait();
      for (int li = 0; li < nI && ok; ++li) {
        const int it = cta + li * grid;
        const int mb = it / per_mb, rem = it - mb * per_mb;
        const int xi = rem / a.n_nblk, nb = rem - xi * a.n_nblk;
        const int tiles = min(kBM, p.T - mb * kBM);
        if (!flag_wait(a.cnt_in + mb, (unsigned)(tiles * cchunks), abort_p)) { ok = false; break; }
        for (int kb = 0; kb < KB; ++kb) {
          const uint32_t sa = s_ring + (uint32_t)s * stage_bytes;
          if (li == 0 && kb < pre) {
            // stage already armed and its U_q half in flight
          } else {
            if (!mbar_wait(bar_empty + 8u * s, ph ^ 1u, abort_p)) { ok = false; break; }
            mbar_expect_tx(bar_full + 8u * s, stage_bytes);
            tma_load_3d(sa + a_bytes, &mapU, bar_full + 8u * s, kb * kStageK, nb * a.BN, xi);
          }
          tma_load_3d(sa, &mapV, bar_full + 8u * s, kb * kStageK, mb * kBM, xi);
          if (++s == a.stages) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) *abort_p = 1u;
    }
  } else if (warp == 3) {
    // =============== GEMM MMAs ===============
    if (lane == 0) {
      const uint32_t idesc = make_idesc_i8(kBM, a.BN);
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      for (int li = 0; li < nI && ok; ++li) {
        const int buf = li & 1;
        const uint32_t aph = (uint32_t)(li >> 1) & 1u;
        if (!mbar_wait(bar_acc_empty + 8u * buf, aph ^ 1u, abort_p)) { ok = false; break; }
        // columns 256..511 hold the transform accumulators until phase A is over
        if (li == 1 && !mbar_wait(bar_tr_done, 0u, abort_p)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tacc = tmem_base + (uint32_t)(buf * 256);
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(bar_full + 8u * s, ph, abort_p)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = s_ring + (uint32_t)s * stage_bytes;
          const uint64_t da = make_desc_sw128(sa), db = make_desc_sw128(sa + a_bytes);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_i8(tacc, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
          mma_commit(bar_empty + 8u * s);
          if (++s == a.stages) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        mma_commit(bar_acc_full + 8u * buf);
      }
      if (!ok) *abort_p = 1u;
    }
  } else {
    // =============== workers ===============
    const int g = (warp - 4) >> 2;              // group
    const int quad = warp & 3;                  // tensor-memory lane quadrant
    const int et = threadIdx.x - 128 - g * 128; // 0..127 inside the group
    const bool leader = et == 0;
    const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
    const int ch = quad * 32 + lane;            // channel inside a 128-channel chunk / row inside an m-block
    griddep_wait();                             // bias may be the previous kernel's output
    for (int k = threadIdx.x - 128; k < p.K; k += kFlThreads - 128)
      bias_s[k] = bias != nullptr ? (float)((double)__ldg(bias + k) / (double)s_Y) : 0.0f;
    asm volatile("bar.sync 5, 512;" ::: "memory");
    uint32_t tuse = 0;                          // uses of this group's transform accumulator
    bool ok = true;

    // ---------------- phase A ----------------
    {
      const float lo = __fadd_rn(p.lo_V, kMagic), hi = __fadd_rn(p.hi_V, kMagic);
      int prev_mb = -1, jj = 0;
      for (int j = g; j < nA; j += 4, ++jj, ++tuse) {
        const int u = cta + j * grid;
        const int tau = u / cchunks, c0 = (u - tau * cchunks) << 7;
        if (leader && !mbar_wait(bar_tacc_full + 8u * g, tuse & 1u, abort_p)) *abort_p = 1u;
        group_barrier(g);
        if (*abort_p != 0u) { ok = false; break; }
        (void)mbar_try_wait(bar_tacc_full + 8u * g, tuse & 1u);
        tc_fence_after();
        const uint32_t tacc = tmem_base + (uint32_t)(256 + g * 64) + lane_off;
        constexpr int N0 = M == 4 ? 32 : 16, N1 = M == 4 ? 4 : 1;
        uint32_t r0[N0], r1[4];
        if constexpr (M == 4) {
          tmem_ld32(tacc, r0);
          fl_tmem_ld4(tacc + 32u, r1);
        } else {
          fl_tmem_ld16(tacc, r0);
        }
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tacc_empty + 8u * g);
        const uint32_t st = s_stage + (uint32_t)(g * 2 + (jj & 1)) * kStageOut;
        auto put = [&](int xi, uint32_t acc) {
          const float r = fminf(fmaxf(__fmaf_rn(__int2float_rn((int)acc), p.mult_V, kMagic), lo), hi);
          asm volatile("st.shared.u8 [%0], %1;" ::"r"(st + (uint32_t)(xi * 128 + ch)), "r"(__float_as_uint(r))
                       : "memory");
        };
#pragma unroll
        for (int q = 0; q < N0; ++q) put(q, r0[q]);
        if constexpr (M == 4) {
#pragma unroll
          for (int q = 0; q < N1; ++q) put(32 + q, r1[q]);
        }
        fence_async_smem();
        group_barrier(g);
        if (leader) {
          tma_store_3d(&mapVst, st, c0, tau, 0);
          bulk_commit();
          fl_bulk_wait_n<1>();                  // the previous unit's store is complete
          if (prev_mb >= 0) flag_add(a.cnt_in + prev_mb);
          prev_mb = tau >> 7;
        }
      }
      if (leader) {
        fl_bulk_wait_n<0>();
        if (prev_mb >= 0) flag_add(a.cnt_in + prev_mb);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tr_done);
    }

    // ---------------- phase B: Q_M epilogue of the GEMM items ----------------
    if (ok) {
      const float lo = __fadd_rn(p.lo_M, kMagic), hi = __fadd_rn(p.hi_M, kMagic);
      for (int li = 0; li < nI; ++li) {
        const int it = cta + li * grid;
        const int mb = it / per_mb, rem = it - mb * per_mb;
        const int xi = rem / a.n_nblk, nb = rem - xi * a.n_nblk;
        const int buf = li & 1;
        const uint32_t aph = (uint32_t)(li >> 1) & 1u;
        if (!__all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8u * buf, aph, abort_p))) {
          *abort_p = 1u;
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t tacc = tmem_base + (uint32_t)(buf * 256) + lane_off;
        const int tau = mb * kBM + ch;
        for (int col = g * 32; col < a.BN; col += 128) {
          uint32_t r[32];
          __syncwarp();
          tmem_ld32(tacc + (uint32_t)col, r);
          tmem_ld_wait();
          const int k0 = nb * a.BN + col;
          if (tau < p.T && k0 < p.K) {
          uint32_t w[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            float f[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
              f[e] = fminf(fmaxf(__fmaf_rn(__int2float_rn((int)r[4 * q + e]), p.mult_M, kMagic), lo), hi);
            const uint32_t l2 = __byte_perm(__float_as_uint(f[0]), __float_as_uint(f[1]), 0x0040u);
            const uint32_t h2 = __byte_perm(__float_as_uint(f[2]), __float_as_uint(f[3]), 0x0040u);
            w[q] = __byte_perm(l2, h2, 0x5410u);
          }
          uint4* dst = reinterpret_cast<uint4*>(mq + ((long)xi * p.T + tau) * p.K + k0);
          dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
          dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(bar_acc_empty + 8u * buf);
          __threadfence();
          flag_add(a.cnt_m + mb);
        }
      }
    }

    __syncwarp();
    if (lane == 0) mbar_arrive(bar_gemm_done);

    // ---------------- phase C ----------------
    if (ok) {
      int jj = 0;
      for (int j = g; j < nC; j += 4, ++jj, ++tuse) {
        const int u = cta + j * grid;
        const int tau = u / kchunks, k0 = (u - tau * kchunks) << 7;
        if (leader && !mbar_wait(bar_tacc_full + 8u * g, tuse & 1u, abort_p)) *abort_p = 1u;
        group_barrier(g);
        if (*abort_p != 0u) { ok = false; break; }
        (void)mbar_try_wait(bar_tacc_full + 8u * g, tuse & 1u);
        tc_fence_after();
        uint32_t v[16];
        fl_tmem_ld16(tmem_base + (uint32_t)(cbuf * 256 + g * 64) + lane_off, v);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tacc_empty + 8u * g);
        const float b_scaled = bias_s[k0 + ch];
        const uint32_t st = s_stage + (uint32_t)(g * 2 + (jj & 1)) * kStageOut;
#pragma unroll
        for (int q = 0; q < MM; ++q) {
          const float yf = __fmaf_rn(__int2float_rn((int)v[q]), p.mult_Y, b_scaled);
          const float r = __fadd_rn(fminf(fmaxf(yf, p.lo_Y), p.hi_Y), kMagic);
          const uint32_t code = (uint32_t)(magic_to_int(r) + p.z_Y);
          asm volatile("st.shared.u8 [%0], %1;" ::"r"(st + (uint32_t)(q * 128 + ch)), "r"(code) : "memory");
        }
        fence_async_smem();
        group_barrier(g);
        if (leader) {
          const int tw = tau % p.TW;
          const int th = (tau / p.TW) % p.TH;
          const int n = tau / (p.TW * p.TH);
          tma_store_4d(&mapY, st, k0, tw * M, th * M, n);
          bulk_commit();
          fl_bulk_wait_read_n<1>();
        }
      }
      if (leader) fl_bulk_wait_n<0>();
    }
    if (!ok) *abort_p = 1u;
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    if (*abort_p != 0u) atomicExch(status, -6);  // WINO_ERR_TIMEOUT
    // the last CTA to get here clears the counters for the next launch
    __threadfence();
    if (atomicAdd(a.ticket, 1u) == (unsigned)grid - 1u) {
      for (int i = 0; i < a.n_mblk; ++i) { a.cnt_in[i] = 0u; a.cnt_m[i] = 0u; }
      *a.ticket = 0u;
      __threadfence();
    }
  }
  if (warp == 3) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512u);
  }
}

// ---------------------------------------------------------------------------
// Host side.
// ---------------------------------------------------------------------------
bool layer_fused_supported(const Params& p, bool std_mats) {
  return std_mats && (p.m == 2 || p.m == 4) && p.C % 128 == 0 && p.K % 128 == 0 && p.z_x == 0 &&
         p.qM_enabled != 0 && p.out_dtype == 0 && (p.T + kBM - 1) / kBM <= kFusedMaxMblk;
}

FusedGeom layer_fused_geometry(const Params& p, int num_sms) {
  FusedGeom g;
  g.BN = p.K >= 256 ? 256 : 128;
  const int t2 = p.t * p.t;
  const size_t slot = (size_t)((t2 + 31) / 32 * 32) * 128;
  const size_t fixed = 1024 + kSlots * slot + 4096 + 8 * (size_t)t2 * 128 + 4224 + 512;
  const size_t stage = (size_t)kBM * kStageK + (size_t)g.BN * kStageK;
  int stages = (int)((227 * 1024 - fixed) / stage);
  if (stages > 8) stages = 8;
  g.stages = stages;
  g.smem = fixed + (size_t)stages * stage;
  g.n_mblk = (p.T + kBM - 1) / kBM;
  g.n_nblk = (p.K + g.BN - 1) / g.BN;
  g.n_items = g.n_mblk * t2 * g.n_nblk;
  g.grid = num_sms;
  return g;
}

namespace {
template <int M>
int fused_launch(const Params& p, const LaunchOpt& o, const FusedGeom& g, const FusedMaps& m,
                 const void* kron, unsigned* counters, int8_t* mq, const float* bias, float s_Y,
                 int* status, cudaStream_t st) {
  static DeviceOnce once;
  if (int rc = set_max_smem(once, o.device, k_layer_fused<M>, 227 * 1024)) return rc;
  FusedArgs a;
  a.BN = g.BN; a.stages = g.stages; a.n_mblk = g.n_mblk; a.n_nblk = g.n_nblk; a.n_items = g.n_items;
  a.units_a = p.T * (p.C >> 7);
  a.units_c = p.T * (p.K >> 7);
  a.cnt_in = counters;
  a.cnt_m = counters + kFusedMaxMblk;
  a.ticket = counters + 2 * kFusedMaxMblk;
  return launch_kernel(k_layer_fused<M>, dim3((unsigned)g.grid), dim3(kFlThreads), g.smem, st, o.pdl,
                       p, *m.x, *m.v_store, *m.v_load, *m.u, *m.m_load, *m.y, a,
                       reinterpret_cast<const uint4*>(kron), mq, bias, s_Y, status);
}
}  // namespace

int launch_layer_fused(const Params& p, const LaunchOpt& o, const FusedGeom& g, const FusedMaps& m,
                       const void* kron, unsigned* counters, int8_t* mq, const float* bias,
                       float s_Y, int* status, cudaStream_t st) {
  if (g.stages < 2) return -2;
  return p.m == 2 ? fused_launch<2>(p, o, g, m, kron, counters, mq, bias, s_Y, status, st)
                  : fused_launch<4>(p, o, g, m, kron, counters, mq, bias, s_Y, status, st);
}

}  // namespace wino
