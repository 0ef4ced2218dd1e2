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
//   cnt_m[mb]   16 per GEMM item of the m-block whose m_q is stored and visible.
// A GEMM item waits for cnt_in of its m-block, an output unit for cnt_m of its
// m-block; nothing in phase A waits for another CTA, so the dependency graph has
// no cycle as long as every CTA is resident (the grid is at most one CTA per SM).
// Every wait is bounded; on expiry the kernel records WINO_ERR_TIMEOUT and unwinds.
// The last CTA to finish clears the counters for the next launch.
//
// Warp roles (800 threads):
//   warp 0   TMA loads of the transform units (x patches, later m_q blocks), one lane
//            per shared-memory slot; the other lanes prefetch x into L2
//   warp 1   transform MMAs, one lane per worker group
//   warp 2   TMA loads of the GEMM operands (U_q, V_q)
//   warp 3   GEMM MMAs (one lane); owns the tensor-memory allocation
//   warp 4   bias / s_Y table at the start, then publisher of cnt_m
//   warps 5-8   one store thread per worker group: TMA stores of the group's staging
//            tile (V_q, later y) and the cnt_in updates.  A store needs the better
//            part of a microsecond to be complete and visible device-wide; these
//            threads, which no arithmetic waits for, pay for that.
//   warps 9-24  four worker groups of four warps (one per tensor-memory lane
//            quadrant): epilogues of A, B and C, in that order.
// A unit's position jj in the CTA's list (A units first, then C units) fixes its worker
// group (jj % 4) and its shared-memory slot (jj % 8), so a slot and an accumulator are
// always reused by the same lanes in program order: no waiter is ever more than one
// barrier phase behind what it waits for.
// While the workers are still quantizing phase A, warps 2 and 3 already run the
// first GEMM item of the CTA into tensor-memory columns 0..255; the transform
// accumulators live in columns 256..511 until phase A is done.
#include "wino_launch.h"
#include "wino_ptx.cuh"

namespace wino {

namespace {

constexpr int kFlThreads = 800;
constexpr int kFlWorker0 = 288;      // first worker thread
constexpr int kSlots = 8;            // transform units in flight per CTA (a multiple of 4)
constexpr int kPrefetchUnits = 96;   // units whose input is requested into L2 at the start
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
// Counter update.  Relaxed on purpose: the updating thread issues ONE __threadfence()
// before its updates (fence + relaxed write = release) instead of paying for a fence
// inside every update (a release update costs ~1500 cycles each).
__device__ __forceinline__ void flag_add(unsigned* p, unsigned v) {
  asm volatile("red.relaxed.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Bounded wait for *p >= target; then order the acquire before later TMA reads.
__device__ __forceinline__ bool flag_wait(const unsigned* p, unsigned target,
                                          volatile uint32_t* abort_flag) {
  if (ld_acquire(p) < target) {
    const long long t0 = clock64();
    for (uint32_t i = 1;; ++i) {
      if (ld_acquire(p) >= target) break;
      __nanosleep(20u);
      if ((i & 63u) == 0u) {
        if (*abort_flag != 0u) return false;
        if (clock64() - t0 > kFlagWaitCycles) return false;
      }
    }
  }
  fence_async_global();
  return true;
}
// Progress counter in shared memory (workers -> publisher).
__device__ __forceinline__ void smem_count_add(uint32_t addr) {
  asm volatile("red.release.cta.shared::cta.add.u32 [%0], 1;" ::"r"(addr) : "memory");
}
__device__ __forceinline__ uint32_t smem_count_read(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}

// Optional time stamps and failure codes (build with -DWINO_TRACE): 16 slots per CTA.
#ifdef WINO_TRACE
__device__ unsigned long long g_trace[256 * 16];
__device__ long long g_trace_clk[256 * 16];
__device__ __forceinline__ void trace(int slot) {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  g_trace[blockIdx.x * 16 + slot] = t;
}
#define WINO_TRACE_AT(slot) trace(slot)
#define WINO_CLK_AT(cond, slot) do { if (cond) g_trace_clk[blockIdx.x * 16 + (slot)] = clock64(); } while (0)
#define WINO_FAIL(code) atomicCAS((unsigned long long*)&g_trace_clk[blockIdx.x * 16 + 15], 0ull, (unsigned long long)(code))
#else
#define WINO_TRACE_AT(slot) ((void)0)
#define WINO_CLK_AT(cond, slot) ((void)0)
#define WINO_FAIL(code) ((void)0)
#endif

struct FusedArgs {
  int BN;             // GEMM block width (128 or 256)
  int stages;         // GEMM ring stages
  int n_mblk, n_nblk, n_items;
  int units_a, units_c;   // T * C/128, T * K/128
  unsigned* cnt_in;   // [n_mblk]
  unsigned* cnt_m;    // [n_mblk]
  unsigned* ticket;   // CTAs that have finished
};

// Positions jj < n of a CTA's unit list that fall to group g (jj % 4 == g).
__device__ __forceinline__ int group_units(int n, int g) { return n > g ? (n - g + 3) >> 2 : 0; }

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
  // a slot holds the t*t rows TMA writes; the MMA reads KROWS rows, running into the next
  // slot (or the pad behind the last one), where the Kronecker matrix has zero columns
  constexpr uint32_t kSlotBytes = (T2 * 128 + 1023) / 1024 * 1024;
  constexpr uint32_t kSlotRegion = kSlots * kSlotBytes + (KROWS * 128 - kSlotBytes);
  constexpr uint32_t kStageOut = T2 * 128;             // staging tile, one per worker group
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  // ---- shared-memory map ----
  const uint32_t a_bytes = kBM * kStageK, b_bytes = (uint32_t)a.BN * kStageK;
  const uint32_t stage_bytes = a_bytes + b_bytes;
  const uint32_t s_ring = base;
  const uint32_t s_slots = s_ring + (uint32_t)a.stages * stage_bytes;
  const uint32_t s_kron = s_slots + kSlotRegion;                        // 64 rows x 64 B
  const uint32_t s_stage = s_kron + 4096u;                              // 4 groups x kStageOut
  const uint32_t s_bias = s_stage + 4u * kStageOut;                     // K floats (<= 1040)
  const uint32_t s_bar = s_bias + 4224u;
  const uint32_t bar_full = s_bar;                        // stages (<= 8)
  const uint32_t bar_empty = bar_full + 64u;
  const uint32_t bar_acc_full = bar_empty + 64u;          // 2
  const uint32_t bar_acc_empty = bar_acc_full + 16u;      // 2
  const uint32_t bar_tin_full = bar_acc_empty + 16u;      // kSlots
  const uint32_t bar_tin_empty = bar_tin_full + 8u * kSlots;
  const uint32_t bar_tacc_full = bar_tin_empty + 8u * kSlots;   // 4
  const uint32_t bar_tacc_empty = bar_tacc_full + 32u;          // 4
  const uint32_t bar_st_full = bar_tacc_empty + 32u;            // 4 staging tiles
  const uint32_t bar_st_empty = bar_st_full + 32u;              // 4
  const uint32_t bar_kron = bar_st_empty + 32u;                 // 1: Kronecker tables are in place
  const uint32_t bar_drain = bar_kron + 8u;                     // 5: last MMAs of an issuing thread are done
  const uint32_t bar_bias = bar_drain + 40u;                    // 1: bias table is in place
  const uint32_t bar_tr_done = bar_bias + 8u;                   // 1
  const uint32_t bar_gemm_done = bar_tr_done + 8u;              // 1
  const uint32_t cnt_items = bar_gemm_done + 8u;                // u32: warps done with a GEMM item
  const uint32_t tmem_slot = cnt_items + 8u;
  const uint32_t abort_slot = tmem_slot + 4u;
  const uint32_t zero_slot = abort_slot + 4u;             // stays 0: "no abort" for the final drains
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gen + (tmem_slot - base));
  volatile uint32_t* abort_p = reinterpret_cast<volatile uint32_t*>(gen + (abort_slot - base));
  volatile uint32_t* zero_p = reinterpret_cast<volatile uint32_t*>(gen + (zero_slot - base));
  float* bias_s = reinterpret_cast<float*>(gen + (s_bias - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grid = (int)gridDim.x, cta = (int)blockIdx.x;
  const int cchunks = p.C >> 7, kchunks = p.K >> 7;
  const int KB = p.C >> 7;                              // GEMM k-stages per item
  const int nA = cta < a.units_a ? (a.units_a - 1 - cta) / grid + 1 : 0;
  const int nC = cta < a.units_c ? (a.units_c - 1 - cta) / grid + 1 : 0;
  const int nI = cta < a.n_items ? (a.n_items - 1 - cta) / grid + 1 : 0;
  const int nU = nA + nC;                               // the CTA's unit list: A units, then C units
  const int per_mb = T2 * a.n_nblk;                     // items per m-block
  const int cbuf = nI & 1;                              // GEMM accumulator buffer phase C borrows

  griddep_launch();
  if (threadIdx.x == 0) {
    WINO_TRACE_AT(0);
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
      mbar_init(bar_st_full + 8u * g, 4);
      mbar_init(bar_st_empty + 8u * g, 1);
    }
    mbar_init(bar_kron, 16);
    mbar_init(bar_bias, 1);
    for (int i = 0; i < 5; ++i) mbar_init(bar_drain + 8u * i, 1);
    mbar_init(bar_tr_done, 16);
    mbar_init(bar_gemm_done, 16);
    *reinterpret_cast<volatile uint32_t*>(gen + (cnt_items - base)) = 0u;
    *abort_p = 0u;
    *zero_p = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 3) tmem_alloc(tmem_slot, 512u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_p;

  if (warp == 0) {
    // =============== transform loads: x patches (A), then m_q blocks (C) ===============
    // Lane l owns slot l and loads every kSlots-th unit: a lone thread spends hundreds of
    // cycles per unit on coordinates and issue, the lanes share that cost.  The lanes never
    // block inside the loop (a lane spinning in a wait would hold the others at the warp's
    // reconvergence point, and what it waits for may depend on them): each pass they test
    // their conditions once and issue if everything is ready.
    if (lane == 0) {
      tma_prefetch_map(&mapX);
      tma_prefetch_map(&mapMld);
    }
    {
      // x comes from HBM: ask for the patches of this CTA's units to be brought into L2 while
      // the preceding kernel is still running (a hint only: nothing reaches the SM before the
      // wait below), so that the loads find them there
      for (int jj = lane; jj < nA && jj < kPrefetchUnits; jj += 32) {
        const int u = cta + jj * grid;
        const int tau = u / cchunks, c0 = (u - tau * cchunks) << 7;
        const int tw = tau % p.TW;
        const int th = (tau / p.TW) % p.TH;
        const int n = tau / (p.TW * p.TH);
        tma_prefetch_l2_4d(&mapX, c0, tw * M - 1, th * M - 1, n);
      }
    }
    griddep_wait();
    if (lane == 0) WINO_TRACE_AT(1);
    if (lane < kSlots) {
      const uint32_t sl = (uint32_t)lane;
      int jj = lane, it = 0;
      const long long t0 = clock64();
      uint32_t spins = 0;
      while (jj < nU) {
        bool ready = it == 0 || mbar_try_wait(bar_tin_empty + 8u * sl, (uint32_t)(it - 1) & 1u);
        int tau = 0, c0 = 0;
        if (ready) {
          const bool in_a = jj < nA;
          const int u = cta + (in_a ? jj : jj - nA) * grid;
          const int chunks = in_a ? cchunks : kchunks;
          tau = u / chunks;
          c0 = (u - tau * chunks) << 7;
          if (!in_a) ready = ld_acquire(a.cnt_m + (tau >> 7)) >= (unsigned)(per_mb * 16);
        }
        if (ready) {
          mbar_expect_tx(bar_tin_full + 8u * sl, (uint32_t)T2 * 128u);
          if (jj < nA) {
            const int tw = tau % p.TW;
            const int th = (tau / p.TW) % p.TH;
            const int n = tau / (p.TW * p.TH);
            tma_load_4d(s_slots + sl * kSlotBytes, &mapX, bar_tin_full + 8u * sl, c0, tw * M - 1, th * M - 1, n);
          } else {
            fence_async_global();     // the counter was read with acquire; order the TMA read after it
            if (jj == nA) WINO_TRACE_AT(12);
            tma_load_3d(s_slots + sl * kSlotBytes, &mapMld, bar_tin_full + 8u * sl, c0, tau, 0);
          }
          jj += kSlots;
          ++it;
        } else if ((++spins & 1023u) == 0u && (*abort_p != 0u || clock64() - t0 > kWaitCycles)) {
          WINO_FAIL(300 + jj);
          *abort_p = 1u;
          break;
        }
      }
    }
  } else if (warp == 1) {
    // =============== transform MMAs: lane g issues for worker group g ===============
    // (same rule as above: no lane blocks inside the loop)
    if (lane < 4) {
      const int g = lane;
      const uint32_t idesc_in = fl_idesc_a_mn(128, NB_IN), idesc_out = fl_idesc_a_mn(128, NB_OUT);
      const uint64_t db_in = fl_desc_kmajor_sw64(s_kron);
      const uint64_t db_out = fl_desc_kmajor_sw64(s_kron + 48u * 64u);
      const int nG = group_units(nU, g);
      const long long t0 = clock64();
      uint32_t spins = 0;
      int n = 0;                                  // n-th unit of group g = n-th use of its accumulator
      bool kron_ok = false, gemm_ok = nI == 0;
      while (n < nG) {
        const int jj = g + 4 * n;                 // position in the CTA's unit list
        const bool ph_c = jj >= nA;
        const uint32_t sl = (uint32_t)(jj % kSlots);
        if (!kron_ok) kron_ok = mbar_try_wait(bar_kron, 0u);        // the workers have copied the tables
        // phase C borrows the columns of a GEMM accumulator buffer: every item of this CTA
        // must have been drained first (a one-phase barrier: no parity to get ahead of)
        if (ph_c && !gemm_ok) gemm_ok = mbar_try_wait(bar_gemm_done, 0u);
        const bool ready = kron_ok && (!ph_c || gemm_ok) &&
                           mbar_try_wait(bar_tin_full + 8u * sl, (uint32_t)(n >> 1) & 1u) &&
                           mbar_try_wait(bar_tacc_empty + 8u * g, ((uint32_t)n & 1u) ^ 1u);
        if (ready) {
          tc_fence_after();
          const uint32_t tcol = tmem_base + (uint32_t)((ph_c ? cbuf : 1) * 256 + g * 64);
          const uint64_t da = fl_desc_mnmajor_sw128(s_slots + sl * kSlotBytes);
#pragma unroll
          for (int ks = 0; ks < KROWS / 32; ++ks)
            mma_i8(tcol, da + (uint64_t)(ks * 256), (ph_c ? db_out : db_in) + (uint64_t)(ks * 2),
                   ph_c ? idesc_out : idesc_in, ks != 0 ? 1u : 0u);
          mma_commit(bar_tin_empty + 8u * sl);
          mma_commit(bar_tacc_full + 8u * g);
          ++n;
        } else if ((++spins & 1023u) == 0u && (*abort_p != 0u || clock64() - t0 > kWaitCycles)) {
          WINO_FAIL(400 + n * 4 + g + (kron_ok ? 0 : 10000) + (ph_c && !gemm_ok ? 20000 : 0));
          *abort_p = 1u;
          break;
        }
      }
      // leave only when every MMA this thread has issued is done (also on the abort path:
      // tensor memory is freed at the end of the kernel)
      mma_commit(bar_drain + 8u * (uint32_t)g);
      (void)mbar_wait<false>(bar_drain + 8u * (uint32_t)g, 0u, zero_p);
    }
  } else if (warp == 2) {
    // =============== GEMM operand loads ===============
    if (lane == 0) {
      tma_prefetch_map(&mapV);
      tma_prefetch_map(&mapU);
      bool ok = true;
      int s = 0; uint32_t ph = 0;
      bool waited = false;     // griddepcontrol.wait done (U_q, a constant, may be fetched before it)
      for (int li = 0; li < nI && ok; ++li) {
        const int it = cta + li * grid;
        const int mb = it / per_mb, rem = it - mb * per_mb;
        const int xi = rem / a.n_nblk, nb = rem - xi * a.n_nblk;
        const int tiles = min(kBM, p.T - mb * kBM);
        // weight halves of as many stages as the ring can take now: no dependency on phase A
        int armed = 0;
        {
          int s2 = s; uint32_t ph2 = ph;
          for (int kb = 0; kb < KB && kb < a.stages; ++kb) {
            if (!mbar_wait<false>(bar_empty + 8u * s2, ph2 ^ 1u, abort_p)) { WINO_FAIL(101); ok = false; break; }
            mbar_expect_tx(bar_full + 8u * s2, stage_bytes);
            tma_load_3d(s_ring + (uint32_t)s2 * stage_bytes + a_bytes, &mapU, bar_full + 8u * s2,
                        kb * kStageK, nb * a.BN, xi);
            armed = kb + 1;
            if (++s2 == a.stages) { s2 = 0; ph2 ^= 1u; }
          }
          if (!ok) break;
        }
        if (!waited) { griddep_wait(); waited = true; }
        if (!flag_wait(a.cnt_in + mb, (unsigned)(tiles * cchunks), abort_p)) { WINO_FAIL(102); ok = false; break; }
        if (li == 0) WINO_TRACE_AT(8);
        if (li == 1) WINO_TRACE_AT(9);
        for (int kb = 0; kb < KB; ++kb) {
          const uint32_t sa = s_ring + (uint32_t)s * stage_bytes;
          if (kb >= armed) {
            if (!mbar_wait<false>(bar_empty + 8u * s, ph ^ 1u, abort_p)) { WINO_FAIL(103); ok = false; break; }
            mbar_expect_tx(bar_full + 8u * s, stage_bytes);
            tma_load_3d(sa + a_bytes, &mapU, bar_full + 8u * s, kb * kStageK, nb * a.BN, xi);
          }
          tma_load_3d(sa, &mapV, bar_full + 8u * s, kb * kStageK, mb * kBM, xi);
          if (++s == a.stages) { s = 0; ph ^= 1u; }
        }
      }
      if (!waited) griddep_wait();
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
        if (!mbar_wait<false>(bar_acc_empty + 8u * buf, aph ^ 1u, abort_p)) { WINO_FAIL(104); ok = false; break; }
        // columns 256..511 hold the transform accumulators until phase A is over
        if (li == 1 && !mbar_wait<false>(bar_tr_done, 0u, abort_p)) { WINO_FAIL(105); ok = false; break; }
        tc_fence_after();
        const uint32_t tacc = tmem_base + (uint32_t)(buf * 256);
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait<false>(bar_full + 8u * s, ph, abort_p)) { WINO_FAIL(106); ok = false; break; }
          tc_fence_after();
          if (kb == 0 && li == 0) WINO_TRACE_AT(10);
          if (kb == 0 && li == 1) WINO_TRACE_AT(11);
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
      mma_commit(bar_drain + 32u);     // leave only when every MMA issued here is done
      (void)mbar_wait<false>(bar_drain + 32u, 0u, zero_p);
    }
  } else if (warp == 4) {
    // =============== bias table, then publisher of cnt_m ===============
    griddep_wait();                             // bias may be the previous kernel's output
    for (int k = lane; k < p.K; k += 32)
      bias_s[k] = bias != nullptr ? (float)((double)__ldg(bias + k) / (double)s_Y) : 0.0f;
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_bias);
    // an item's m_q is in place once all 16 epilogue warps have stored their share; one
    // fence covers every item that finished in the meantime (fence + relaxed update = release)
    if (lane == 0) {
      const long long t0 = clock64();
      uint32_t spins = 0;
      int pub = 0;
      while (pub < nI) {
        const int fin = (int)(smem_count_read(cnt_items) >> 4);
        if (fin > pub) {
          __threadfence();
          fence_async_global();
          for (; pub < fin; ++pub) flag_add(a.cnt_m + (cta + pub * grid) / per_mb, 16u);
        } else if ((++spins & 255u) == 0u && (*abort_p != 0u || clock64() - t0 > kWaitCycles)) {
          WINO_FAIL(500 + pub);
          *abort_p = 1u;
          break;
        }
      }
    }
  } else if (warp < 9) {
    // =============== store thread of worker group g ===============
    if (lane == 0) {
      const int g = warp - 5;
      tma_prefetch_map(&mapVst);
      tma_prefetch_map(&mapY);
      const int nG = group_units(nU, g);
      const uint32_t st = s_stage + (uint32_t)g * kStageOut;
      bool ok = true;
      // cnt_in updates are batched: waiting for a store to complete and fencing costs about
      // two unit times, so it is done once per two tiles (and at the end of phase A), while
      // the staging tile is handed back as soon as the store has read it
      int pend = 0, pend_mb[4];
      auto flush = [&]() {
        if (pend == 0) return;
        bulk_wait_all();                           // the V_q bytes are in place
        __threadfence();
        fence_async_global();
        for (int i = 0; i < pend; ++i) {
          unsigned cnt = 1u;
          while (i + 1 < pend && pend_mb[i + 1] == pend_mb[i]) { ++cnt; ++i; }
          flag_add(a.cnt_in + pend_mb[i], cnt);
        }
        pend = 0;
      };
      for (int n = 0; n < nG; ++n) {               // n-th tile of this group
        const int jj = g + 4 * n;
        if (!mbar_wait<false>(bar_st_full + 8u * (uint32_t)g, (uint32_t)n & 1u, abort_p)) { WINO_FAIL(600 + n); ok = false; break; }
        if (jj < nA) {
          const int u = cta + jj * grid;
          const int tau = u / cchunks, c0 = (u - tau * cchunks) << 7;
          tma_store_3d(&mapVst, st, c0, tau, 0);
          bulk_commit();
          bulk_wait_read();                        // the staging tile may be refilled
          mbar_arrive(bar_st_empty + 8u * (uint32_t)g);
          pend_mb[pend++] = tau >> 7;
          if (pend == 2 || jj + 4 >= nA) flush();
          if (g == 0 && jj + 4 >= nA) WINO_TRACE_AT(13);
        } else {
          // y tile (pixels past the image edge are clipped by the TMA unit)
          const int u = cta + (jj - nA) * grid;
          const int tau = u / kchunks, k0 = (u - tau * kchunks) << 7;
          const int tw = tau % p.TW;
          const int th = (tau / p.TW) % p.TH;
          const int n_img = tau / (p.TW * p.TH);
          tma_store_4d(&mapY, st, k0, tw * M, th * M, n_img);
          bulk_commit();
          bulk_wait_read();
          mbar_arrive(bar_st_empty + 8u * (uint32_t)g);
        }
      }
      flush();
      bulk_wait_read();   // the y stores have read their tiles; the end of the grid publishes them
      if (!ok) *abort_p = 1u;
    }
  } else {
    // =============== workers ===============
    const int g = (warp - 9) >> 2;              // group
    const int quad = warp & 3;                  // tensor-memory lane quadrant
    const int et = threadIdx.x - kFlWorker0 - g * 128;   // 0..127 inside the group
    const bool leader = et == 0;
    const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
    const int ch = quad * 32 + lane;            // channel inside a 128-channel chunk / row inside an m-block
    // Kronecker tables (plan constants): rows 0..47 input side, 48..63 output side
    for (int idx = threadIdx.x - kFlWorker0; idx < 64 * 4; idx += kFlThreads - kFlWorker0)
      *reinterpret_cast<uint4*>(gen + (s_kron - base) + fl_sw64_off(idx >> 2, (idx & 3) * 16)) =
          __ldg(kron + idx);
    fence_async_smem();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_kron);
    const uint32_t st = s_stage + (uint32_t)g * kStageOut;
    uint8_t* sp = gen + (st - base) + ch;       // this thread's column of the staging tile
    uint32_t tuse = 0;                          // units this group has processed (A and C together)
    int jj = g;                                 // position in the CTA's unit list
    bool ok = true;

    // wait (every thread, bounded) until the store thread has read the previous tile out of
    // the staging buffer; placed after the arithmetic, so it has normally long happened
    auto staging_free = [&]() -> bool {
      if (tuse == 0) return true;
      return mbar_wait<false>(bar_st_empty + 8u * (uint32_t)g, (tuse & 1u) ^ 1u, abort_p);
    };

    // ---------------- phase A ----------------
    {
      const float lo = __fadd_rn(p.lo_V, kMagic), hi = __fadd_rn(p.hi_V, kMagic);
      for (; jj < nA; jj += 4, ++tuse) {
        WINO_CLK_AT(leader && g == 0 && tuse == 1, 0);
        if (leader && !mbar_wait<false>(bar_tacc_full + 8u * g, tuse & 1u, abort_p)) { WINO_FAIL(201); *abort_p = 1u; }
        if (leader && g == 0 && tuse == 0) WINO_TRACE_AT(2);
        WINO_CLK_AT(leader && g == 0 && tuse == 1, 1);
        group_barrier(g);
        WINO_CLK_AT(leader && g == 0 && tuse == 1, 2);
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
        WINO_CLK_AT(leader && g == 0 && tuse == 1, 3);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tacc_empty + 8u * g);
        // all codes first (independent chains the compiler can interleave), then the stores
        auto code = [&](uint32_t acc) {
          return __float_as_uint(fminf(fmaxf(__fmaf_rn(__int2float_rn((int)acc), p.mult_V, kMagic), lo), hi));
        };
#pragma unroll
        for (int q = 0; q < N0; ++q) r0[q] = code(r0[q]);
        if constexpr (M == 4) {
#pragma unroll
          for (int q = 0; q < N1; ++q) r1[q] = code(r1[q]);
        }
        if (!staging_free()) { WINO_FAIL(202); *abort_p = 1u; }
#pragma unroll
        for (int q = 0; q < N0; ++q) sp[q * 128] = (uint8_t)r0[q];
        if constexpr (M == 4) {
#pragma unroll
          for (int q = 0; q < N1; ++q) sp[(32 + q) * 128] = (uint8_t)r1[q];
        }
        WINO_CLK_AT(leader && g == 0 && tuse == 1, 4);
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_st_full + 8u * (uint32_t)g);   // the group's store thread takes over
        WINO_CLK_AT(leader && g == 0 && tuse == 1, 5);
      }
      if (leader && g == 0) WINO_TRACE_AT(3);
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
        if (!__all_sync(0xffffffffu, mbar_wait<false>(bar_acc_full + 8u * buf, aph, abort_p))) {
          WINO_FAIL(203);
          *abort_p = 1u;
          ok = false;
          break;
        }
        tc_fence_after();
        if (leader && g == 0 && li == 0) WINO_TRACE_AT(4);
        if (leader && g == 0 && li == 1) WINO_TRACE_AT(5);
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
            if (p.hi_M == 127.0f) {
#pragma unroll
              for (int q = 0; q < 8; ++q)
                w[q] = quant_pack4<true>(__int2float_rn((int)r[4 * q]), __int2float_rn((int)r[4 * q + 1]),
                                         __int2float_rn((int)r[4 * q + 2]), __int2float_rn((int)r[4 * q + 3]),
                                         p.mult_M, lo, hi);
            } else {
#pragma unroll
              for (int q = 0; q < 8; ++q)
                w[q] = quant_pack4<false>(__int2float_rn((int)r[4 * q]), __int2float_rn((int)r[4 * q + 1]),
                                          __int2float_rn((int)r[4 * q + 2]), __int2float_rn((int)r[4 * q + 3]),
                                          p.mult_M, lo, hi);
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
          smem_count_add(cnt_items);                 // release: this warp's m_q stores precede it
        }
      }
    }
    if (leader && g == 0) WINO_TRACE_AT(6);
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_gemm_done);

    // ---------------- phase C ----------------
    if (ok && !mbar_wait<false>(bar_bias, 0u, abort_p)) { WINO_FAIL(206); ok = false; }
    if (ok) {
      bool first = true;
      for (; jj < nU; jj += 4, ++tuse) {
        const int u = cta + (jj - nA) * grid;
        const int tau = u / kchunks, k0 = (u - tau * kchunks) << 7;
        if (leader && !mbar_wait<false>(bar_tacc_full + 8u * g, tuse & 1u, abort_p)) { WINO_FAIL(204); *abort_p = 1u; }
        if (leader && g == 0 && first) WINO_TRACE_AT(7);
        first = false;
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
#pragma unroll
        for (int q = 0; q < MM; ++q) {
          const float yf = __fmaf_rn(__int2float_rn((int)v[q]), p.mult_Y, b_scaled);
          const float r = __fadd_rn(fminf(fmaxf(yf, p.lo_Y), p.hi_Y), kMagic);
          v[q] = (uint32_t)(magic_to_int(r) + p.z_Y);
        }
        if (!staging_free()) { WINO_FAIL(205); *abort_p = 1u; }
#pragma unroll
        for (int q = 0; q < MM; ++q) sp[q * 128] = (uint8_t)v[q];
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_st_full + 8u * (uint32_t)g);
      }
    }
    if (leader && g == 0) WINO_TRACE_AT(15);
    if (!ok) *abort_p = 1u;
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    WINO_TRACE_AT(14);
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
  const size_t krows = (size_t)(t2 + 31) / 32 * 32;
  const size_t slot = ((size_t)t2 * 128 + 1023) / 1024 * 1024;
  const size_t slot_region = kSlots * slot + (krows * 128 - slot);
  const size_t fixed = 1024 + slot_region + 4096 + 4 * (size_t)t2 * 128 + 4224 + 640;
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

#ifdef WINO_TRACE
extern "C" int wino_trace_read(unsigned long long* host_out) {
  return cudaMemcpyFromSymbol(host_out, g_trace, sizeof(g_trace)) == cudaSuccess ? 0 : -5;
}
extern "C" int wino_trace_read_clk(long long* host_out) {
  return cudaMemcpyFromSymbol(host_out, g_trace_clk, sizeof(g_trace_clk)) == cudaSuccess ? 0 : -5;
}
#endif

int launch_layer_fused(const Params& p, const LaunchOpt& o, const FusedGeom& g, const FusedMaps& m,
                       const void* kron, unsigned* counters, int8_t* mq, const float* bias,
                       float s_Y, int* status, cudaStream_t st) {
  if (g.stages < 2) return -2;
  return p.m == 2 ? fused_launch<2>(p, o, g, m, kron, counters, mq, bias, s_Y, status, st)
                  : fused_launch<4>(p, o, g, m, kron, counters, mq, bias, s_Y, status, st);
}

}  // namespace wino
