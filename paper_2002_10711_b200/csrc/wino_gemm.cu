// Hadamard stage of the Winograd-aware layer as t*t independent int8 GEMMs over
// channels with int32 accumulation (paper: Sections 1 and 5.3, where the
// position-wise products are carried out as GEMMs):   M[xi][tau][k] = sum_c V_q[xi][tau][c] * U_q[xi][k][c]
// followed by the quantizer of the Hadamard output (paper: Fig. 2).
//
//   k_gemm_tc   : persistent, warp-specialised tcgen05 kernel.  int8 operands are
//                 staged in shared memory by TMA (128-byte swizzle), MMAs of
//                 kind::i8 accumulate in int32 in tensor memory, two accumulator
//                 buffers let the epilogue of one block overlap the MMAs of the
//                 next.
//   k_gemm_dp4a : the same contraction with 4-way integer dot products on the
//                 ALUs; fallback for channel counts the TMA path cannot take.
#include "wino_launch.h"
#include "wino_ptx.cuh"
#include "wino_trace.cuh"

namespace wino {

// ---------------------------------------------------------------------------
// ALU fallback.  Thread = (xi, tau, 4 consecutive k).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
k_gemm_dp4a(const __grid_constant__ Params p, const int8_t* __restrict__ Vq,
            const int8_t* __restrict__ Uq, void* __restrict__ out, int out_mode,
            unsigned* __restrict__ absmaxM, const float* __restrict__ chan) {
  const int C4 = p.C >> 2, K4 = p.K >> 2;
  const int xi = blockIdx.z;
  const long idx = blockIdx.x * (long)blockDim.x + threadIdx.x;
  float vmax = 0.0f;
  griddep_launch();
  griddep_wait();
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
      *reinterpret_cast<int4*>(reinterpret_cast<int*>(out) + o) =
          make_int4(acc[0], acc[1], acc[2], acc[3]);
    } else {
      uint32_t wv = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float r = quant_magic(__int2float_rn(acc[j]), chan_or(chan, p.K, kChMultM, k4 * 4 + j, p.mult_M),
                              p.lo_M, p.hi_M);
        wv |= (__float_as_uint(r) & 0xFFu) << (8 * j);
      }
      *reinterpret_cast<uint32_t*>(reinterpret_cast<int8_t*>(out) + o) = wv;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) vmax = fmaxf(vmax, fabsf(__int2float_rn(acc[j])));
  }
  if (absmaxM != nullptr) atomic_absmax(absmaxM, vmax);
}

int launch_gemm_dp4a(const Params& p, const LaunchOpt& o, const int8_t* Vq, const int8_t* Uq,
                     void* out, int out_mode, unsigned* absmaxM, cudaStream_t st) {
  const long total = (long)p.T * (p.K / 4);
  dim3 grid((unsigned)((total + 127) / 128), 1, (unsigned)(p.t * p.t));
  return launch_kernel(k_gemm_dp4a, grid, dim3(128), 0, st, o.pdl, p, Vq, Uq, out, out_mode,
                       absmaxM, o.chan);
}

// ---------------------------------------------------------------------------
// tcgen05 GEMM.  Work item = one 128 (tau) x BN (k) block of one xi; CTAs walk
// the item list with stride gridDim.x (m-block fastest, so CTAs running
// together share the same U_q tile in L2).
//   warp 0   : TMA producer (one lane)
//   warp 1   : tensor-memory owner; one lane issues the MMAs
//   warps 2-17: epilogue.  Warp w reads TMEM lanes 32*(w%4) .. +31 (its hardware
//              quadrant) and every fourth 32-column chunk, by (w-2)/4.
// A stage holds 128 channels: A tile 128 x 128 B, B tile BN x 128 B; one MMA
// consumes 32 channels.
// ---------------------------------------------------------------------------

#ifdef WINO_TRACE
static __device__ TraceTable g_gemm_trace;
#endif
WINO_ST_READER(wino_trace_gemm, g_gemm_trace)

constexpr int kEpiWarps = 16;
constexpr int kGemmThreads = 64 + 32 * kEpiWarps;

struct GemmTcArgs {
  int BN;          // multiple of 16, <= 256
  int stages;
  int tmem_cols;   // power of two >= 32, >= 2 * acc_stride
  int acc_stride;  // columns between the two accumulator buffers
  int out_mode;
  int MB;          // m-blocks (128 tiles each) per work item, sharing one U_q tile
  int n_mblk, n_nblk, n_items;   // n_mblk counts groups of MB m-blocks
  int wide_store;  // 1: the output rows are 32-byte aligned (one 256-bit store per row piece)
  const float* chan;  // per-output-channel multipliers [5][K], or null
  int chan_smem;      // 1: the block keeps the K multipliers of Q_M in shared memory
};

template <bool SMALL>
__device__ __forceinline__ float acc_to_float(uint32_t v) {
  if constexpr (SMALL) return small_int_to_float((int)v);
  else return __int2float_rn((int)v);
}

// Epilogue of one 32-column chunk of one accumulator row.  FULL: all 32 columns
// are inside K (no per-element guards).  STATS: track max |M| for calibration.  PK: the
// multiplier of Q_M varies per output channel (column).
template <bool SMALL, bool FULL, bool STATS, bool PK, bool LEAN = false>
__device__ __forceinline__ void epilogue_chunk(const Params& p, const uint32_t (&r)[32], int k0,
                                               long o, int out_mode, void* out, float& vmax,
                                               bool wide_store, const float* mult_k) {
  if constexpr (LEAN) {
    // the one configuration the lean kernel is launched for: int8 codes, upper bound 127
    // (saturating pack), 32-byte aligned rows
    const float lo_m = __fadd_rn(p.lo_M, kMagic), hi_m = __fadd_rn(p.hi_M, kMagic);
    uint32_t w[8];
#pragma unroll
    for (int q = 0; q < 8; ++q)
      w[q] = quant_pack4<true>(acc_to_float<SMALL>(r[4 * q + 0]), acc_to_float<SMALL>(r[4 * q + 1]),
                               acc_to_float<SMALL>(r[4 * q + 2]), acc_to_float<SMALL>(r[4 * q + 3]),
                               p.mult_M, lo_m, hi_m);
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(
                     reinterpret_cast<int8_t*>(out) + o),
                 "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
    return;
  }
  if constexpr (STATS) {
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (FULL || k0 + j < p.K) vmax = fmaxf(vmax, fabsf(__int2float_rn((int)r[j])));
  }
  if (out_mode == kOutI32) {
    int4* dst = reinterpret_cast<int4*>(reinterpret_cast<int*>(out) + o);
#pragma unroll
    for (int q = 0; q < 8; ++q)
      if (FULL || k0 + q * 4 < p.K)
        dst[q] = make_int4((int)r[4 * q], (int)r[4 * q + 1], (int)r[4 * q + 2], (int)r[4 * q + 3]);
  } else {
    uint32_t w[8];
    const float lo_m = __fadd_rn(p.lo_M, kMagic), hi_m = __fadd_rn(p.hi_M, kMagic);
    if constexpr (PK) {
      // every lane reads the same 32 multipliers (one broadcast request per four); mult_k
      // is the block's copy in shared memory, or the table in global memory
      const float4* mp = reinterpret_cast<const float4*>(mult_k + k0);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const float4 mm = (FULL || k0 + q * 4 < p.K) ? mp[q] : make_float4(0.f, 0.f, 0.f, 0.f);
        if (p.hi_M == 127.0f) {   // upper bound by the saturating pack, as in quant_pack4
          const int c0 = magic_to_int(fmaxf(__fmaf_rn(acc_to_float<SMALL>(r[4 * q + 0]), mm.x, kMagic), lo_m));
          const int c1 = magic_to_int(fmaxf(__fmaf_rn(acc_to_float<SMALL>(r[4 * q + 1]), mm.y, kMagic), lo_m));
          const int c2 = magic_to_int(fmaxf(__fmaf_rn(acc_to_float<SMALL>(r[4 * q + 2]), mm.z, kMagic), lo_m));
          const int c3 = magic_to_int(fmaxf(__fmaf_rn(acc_to_float<SMALL>(r[4 * q + 3]), mm.w, kMagic), lo_m));
          w[q] = pack_sat_s8(c1, c0, pack_sat_s8(c3, c2, 0u));
          continue;
        }
        const uint32_t b0 = __float_as_uint(quant_magic(acc_to_float<SMALL>(r[4 * q + 0]), mm.x, p.lo_M, p.hi_M));
        const uint32_t b1 = __float_as_uint(quant_magic(acc_to_float<SMALL>(r[4 * q + 1]), mm.y, p.lo_M, p.hi_M));
        const uint32_t b2 = __float_as_uint(quant_magic(acc_to_float<SMALL>(r[4 * q + 2]), mm.z, p.lo_M, p.hi_M));
        const uint32_t b3 = __float_as_uint(quant_magic(acc_to_float<SMALL>(r[4 * q + 3]), mm.w, p.lo_M, p.hi_M));
        w[q] = __byte_perm(__byte_perm(b0, b1, 0x0040u), __byte_perm(b2, b3, 0x0040u), 0x5410u);
      }
    } else if (p.hi_M == 127.0f) {
#pragma unroll
      for (int q = 0; q < 8; ++q)
        w[q] = quant_pack4<true>(acc_to_float<SMALL>(r[4 * q + 0]), acc_to_float<SMALL>(r[4 * q + 1]),
                                 acc_to_float<SMALL>(r[4 * q + 2]), acc_to_float<SMALL>(r[4 * q + 3]),
                                 p.mult_M, lo_m, hi_m);
    } else {
#pragma unroll
      for (int q = 0; q < 8; ++q)
        w[q] = quant_pack4<false>(acc_to_float<SMALL>(r[4 * q + 0]), acc_to_float<SMALL>(r[4 * q + 1]),
                                  acc_to_float<SMALL>(r[4 * q + 2]), acc_to_float<SMALL>(r[4 * q + 3]),
                                  p.mult_M, lo_m, hi_m);
    }
    uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<int8_t*>(out) + o);
    if (FULL && wide_store) {
      // the whole 32-byte sector of this row in one request
      asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]),
                   "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                   : "memory");
    } else {
      if (FULL || k0 < p.K) dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
      if (FULL || k0 + 16 < p.K) dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
  }
}

// The epilogue warps' loop over their work items.
template <bool SMALL, bool FULL, bool STATS, bool PK = false, bool LEAN = false>
__device__ __forceinline__ void epilogue_loop(const Params& p, const GemmTcArgs& a, void* out,
                                              unsigned* absmaxM, uint32_t tmem_base,
                                              uint32_t bar_acc_full, uint32_t bar_acc_empty,
                                              volatile uint32_t* abort_p, int warp, int lane,
                                              int trace_step, const float* mult_k = nullptr) {
  (void)trace_step;
  const int quad = warp & 3;
  const int sub = (warp - 2) >> 2;
  const int per_xi = a.n_mblk * a.n_nblk;
  float vmax = 0.0f;
  int li = 0;
  for (int it = blockIdx.x; it < a.n_items; it += gridDim.x, ++li) {
    const int xi = it / per_xi, rem = it - xi * per_xi;
    const int nb = rem / a.n_mblk, mb = rem - nb * a.n_mblk;
    const int buf = li & 1;
    const uint32_t aph = (uint32_t)(li >> 1) & 1u;
    if (!__all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8u * buf, aph, abort_p))) {
      *abort_p = 1u;
      break;
    }
    if (warp == 2 && lane == 0 && li < 2) WINO_ST(g_gemm_trace, trace_step, 5 + 2 * li);
    tc_fence_after();
    const uint32_t tacc = tmem_base + (uint32_t)(buf * a.acc_stride) + ((uint32_t)(quad * 32) << 16);
    // the accumulator holds MB blocks of BN columns side by side; one chunk at a
    // time per warp, the four warps of a scheduler hide each other's
    // tensor-memory load latency
    auto chunk = [&](const uint32_t (&r)[32], int col) {
      const int j = a.MB > 1 ? col / a.BN : 0;
      const int kcol = col - j * a.BN;
      const int tau = (mb * a.MB + j) * kBM + quad * 32 + lane;
      if (tau >= p.T) return;
      const int k0 = nb * a.BN + kcol;
      const long o = ((long)xi * p.T + tau) * p.K + k0;
      epilogue_chunk<SMALL, FULL, STATS, PK, LEAN>(p, r, k0, o, a.out_mode, out, vmax, a.wide_store != 0, mult_k);
    };
    for (int col = sub * 32; col < a.MB * a.BN; col += 128) {
      uint32_t r0[32];
      tmem_ld32(tacc + (uint32_t)col, r0);
      tmem_ld_wait();
      chunk(r0, col);
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_acc_empty + 8u * buf);
    if (warp == 2 && lane == 0 && li < 2) WINO_ST(g_gemm_trace, trace_step, 6 + 2 * li);
  }
  if constexpr (STATS) atomic_absmax(absmaxM, vmax);
}

// PK: Q_M takes one multiplier per output channel (a build of its own, so that the
// per-layer kernel carries none of that code).
// LEAN: only the epilogue of the common case is compiled in (Q_M to int8 codes with upper
// bound 127, C <= 260, whole 32-column chunks, 32-byte aligned rows); the kernel's code is a
// third of the general one's, which shows at every launch.
template <bool PK, bool LEAN = false>
__device__ __forceinline__ void gemm_tc_body(const Params& p, const CUtensorMap* mapV,
                                             const CUtensorMap* mapU, const GemmTcArgs& a,
                                             void* __restrict__ out, unsigned* __restrict__ absmaxM,
                                             int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  // tiles need 1024-byte alignment for the 128-byte swizzle
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t a_bytes = kBM * kStageK, b_bytes = (uint32_t)a.BN * kStageK;
  const uint32_t stage_bytes = (uint32_t)a.MB * a_bytes + b_bytes;
  const uint32_t bars = base + (uint32_t)a.stages * stage_bytes;
  const uint32_t bar_full = bars;                           // stages x 8 B
  const uint32_t bar_empty = bar_full + 8u * a.stages;      // stages x 8 B
  const uint32_t bar_acc_full = bar_empty + 8u * a.stages;  // 2 x 8 B
  const uint32_t bar_acc_empty = bar_acc_full + 16u;        // 2 x 8 B
  const uint32_t tmem_slot = bar_acc_empty + 16u;
  const uint32_t abort_slot = tmem_slot + 4u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gen + (tmem_slot - base));
  volatile uint32_t* abort_p = reinterpret_cast<volatile uint32_t*>(gen + (abort_slot - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KB = (p.C + kStageK - 1) / kStageK;
  const int per_xi = a.n_mblk * a.n_nblk;

  int trace_step = 0;
#ifdef WINO_TRACE
  int& trace_step_s = *reinterpret_cast<int*>(gen + (abort_slot + 4u - base));
  if (threadIdx.x == 0) {
    WINO_ST_BEGIN(g_gemm_trace, trace_step_s);
    WINO_ST(g_gemm_trace, trace_step_s, 0);
  }
#endif
  griddep_launch();
  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      mbar_init(bar_full + 8u * s, 1);
      mbar_init(bar_empty + 8u * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_acc_full + 8u * b, 1);
      mbar_init(bar_acc_empty + 8u * b, kEpiWarps);
    }
    *abort_p = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, (uint32_t)a.tmem_cols);
#ifdef WINO_TRACE
    if (lane == 0) *reinterpret_cast<unsigned long long*>(gen + (tmem_slot + 16u - base)) = trace_now();
#endif
  }
  if (warp == 0 && lane == 0) {   // descriptors do not depend on the previous kernel
    tma_prefetch_map(mapV);
    tma_prefetch_map(mapU);

  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_p;
#ifdef WINO_TRACE
  trace_step = trace_step_s;
  if (threadIdx.x == 0) {
    WINO_ST(g_gemm_trace, trace_step, 1);
    g_gemm_trace.t[trace_step][blockIdx.x][13] = *reinterpret_cast<unsigned long long*>(gen + (tmem_slot + 16u - base));
  }
#endif
  // Each role waits for the preceding kernels itself, as late as it can: the producer just
  // before its first load (its index arithmetic is done by then), the epilogue warps before
  // they write; the MMA thread touches no global memory.
  if (warp == 0) {
    if (lane == 0) {
      int s = 0, issued = 0; uint32_t ph = 0;
      int xi = blockIdx.x / per_xi, rem = blockIdx.x - xi * per_xi;
      int nb = rem / a.n_mblk, mb = rem - nb * a.n_mblk;
      // A lone thread retires an instruction every ten to twenty cycles, and the first loads
      // after the wait are the step's critical path (the generic loop took 0.6 us to get them
      // out).  So the operands of the first item's first one or two stages are computed, and
      // pinned in registers, before the wait; after it only the copy instructions themselves
      // are issued, and the generic loop takes over from there.
      const int n_first = (KB >= 2 && a.stages >= 2) ? 2 : 1;
      uint32_t f_bytes = stage_bytes, f_dst = base, f_b_off = (uint32_t)a.MB * a_bytes, f_a_bytes = a_bytes;
      int f_row_a = (mb * a.MB) * kBM, f_row_b = nb * a.BN, f_xi = xi, f_mb = a.MB, f_n = n_first;
      asm volatile("" : "+r"(f_bytes), "+r"(f_dst), "+r"(f_b_off), "+r"(f_a_bytes), "+r"(f_row_a),
                        "+r"(f_row_b), "+r"(f_xi), "+r"(f_mb), "+r"(f_n));
      griddep_wait();
      WINO_ST(g_gemm_trace, trace_step, 2);
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        if (q < f_n) {
          const uint32_t fb = bar_full + 8u * (uint32_t)q, fd = f_dst + (uint32_t)q * f_bytes;
          mbar_expect_tx(fb, f_bytes);
          tma_load_3d(fd, mapV, fb, q * kStageK, f_row_a, f_xi);
          tma_load_3d(fd + f_b_off, mapU, fb, q * kStageK, f_row_b, f_xi);
          for (int j = 1; j < f_mb; ++j)   // rows past T are filled with zeros by the TMA unit
            tma_load_3d(fd + (uint32_t)j * f_a_bytes, mapV, fb, q * kStageK, f_row_a + j * kBM, f_xi);
          if (q == 0) WINO_ST(g_gemm_trace, trace_step, 15);
        }
      }
      issued = n_first;
      s = n_first;
      if (s == a.stages) { s = 0; ph ^= 1u; }
      for (int it = blockIdx.x; it < a.n_items; it += gridDim.x) {
        if (it != blockIdx.x) {
          xi = it / per_xi; rem = it - xi * per_xi;
          nb = rem / a.n_mblk; mb = rem - nb * a.n_mblk;
        }
        bool ok = true;
        for (int kb = (it == (int)blockIdx.x ? n_first : 0); kb < KB; ++kb) {
          // the ring's first pass finds every stage free
          if (issued >= a.stages && !mbar_wait(bar_empty + 8u * s, ph ^ 1u, abort_p)) { ok = false; break; }
          ++issued;
          const uint32_t sa = base + (uint32_t)s * stage_bytes;
          mbar_expect_tx(bar_full + 8u * s, stage_bytes);
          for (int j = 0; j < a.MB; ++j)   // rows past T are filled with zeros by the TMA unit
            tma_load_3d(sa + (uint32_t)j * a_bytes, mapV, bar_full + 8u * s, kb * kStageK,
                        (mb * a.MB + j) * kBM, xi);
          tma_load_3d(sa + (uint32_t)a.MB * a_bytes, mapU, bar_full + 8u * s, kb * kStageK,
                      nb * a.BN, xi);
          if (++s == a.stages) { s = 0; ph ^= 1u; }
        }
        if (!ok) { *abort_p = 1u; break; }
      }
    }
  } else if (warp == 1) {
    // The whole warp walks the loop so that stage addresses and descriptors are warp-uniform
    // values; one elected lane issues the MMAs and the commits.
    const bool leader = elect_one();
    const uint32_t idesc = make_idesc_i8(kBM, a.BN);
    // What does not change from stage to stage is computed once: this warp's every
    // instruction costs ten to twenty cycles and a stage's MMAs take five hundred.  Descriptors
    // are linear in the tile address (units of 16 bytes), so a stage's are the first stage's
    // plus a multiple of the stage size.
    const uint64_t da_first = make_desc_sw128(base);
    const uint32_t stage_units = stage_bytes >> 4, a_units = a_bytes >> 4;
    const uint32_t b_units = (uint32_t)a.MB * a_units;
    const int last_ksteps = (p.C - (KB - 1) * kStageK + 31) / 32;   // 1..4
    uint32_t s_units = 0;   // s * stage_units
    int s = 0; uint32_t ph = 0;
    int li = 0;
    for (int it = blockIdx.x; it < a.n_items; it += gridDim.x, ++li) {
      const int buf = li & 1;
      const uint32_t aph = (uint32_t)(li >> 1) & 1u;
      bool ok = __all_sync(0xffffffffu, mbar_wait(bar_acc_empty + 8u * buf, aph ^ 1u, abort_p));
      tc_fence_after();
      const uint32_t tacc = tmem_base + (uint32_t)(buf * a.acc_stride);
      for (int kb = 0; kb < KB && ok; ++kb) {
        if (!__all_sync(0xffffffffu, mbar_wait(bar_full + 8u * s, ph, abort_p))) { ok = false; break; }
        if (leader && li == 0 && kb == 0) WINO_ST(g_gemm_trace, trace_step, 3);
        if (leader && li == 0 && kb == KB - 1) WINO_ST(g_gemm_trace, trace_step, 4);
        if (leader && li == 1 && kb == 0) WINO_ST(g_gemm_trace, trace_step, 10);
        if (leader && li == 1 && kb == KB - 1) WINO_ST(g_gemm_trace, trace_step, 11);
        tc_fence_after();
        const uint64_t da0 = da_first + s_units;
        const uint64_t db = da0 + b_units;
        const int ksteps = kb == KB - 1 ? last_ksteps : 4;
        for (int j = 0; j < a.MB; ++j) {
          const uint64_t da = da0 + (uint64_t)(j * (int)a_units);
          const uint32_t td = tacc + (uint32_t)(j * a.BN);
          if (leader) {
            if (ksteps == 4) {
              mma_i8(td, da, db, idesc, kb != 0 ? 1u : 0u);
              mma_i8(td, da + 2u, db + 2u, idesc, 1u);
              mma_i8(td, da + 4u, db + 4u, idesc, 1u);
              mma_i8(td, da + 6u, db + 6u, idesc, 1u);
            } else {
              for (int k = 0; k < ksteps; ++k)
                mma_i8(td, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
            }
          }
        }
        if (leader) mma_commit(bar_empty + 8u * s);   // frees the stage when these MMAs retire
        __syncwarp();
        s_units += stage_units;
        if (++s == a.stages) { s = 0; s_units = 0; ph ^= 1u; }
      }
      if (!ok) { *abort_p = 1u; break; }
      if (leader) mma_commit(bar_acc_full + 8u * buf);  // accumulator complete
      __syncwarp();
    }
  } else {
    // epilogue warps.  small: |M| <= 127^2 * C < 2^22; full: every 32-column chunk
    // of every column block lies inside K (the last block is not ragged).
    const bool small = p.C <= 260;
    const bool full = (p.K % a.BN) == 0 && (a.BN % 32) == 0;
    const bool per_channel = PK;
    // Per-channel multipliers of Q_M: the block's own copy in shared memory (the L1 left
    // beside 200 KB of operand ring does not keep the table while the epilogue's stores
    // stream through it).  The table is written by the host before any launch, so it is
    // read ahead of the dependency wait.
    const float* mult_k = PK ? a.chan + (long)kChMultM * p.K : nullptr;
    if (PK && a.chan_smem) {
      float* tab = reinterpret_cast<float*>(gen + (bars + 16u * (uint32_t)a.stages + 64u - base));
      for (int i = (int)threadIdx.x - 64; i < p.K; i += 32 * kEpiWarps) tab[i] = __ldg(mult_k + i);
      asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
      mult_k = tab;
    }
    griddep_wait();
    if constexpr (LEAN) {
      (void)per_channel; (void)small; (void)full;
      epilogue_loop<true, true, false, false, true>(p, a, out, absmaxM, tmem_base, bar_acc_full,
                                                    bar_acc_empty, abort_p, warp, lane, trace_step);
    } else if constexpr (PK) {
      (void)per_channel;
      if (absmaxM != nullptr)
        epilogue_loop<false, false, true, true>(p, a, out, absmaxM, tmem_base, bar_acc_full,
                                                bar_acc_empty, abort_p, warp, lane, trace_step, mult_k);
      else if (small && full)
        epilogue_loop<true, true, false, true>(p, a, out, absmaxM, tmem_base, bar_acc_full,
                                               bar_acc_empty, abort_p, warp, lane, trace_step, mult_k);
      else
        epilogue_loop<false, false, false, true>(p, a, out, absmaxM, tmem_base, bar_acc_full,
                                                 bar_acc_empty, abort_p, warp, lane, trace_step, mult_k);
    } else if (absmaxM != nullptr)
      epilogue_loop<false, false, true>(p, a, out, absmaxM, tmem_base, bar_acc_full, bar_acc_empty,
                                        abort_p, warp, lane, trace_step);
    else if (small && full)
      epilogue_loop<true, true, false>(p, a, out, absmaxM, tmem_base, bar_acc_full, bar_acc_empty,
                                       abort_p, warp, lane, trace_step);
    else if (full)
      epilogue_loop<false, true, false>(p, a, out, absmaxM, tmem_base, bar_acc_full, bar_acc_empty,
                                        abort_p, warp, lane, trace_step);
    else
      epilogue_loop<false, false, false>(p, a, out, absmaxM, tmem_base, bar_acc_full,
                                         bar_acc_empty, abort_p, warp, lane, trace_step);
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_p != 0u && threadIdx.x == 0) atomicExch(status, -6);  // WINO_ERR_TIMEOUT
  if (threadIdx.x == 0) WINO_ST(g_gemm_trace, trace_step, 9);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)a.tmem_cols);
  }
}

__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_tc(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap mapV,
          const __grid_constant__ CUtensorMap mapU, const GemmTcArgs a, void* __restrict__ out,
          unsigned* __restrict__ absmaxM, int* __restrict__ status) {
  gemm_tc_body<false>(p, &mapV, &mapU, a, out, absmaxM, status);
}
__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_tc_lean(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap mapV,
               const __grid_constant__ CUtensorMap mapU, const GemmTcArgs a, void* __restrict__ out,
               unsigned* __restrict__ absmaxM, int* __restrict__ status) {
  gemm_tc_body<false, true>(p, &mapV, &mapU, a, out, absmaxM, status);
}
__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_tc_per_channel(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap mapV,
                      const __grid_constant__ CUtensorMap mapU, const GemmTcArgs a,
                      void* __restrict__ out, unsigned* __restrict__ absmaxM,
                      int* __restrict__ status) {
  gemm_tc_body<true>(p, &mapV, &mapU, a, out, absmaxM, status);
}

TcGeom tc_geometry(const Params& p, int num_sms) {
  TcGeom g;
  g.BN = p.K >= 256 ? 256 : (p.K + 15) / 16 * 16;
  // narrow layers: several m-blocks share one U_q tile and one 256-column accumulator
  g.MB = (g.BN == 64 || g.BN == 128) ? 256 / g.BN : 1;
  const int n_mblk = (p.T + kBM - 1) / kBM;
  // ... as long as that leaves every CTA at least three items to pipeline
  const int n_nblk0 = (p.K + g.BN - 1) / g.BN;
  while (g.MB > 1 && (p.t * p.t) * ((n_mblk + g.MB - 1) / g.MB) * n_nblk0 < 3 * num_sms) g.MB /= 2;
  const size_t per_stage = (size_t)g.MB * kBM * kStageK + (size_t)g.BN * kStageK;
  g.stages = (int)((196 * 1024) / per_stage);
  const int KB = (p.C + kStageK - 1) / kStageK;
  // one and a half items' worth: with two whole items in the ring the second item's operands
  // compete with the first item's for the path from L2 and delay its accumulator (cfg3: 5.87 us
  // with four stages, 5.74 with three, 6.12 with two)
  if (g.stages > (3 * KB + 1) / 2) g.stages = (3 * KB + 1) / 2;
  if (g.stages > 8) g.stages = 8;
  if (g.stages < 1) g.stages = 1;
  int acc_stride = 32;
  while (acc_stride < g.MB * g.BN) acc_stride *= 2;
  g.tmem_cols = 2 * acc_stride;
  g.smem = 1024 + g.stages * per_stage + 16 * g.stages + 64;
  const int n_mgrp = (n_mblk + g.MB - 1) / g.MB;
  const int items = (p.t * p.t) * n_mgrp * ((p.K + g.BN - 1) / g.BN);
  g.grid = items < num_sms ? items : num_sms;
  return g;
}

int launch_gemm_tc(const Params& p, const LaunchOpt& o, const TcGeom& g, const CUtensorMap& mapV,
                   const CUtensorMap& mapU, void* out, int out_mode, unsigned* absmaxM,
                   int* status, cudaStream_t st) {
  static DeviceOnce once;
  if (int rc = set_max_smem(once, o.device, k_gemm_tc, 227 * 1024)) return rc;
  GemmTcArgs a;
  a.BN = g.BN; a.stages = g.stages; a.tmem_cols = g.tmem_cols; a.acc_stride = g.tmem_cols / 2;
  a.out_mode = out_mode;
  a.MB = g.MB;
  a.n_mblk = ((p.T + kBM - 1) / kBM + g.MB - 1) / g.MB;
  a.n_nblk = (p.K + g.BN - 1) / g.BN;
  a.n_items = p.t * p.t * a.n_mblk * a.n_nblk;
  a.wide_store = (reinterpret_cast<uintptr_t>(out) & 31u) == 0 ? 1 : 0;
  a.chan = o.chan;
  // room for the multipliers behind the ring and the barriers (the ring stops at 196 KB)
  a.chan_smem = (o.chan != nullptr && (size_t)p.K * 4 <= 24 * 1024) ? 1 : 0;
  if (o.chan != nullptr) {
    static DeviceOnce once_pk;
    if (int rc = set_max_smem(once_pk, o.device, k_gemm_tc_per_channel, 227 * 1024)) return rc;
    const size_t smem = g.smem + (a.chan_smem ? (size_t)p.K * 4 : 0);
    return launch_kernel(k_gemm_tc_per_channel, dim3((unsigned)g.grid), dim3(kGemmThreads), smem, st,
                         o.pdl, p, mapV, mapU, a, out, absmaxM, status);
  }
  const bool lean = absmaxM == nullptr && out_mode == kOutMq && p.hi_M == 127.0f && a.wide_store &&
                    p.C <= 260 && p.K % a.BN == 0 && a.BN % 32 == 0;
  if (lean) {
    static DeviceOnce once_lean;
    if (int rc = set_max_smem(once_lean, o.device, k_gemm_tc_lean, 227 * 1024)) return rc;
    return launch_kernel(k_gemm_tc_lean, dim3((unsigned)g.grid), dim3(kGemmThreads), g.smem, st, o.pdl,
                         p, mapV, mapU, a, out, absmaxM, status);
  }
  return launch_kernel(k_gemm_tc, dim3((unsigned)g.grid), dim3(kGemmThreads), g.smem, st, o.pdl, p,
                       mapV, mapU, a, out, absmaxM, status);
}

}  // namespace wino
