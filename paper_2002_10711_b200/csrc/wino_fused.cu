// Fully fused F(2x2, 3x3) layer (paper: Eq. 1 with the quantizers of Fig. 2) for
// narrow layers: C in {32, 64}, K <= 64, Cook-Toom matrices.  One kernel does
// input transform, Q_V, the sixteen channel contractions on tcgen05, Q_M, the
// output transform, bias and Q_Y; V_q and m_q never leave the SM.
//
// Why F2 only: the output transform of a (tile, k) pair needs all t*t Hadamard
// sums of that pair, so a fused CTA has to hold t*t accumulators of its
// (tile-block x k-block) in tensor memory at once.  128 lanes x 512 columns give
// 16 accumulators x 32 columns for F2; F4 and F6 would be left with 14 and 8
// columns, below the smallest MMA.
//
// A CTA owns blocks of 128 consecutive tiles (persistent, stride gridDim.x):
//   workers (16 warps)  B^T d B for all 16 positions from registers (inputs read
//                       straight from global memory, padding by predicate), Q_V,
//                       int8 A-operand tiles written to shared memory in the
//                       64-byte-swizzled K-major layout the MMA expects;
//   control warp        U_q for all positions fetched once by TMA (same
//                       swizzle); per 32 output channels: 16 x (C/32) MMAs
//                       128x32x32 of kind::i8, one TMEM accumulator per position;
//   workers             tcgen05.ld per row of positions, Q_M, R = m A, Y = A^T R
//                       in the contract's chain order, bias, Q_Y, stores.
#include "wino_launch.h"
#include "wino_ptx.cuh"
#include "wino_transform_math.cuh"

namespace wino {

namespace {

constexpr int kFusedWorkers = 16;                       // warps
constexpr int kFusedThreads = 32 * (1 + kFusedWorkers);
constexpr uint32_t kATile = 128 * 64;                   // one position: 128 tiles x 64 B
constexpr uint32_t kBTile = 64 * 64;                    // one position: 64 k x 64 B

// K-major operand tile of 64-byte rows with the 64-byte swizzle: start / 16,
// 8-row group stride 512 B, descriptor version 1, layout 4.
__device__ __forceinline__ uint64_t make_desc_sw64(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (32ull << 32) | (1ull << 46) |
         (4ull << 61);
}
// Byte offset of (row, byte) inside such a tile: 16-byte chunk index XOR row bits 1..2.
__device__ __forceinline__ uint32_t sw64_offset(int row, int byte) {
  const int chunk = (byte >> 4) ^ ((row >> 1) & 3);
  return (uint32_t)(row * 64 + chunk * 16 + (byte & 15));
}
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t (&r)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr)
               : "memory");
}

}  // namespace

__global__ void __launch_bounds__(kFusedThreads, 1)
k_fused_f2(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap mapU,
           const int8_t* __restrict__ x, const float* __restrict__ bias, void* __restrict__ y,
           float s_Y, int n_mblk, int* __restrict__ status, int* __restrict__ dbgM) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = base;                         // 16 x kATile
  const uint32_t sB = sA + 16u * kATile;            // 16 x kBTile
  const uint32_t sBias = sB + 16u * kBTile;         // 64 floats: bias / s_Y
  const uint32_t bar_b = sBias + 256u;              // U_q landed
  const uint32_t bar_a_full = bar_b + 8u;           // workers -> control: A tiles written
  const uint32_t bar_acc = bar_a_full + 8u;         // control -> workers: 4 barriers, one per row of positions
  const uint32_t bar_tmem_free = bar_acc + 32u;     // workers -> control: accumulators drained
  const uint32_t tmem_slot = bar_tmem_free + 8u;
  const uint32_t abort_slot = tmem_slot + 4u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gen + (tmem_slot - base));
  volatile uint32_t* abort_p = reinterpret_cast<volatile uint32_t*>(gen + (abort_slot - base));
  float* bias_s = reinterpret_cast<float*>(gen + (sBias - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ksteps = p.C / 32;                      // 1 or 2
  const int n_nblk = (p.K + 31) / 32;               // 1 or 2

  griddep_launch();
  if (threadIdx.x == 0) {
    mbar_init(bar_b, 1);
    mbar_init(bar_a_full, kFusedWorkers);
    for (int i = 0; i < 4; ++i) mbar_init(bar_acc + 8u * i, 1);
    mbar_init(bar_tmem_free, kFusedWorkers);
    *abort_p = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) tmem_alloc(tmem_slot, 512u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_p;
  griddep_wait();

  if (warp == 0) {
    // ---------------- control warp: TMA for U_q, MMA issue ----------------
    if (lane == 0) {
      mbar_expect_tx(bar_b, 16u * kBTile);
      for (int xi = 0; xi < 16; ++xi) tma_load_3d(sB + (uint32_t)xi * kBTile, &mapU, bar_b, 0, 0, xi);
      bool ok = mbar_wait(bar_b, 0u, abort_p);
      const uint32_t idesc = make_idesc_i8(128, 32);
      uint32_t it = 0, round = 0;   // round counts (m-block, n-block) pairs
      for (int mb = blockIdx.x; mb < n_mblk && ok; mb += gridDim.x, ++it) {
        if (!mbar_wait(bar_a_full, it & 1u, abort_p)) { ok = false; break; }
        tc_fence_after();
        for (int nb = 0; nb < n_nblk; ++nb, ++round) {
          // the previous round's accumulators must have been read out
          if (round > 0 && !mbar_wait(bar_tmem_free, (round - 1u) & 1u, abort_p)) { ok = false; break; }
          tc_fence_after();
          for (int xi = 0; xi < 16; ++xi) {
            const uint64_t da = make_desc_sw64(sA + (uint32_t)xi * kATile);
            const uint64_t db = make_desc_sw64(sB + (uint32_t)xi * kBTile + (uint32_t)nb * (32u * 64u));
            for (int k = 0; k < ksteps; ++k)
              mma_i8(tmem_base + (uint32_t)(xi * 32), da + (uint64_t)(k * 2), db + (uint64_t)(k * 2),
                     idesc, k != 0 ? 1u : 0u);
            // a row of four positions is complete: its epilogue may start while the
            // remaining rows are still being multiplied
            if ((xi & 3) == 3) mma_commit(bar_acc + 8u * (uint32_t)(xi >> 2));
          }
        }
      }
      if (!ok) *abort_p = 1u;
    }
  } else {
    // ---------------- worker warps ----------------
    const int wid = threadIdx.x - 32;               // 0 .. 511
    for (int k = wid; k < 64; k += 32 * kFusedWorkers)
      bias_s[k] = (bias != nullptr && k < p.K && p.out_dtype == 0)
                      ? (float)((double)__ldg(bias + k) / (double)s_Y) : 0.0f;
    asm volatile("bar.sync 1, 512;" ::: "memory");   // workers only: bias_s is complete
    const int C4 = p.C >> 2;
    const int tasks = 128 * C4;                     // (tile, 4-channel group) pairs per block
    const uint32_t* x32 = reinterpret_cast<const uint32_t*>(x);
    const uint32_t zword = ((uint32_t)(p.z_x & 0xFF) * 0x01010101u) ^ 0x80808080u;
    const float ubias = 8388736.0f + (float)p.z_x;
    const int quad = warp & 3;
    const int sub = (warp - 1) >> 2;                // 8 output channels per sub
    uint32_t it = 0, round = 0;
    bool ok = true;
    for (int mb = blockIdx.x; mb < n_mblk && ok; mb += gridDim.x, ++it) {
      // the MMAs of the previous block must be done reading the A tiles
      // (implied: its last accumulator round was observed complete below)
      // ---- input transform: A tiles for all 16 positions ----
      // loads of the next task are issued before the current one is transformed
      auto load_task = [&](int task, uint32_t (&wd)[16]) {
        const int c4 = task % C4, tau = mb * 128 + task / C4;
        if (task >= tasks || tau >= p.T) {
#pragma unroll
          for (int i = 0; i < 16; ++i) wd[i] = zword;
          return;
        }
        const int tw = tau % p.TW;
        const int th = (tau / p.TW) % p.TH;
        const int n = tau / (p.TW * p.TH);
        // one 64-bit base; row / column offsets are 32-bit, coordinates clamped
        // into the image and validity applied as a mask afterwards
        const uint32_t* xb = x32 + (long)n * p.H * p.W * C4 + c4;
        int roff[4], coff[4];
        uint32_t rmask[4], cmask[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          const int h = th * 2 - 1 + a, wv = tw * 2 - 1 + a;
          rmask[a] = (h >= 0 && h < p.H) ? 0xFFFFFFFFu : 0u;
          cmask[a] = (wv >= 0 && wv < p.W) ? 0xFFFFFFFFu : 0u;
          roff[a] = min(max(h, 0), p.H - 1) * p.W * C4;
          coff[a] = min(max(wv, 0), p.W - 1) * C4;
        }
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            const uint32_t v = __ldg(xb + (roff[a] + coff[b])) ^ 0x80808080u;
            const uint32_t mk = rmask[a] & cmask[b];
            wd[a * 4 + b] = (v & mk) | (zword & ~mk);
          }
      };
      uint32_t wd[16];
      load_task(wid, wd);
      for (int task = wid; task < tasks; task += 32 * kFusedWorkers) {
        const int c4 = task % C4, tl = task / C4;
        uint32_t wn[16];
        load_task(task + 32 * kFusedWorkers, wn);
        uint32_t out[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) out[i] = 0u;
        // tiles past the end carry zero patches; their rows are never stored
#pragma unroll 1
        for (int ch = 0; ch < 4; ++ch) {
          const uint32_t sel_in = 0x7440u | (uint32_t)ch;
          const uint32_t sel_out = insert_selector(ch);
          float V[16];
          input_transform_2d<2, kExact>(p, [&](int l, float (&dcol)[4]) {
#pragma unroll
            for (int a = 0; a < 4; ++a) dcol[a] = byte_to_float_sel(wd[a * 4 + l], sel_in, ubias);
          }, V);
#pragma unroll
          for (int xi = 0; xi < 16; ++xi) {
            const float r = quant_magic(V[xi], p.mult_V, p.lo_V, p.hi_V);
            out[xi] = __byte_perm(out[xi], __float_as_uint(r), sel_out);
          }
        }
        const uint32_t off = sw64_offset(tl, c4 * 4);
#pragma unroll
        for (int xi = 0; xi < 16; ++xi) sts32(sA + (uint32_t)xi * kATile + off, out[xi]);
#pragma unroll
        for (int i = 0; i < 16; ++i) wd[i] = wn[i];
      }
      fence_async_smem();      // generic-proxy writes -> visible to the tensor core's async reads
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_a_full);

      // ---- per 32 output channels: drain accumulators, output transform, store ----
      const int tau = mb * 128 + quad * 32 + lane;
      const bool row_ok = tau < p.T;
      const int tw = tau % p.TW;
      const int th = (tau / p.TW) % p.TH;
      const int n = tau / (p.TW * p.TH);
      const long obase = (((long)n * p.H + th * 2) * p.W + tw * 2) * p.K;   // pixel (0,0) of the tile
      for (int nb = 0; nb < n_nblk; ++nb, ++round) {
        // wait for a row of positions: lane 0 polls (bounded), every lane then
        // observes the completed phase once
        auto wait_row = [&](int i) -> bool {
          int got = 1;
          if (lane == 0) got = mbar_wait(bar_acc + 8u * (uint32_t)i, round & 1u, abort_p) ? 1 : 0;
          if (__shfl_sync(0xffffffffu, got, 0) == 0) return false;
          (void)mbar_try_wait(bar_acc + 8u * (uint32_t)i, round & 1u);
          tc_fence_after();
          return true;
        };
        const uint32_t tlane = tmem_base + ((uint32_t)(quad * 32) << 16);
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          const int kc = nb * 32 + sub * 8 + half * 4;         // first of 4 output channels
          float Y[2][2][4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {                        // row of positions (i, 0..3)
            if (half == 0 && !wait_row(i)) { ok = false; break; }
            uint32_t acc[4][4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
              tmem_ld4(tlane + (uint32_t)((i * 4 + j) * 32 + sub * 8 + half * 4), acc[j]);
            tmem_ld_wait();
            if (dbgM != nullptr && row_ok) {   // debugging aid: the int32 sums M[xi][tau][k]
#pragma unroll
              for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int q = 0; q < 4; ++q)
                  if (kc + q < p.K)
                    dbgM[((long)(i * 4 + j) * p.T + tau) * p.K + kc + q] = (int)acc[j][q];
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              float mrow[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                // |M| <= 127^2 * 64 < 2^22: exact conversion by one add and one subtract
                const float f = small_int_to_float((int)acc[j][q]);
                mrow[j] = p.qM_enabled ? magic_to_float(quant_magic(f, p.mult_M, p.lo_M, p.hi_M)) : f;
              }
              // R = m A (right factor first): chains over j with A^T rows (1,1,1,0), (0,1,-1,1)
              const float R0 = __fadd_rn(__fadd_rn(mrow[0], mrow[1]), mrow[2]);
              const float R1 = __fadd_rn(__fsub_rn(mrow[1], mrow[2]), mrow[3]);
              // Y = A^T R: chains over i in ascending order
              if (i == 0) {
                Y[0][0][q] = R0; Y[0][1][q] = R1;
              } else if (i == 1) {
                Y[0][0][q] = __fadd_rn(Y[0][0][q], R0); Y[0][1][q] = __fadd_rn(Y[0][1][q], R1);
                Y[1][0][q] = R0; Y[1][1][q] = R1;
              } else if (i == 2) {
                Y[0][0][q] = __fadd_rn(Y[0][0][q], R0); Y[0][1][q] = __fadd_rn(Y[0][1][q], R1);
                Y[1][0][q] = __fsub_rn(Y[1][0][q], R0); Y[1][1][q] = __fsub_rn(Y[1][1][q], R1);
              } else {
                Y[1][0][q] = __fadd_rn(Y[1][0][q], R0); Y[1][1][q] = __fadd_rn(Y[1][1][q], R1);
              }
            }
          }
          if (!ok) break;
          if (row_ok && kc < p.K) {
#pragma unroll
            for (int ip = 0; ip < 2; ++ip)
#pragma unroll
              for (int jp = 0; jp < 2; ++jp) {
                const int h = th * 2 + ip, wv = tw * 2 + jp;
                if (h >= p.H || wv >= p.W) continue;
                const long o = obase + (long)((ip * p.W + jp) * p.K + kc);
                if (p.out_dtype == 0) {
                  uint32_t word = 0u;
#pragma unroll
                  for (int q = 0; q < 4; ++q) {
                    const float yf = __fmaf_rn(Y[ip][jp][q], p.mult_Y, bias_s[kc + q]);
                    const float r = __fadd_rn(fminf(fmaxf(yf, p.lo_Y), p.hi_Y), kMagic);
                    word |= ((uint32_t)(magic_to_int(r) + p.z_Y) & 0xFFu) << (8 * q);
                  }
                  *reinterpret_cast<uint32_t*>(reinterpret_cast<int8_t*>(y) + o) = word;
                } else {
#pragma unroll
                  for (int q = 0; q < 4; ++q) {
                    const float b = bias != nullptr ? __ldg(bias + kc + q) : 0.0f;
                    reinterpret_cast<float*>(y)[o + q] = __fmaf_rn(Y[ip][jp][q], p.s_acc, b);
                  }
                }
              }
          }
        }
        if (!ok) break;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tmem_free);
      }
    }
    if (!ok) *abort_p = 1u;
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_p != 0u && threadIdx.x == 0) atomicExch(status, -6);  // WINO_ERR_TIMEOUT
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512u);
  }
}

bool fused_f2_supported(const Params& p, bool std_mats) {
  return p.m == 2 && std_mats && (p.C == 32 || p.C == 64) && p.K % 16 == 0 && p.K <= 64;
}

int launch_fused_f2(const Params& p, const LaunchOpt& o, const CUtensorMap& mapU, const int8_t* x,
                    const float* bias, void* y, float s_Y, int num_sms, int* status, int* dbgM,
                    cudaStream_t st) {
  const size_t smem = 1024 + 16 * (size_t)kATile + 16 * (size_t)kBTile + 256 + 128;
  static DeviceOnce once;
  if (int rc = set_max_smem(once, o.device, k_fused_f2, smem)) return rc;
  const int n_mblk = (p.T + 127) / 128;
  const int grid = n_mblk < num_sms ? n_mblk : num_sms;
  return launch_kernel(k_fused_f2, dim3((unsigned)grid), dim3(kFusedThreads), smem, st, o.pdl, p,
                       mapU, x, bias, y, s_Y, n_mblk, status, dbgM);
}

}  // namespace wino
