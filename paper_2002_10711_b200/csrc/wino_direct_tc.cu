// Direct int8 3x3 convolution, stride 1 or 2, as an implicit GEMM on the tensor cores
// (the lossless "im2row" candidate of the paper's search space, Section 4, without ever
// forming the im2row matrix).  For an output tile of 128 pixels and a block of BN output
// channels,
//     acc[pixel][k] = sum over the nine taps (a, b) and over c of x[n][s*h-1+a][s*w-1+b][c] * w[k][a][b][c],
// i.e. nine GEMM K-slices per channel block.  The A operand of tap (a, b) is the input box
// of the tile shifted by (a-1, b-1), fetched by one 4-D TMA load whose out-of-image part is
// filled with zeros by the hardware (= the zero padding); the B operand is the tap's
// [BN][channels] slice of the weights.  Both land in shared memory as K-major rows of 64 or
// 128 channel bytes with the matching swizzle, `tcgen05.mma.kind::i8` accumulates all
// 9 * C / 32 steps of an item in one tensor-memory accumulator, and sixteen epilogue warps
// apply the output quantizer (or the float output) and write 32-byte row pieces.
//
//   warp 0    : TMA producer (one lane)
//   warp 1    : tensor-memory owner; walks the MMA loop as a whole warp, one elected lane issues
//   warps 2-17: epilogue; warp w reads TMEM lanes 32*(w%4) .. +31 and every fourth 32-column chunk
//
// For stride 2 (even H and W) the input is addressed as [N][H/2][2][W/2][2*C]: a tap then reads
// one row parity and one column parity, again a dense box.
// Narrow layers (one block of output channels, 9 * C * K bytes of weights that fit beside the
// input ring; the 64- and 128-channel layers of the network): the weights are fetched once per
// block and stay in shared memory, and the ring's stages carry input boxes only, three taps
// (one row of the filter) per stage where that fits.  The producer and the MMA warp are
// single threads of control whose every instruction costs ten to twenty cycles, so what
// bounds these layers is the number of copies, waits and commits per item, which this halves.
// Zero points on x or w, odd sizes at stride 2 and channel counts that are not multiples of
// 64 / 32 stay on the ALU kernel (wino_direct.cu).
#include "wino_launch.h"
#include "wino_ptx.cuh"

namespace wino {

namespace {

constexpr int kDtEpiWarps = 16;
constexpr int kDtThreads = 64 + 32 * kDtEpiWarps;

// K-major tile of 64-byte rows with the 64-byte swizzle: start / 16, 8-row group stride
// 512 B, descriptor version 1, layout 4.
__device__ __forceinline__ uint64_t desc_sw64(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (32ull << 32) | (1ull << 46) |
         (4ull << 61);
}

// PK: the weight and output scales vary per output channel (a build of its own: the per-layer
// kernel keeps its one multiplier in a register).
template <bool PK, bool RW>
__device__ __forceinline__ void direct_conv_tc_body(const CUtensorMap& mapX, const CUtensorMap& mapW,
                                                    const DirectTcArgs& a, const float* __restrict__ bias,
                                                    void* __restrict__ y, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t a_bytes = 128u * (uint32_t)a.cB, b_bytes = (uint32_t)a.BN * (uint32_t)a.cB;
  // RW: [9 * KB weight slices][stages x taps_per_stage * KB input boxes]; else [stages x (A, B)]
  const uint32_t res_bytes = RW ? 9u * (uint32_t)a.KB * b_bytes : 0u;
  const uint32_t stage_bytes = RW ? (uint32_t)(a.taps_per_stage * a.KB) * a_bytes : a_bytes + b_bytes;
  const uint32_t ring = base + res_bytes;
  const uint32_t s_bias = ring + (uint32_t)a.stages * stage_bytes;   // K floats
  const uint32_t bars = s_bias + (uint32_t)a.K * (PK ? 8u : 4u);   // PK: K multipliers follow
  const uint32_t bar_full = bars;                           // stages x 8 B
  const uint32_t bar_empty = bar_full + 8u * a.stages;      // stages x 8 B
  const uint32_t bar_acc_full = bar_empty + 8u * a.stages;  // 2 x 8 B
  const uint32_t bar_acc_empty = bar_acc_full + 16u;        // 2 x 8 B
  const uint32_t tmem_slot = bar_acc_empty + 16u;
  const uint32_t abort_slot = tmem_slot + 4u;
  const uint32_t bar_w = bar_acc_empty + 32u;               // RW: the resident weights have landed
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_p = reinterpret_cast<volatile uint32_t*>(gen + (tmem_slot - base));
  volatile uint32_t* abort_p = reinterpret_cast<volatile uint32_t*>(gen + (abort_slot - base));
  float* bias_tab = reinterpret_cast<float*>(gen + (s_bias - base));
  float* mult_tab = bias_tab + a.K;   // PK only
  (void)mult_tab;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tiles = a.nW * a.nH * a.nI;
  const int steps = RW ? 9 / a.taps_per_stage : 9 * a.KB;   // stages per item

  griddep_launch();
  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      mbar_init(bar_full + 8u * s, 1);
      mbar_init(bar_empty + 8u * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_acc_full + 8u * b, 1);
      mbar_init(bar_acc_empty + 8u * b, kDtEpiWarps);
    }
    if (RW) mbar_init(bar_w, 1);
    *abort_p = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tma_prefetch_map(&mapX);
    tma_prefetch_map(&mapW);
  }
  if (warp == 1) tmem_alloc(tmem_slot, (uint32_t)a.tmem_cols);
  // bias in output-code units (or as it is, for the float output); the bias is a parameter of
  // the layer, not an output of the preceding kernel
  for (int k = threadIdx.x; k < a.K; k += blockDim.x) {
    float s_Y_k = a.s_Y;
    if constexpr (PK) {
      // channel k: accumulator scale s_x * s_w[k] (exact in double), output scale s_Y[k]
      const double s_in_k = (double)a.s_x * (double)(a.s_w_K != nullptr ? __ldg(a.s_w_K + k) : a.s_w);
      if (a.s_Y_K != nullptr) s_Y_k = __ldg(a.s_Y_K + k);
      mult_tab[k] = a.out_dtype == 0 ? (float)(s_in_k / (double)s_Y_k) : (float)s_in_k;
    }
    float b = 0.0f;
    if (bias != nullptr)
      b = a.out_dtype == 0 ? (float)((double)__ldg(bias + k) / (double)s_Y_k) : __ldg(bias + k);
    bias_tab[k] = b;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_p;

  if (warp == 0) {
    if (lane == 0) {
      int s = 0, issued = 0; uint32_t ph = 0;
      griddep_wait();
      // (a lone thread retires an instruction every ten to twenty cycles, and a stage's MMAs take
      // about five hundred: everything that does not change inside an item is computed once per
      // item, and the loops carry running coordinates instead of multiplying)
      const int n_stages = a.stages, kblocks = a.KB, cb = a.cB, strided = a.stride != 1;
      if constexpr (RW) {
        // the whole weight tensor, once: slice (tap, channel block) at res + (tap * KB + kb) * b_bytes
        mbar_expect_tx(bar_w, res_bytes);
        uint32_t dst = base;
        for (int tap = 0; tap < 9; ++tap)
          for (int kb = 0; kb < kblocks; ++kb, dst += b_bytes)
            tma_load_3d(dst, &mapW, bar_w, kb * cb, tap, 0);
      }
      const int tps = RW ? a.taps_per_stage : 1;
      // item -> (channel block, tile column, tile row, image group): divided out once, then
      // advanced by the grid's stride with carries (an integer division costs this thread some
      // forty instructions, and narrow layers have a dozen items per block)
      const int nW = a.nW, nH = a.nH, nI = a.nI;
      int nb = (int)blockIdx.x / n_tiles;
      int tw, th, ti;
      {
        const int tile = (int)blockIdx.x - nb * n_tiles;
        tw = tile % nW; th = (tile / nW) % nH; ti = tile / (nW * nH);
      }
      const int step_nb = (int)gridDim.x / n_tiles, step_r = (int)gridDim.x - step_nb * n_tiles;
      const int d_w = step_r % nW, d_h = (step_r / nW) % nH, d_i = step_r / (nW * nH);
      int in_stage = 0;
      for (int it = blockIdx.x; it < a.n_items; it += gridDim.x) {
        const int w0 = tw * a.BW, h0 = th * a.BH, i0 = ti * a.BI, k_row = nb * a.BN;
        tw += d_w; if (tw >= nW) { tw -= nW; ++th; }
        th += d_h; if (th >= nH) { th -= nH; ++ti; }
        ti += d_i; nb += step_nb; if (ti >= nI) { ti -= nI; ++nb; }
        bool ok = true;
        int tap = 0;
        for (int ta = 0; ta < 3 && ok; ++ta) {
          // stride 1: input row h0 - 1 + ta.  Stride 2: input row 2*ho - 1 + ta, i.e. (half-row
          // ho - 1, parity 1), (ho, 0), (ho, 1) for ta = 0, 1, 2
          const int hc = strided ? h0 + (ta == 0 ? -1 : 0) : h0 - 1 + ta;
          const int prow = ta == 1 ? 0 : 1;
          for (int tb = 0; tb < 3 && ok; ++tb, ++tap) {
            const int wc = strided ? w0 + (tb == 0 ? -1 : 0) : w0 - 1 + tb;
            const int c_base = strided ? (tb == 1 ? 0 : a.C) : 0;
            int c_off = 0;
            if constexpr (RW) {
              // a stage holds the boxes of `tps` consecutive taps: it is opened by its first
              // tap and advanced after its last
              const uint32_t fb = bar_full + 8u * s;
              if (in_stage == 0) {
                if (issued >= n_stages && !mbar_wait(bar_empty + 8u * s, ph ^ 1u, abort_p)) { ok = false; break; }
                ++issued;
                mbar_expect_tx(fb, stage_bytes);
              }
              uint32_t sa = ring + (uint32_t)s * stage_bytes + (uint32_t)(in_stage * kblocks) * a_bytes;
              for (int kb = 0; kb < kblocks; ++kb, c_off += cb, sa += a_bytes) {
                if (!strided) tma_load_4d(sa, &mapX, fb, c_off, wc, hc, i0);
                else tma_load_5d(sa, &mapX, fb, c_base + c_off, wc, prow, hc, i0);
              }
              if (++in_stage == tps) {
                in_stage = 0;
                if (++s == n_stages) { s = 0; ph ^= 1u; }
              }
              continue;
            }
            for (int kb = 0; kb < kblocks; ++kb, c_off += cb) {
              if (issued >= n_stages && !mbar_wait(bar_empty + 8u * s, ph ^ 1u, abort_p)) { ok = false; break; }
              ++issued;
              const uint32_t sa = base + (uint32_t)s * stage_bytes;
              const uint32_t fb = bar_full + 8u * s;
              mbar_expect_tx(fb, stage_bytes);
              // pixels outside the image (the padding ring, ragged tile edges, images past N)
              // arrive as zeros
              if (!strided) tma_load_4d(sa, &mapX, fb, c_off, wc, hc, i0);
              else tma_load_5d(sa, &mapX, fb, c_base + c_off, wc, prow, hc, i0);
              tma_load_3d(sa + a_bytes, &mapW, fb, c_off, tap, k_row);
              if (++s == n_stages) { s = 0; ph ^= 1u; }
            }
          }
        }
        if (!ok) { *abort_p = 1u; break; }
      }
    }
  } else if (warp == 1) {
    const bool leader = elect_one();
    const uint32_t idesc = make_idesc_i8(128, a.BN);
    const int ksteps = a.cB / 32;
    // descriptors are linear in the tile address (units of 16 bytes): the first tile's, once,
    // plus running offsets, instead of rebuilding them in every stage
    const uint64_t d_first = a.cB == 128 ? make_desc_sw128(base) : desc_sw64(base);
    const uint32_t a_units = a_bytes >> 4, b_units = b_bytes >> 4, stage_units = stage_bytes >> 4;
    const uint32_t ring_units = (ring - base) >> 4;
    uint32_t s_units = 0;   // s * stage_units
    int s = 0; uint32_t ph = 0;
    int li = 0;
    bool w_ok = true;
    if constexpr (RW) w_ok = __all_sync(0xffffffffu, mbar_wait(bar_w, 0u, abort_p));
    if (!w_ok) *abort_p = 1u;
    for (int it = blockIdx.x; it < a.n_items && w_ok; it += gridDim.x, ++li) {
      const int buf = li & 1;
      const uint32_t aph = (uint32_t)(li >> 1) & 1u;
      bool ok = __all_sync(0xffffffffu, mbar_wait(bar_acc_empty + 8u * buf, aph ^ 1u, abort_p));
      tc_fence_after();
      const uint32_t tacc = tmem_base + (uint32_t)(buf * a.acc_stride);
      for (int st = 0; st < steps && ok; ++st) {
        if (!__all_sync(0xffffffffu, mbar_wait(bar_full + 8u * s, ph, abort_p))) { ok = false; break; }
        tc_fence_after();
        if constexpr (RW) {
          // the stage's boxes in tap order against the resident slices of the same taps
          const int per_stage = a.taps_per_stage * a.KB;
          uint64_t da = d_first + (ring_units + s_units);
          uint64_t db = d_first + (uint32_t)(st * per_stage) * b_units;
          for (int j = 0; j < per_stage; ++j, da += a_units, db += b_units) {
            if (leader)
              for (int k = 0; k < ksteps; ++k)
                mma_i8(tacc, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (st | j | k) != 0 ? 1u : 0u);
          }
          if (leader) mma_commit(bar_empty + 8u * s);
          __syncwarp();
          s_units += stage_units;
          if (++s == a.stages) { s = 0; s_units = 0; ph ^= 1u; }
          continue;
        }
        const uint64_t da = d_first + s_units;
        const uint64_t db = da + a_units;
        if (leader) {
          for (int k = 0; k < ksteps; ++k)
            mma_i8(tacc, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (st | k) != 0 ? 1u : 0u);
          mma_commit(bar_empty + 8u * s);   // frees the stage when these MMAs retire
        }
        __syncwarp();
        s_units += stage_units;
        if (++s == a.stages) { s = 0; s_units = 0; ph ^= 1u; }
      }
      if (!ok) { *abort_p = 1u; break; }
      if (leader) mma_commit(bar_acc_full + 8u * buf);  // accumulator complete
      __syncwarp();
    }
  } else {
    const int quad = warp & 3;
    const int sub = (warp - 2) >> 2;
    const int r = quad * 32 + lane;
    const int wi = r % a.BW, hi = (r / a.BW) % a.BH, ii = r / (a.BW * a.BH);
    const float lo = a.lo_Y, hi_c = a.hi_Y;
    griddep_wait();
    int li = 0;
    for (int it = blockIdx.x; it < a.n_items; it += gridDim.x, ++li) {
      const int nb = it / n_tiles, tile = it - nb * n_tiles;
      const int tw = tile % a.nW, th = (tile / a.nW) % a.nH, ti = tile / (a.nW * a.nH);
      const int n = ti * a.BI + ii, ho = th * a.BH + hi, wo = tw * a.BW + wi;
      const bool valid = n < a.N && ho < a.H && wo < a.W;
      const long pix = ((long)n * a.H + ho) * a.W + wo;
      const int buf = li & 1;
      const uint32_t aph = (uint32_t)(li >> 1) & 1u;
      if (!__all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8u * buf, aph, abort_p))) {
        *abort_p = 1u;
        break;
      }
      tc_fence_after();
      const uint32_t tacc = tmem_base + (uint32_t)(buf * a.acc_stride) + ((uint32_t)(quad * 32) << 16);
      for (int col = sub * 32; col < a.BN; col += 128) {
        uint32_t acc[32];
        tmem_ld32(tacc + (uint32_t)col, acc);
        tmem_ld_wait();
        if (!valid) continue;
        const int k0 = nb * a.BN + col;
        if (a.out_dtype == 0) {
          uint32_t w[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            uint32_t word = 0u;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float yf = __fmaf_rn(__int2float_rn((int)acc[4 * q + e]),
                                         PK ? mult_tab[k0 + 4 * q + e] : a.mult, bias_tab[k0 + 4 * q + e]);
              const float rr = __fadd_rn(fminf(fmaxf(yf, lo), hi_c), kMagic);
              word |= ((uint32_t)(magic_to_int(rr) + a.z_Y) & 0xFFu) << (8 * e);
            }
            w[q] = word;
          }
          uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<int8_t*>(y) + pix * a.K + k0);
          asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]),
                       "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                       : "memory");
        } else {
          float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(y) + pix * a.K + k0);
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            float4 v;
            v.x = __fmaf_rn(__int2float_rn((int)acc[4 * q + 0]), PK ? mult_tab[k0 + 4 * q + 0] : a.s_in, bias_tab[k0 + 4 * q + 0]);
            v.y = __fmaf_rn(__int2float_rn((int)acc[4 * q + 1]), PK ? mult_tab[k0 + 4 * q + 1] : a.s_in, bias_tab[k0 + 4 * q + 1]);
            v.z = __fmaf_rn(__int2float_rn((int)acc[4 * q + 2]), PK ? mult_tab[k0 + 4 * q + 2] : a.s_in, bias_tab[k0 + 4 * q + 2]);
            v.w = __fmaf_rn(__int2float_rn((int)acc[4 * q + 3]), PK ? mult_tab[k0 + 4 * q + 3] : a.s_in, bias_tab[k0 + 4 * q + 3]);
            dst[q] = v;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_acc_empty + 8u * buf);
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_p != 0u && threadIdx.x == 0) atomicExch(status, -6);  // WINO_ERR_TIMEOUT
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)a.tmem_cols);
  }
}

__global__ void __launch_bounds__(kDtThreads, 1)
k_direct_conv_tc(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW,
                 const DirectTcArgs a, const float* __restrict__ bias, void* __restrict__ y,
                 int* __restrict__ status) {
  direct_conv_tc_body<false, false>(mapX, mapW, a, bias, y, status);
}
__global__ void __launch_bounds__(kDtThreads, 1)
k_direct_conv_tc_resident(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW,
                          const DirectTcArgs a, const float* __restrict__ bias, void* __restrict__ y,
                          int* __restrict__ status) {
  direct_conv_tc_body<false, true>(mapX, mapW, a, bias, y, status);
}
__global__ void __launch_bounds__(kDtThreads, 1)
k_direct_conv_tc_resident_per_channel(const __grid_constant__ CUtensorMap mapX,
                                      const __grid_constant__ CUtensorMap mapW, const DirectTcArgs a,
                                      const float* __restrict__ bias, void* __restrict__ y,
                                      int* __restrict__ status) {
  direct_conv_tc_body<true, true>(mapX, mapW, a, bias, y, status);
}
__global__ void __launch_bounds__(kDtThreads, 1)
k_direct_conv_tc_per_channel(const __grid_constant__ CUtensorMap mapX,
                             const __grid_constant__ CUtensorMap mapW, const DirectTcArgs a,
                             const float* __restrict__ bias, void* __restrict__ y,
                             int* __restrict__ status) {
  direct_conv_tc_body<true, false>(mapX, mapW, a, bias, y, status);
}

// One status word per device for the plan-less direct convolution.
__device__ int g_direct_status;

}  // namespace

bool direct_tc_supported(int C, int K, int H, int W, int stride, int z_x, int z_w) {
  if (z_x != 0 || z_w != 0 || C % 64 != 0 || K % 32 != 0 || K > 2048) return false;
  return stride == 1 || (stride == 2 && H % 2 == 0 && W % 2 == 0);
}

DirectTcArgs direct_tc_geometry(int N, int C, int H_in, int W_in, int K, int stride, int num_sms) {
  DirectTcArgs a = {};
  const int H = (H_in - 1) / stride + 1, W = (W_in - 1) / stride + 1;   // output size
  a.N = N; a.C = C; a.H = H; a.W = W; a.K = K; a.stride = stride;
  auto pow2_ceil = [](int v) { int p = 1; while (p < v) p *= 2; return p; };
  a.BW = pow2_ceil(W) < 16 ? pow2_ceil(W) : 16;
  a.BH = pow2_ceil(H) < 128 / a.BW ? pow2_ceil(H) : 128 / a.BW;
  a.BI = 128 / (a.BW * a.BH);
  a.nW = (W + a.BW - 1) / a.BW; a.nH = (H + a.BH - 1) / a.BH; a.nI = (N + a.BI - 1) / a.BI;
  a.cB = C % 128 == 0 ? 128 : 64;
  a.KB = C / a.cB;
  a.BN = K % 256 == 0 ? 256 : K % 128 == 0 ? 128 : K % 64 == 0 ? 64 : 32;
  const int tiles = a.nW * a.nH * a.nI;
  // enough items for every SM, as long as the blocks stay at least 64 channels wide
  while (a.BN > 64 && tiles * (K / a.BN) < (num_sms * 4) / 5) a.BN /= 2;
  a.n_nblk = K / a.BN;
  a.n_items = tiles * a.n_nblk;
  const size_t a_bytes = (size_t)128 * a.cB, b_bytes = (size_t)a.BN * a.cB;
  const size_t stage = a_bytes + b_bytes;
  a.stages = (int)((192 * 1024) / stage);
  if (a.stages > 8) a.stages = 8;
  // resident weights: one block of output channels, and room for at least three stages of
  // three taps each beside them (with less room the shallower ring costs more than the saved
  // copies gain: 19.1 against 17.8 us on the 128-channel 16x16 layer at batch 256)
  const size_t budget = 200 * 1024, res = 9 * (size_t)a.KB * b_bytes;
  const size_t st3 = 3 * (size_t)a.KB * a_bytes;
  a.w_resident = 0;
  a.taps_per_stage = 1;
  // (a whole item, nine taps, per stage measured the same as three: 36.2 against 36.6 us on
  // the 64-channel 32x32 layer.  What then bounds these layers is the rate at which the copy
  // engine delivers box rows, about one per two cycles per SM whatever their width, and
  // 64-channel rows are 64 bytes)
  if (a.n_nblk == 1 && res + 3 * st3 <= budget) {
    a.w_resident = 1;
    a.taps_per_stage = 3;
    a.stages = (int)((budget - res) / st3);
    if (a.stages > 8) a.stages = 8;
  }
  int acc_stride = 32;
  while (acc_stride < a.BN) acc_stride *= 2;
  a.acc_stride = acc_stride;
  a.tmem_cols = 2 * acc_stride;
  return a;
}

int* direct_tc_status_word(int device) {
  static std::mutex mu;
  static int* addr[64];
  std::lock_guard<std::mutex> lock(mu);
  const int d = device >= 0 && device < 64 ? device : 0;
  if (addr[d] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_direct_status) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    addr[d] = static_cast<int*>(p);
  }
  return addr[d];
}

int launch_direct_conv_tc(const DirectTcArgs& a, int device, int num_sms, const CUtensorMap& mapX,
                          const CUtensorMap& mapW, const float* bias, void* y, cudaStream_t st) {
  int* status = direct_tc_status_word(device);
  if (status == nullptr) return -5;
  const size_t a_bytes = (size_t)128 * a.cB, b_bytes = (size_t)a.BN * a.cB;
  const size_t ring = a.w_resident
                          ? 9 * (size_t)a.KB * b_bytes + (size_t)a.stages * a.taps_per_stage * a.KB * a_bytes
                          : (size_t)a.stages * (a_bytes + b_bytes);
  const bool pk = a.s_w_K != nullptr || a.s_Y_K != nullptr;
  const size_t smem = 1024 + ring + (size_t)a.K * (pk ? 8 : 4) + 16 * (size_t)a.stages + 64;
  const int grid = a.n_items < num_sms ? a.n_items : num_sms;
  auto go = [&](auto kernel, DeviceOnce& once) -> int {
    if (int rc = set_max_smem(once, device, kernel, 227 * 1024)) return rc;
    return launch_kernel(kernel, dim3((unsigned)grid), dim3(kDtThreads), smem, st, true, mapX, mapW, a,
                         bias, y, status);
  };
  static DeviceOnce once, once_pk, once_rw, once_rw_pk;
  if (a.w_resident) return pk ? go(k_direct_conv_tc_resident_per_channel, once_rw_pk)
                              : go(k_direct_conv_tc_resident, once_rw);
  return pk ? go(k_direct_conv_tc_per_channel, once_pk) : go(k_direct_conv_tc, once);
}

}  // namespace wino
