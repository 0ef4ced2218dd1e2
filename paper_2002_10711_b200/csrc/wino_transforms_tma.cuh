// TMA-staged variants of the input and output transform kernels (paper: Eq. 1,
// Fig. 2, stages 1 and 4).  A block owns G consecutive tiles x CC channels:
//   - the (m+2)x(m+2)xCC input patches (or the t*t x G x CC block of m_q) arrive
//     in shared memory by TMA; for the input, coordinates may start at -1 and
//     run past the image: the hardware fills those bytes with zero, which is
//     the padding (valid when the input zero point is 0);
//   - every thread transforms four channels from registers, reading and writing
//     shared memory at compile-time offsets;
//   - the result leaves by one TMA store (rows past the last tile, or pixels past
//     the image edge, are clipped by the hardware).
// Compared with the pointer-based kernels this removes nearly all integer
// address arithmetic, which was a third of their instructions.
#pragma once
#include "wino_ptx.cuh"
#include "wino_trace.cuh"

namespace wino {

template <int CPT>
__device__ __forceinline__ uint32_t lds_pack(uint32_t addr) {
  if constexpr (CPT == 4) return lds32(addr);
  else if constexpr (CPT == 2) {
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
    return (uint32_t)v;
  } else {
    uint32_t v;   // one channel per thread: the sign-extended code itself
    asm volatile("ld.shared.s8 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
  }
}
template <int CPT>
__device__ __forceinline__ void sts_pack(uint32_t addr, uint32_t v) {
  if constexpr (CPT == 4) sts32(addr, v);
  else if constexpr (CPT == 2) {
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"((uint16_t)v) : "memory");
  } else {
    asm volatile("st.shared.u8 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
  }
}

#ifdef WINO_TRACE
static __device__ TraceTable g_in_trace, g_out_trace;
#endif
#if WINO_M == 4
WINO_ST_READER(wino_trace_input, g_in_trace)
WINO_ST_READER(wino_trace_output, g_out_trace)
#endif

// Blocks per SM asked of the compiler.  One channel per thread: a full SM of threads (2048),
// i.e. at most 32 registers each.  The F2 and F4 output transforms fit that without spilling
// (F6 does not and is left alone).  The input
// transform does not (it spills some sixty words), so it exists in two builds and the launcher
// takes the 32-register one only where it turns a grid of slightly more than one wave into a
// single wave: the 2048 blocks of a 256-channel, 1024-tile layer are then resident together,
// where otherwise a second, nearly empty wave lengthened the kernel by a quarter.
constexpr int tma_min_blocks(int threads, int cpt, bool cap) {
  return (cpt == 1 && cap) ? (2048 / threads > 32 ? 32 : 2048 / threads) : 1;
}

template <int M, int MODE, int CC, int G, int CPT, bool CAP>
__global__ void __launch_bounds__((CC / CPT) * G, tma_min_blocks((CC / CPT) * G, CPT, CAP))
k_input_transform_tma(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap mapX,
                      const __grid_constant__ CUtensorMap mapV, int* __restrict__ status,
                      const uint8_t* __restrict__ l2_hint, uint32_t l2_hint_bytes) {
  constexpr int T_ = M + 2, T2 = T_ * T_, TPT = CC / CPT;
  constexpr uint32_t kTileBytes = T2 * CC;
  constexpr uint32_t kTileStride = (kTileBytes + 127u) & ~127u;   // TMA destinations stay 128-byte aligned
  constexpr uint32_t kUnitBytes = G * kTileStride;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
  const uint32_t s_in = base;                 // [G][T2][CC]
  const uint32_t s_out = base + kUnitBytes;   // [T2][G][CC]
  const uint32_t bar = s_out + kUnitBytes;
  __shared__ uint32_t abort_flag;

  // unit = (tile group, channel chunk).  Blocks of several tiles (G > 1) are launched as a
  // two-dimensional grid (x: chunk, y: group) where the group count fits, which spares every
  // thread the division (2 % on the 64-channel layers; one-tile blocks measured slower that way)
  const int cchunks = p.C / CC;
  int group, chunk;
  if (G > 1 && gridDim.y > 1) {
    chunk = blockIdx.x; group = blockIdx.y;
  } else {
    group = (int)blockIdx.x / cchunks; chunk = (int)blockIdx.x - group * cchunks;
  }
  const int tau0 = group * G;
  const int c0 = chunk * CC;
  const int g = threadIdx.x / TPT, c4 = threadIdx.x % TPT;
  const int ntile = min(G, p.T - tau0);

  int trace_step = 0;
  (void)trace_step;
  if (threadIdx.x == 0) {
    WINO_ST_BEGIN(g_in_trace, trace_step);
    WINO_ST(g_in_trace, trace_step, 0);
  }
  griddep_launch();
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    tma_prefetch_map(&mapX);
    tma_prefetch_map(&mapV);
    // patch coordinates first: nothing but the loads themselves is left for after the wait
    int cw[G], ch[G], cn[G];
#pragma unroll
    for (int i = 0; i < G; ++i) {
      const int tau = tau0 + i;
      cw[i] = (tau % p.TW) * M - 1;
      ch[i] = ((tau / p.TW) % p.TH) * M - 1;
      cn[i] = tau / (p.TW * p.TH);
    }
    // ask for the patches to be brought into L2 while the preceding kernel is still running
    // (a hint only: nothing is read into the SM before the wait below)
#pragma unroll
    for (int i = 0; i < G; ++i)
      if (i < ntile) tma_prefetch_l2_4d(&mapX, c0, cw[i], ch[i], cn[i]);
    l2_hint_slice(l2_hint, l2_hint_bytes);   // what the next kernel will want from HBM
    griddep_wait();   // only this thread reads or writes buffers that other kernels touch
    WINO_ST(g_in_trace, trace_step, 1);
    mbar_expect_tx(bar, (uint32_t)ntile * kTileBytes);
#pragma unroll
    for (int i = 0; i < G; ++i)
      if (i < ntile) tma_load_4d(s_in + (uint32_t)i * kTileStride, &mapX, bar, c0, cw[i], ch[i], cn[i]);
    // one thread polls (bounded); the others sleep in the barrier below
    if (!mbar_wait(bar, 0u, &abort_flag)) {
      abort_flag = 1u;
      atomicExch(status, -6);  // WINO_ERR_TIMEOUT
    }
    WINO_ST(g_in_trace, trace_step, 2);
  }
  __syncthreads();
  if (*(volatile uint32_t*)&abort_flag != 0u) return;
  (void)mbar_try_wait(bar, 0u);   // every thread observes the completed phase itself
  if (g < ntile) {
    const uint32_t rd = s_in + (uint32_t)g * kTileStride + (uint32_t)(CPT * c4);
    uint32_t wd[T2];
#pragma unroll
    for (int ab = 0; ab < T2; ++ab)
      wd[ab] = lds_pack<CPT>(rd + (uint32_t)ab * CC) ^ (CPT == 1 ? 0u : 0x80808080u);
    uint32_t out[T2];
#pragma unroll
    for (int i = 0; i < T2; ++i) out[i] = 0u;
#pragma unroll 1
    for (int ch = 0; ch < CPT; ++ch) {
      const uint32_t sel_in = 0x7440u | (uint32_t)ch;
      const uint32_t sel_out = insert_selector(ch);
      float V[T2];
      input_transform_2d<M, MODE>(p, [&](int l, float (&dcol)[T_]) {
#pragma unroll
        for (int a = 0; a < T_; ++a)
          dcol[a] = CPT == 1 ? small_int_to_float((int)wd[a * T_ + l])
                             : byte_to_float_sel(wd[a * T_ + l], sel_in, 8388736.0f);
      }, V);
#pragma unroll
      for (int xi = 0; xi < T2; ++xi) {
        const float r = quant_magic(V[xi], p.mult_V, p.lo_V, p.hi_V);
        out[xi] = CPT == 1 ? __float_as_uint(r) : __byte_perm(out[xi], __float_as_uint(r), sel_out);
      }
    }
    const uint32_t wr = s_out + ((uint32_t)g * CC + (uint32_t)(CPT * c4));
#pragma unroll
    for (int xi = 0; xi < T2; ++xi) sts_pack<CPT>(wr + (uint32_t)xi * (G * CC), out[xi]);
  }
  fence_async_smem();
  __syncthreads();
  if (threadIdx.x == 0) {
    WINO_ST(g_in_trace, trace_step, 3);
    tma_store_3d(&mapV, s_out, c0, tau0, 0);
    bulk_commit();
    bulk_wait_all();    // the bytes are in place before the block leaves
    WINO_ST(g_in_trace, trace_step, 4);
  }
}

// Variant with UPB units per block for grids of several waves: all loads are issued
// up front, so a later unit's load and an earlier unit's store overlap the arithmetic.
// (For a single wave the one-unit kernel above is faster: more blocks, better balance.)
template <int M, int MODE, int CC, int G, int CPT, int UPB>
__global__ void __launch_bounds__((CC / CPT) * G)
k_input_transform_tma_multi(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap mapX,
                            const __grid_constant__ CUtensorMap mapV, int* __restrict__ status,
                      const uint8_t* __restrict__ l2_hint, uint32_t l2_hint_bytes) {
  constexpr int T_ = M + 2, T2 = T_ * T_, TPT = CC / CPT;
  constexpr uint32_t kTileBytes = T2 * CC;
  constexpr uint32_t kTileStride = (kTileBytes + 127u) & ~127u;
  constexpr uint32_t kUnitBytes = G * kTileStride;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
  const uint32_t s_in0 = base;                      // UPB x [G][T2][CC]
  const uint32_t s_out0 = base + UPB * kUnitBytes;  // UPB x [T2][G][CC]
  const uint32_t bar0 = s_out0 + UPB * kUnitBytes;  // UPB barriers
  __shared__ uint32_t abort_flag;
  const int cchunks = p.C / CC;
  const int n_units = ((p.T + G - 1) / G) * cchunks;
  const int g = threadIdx.x / TPT, c4 = threadIdx.x % TPT;
  auto issue = [&](int unit, int st) {
    const int tau0 = (unit / cchunks) * G, c0 = (unit % cchunks) * CC;
    const int ntile = min(G, p.T - tau0);
    mbar_expect_tx(bar0 + 8u * st, (uint32_t)ntile * kTileBytes);
    for (int i = 0; i < ntile; ++i) {
      const int tau = tau0 + i;
      const int tw = tau % p.TW;
      const int th = (tau / p.TW) % p.TH;
      const int n = tau / (p.TW * p.TH);
      tma_load_4d(s_in0 + (uint32_t)st * kUnitBytes + (uint32_t)i * kTileStride, &mapX, bar0 + 8u * st,
                  c0, tw * M - 1, th * M - 1, n);
    }
  };
  griddep_launch();
  if (threadIdx.x == 0) {
    for (int r = 0; r < UPB; ++r) mbar_init(bar0 + 8u * r, 1);
    abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const int u0 = blockIdx.x * UPB;
  if (threadIdx.x == 0) {
    tma_prefetch_map(&mapX);
    tma_prefetch_map(&mapV);
    l2_hint_slice(l2_hint, l2_hint_bytes);
    griddep_wait();   // only this thread reads or writes buffers that other kernels touch
#pragma unroll
    for (int r = 0; r < UPB; ++r)
      if (u0 + r < n_units) issue(u0 + r, r);
  }
#pragma unroll
  for (int r = 0; r < UPB; ++r) {
    const int unit = u0 + r;
    if (unit >= n_units) break;
    const int tau0 = (unit / cchunks) * G, c0 = (unit % cchunks) * CC;
    const int ntile = min(G, p.T - tau0);
    const uint32_t s_in = s_in0 + (uint32_t)r * kUnitBytes, s_out = s_out0 + (uint32_t)r * kUnitBytes;
    if (threadIdx.x == 0 && !mbar_wait(bar0 + 8u * r, 0u, &abort_flag)) {
      abort_flag = 1u;
      atomicExch(status, -6);  // WINO_ERR_TIMEOUT
    }
    __syncthreads();
    if (*(volatile uint32_t*)&abort_flag != 0u) return;
    (void)mbar_try_wait(bar0 + 8u * r, 0u);
    if (g < ntile) {
      const uint32_t rd = s_in + (uint32_t)g * kTileStride + (uint32_t)(CPT * c4);
      uint32_t wd[T2];
#pragma unroll
      for (int ab = 0; ab < T2; ++ab)
        wd[ab] = lds_pack<CPT>(rd + (uint32_t)ab * CC) ^ (CPT == 1 ? 0u : 0x80808080u);
      uint32_t out[T2];
#pragma unroll
      for (int i = 0; i < T2; ++i) out[i] = 0u;
#pragma unroll 1
      for (int ch = 0; ch < CPT; ++ch) {
        const uint32_t sel_in = 0x7440u | (uint32_t)ch;
        const uint32_t sel_out = insert_selector(ch);
        float V[T2];
        input_transform_2d<M, MODE>(p, [&](int l, float (&dcol)[T_]) {
#pragma unroll
          for (int a = 0; a < T_; ++a)
            dcol[a] = CPT == 1 ? small_int_to_float((int)wd[a * T_ + l])
                               : byte_to_float_sel(wd[a * T_ + l], sel_in, 8388736.0f);
        }, V);
#pragma unroll
        for (int xi = 0; xi < T2; ++xi) {
          const float rr = quant_magic(V[xi], p.mult_V, p.lo_V, p.hi_V);
          out[xi] = CPT == 1 ? __float_as_uint(rr) : __byte_perm(out[xi], __float_as_uint(rr), sel_out);
        }
      }
      const uint32_t wr = s_out + ((uint32_t)g * CC + (uint32_t)(CPT * c4));
#pragma unroll
      for (int xi = 0; xi < T2; ++xi) sts_pack<CPT>(wr + (uint32_t)xi * (G * CC), out[xi]);
    }
    fence_async_smem();
    __syncthreads();
    if (threadIdx.x == 0) {
      tma_store_3d(&mapV, s_out, c0, tau0, 0);
      bulk_commit();
    }
  }
  // shared memory may be released once the stores have read it; the grid's completion
  // publishes the data
  if (threadIdx.x == 0) bulk_wait_all();
}

// PK: the output scale varies per output channel (`chan`, rows kChMultY and kChSY; one
// channel per thread only).
template <int M, int MODE, int KC, int G, int CPT, bool PK = false>
__global__ void __launch_bounds__((KC / CPT) * G, tma_min_blocks((KC / CPT) * G, CPT, M <= 4))
k_output_transform_tma(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap mapM,
                       const __grid_constant__ CUtensorMap mapY, const float* __restrict__ bias,
                       float s_Y, int* __restrict__ status, const float* __restrict__ chan) {
  static_assert(!PK || CPT == 1, "per-channel scales: one channel per thread");
  constexpr int T_ = M + 2, T2 = T_ * T_, TPT = KC / CPT;
  constexpr uint32_t kInBytes = T2 * G * KC;          // [T2][G][KC]
  constexpr uint32_t kTileOutBytes = M * M * KC;      // [M][M][KC] per tile
  constexpr uint32_t kTileOut = (kTileOutBytes + 127u) & ~127u;   // stride: TMA sources 128-byte aligned
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
  const uint32_t s_in = base;
  const uint32_t s_out = base + kInBytes;             // [G][M][M][KC]
  const uint32_t bar = s_out + G * kTileOut;
  __shared__ uint32_t abort_flag;

  const int kchunks = p.K / KC;
  int group, chunk;   // as in the input transform
  if (G > 1 && gridDim.y > 1) {
    chunk = blockIdx.x; group = blockIdx.y;
  } else {
    group = (int)blockIdx.x / kchunks; chunk = (int)blockIdx.x - group * kchunks;
  }
  const int tau0 = group * G;
  const int k0 = chunk * KC;
  const int g = threadIdx.x / TPT, k4 = threadIdx.x % TPT;
  const int ntile = min(G, p.T - tau0);

  int trace_step = 0;
  (void)trace_step;
  if (threadIdx.x == 0) {
    WINO_ST_BEGIN(g_out_trace, trace_step);
    WINO_ST(g_out_trace, trace_step, 0);
  }
  griddep_launch();
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    tma_prefetch_map(&mapM);
    tma_prefetch_map(&mapY);
    griddep_wait();
    WINO_ST(g_out_trace, trace_step, 1);
    mbar_expect_tx(bar, kInBytes);   // the full box counts, clipped rows included
    tma_load_3d(s_in, &mapM, bar, k0, tau0, 0);
  } else {
    griddep_wait();
  }
  // while the block's m_q is in flight: the pixel coordinates of the block's stores (thread 0)
  // and this thread's bias in output-code units (a double-precision division, some forty
  // instructions), which would otherwise follow the load
  __shared__ int store_at[3 * G];   // written and read by thread 0 only (no registers held by the rest)
  if (threadIdx.x == 0) {
#pragma unroll
    for (int i = 0; i < G; ++i) {
      const int tau = tau0 + i;
      store_at[3 * i + 0] = (tau % p.TW) * M;
      store_at[3 * i + 1] = ((tau / p.TW) % p.TH) * M;
      store_at[3 * i + 2] = tau / (p.TW * p.TH);
    }
  }
  float b_pre[CPT];
  float mult_Y = p.mult_Y;
  if constexpr (PK) {
    mult_Y = __ldg(chan + (long)kChMultY * p.K + k0 + k4);
    s_Y = __ldg(chan + (long)kChSY * p.K + k0 + k4);
  }
#pragma unroll
  for (int ch = 0; ch < CPT; ++ch) {
    const int k = k0 + k4 * CPT + ch;
    b_pre[ch] = (bias != nullptr && g < ntile) ? (float)((double)__ldg(bias + k) / (double)s_Y) : 0.0f;
  }
  if (threadIdx.x == 0) {
    if (!mbar_wait(bar, 0u, &abort_flag)) {
      abort_flag = 1u;
      atomicExch(status, -6);  // WINO_ERR_TIMEOUT
    }
    WINO_ST(g_out_trace, trace_step, 2);
  }
  __syncthreads();
  if (*(volatile uint32_t*)&abort_flag != 0u) return;
  (void)mbar_try_wait(bar, 0u);
  if (g < ntile) {
    const uint32_t rd = s_in + ((uint32_t)g * KC + (uint32_t)(CPT * k4));
    uint32_t wd[T2];
#pragma unroll
    for (int xi = 0; xi < T2; ++xi)
      wd[xi] = lds_pack<CPT>(rd + (uint32_t)xi * (G * KC)) ^ (CPT == 1 ? 0u : 0x80808080u);
    uint32_t outw[M * M];
#pragma unroll
    for (int i = 0; i < M * M; ++i) outw[i] = 0u;
#pragma unroll 1
    for (int ch = 0; ch < CPT; ++ch) {
      const uint32_t sel_in = 0x7440u | (uint32_t)ch;
      const uint32_t sel_out = insert_selector(ch);
      float Y[M * M];
      output_transform_2d<M, MODE>(p, [&](int i, float (&mrow)[T_]) {
#pragma unroll
        for (int j = 0; j < T_; ++j)
          mrow[j] = CPT == 1 ? small_int_to_float((int)wd[i * T_ + j])
                             : byte_to_float_sel(wd[i * T_ + j], sel_in, 8388736.0f);
      }, Y);
      const float b_scaled = b_pre[ch];
#pragma unroll
      for (int q = 0; q < M * M; ++q) {
        const float yf = __fmaf_rn(Y[q], PK ? mult_Y : p.mult_Y, b_scaled);
        const float r = __fadd_rn(fminf(fmaxf(yf, p.lo_Y), p.hi_Y), kMagic);
        const uint32_t code = (uint32_t)(magic_to_int(r) + p.z_Y);
        outw[q] = CPT == 1 ? code : __byte_perm(outw[q], code, sel_out);
      }
    }
    const uint32_t wr = s_out + (uint32_t)g * kTileOut + (uint32_t)(CPT * k4);
#pragma unroll
    for (int q = 0; q < M * M; ++q) sts_pack<CPT>(wr + (uint32_t)q * KC, outw[q]);
  }
  fence_async_smem();
  __syncthreads();
  if (threadIdx.x == 0) {
    WINO_ST(g_out_trace, trace_step, 3);
#pragma unroll
    for (int i = 0; i < G; ++i)
      if (i < ntile)
        tma_store_4d(&mapY, s_out + (uint32_t)i * kTileOut, k0, store_at[3 * i], store_at[3 * i + 1],
                     store_at[3 * i + 2]);
    bulk_commit();
    bulk_wait_all();
    WINO_ST(g_out_trace, trace_step, 4);
  }
}

// ---------------------------------------------------------------------------
// Launchers.  CC (or KC) is the largest of 128 / 64 / 32 / 16 that divides the
// channel count; narrower chunks take several tiles per block.
// ---------------------------------------------------------------------------
namespace {

// Channels per thread.  One channel per thread needs the fewest registers (so the
// most resident warps) and no byte-insert step; it is used unless the grid is so
// large that four channels per thread still fill every SM many warps deep.
inline int tma_cpt(long tiles_times_channels) {
  return tiles_times_channels / (4 * 32) >= 148l * 64 ? 4 : 1;
}

// Resident blocks per SM of a kernel, asked once per instantiation and device.
template <auto kernel>
int resident_blocks(int threads, size_t smem, int device) {
  static std::mutex mu;
  static int cache[64];   // 0: not asked yet
  std::lock_guard<std::mutex> lock(mu);
  const int d = device >= 0 && device < 64 ? device : 0;
  if (cache[d] == 0) {
    int nb = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kernel, threads, smem) != cudaSuccess || nb < 1) {
      cudaGetLastError();
      nb = 1;
    }
    cache[d] = nb;
  }
  return cache[d];
}

template <int M, int MODE, int CC, int G, int CPT, int UPB>
int input_tma_launch_u(const Params& p, const LaunchOpt& o, const CUtensorMap& mapX, const CUtensorMap& mapV,
                       int* status, cudaStream_t st) {
  constexpr size_t smem =
      2 * (size_t)UPB * G * ((((M + 2) * (M + 2) * CC) + 127) / 128 * 128) + 128 + 16 * UPB;
  constexpr int threads = (CC / CPT) * G;
  const int cchunks = p.C / CC, groups = (p.T + G - 1) / G;
  const int units = groups * cchunks;
  auto grid2 = [&](int n_units) {
    return G > 1 && groups > 1 && groups <= 65535 ? dim3((unsigned)cchunks, (unsigned)groups)
                                                  : dim3((unsigned)n_units);
  };
  if constexpr (UPB == 1 && CPT == 1 && M <= 4) {   // (F6 would spill an eighth of its work at 32 registers)
    // the 32-register build only where it saves a second wave
    static DeviceOnce once_a, once_b;
    auto ka = k_input_transform_tma<M, MODE, CC, G, CPT, false>;
    auto kb = k_input_transform_tma<M, MODE, CC, G, CPT, true>;
    if (int rc = set_max_smem(once_a, o.device, ka, smem)) return rc;
    if (int rc = set_max_smem(once_b, o.device, kb, smem)) return rc;
    const int na = resident_blocks<k_input_transform_tma<M, MODE, CC, G, CPT, false>>(threads, smem, o.device) * o.num_sms;
    const int nb = resident_blocks<k_input_transform_tma<M, MODE, CC, G, CPT, true>>(threads, smem, o.device) * o.num_sms;
    const bool cap = units > na && units <= nb;
    return launch_kernel(cap ? kb : ka, grid2(units), dim3(threads), smem, st, o.pdl, p, mapX,
                         mapV, status, static_cast<const uint8_t*>(o.l2_hint), (uint32_t)o.l2_hint_bytes);
  } else {
    auto kernel = [] {
      if constexpr (UPB == 1) return k_input_transform_tma<M, MODE, CC, G, CPT, false>;
      else return k_input_transform_tma_multi<M, MODE, CC, G, CPT, UPB>;
    }();
    static DeviceOnce once;   // one per instantiation
    if (int rc = set_max_smem(once, o.device, kernel, smem)) return rc;
    return launch_kernel(kernel, UPB == 1 ? grid2(units) : dim3((unsigned)((units + UPB - 1) / UPB)),
                         dim3(threads), smem, st, o.pdl,
                         p, mapX, mapV, status, static_cast<const uint8_t*>(o.l2_hint),
                         (uint32_t)o.l2_hint_bytes);
  }
}
template <int M, int MODE, int CC, int G, int CPT>
int input_tma_launch(const Params& p, const LaunchOpt& o, const CUtensorMap& mapX, const CUtensorMap& mapV,
                     int* status, cudaStream_t st) {
  // two units per block once the grid is several waves deep (measured: 8 % faster at four
  // times the cfg3 batch, 15 % slower at the cfg3 batch itself)
  const long threads = (long)((p.T + G - 1) / G) * (p.C / CC) * ((CC / CPT) * G);
  if (threads >= 3l * 148 * 2048)
    return input_tma_launch_u<M, MODE, CC, G, CPT, 2>(p, o, mapX, mapV, status, st);
  return input_tma_launch_u<M, MODE, CC, G, CPT, 1>(p, o, mapX, mapV, status, st);
}
template <int M, int MODE>
int input_tma_mode(const Params& p, const LaunchOpt& o, const CUtensorMap& mapX, const CUtensorMap& mapV,
                   int* status, cudaStream_t st) {
  const int cc = tma_chunk(p.C);
  if (tma_cpt((long)p.T * p.C) == 4)
    return cc == 128 ? input_tma_launch<M, MODE, 128, 1, 4>(p, o, mapX, mapV, status, st)
         : cc == 64 ? input_tma_launch<M, MODE, 64, 4, 4>(p, o, mapX, mapV, status, st)
         : cc == 32 ? input_tma_launch<M, MODE, 32, 4, 4>(p, o, mapX, mapV, status, st)
                    : input_tma_launch<M, MODE, 16, 8, 4>(p, o, mapX, mapV, status, st);
  if (tma_cpt((long)p.T * p.C) == 1)
    return cc == 128 ? input_tma_launch<M, MODE, 128, 1, 1>(p, o, mapX, mapV, status, st)
         : cc == 64 ? input_tma_launch<M, MODE, 64, 4, 1>(p, o, mapX, mapV, status, st)
         : cc == 32 ? input_tma_launch<M, MODE, 32, 4, 1>(p, o, mapX, mapV, status, st)
                    : input_tma_launch<M, MODE, 16, 8, 1>(p, o, mapX, mapV, status, st);
  return cc == 128 ? input_tma_launch<M, MODE, 128, 1, 2>(p, o, mapX, mapV, status, st)
         : cc == 64 ? input_tma_launch<M, MODE, 64, 4, 2>(p, o, mapX, mapV, status, st)
         : cc == 32 ? input_tma_launch<M, MODE, 32, 4, 2>(p, o, mapX, mapV, status, st)
                    : input_tma_launch<M, MODE, 16, 8, 2>(p, o, mapX, mapV, status, st);
}

template <int M, int MODE, int KC, int G, int CPT, bool PK = false>
int output_tma_launch(const Params& p, const LaunchOpt& o, const CUtensorMap& mapM, const CUtensorMap& mapY,
                      const float* bias, float s_Y, int* status, cudaStream_t st) {
  constexpr size_t smem = (size_t)G * ((M + 2) * (M + 2) * KC + ((M * M * KC + 127) / 128 * 128)) + 128 + 16;
  static DeviceOnce once;   // one per instantiation
  if (int rc = set_max_smem(once, o.device, k_output_transform_tma<M, MODE, KC, G, CPT, PK>, smem)) return rc;
  const int kchunks = p.K / KC, groups = (p.T + G - 1) / G;
  const dim3 grid = G > 1 && groups > 1 && groups <= 65535 ? dim3((unsigned)kchunks, (unsigned)groups)
                                                           : dim3((unsigned)(groups * kchunks));
  return launch_kernel(k_output_transform_tma<M, MODE, KC, G, CPT, PK>, grid,
                       dim3((KC / CPT) * G), smem, st, o.pdl, p, mapM, mapY, bias, s_Y, status,
                       PK ? o.chan : nullptr);
}
template <int M, int MODE>
int output_tma_mode(const Params& p, const LaunchOpt& o, const CUtensorMap& mapM, const CUtensorMap& mapY,
                    const float* bias, float s_Y, int* status, cudaStream_t st) {
  const int kc = tma_chunk(p.K);
  if (o.chan != nullptr)   // per-output-channel scales: the one-channel-per-thread build
    return kc == 128 ? output_tma_launch<M, MODE, 128, 1, 1, true>(p, o, mapM, mapY, bias, s_Y, status, st)
         : kc == 64 ? output_tma_launch<M, MODE, 64, 4, 1, true>(p, o, mapM, mapY, bias, s_Y, status, st)
         : kc == 32 ? output_tma_launch<M, MODE, 32, 4, 1, true>(p, o, mapM, mapY, bias, s_Y, status, st)
                    : output_tma_launch<M, MODE, 16, 8, 1, true>(p, o, mapM, mapY, bias, s_Y, status, st);
  if (tma_cpt((long)p.T * p.K) == 4)
    return kc == 128 ? output_tma_launch<M, MODE, 128, 1, 4>(p, o, mapM, mapY, bias, s_Y, status, st)
         : kc == 64 ? output_tma_launch<M, MODE, 64, 4, 4>(p, o, mapM, mapY, bias, s_Y, status, st)
         : kc == 32 ? output_tma_launch<M, MODE, 32, 4, 4>(p, o, mapM, mapY, bias, s_Y, status, st)
                    : output_tma_launch<M, MODE, 16, 8, 4>(p, o, mapM, mapY, bias, s_Y, status, st);
  if (tma_cpt((long)p.T * p.K) == 1)
    return kc == 128 ? output_tma_launch<M, MODE, 128, 1, 1>(p, o, mapM, mapY, bias, s_Y, status, st)
         : kc == 64 ? output_tma_launch<M, MODE, 64, 4, 1>(p, o, mapM, mapY, bias, s_Y, status, st)
         : kc == 32 ? output_tma_launch<M, MODE, 32, 4, 1>(p, o, mapM, mapY, bias, s_Y, status, st)
                    : output_tma_launch<M, MODE, 16, 8, 1>(p, o, mapM, mapY, bias, s_Y, status, st);
  return kc == 128 ? output_tma_launch<M, MODE, 128, 1, 2>(p, o, mapM, mapY, bias, s_Y, status, st)
         : kc == 64 ? output_tma_launch<M, MODE, 64, 4, 2>(p, o, mapM, mapY, bias, s_Y, status, st)
         : kc == 32 ? output_tma_launch<M, MODE, 32, 4, 2>(p, o, mapM, mapY, bias, s_Y, status, st)
                    : output_tma_launch<M, MODE, 16, 8, 2>(p, o, mapM, mapY, bias, s_Y, status, st);
}

}  // namespace

int WINO_CAT(launch_input_transform_tma_m, WINO_M)(const Params& p, const LaunchOpt& o,
                                                    const CUtensorMap& mapX,
                                                    const CUtensorMap& mapV, int* status,
                                                    cudaStream_t st) {
  if (!o.std_mats) return input_tma_mode<WINO_M, kDense>(p, o, mapX, mapV, status, st);
  return input_tma_mode<WINO_M, kExact>(p, o, mapX, mapV, status, st);
}
int WINO_CAT(launch_output_transform_tma_m, WINO_M)(const Params& p, const LaunchOpt& o,
                                                     const CUtensorMap& mapM,
                                                     const CUtensorMap& mapY, const float* bias,
                                                     float s_Y, int* status, cudaStream_t st) {
  if (!o.std_mats) return output_tma_mode<WINO_M, kDense>(p, o, mapM, mapY, bias, s_Y, status, st);
  if (WINO_M != 6) return output_tma_mode<WINO_M, kExact>(p, o, mapM, mapY, bias, s_Y, status, st);
  return output_tma_mode<WINO_M, kSparse>(p, o, mapM, mapY, bias, s_Y, status, st);
}

}  // namespace wino
