// Fused small-channel path (C <= 32, K <= 32): the whole layer of Eq. 1 in one
// kernel built on warp shuffles.  With few channels the transforms dominate the
// layer's cost (paper: Sections 3.1 "Compute" and 5.3) and no tensor-core tile
// would be filled; instead a warp holds 32 / LPT tiles, LPT = 8, 16 or 32 lanes
// per tile (the smallest that covers max(C, K)), and inside a tile's lane group
//   - lane = input channel c for the input transform B^T d B and Q_V;
//   - the codes of four neighbouring lanes are packed into one word with two
//     shuffles;
//   - lane = output channel k for the Hadamard stage: the packed words are
//     broadcast lane to lane by shuffle and contracted with 4-way integer dot
//     products against U_q held in shared memory;
//   - lane = k for Q_M, the output transform A^T m A, bias and Q_Y.
// Nothing but x, U_q and y touches global memory.  Blocks are persistent (they
// stage U_q once and then walk over tile groups).
#include "wino_launch.h"
#include "wino_transform_math.cuh"

namespace wino {

template <int M, bool STD, int LPT>
__global__ void __launch_bounds__(128)
k_smallc(const __grid_constant__ Params p, const int8_t* __restrict__ x,
         const int8_t* __restrict__ Uq, const float* __restrict__ bias, void* __restrict__ y,
         float s_Y, int* __restrict__ dbgM) {
  constexpr int T_ = M + 2, T2 = T_ * T_;
  constexpr int TPW = 32 / LPT;                   // tiles per warp
  constexpr int MODE = STD ? kSparse : kDense;
  constexpr int L4 = LPT / 4;                     // words per filter row, zero padded
  extern __shared__ uint32_t sU[];                // [T2][L4][LPT]: word L of filter (xi, k)
  const int C4 = p.C >> 2, K = p.K;
  griddep_launch();
  griddep_wait();
  {
    // zero padding in both directions makes the contraction loop branch-free:
    // channels past C multiply zeros, lanes past K read zeros
    for (int i = threadIdx.x; i < T2 * L4 * LPT; i += blockDim.x) sU[i] = 0u;
    __syncthreads();
    const uint32_t* U32 = reinterpret_cast<const uint32_t*>(Uq);
    const int per_xi = K * C4;
    for (int xi = 0; xi < T2; ++xi)
      for (int i = threadIdx.x; i < per_xi; i += blockDim.x) {
        const int k = i / C4, L = i - k * C4;
        sU[(xi * L4 + L) * LPT + k] = __ldg(U32 + xi * per_xi + i);
      }
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = blockDim.x >> 5;
  const int ts = lane / LPT, l = lane % LPT;      // tile slot in the warp, lane in the tile
  const int tbase = ts * LPT;
  const bool c_ok = l < p.C, k_ok = l < K;
  const int kk = k_ok ? l : 0;
  const float b_real = (bias != nullptr && k_ok) ? __ldg(bias + kk) : 0.0f;
  float b_scaled = 0.0f;
  if (p.out_dtype == 0 && bias != nullptr) b_scaled = (float)((double)b_real / (double)s_Y);
  const int groups = (p.T + TPW - 1) / TPW;
  const uint32_t* su = sU + l;                    // this lane's column of the padded U_q

  for (int grp = blockIdx.x * wpb + warp; grp < groups; grp += gridDim.x * wpb) {
    const int tau = grp * TPW + ts;
    const bool t_ok = tau < p.T;
    const int tq = t_ok ? tau : 0;
    const int tw = tq % p.TW;
    const int th = (tq / p.TW) % p.TH;
    const int n = tq / (p.TW * p.TH);
    // ---- input transform, lane = c: coordinates clamped into the image, padding by select ----
    const int8_t* xb = x + (long)n * p.H * p.W * p.C + (c_ok ? l : 0);
    int roff[T_], coff[T_];
    bool rv[T_], cv[T_];
#pragma unroll
    for (int a = 0; a < T_; ++a) {
      const int h = th * M - 1 + a, wv = tw * M - 1 + a;
      rv[a] = h >= 0 && h < p.H;
      cv[a] = wv >= 0 && wv < p.W;
      roff[a] = min(max(h, 0), p.H - 1) * p.W * p.C;
      coff[a] = min(max(wv, 0), p.W - 1) * p.C;
    }
    float V[T2];
    input_transform_2d<M, MODE>(p, [&](int b, float (&dcol)[T_]) {
#pragma unroll
      for (int a = 0; a < T_; ++a) {
        const int code = (int)__ldg(xb + (roff[a] + coff[b]));
        dcol[a] = __int2float_rn((rv[a] && cv[b] && c_ok && t_ok) ? code - p.z_x : 0);
      }
    }, V);
    // ---- per xi: Q_V, pack, Hadamard (lane = k), Q_M ----
    float mf[T2];
#pragma unroll
    for (int xi = 0; xi < T2; ++xi) {
      const float r = quant_magic(V[xi], p.mult_V, p.lo_V, p.hi_V);
      const uint32_t b = c_ok ? (__float_as_uint(r) & 0xFFu) : 0u;
      const uint32_t h2 = b | (__shfl_down_sync(0xffffffffu, b, 1) << 8);
      const uint32_t w4 = h2 | (__shfl_down_sync(0xffffffffu, h2, 2) << 16);  // lanes l % 4 == 0
      int macc = 0;
#pragma unroll
      for (int L = 0; L < L4; ++L) {
        const int vv = (int)__shfl_sync(0xffffffffu, w4, tbase + 4 * L);
        macc = __dp4a(vv, (int)su[(xi * L4 + L) * LPT], macc);
      }
      // debugging aid: the int32 Hadamard sum itself, M[xi][tau][k]
      if (dbgM != nullptr && k_ok && t_ok) dbgM[((long)xi * p.T + tau) * K + l] = macc;
      float mval = __int2float_rn(macc);
      if (p.qM_enabled) mval = magic_to_float(quant_magic(mval, p.mult_M, p.lo_M, p.hi_M));
      mf[xi] = mval;
    }
    // ---- output transform, lane = k ----
    float Y[M * M];
    output_transform_2d<M, MODE>(p, [&](int i, float (&mrow)[T_]) {
#pragma unroll
      for (int j = 0; j < T_; ++j) mrow[j] = mf[i * T_ + j];
    }, Y);
    if (k_ok && t_ok) {
      const long obase = (((long)n * p.H + th * M) * p.W + tw * M) * K + l;
      const int rstep = p.W * K;
#pragma unroll
      for (int ip = 0; ip < M; ++ip)
#pragma unroll
        for (int jp = 0; jp < M; ++jp) {
          if (th * M + ip >= p.H || tw * M + jp >= p.W) continue;
          const float acc = Y[ip * M + jp];
          const long o = obase + ip * rstep + jp * K;
          if (p.out_dtype == 0) {
            const float yf = __fmaf_rn(acc, p.mult_Y, b_scaled);
            const float r = __fadd_rn(fminf(fmaxf(yf, p.lo_Y), p.hi_Y), kMagic);
            reinterpret_cast<int8_t*>(y)[o] = (int8_t)(magic_to_int(r) + p.z_Y);
          } else {
            reinterpret_cast<float*>(y)[o] = __fmaf_rn(acc, p.s_acc, b_real);
          }
        }
    }
  }
}

namespace {

template <int M, bool STD, int LPT>
int smallc_launch(const Params& p, const LaunchOpt& o, const int8_t* x, const int8_t* Uq, const float* bias,
                  void* y, float s_Y, int* dbgM, cudaStream_t st) {
  constexpr int T2 = (M + 2) * (M + 2);
  const size_t smem = (size_t)T2 * (LPT / 4) * LPT * 4;
  static DeviceOnce once;   // one per instantiation
  if (int rc = set_max_smem(once, o.device, k_smallc<M, STD, LPT>, smem)) return rc;
  const int groups = (p.T + (32 / LPT) - 1) / (32 / LPT);
  int blocks = (groups + 3) / 4;
  if (blocks > 148 * 8) blocks = 148 * 8;
  return launch_kernel(k_smallc<M, STD, LPT>, dim3((unsigned)blocks), dim3(128), smem, st, o.pdl, p, x,
                       Uq, bias, y, s_Y, dbgM);
}
template <int M, bool STD>
int smallc_lpt(const Params& p, const LaunchOpt& o, const int8_t* x, const int8_t* Uq, const float* bias,
               void* y, float s_Y, int* dbgM, cudaStream_t st) {
  const int wide = p.C > p.K ? p.C : p.K;
  return wide <= 8  ? smallc_launch<M, STD, 8>(p, o, x, Uq, bias, y, s_Y, dbgM, st)
       : wide <= 16 ? smallc_launch<M, STD, 16>(p, o, x, Uq, bias, y, s_Y, dbgM, st)
                    : smallc_launch<M, STD, 32>(p, o, x, Uq, bias, y, s_Y, dbgM, st);
}
template <int M>
int smallc_m(const Params& p, const LaunchOpt& o, const int8_t* x, const int8_t* Uq,
             const float* bias, void* y, float s_Y, int* dbgM, cudaStream_t st) {
  return o.std_mats ? smallc_lpt<M, true>(p, o, x, Uq, bias, y, s_Y, dbgM, st)
                    : smallc_lpt<M, false>(p, o, x, Uq, bias, y, s_Y, dbgM, st);
}
}  // namespace

int launch_smallc(const Params& p, const LaunchOpt& o, const int8_t* x, const int8_t* Uq,
                  const float* bias, void* y, float s_Y, int* dbgM, cudaStream_t st) {
  return p.m == 2 ? smallc_m<2>(p, o, x, Uq, bias, y, s_Y, dbgM, st)
       : p.m == 4 ? smallc_m<4>(p, o, x, Uq, bias, y, s_Y, dbgM, st)
                  : smallc_m<6>(p, o, x, Uq, bias, y, s_Y, dbgM, st);
}

}  // namespace wino
