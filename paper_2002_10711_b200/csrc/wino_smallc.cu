// Fused small-channel path (C <= 32, K <= 32): the whole layer of Eq. 1 in one
// kernel, one warp per tile.  With few channels the transforms dominate the
// layer's cost (paper: Sections 3.1 "Compute" and 5.3), so no tensor-core tile
// would be filled; instead
//   - lane = input channel c for the input transform B^T d B and Q_V;
//   - the quantized codes of four neighbouring lanes are packed into one word
//     with two shuffles;
//   - lane = output channel k for the Hadamard stage: the packed words are
//     broadcast lane to lane by shuffle and contracted with 4-way integer dot
//     products against U_q held in shared memory;
//   - lane = k for Q_M, the output transform A^T m A, bias and Q_Y.
// Nothing but x, U_q and y touches global memory.
#include "wino_launch.h"

namespace wino {

template <int M, bool STD>
__global__ void __launch_bounds__(128)
k_smallc(const __grid_constant__ Params p, const int8_t* __restrict__ x,
         const int8_t* __restrict__ Uq, const float* __restrict__ bias, void* __restrict__ y,
         float s_Y) {
  constexpr int T_ = M + 2, T2 = T_ * T_;
  using MT = Mat<M, STD>;
  extern __shared__ uint32_t sU[];  // [T2][C4][K]: word L of filter (xi, k)
  const int C4 = p.C >> 2, K = p.K;
  griddep_launch();
  griddep_wait();
  {
    const uint32_t* U32 = reinterpret_cast<const uint32_t*>(Uq);
    const int per_xi = K * C4;
    for (int i = threadIdx.x; i < T2 * per_xi; i += blockDim.x) {
      const int xi = i / per_xi, rem = i - xi * per_xi;
      const int k = rem / C4, L = rem - k * C4;
      sU[(xi * C4 + L) * K + k] = __ldg(U32 + i);
    }
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = blockDim.x >> 5;
  const bool c_ok = lane < p.C, k_ok = lane < K;
  const int kk = k_ok ? lane : 0;
  const float b_real = (bias != nullptr && k_ok) ? __ldg(bias + kk) : 0.0f;
  float b_scaled = 0.0f;
  if (p.out_dtype == 0 && bias != nullptr) b_scaled = (float)((double)b_real / (double)s_Y);

  for (int tau = blockIdx.x * wpb + warp; tau < p.T; tau += gridDim.x * wpb) {
    const int tw = tau % p.TW;
    const int th = (tau / p.TW) % p.TH;
    const int n = tau / (p.TW * p.TH);
    // ---- input transform, lane = c ----
    float P[T_][T_];
#pragma unroll
    for (int l = 0; l < T_; ++l) {
      float dcol[T_];
      const int wv = tw * M - 1 + l;
#pragma unroll
      for (int a = 0; a < T_; ++a) {
        const int h = th * M - 1 + a;
        const bool in = c_ok && h >= 0 && h < p.H && wv >= 0 && wv < p.W;
        int code = p.z_x;
        if (in) code = (int)__ldg(x + (((long)n * p.H + h) * p.W + wv) * p.C + lane);
        dcol[a] = (float)(code - p.z_x);
      }
#pragma unroll
      for (int i = 0; i < T_; ++i) {
        float acc = 0.0f;
#pragma unroll
        for (int k = 0; k < T_; ++k) acc = chain<STD>(MT::bt(p, i, k), dcol[k], acc);
        P[i][l] = acc;
      }
    }
    // ---- per xi: Q_V, pack, Hadamard (lane = k), Q_M ----
    float mf[T2];
#pragma unroll
    for (int i = 0; i < T_; ++i)
#pragma unroll
      for (int j = 0; j < T_; ++j) {
        float acc = 0.0f;
#pragma unroll
        for (int l = 0; l < T_; ++l) acc = chain<STD>(MT::bt(p, j, l), P[i][l], acc);
        const float r = quant_magic(acc, p.mult_V, p.lo_V, p.hi_V);
        const uint32_t b = c_ok ? (__float_as_uint(r) & 0xFFu) : 0u;
        const uint32_t h2 = b | (__shfl_down_sync(0xffffffffu, b, 1) << 8);
        const uint32_t w4 = h2 | (__shfl_down_sync(0xffffffffu, h2, 2) << 16);  // lanes % 4 == 0
        const int xi = i * T_ + j;
        int macc = 0;
        for (int L = 0; L < C4; ++L) {
          const int vv = (int)__shfl_sync(0xffffffffu, w4, 4 * L);
          macc = __dp4a(vv, (int)sU[(xi * C4 + L) * K + kk], macc);
        }
        float mval = __int2float_rn(macc);
        if (p.qM_enabled) mval = magic_to_float(quant_magic(mval, p.mult_M, p.lo_M, p.hi_M));
        mf[xi] = mval;
      }
    // ---- output transform, lane = k ----
    float R[T_][M];
#pragma unroll
    for (int i = 0; i < T_; ++i)
#pragma unroll
      for (int jp = 0; jp < M; ++jp) {
        float acc = 0.0f;
#pragma unroll
        for (int j = 0; j < T_; ++j) acc = chain<STD>(MT::at(p, jp, j), mf[i * T_ + j], acc);
        R[i][jp] = acc;
      }
#pragma unroll
    for (int ip = 0; ip < M; ++ip)
#pragma unroll
      for (int jp = 0; jp < M; ++jp) {
        float acc = 0.0f;
#pragma unroll
        for (int i = 0; i < T_; ++i) acc = chain<STD>(MT::at(p, ip, i), R[i][jp], acc);
        const int h = th * M + ip, wv = tw * M + jp;
        if (!k_ok || h >= p.H || wv >= p.W) continue;
        const long o = (((long)n * p.H + h) * p.W + wv) * K + lane;
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

namespace {
template <int M, bool STD>
int smallc_launch(const Params& p, bool pdl, const int8_t* x, const int8_t* Uq, const float* bias,
                  void* y, float s_Y, cudaStream_t st) {
  constexpr int T2 = (M + 2) * (M + 2);
  const size_t smem = (size_t)T2 * (p.C / 4) * p.K * 4;
  static bool attr_set = false;   // one flag per instantiation
  if (!attr_set) {
    if (cudaFuncSetAttribute(k_smallc<M, STD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             64 * 32 * 8 * 4) != cudaSuccess) return -5;
    attr_set = true;
  }
  int blocks = (p.T + 3) / 4;
  if (blocks > 148 * 8) blocks = 148 * 8;
  return launch_kernel(k_smallc<M, STD>, dim3((unsigned)blocks), dim3(128), smem, st, pdl, p, x, Uq,
                       bias, y, s_Y);
}
template <int M>
int smallc_m(const Params& p, const LaunchOpt& o, const int8_t* x, const int8_t* Uq,
             const float* bias, void* y, float s_Y, cudaStream_t st) {
  return o.std_mats ? smallc_launch<M, true>(p, o.pdl, x, Uq, bias, y, s_Y, st)
                    : smallc_launch<M, false>(p, o.pdl, x, Uq, bias, y, s_Y, st);
}
}  // namespace

int launch_smallc(const Params& p, const LaunchOpt& o, const int8_t* x, const int8_t* Uq,
                  const float* bias, void* y, float s_Y, cudaStream_t st) {
  return p.m == 2 ? smallc_m<2>(p, o, x, Uq, bias, y, s_Y, st)
       : p.m == 4 ? smallc_m<4>(p, o, x, Uq, bias, y, s_Y, st)
                  : smallc_m<6>(p, o, x, Uq, bias, y, s_Y, st);
}

}  // namespace wino
