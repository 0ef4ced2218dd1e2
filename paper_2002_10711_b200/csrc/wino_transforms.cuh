// Transform kernels of the Winograd-aware quantized layer (paper: Eq. 1, Fig. 2):
//   k_weight_transform : U_q = Q(G g G^T)          (stage 2, offline)
//   k_input_transform  : V_q = Q(B^T d B)          (stage 1)
//   k_output_transform : y   = Q(A^T m A + bias)   (stage 4)
// All are streaming kernels: each thread owns four consecutive channels of one
// tile (or filter), reads and writes 32-bit words that are coalesced across the
// warp along the channel axis, and keeps the whole patch in registers.
#pragma once
#include "wino_common.cuh"

namespace wino {

// Insert the low byte of `bits` at byte position `ch` of `word`.
__device__ __forceinline__ uint32_t insert_byte(uint32_t word, uint32_t bits, int ch) {
  const uint32_t sel = ch == 0 ? 0x3214u : ch == 1 ? 0x3240u : ch == 2 ? 0x3410u : 0x4210u;
  return __byte_perm(word, bits, sel);
}

// ---------------------------------------------------------------------------
// Stage 2: filters.  w [K][3][3][C] int8 -> U_q [t*t][K][C] int8.
// ---------------------------------------------------------------------------
template <int M>
__global__ void __launch_bounds__(128)
k_weight_transform(const __grid_constant__ Params p, const int8_t* __restrict__ w,
                   int8_t* __restrict__ Uq, unsigned* __restrict__ absmax) {
  constexpr int T_ = M + 2;
  const int C4 = p.C >> 2;
  const long total = (long)p.K * C4;
  const long idx = blockIdx.x * (long)blockDim.x + threadIdx.x;
  float vmax = 0.0f;
  if (idx < total) {
    const int c4 = (int)(idx % C4);
    const int k = (int)(idx / C4);
    const uint32_t* w32 = reinterpret_cast<const uint32_t*>(w);
    uint32_t wd[9];
#pragma unroll
    for (int ab = 0; ab < 9; ++ab) wd[ab] = __ldg(w32 + ((long)k * 9 + ab) * C4 + c4) ^ 0x80808080u;
    uint32_t out[T_ * T_];
#pragma unroll
    for (int i = 0; i < T_ * T_; ++i) out[i] = 0u;
    const float ubias = 8388736.0f + (float)p.z_w;
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
      float g[9];
#pragma unroll
      for (int ab = 0; ab < 9; ++ab) g[ab] = byte_to_float(wd[ab], ch, ubias);
      float P[T_][3];
#pragma unroll
      for (int i = 0; i < T_; ++i)
#pragma unroll
        for (int l = 0; l < 3; ++l) {
          float acc = 0.0f;
#pragma unroll
          for (int kk = 0; kk < 3; ++kk) acc = __fmaf_rn(p.G[i * 3 + kk], g[kk * 3 + l], acc);
          P[i][l] = acc;
        }
#pragma unroll
      for (int i = 0; i < T_; ++i)
#pragma unroll
        for (int j = 0; j < T_; ++j) {
          float acc = 0.0f;
#pragma unroll
          for (int l = 0; l < 3; ++l) acc = __fmaf_rn(P[i][l], p.G[j * 3 + l], acc);
          vmax = fmaxf(vmax, fabsf(acc));
          float r = quant_magic(acc, p.mult_U, p.lo_U, p.hi_U);
          out[i * T_ + j] = insert_byte(out[i * T_ + j], __float_as_uint(r), ch);
        }
    }
    uint32_t* U32 = reinterpret_cast<uint32_t*>(Uq);
#pragma unroll
    for (int xi = 0; xi < T_ * T_; ++xi) U32[((long)xi * p.K + k) * C4 + c4] = out[xi];
  }
  if (absmax != nullptr) atomic_absmax(absmax, vmax);
}

// ---------------------------------------------------------------------------
// Stage 1: activations.  x [N][H][W][C] int8 -> V_q [t*t][T][C] int8.
// Zero padding is the code z_x (real zero).
// ---------------------------------------------------------------------------
template <int M, bool STD>
__global__ void __launch_bounds__(128)
k_input_transform(const __grid_constant__ Params p, const int8_t* __restrict__ x,
                  int8_t* __restrict__ Vq, unsigned* __restrict__ absmax) {
  constexpr int T_ = M + 2;
  using MT = Mat<M, STD>;
  const int C4 = p.C >> 2;
  const long total = (long)p.T * C4;
  const long idx = blockIdx.x * (long)blockDim.x + threadIdx.x;
  float vmax = 0.0f;
  if (idx < total) {
    const int c4 = (int)(idx % C4);
    const int tau = (int)(idx / C4);
    const int tw = tau % p.TW;
    const int th = (tau / p.TW) % p.TH;
    const int n = tau / (p.TW * p.TH);
    const uint32_t* x32 = reinterpret_cast<const uint32_t*>(x);
    const uint32_t zword = ((uint32_t)(p.z_x & 0xFF) * 0x01010101u) ^ 0x80808080u;
    uint32_t wd[T_ * T_];
#pragma unroll
    for (int a = 0; a < T_; ++a) {
      const int h = th * M - 1 + a;
#pragma unroll
      for (int b = 0; b < T_; ++b) {
        const int wv = tw * M - 1 + b;
        const bool in = (h >= 0) && (h < p.H) && (wv >= 0) && (wv < p.W);
        wd[a * T_ + b] =
            in ? (__ldg(x32 + (((long)n * p.H + h) * p.W + wv) * C4 + c4) ^ 0x80808080u) : zword;
      }
    }
    uint32_t out[T_ * T_];
#pragma unroll
    for (int i = 0; i < T_ * T_; ++i) out[i] = 0u;
    const float ubias = 8388736.0f + (float)p.z_x;
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
      float P[T_][T_];
#pragma unroll
      for (int l = 0; l < T_; ++l) {
        float dcol[T_];
#pragma unroll
        for (int a = 0; a < T_; ++a) dcol[a] = byte_to_float(wd[a * T_ + l], ch, ubias);
#pragma unroll
        for (int i = 0; i < T_; ++i) {
          float acc = 0.0f;
#pragma unroll
          for (int k = 0; k < T_; ++k) acc = chain<STD>(MT::bt(p, i, k), dcol[k], acc);
          P[i][l] = acc;
        }
      }
#pragma unroll
      for (int i = 0; i < T_; ++i)
#pragma unroll
        for (int j = 0; j < T_; ++j) {
          float acc = 0.0f;
#pragma unroll
          for (int l = 0; l < T_; ++l) acc = chain<STD>(MT::bt(p, j, l), P[i][l], acc);
          vmax = fmaxf(vmax, fabsf(acc));
          float r = quant_magic(acc, p.mult_V, p.lo_V, p.hi_V);
          out[i * T_ + j] = insert_byte(out[i * T_ + j], __float_as_uint(r), ch);
        }
    }
    uint32_t* V32 = reinterpret_cast<uint32_t*>(Vq);
#pragma unroll
    for (int xi = 0; xi < T_ * T_; ++xi) V32[((long)xi * p.T + tau) * C4 + c4] = out[xi];
  }
  if (absmax != nullptr) atomic_absmax(absmax, vmax);
}

// ---------------------------------------------------------------------------
// Stage 4: outputs.  m_q [t*t][T][K] int8 (QM) or M [t*t][T][K] int32 (!QM)
// -> y [N][H][W][K] int8 or float.  Right factor first (R = m A), then
// Y = A^T R; bias and the output quantizer follow.
// absmax2 (nullable): [0] = max|Y|, [1] = max|fmaf(Y, s_acc, bias)|.
// ---------------------------------------------------------------------------
template <int M, bool STD, bool QM>
__global__ void __launch_bounds__(128)
k_output_transform(const __grid_constant__ Params p, const void* __restrict__ mbuf,
                   const float* __restrict__ bias, void* __restrict__ y, float s_Y,
                   unsigned* __restrict__ absmax2) {
  constexpr int T_ = M + 2;
  using MT = Mat<M, STD>;
  const int K4 = p.K >> 2;
  const long total = (long)p.T * K4;
  const long idx = blockIdx.x * (long)blockDim.x + threadIdx.x;
  float ymax = 0.0f, fmax_ = 0.0f;
  if (idx < total) {
    const int k4 = (int)(idx % K4);
    const int tau = (int)(idx / K4);
    const int tw = tau % p.TW;
    const int th = (tau / p.TW) % p.TH;
    const int n = tau / (p.TW * p.TH);
    uint32_t wd[QM ? T_ * T_ : 1];
    if constexpr (QM) {
      const uint32_t* m32 = reinterpret_cast<const uint32_t*>(mbuf);
#pragma unroll
      for (int xi = 0; xi < T_ * T_; ++xi)
        wd[xi] = __ldg(m32 + ((long)xi * p.T + tau) * K4 + k4) ^ 0x80808080u;
    }
    uint32_t outw[M * M];
#pragma unroll
    for (int i = 0; i < M * M; ++i) outw[i] = 0u;
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
      const int k = k4 * 4 + ch;
      float R[T_][M];
#pragma unroll
      for (int i = 0; i < T_; ++i) {
        float mrow[T_];
#pragma unroll
        for (int j = 0; j < T_; ++j) {
          if constexpr (QM) {
            mrow[j] = byte_to_float(wd[i * T_ + j], ch, 8388736.0f);
          } else {
            const int* Mi = reinterpret_cast<const int*>(mbuf);
            mrow[j] = __int2float_rn(__ldg(Mi + ((long)(i * T_ + j) * p.T + tau) * p.K + k));
          }
        }
#pragma unroll
        for (int jp = 0; jp < M; ++jp) {
          float acc = 0.0f;
#pragma unroll
          for (int j = 0; j < T_; ++j) acc = chain<STD>(MT::at(p, jp, j), mrow[j], acc);
          R[i][jp] = acc;
        }
      }
      const float b_real = bias != nullptr ? __ldg(bias + k) : 0.0f;
      float b_scaled = 0.0f;
      if (p.out_dtype == 0 && bias != nullptr) b_scaled = (float)((double)b_real / (double)s_Y);
#pragma unroll
      for (int ip = 0; ip < M; ++ip)
#pragma unroll
        for (int jp = 0; jp < M; ++jp) {
          float acc = 0.0f;
#pragma unroll
          for (int i = 0; i < T_; ++i) acc = chain<STD>(MT::at(p, ip, i), R[i][jp], acc);
          const int h = th * M + ip, wv = tw * M + jp;
          if (absmax2 != nullptr) {
            ymax = fmaxf(ymax, fabsf(acc));
            if (h < p.H && wv < p.W) fmax_ = fmaxf(fmax_, fabsf(__fmaf_rn(acc, p.s_acc, b_real)));
          }
          if (p.out_dtype == 0) {
            const float yf = __fmaf_rn(acc, p.mult_Y, b_scaled);
            const float r = __fadd_rn(fminf(fmaxf(yf, p.lo_Y), p.hi_Y), kMagic);
            outw[ip * M + jp] =
                insert_byte(outw[ip * M + jp], (uint32_t)(magic_to_int(r) + p.z_Y), ch);
          } else if (y != nullptr && h < p.H && wv < p.W) {
            reinterpret_cast<float*>(y)[(((long)n * p.H + h) * p.W + wv) * p.K + k] =
                __fmaf_rn(acc, p.s_acc, b_real);
          }
        }
    }
    if (p.out_dtype == 0 && y != nullptr) {
      uint32_t* y32 = reinterpret_cast<uint32_t*>(y);
#pragma unroll
      for (int ip = 0; ip < M; ++ip)
#pragma unroll
        for (int jp = 0; jp < M; ++jp) {
          const int h = th * M + ip, wv = tw * M + jp;
          if (h < p.H && wv < p.W)
            y32[(((long)n * p.H + h) * p.W + wv) * K4 + k4] = outw[ip * M + jp];
        }
    }
  }
  if (absmax2 != nullptr) {
    atomic_absmax(absmax2 + 0, ymax);
    atomic_absmax(absmax2 + 1, fmax_);
  }
}

}  // namespace wino
