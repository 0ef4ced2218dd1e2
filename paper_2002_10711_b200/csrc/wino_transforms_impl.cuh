// Transform kernels of the Winograd-aware quantized layer (paper: Eq. 1, Fig. 2):
//   k_weight_transform : U_q = Q(G g G^T)          (stage 2, offline)
//   k_input_transform  : V_q = Q(B^T d B)          (stage 1)
//   k_output_transform : y   = Q(A^T m A + bias)   (stage 4)
// Streaming kernels: a thread owns CPT consecutive channels (1, 2 or 4) of one
// tile, keeps the patch in registers and reads / writes CPT-byte elements that
// are contiguous across the warp along the channel axis.  CPT is chosen at
// launch so that the grid fills the SMs several warps deep.
//
// Transform modes:
//   kDense  : matrices are data (learnt "flex" transforms); every entry is used,
//             fused-multiply-add chains in the contract's order.
//   kSparse : the built-in Cook-Toom matrices as compile-time constants; zero
//             entries vanish (the chain's value does not change).
//   kExact  : Cook-Toom F4 with every intermediate an integer below 2^24, so
//             any summation order gives the same bits; shared sub-expressions
//             are factored out (12 instead of 22 operations per 1-D transform).
#pragma once
#include <cstdlib>
#include "wino_launch.h"
#include "wino_transform_math.cuh"

#define WINO_CAT_(a, b) a##b
#define WINO_CAT(a, b) WINO_CAT_(a, b)

namespace wino {

// ---------------------------------------------------------------------------
// Stage 2: filters.  w [K][3][3][C] int8 -> U_q [t*t][K][C] int8.
// ---------------------------------------------------------------------------
template <int M, int CPT>
__global__ void __launch_bounds__(128)
k_weight_transform(const __grid_constant__ Params p, const float* __restrict__ chan,
                   const int8_t* __restrict__ w, int8_t* __restrict__ Uq,
                   unsigned* __restrict__ absmax, unsigned* __restrict__ absmax_K) {
  constexpr int T_ = M + 2;
  typedef typename Pack<CPT>::type PT;
  const int CG = p.C / CPT;
  const long total = (long)p.K * CG;
  const long idx = blockIdx.x * (long)blockDim.x + threadIdx.x;
  float vmax = 0.0f;
  griddep_wait();
  if (idx < total) {
    const int cg = (int)(idx % CG);
    const int k = (int)(idx / CG);
    const PT* wp = reinterpret_cast<const PT*>(w);
    uint32_t wd[9];
#pragma unroll
    for (int ab = 0; ab < 9; ++ab)
      wd[ab] = (uint32_t)__ldg(wp + ((long)k * 9 + ab) * CG + cg) ^ 0x80808080u;
    uint32_t out[T_ * T_];
#pragma unroll
    for (int i = 0; i < T_ * T_; ++i) out[i] = 0u;
    const float ubias = 8388736.0f + (float)p.z_w;
    const float mult_U = chan_or(chan, p.K, kChMultU, k, p.mult_U);
#pragma unroll
    for (int ch = 0; ch < CPT; ++ch) {
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
          float r = quant_magic(acc, mult_U, p.lo_U, p.hi_U);
          out[i * T_ + j] = insert_byte(out[i * T_ + j], __float_as_uint(r), ch);
        }
    }
    PT* Up = reinterpret_cast<PT*>(Uq);
#pragma unroll
    for (int xi = 0; xi < T_ * T_; ++xi) Up[((long)xi * p.K + k) * CG + cg] = (PT)out[xi];
    if (absmax_K != nullptr) atomic_absmax(absmax_K + k, vmax);   // this thread's filter only
  }
  if (absmax != nullptr) atomic_absmax(absmax, vmax);
}

// ---------------------------------------------------------------------------
// Stage 1: activations.  x [N][H][W][C] int8 -> V_q [t*t][T][C] int8.
// Zero padding is the code z_x (real zero).
// ---------------------------------------------------------------------------
template <int M, int MODE, int CPT, bool STATS>
__global__ void __launch_bounds__(128)
k_input_transform(const __grid_constant__ Params p, const int8_t* __restrict__ x,
                  int8_t* __restrict__ Vq, unsigned* __restrict__ absmax) {
  constexpr int T_ = M + 2;
  typedef typename Pack<CPT>::type PT;
  const int CG = p.C / CPT;
  const long total = (long)p.T * CG;
  const long idx = blockIdx.x * (long)blockDim.x + threadIdx.x;
  float vmax = 0.0f;
  griddep_launch();
  griddep_wait();
  if (idx < total) {
    const int cg = (int)(idx % CG);
    const int tau = (int)(idx / CG);
    const int tw = tau % p.TW;
    const int th = (tau / p.TW) % p.TH;
    const int n = tau / (p.TW * p.TH);
    // one 64-bit base per thread; per-element offsets are 32-bit sums of a
    // row part and a column part (coordinates clamped into the image, validity
    // applied afterwards as an all-ones / all-zeros mask)
    const PT* xbase = reinterpret_cast<const PT*>(x) + (long)n * p.H * p.W * CG + cg;
    const uint32_t zword = ((uint32_t)(p.z_x & 0xFF) * 0x01010101u) ^ 0x80808080u;
    int roff[T_], coff[T_];
    uint32_t rmask[T_], cmask[T_];
#pragma unroll
    for (int a = 0; a < T_; ++a) {
      const int h = th * M - 1 + a, wv = tw * M - 1 + a;
      rmask[a] = (h >= 0 && h < p.H) ? 0xFFFFFFFFu : 0u;
      cmask[a] = (wv >= 0 && wv < p.W) ? 0xFFFFFFFFu : 0u;
      roff[a] = min(max(h, 0), p.H - 1) * p.W * CG;
      coff[a] = min(max(wv, 0), p.W - 1) * CG;
    }
    uint32_t wd[T_ * T_];
#pragma unroll
    for (int a = 0; a < T_; ++a)
#pragma unroll
      for (int b = 0; b < T_; ++b) {
        const uint32_t v = (uint32_t)__ldg(xbase + (roff[a] + coff[b])) ^ 0x80808080u;
        const uint32_t mk = rmask[a] & cmask[b];
        wd[a * T_ + b] = (v & mk) | (zword & ~mk);
      }
    uint32_t out[T_ * T_];
#pragma unroll
    for (int i = 0; i < T_ * T_; ++i) out[i] = 0u;
    const float ubias = 8388736.0f + (float)p.z_x;
    // the channel loop stays rolled: the body is large and instruction-cache
    // misses cost more than the loop overhead
#pragma unroll 1
    for (int ch = 0; ch < CPT; ++ch) {
      const uint32_t sel_in = 0x7440u | (uint32_t)ch;
      const uint32_t sel_out = insert_selector(ch);
      float V[T_ * T_];
      input_transform_2d<M, MODE>(p, [&](int l, float (&dcol)[T_]) {
#pragma unroll
        for (int a = 0; a < T_; ++a) dcol[a] = byte_to_float_sel(wd[a * T_ + l], sel_in, ubias);
      }, V);
#pragma unroll
      for (int xi = 0; xi < T_ * T_; ++xi) {
        if constexpr (STATS) vmax = fmaxf(vmax, fabsf(V[xi]));
        float r = quant_magic(V[xi], p.mult_V, p.lo_V, p.hi_V);
        out[xi] = CPT == 1 ? __float_as_uint(r) : __byte_perm(out[xi], __float_as_uint(r), sel_out);
      }
    }
    PT* Vp = reinterpret_cast<PT*>(Vq) + (long)tau * CG + cg;
    const long plane = (long)p.T * CG;
#pragma unroll
    for (int xi = 0; xi < T_ * T_; ++xi) { *Vp = (PT)out[xi]; Vp += plane; }
  }
  if constexpr (STATS) atomic_absmax(absmax, vmax);
}

// ---------------------------------------------------------------------------
// Stage 4: outputs.  m_q [t*t][T][K] int8 (QM) or M [t*t][T][K] int32 (!QM)
// -> y [N][H][W][K] int8 or float.  absmax2 (nullable): [0] = max|Y|,
// [1] = max|fmaf(Y, s_acc, bias)|.
// ---------------------------------------------------------------------------
template <int M, int MODE, bool QM, int CPT, bool STATS>
__global__ void __launch_bounds__(128)
k_output_transform(const __grid_constant__ Params p, const void* __restrict__ mbuf,
                   const float* __restrict__ bias, void* __restrict__ y, float s_Y,
                   unsigned* __restrict__ absmax2, const float* __restrict__ chan) {
  constexpr int T_ = M + 2;
  typedef typename Pack<CPT>::type PT;
  const int KG = p.K / CPT;
  const long total = (long)p.T * KG;
  const long idx = blockIdx.x * (long)blockDim.x + threadIdx.x;
  float ymax = 0.0f, fmax_ = 0.0f;
  griddep_launch();
  griddep_wait();
  if (idx < total) {
    const int kg = (int)(idx % KG);
    const int tau = (int)(idx / KG);
    const int tw = tau % p.TW;
    const int th = (tau / p.TW) % p.TH;
    const int n = tau / (p.TW * p.TH);
    uint32_t wd[QM ? T_ * T_ : 1];
    if constexpr (QM) {
      const PT* mp = reinterpret_cast<const PT*>(mbuf) + (long)tau * KG + kg;
      const long plane = (long)p.T * KG;
#pragma unroll
      for (int xi = 0; xi < T_ * T_; ++xi) { wd[xi] = (uint32_t)__ldg(mp) ^ 0x80808080u; mp += plane; }
    }
    uint32_t outw[M * M];
#pragma unroll
    for (int i = 0; i < M * M; ++i) outw[i] = 0u;
#pragma unroll 1
    for (int ch = 0; ch < CPT; ++ch) {
      const int k = kg * CPT + ch;
      const uint32_t sel_in = 0x7440u | (uint32_t)ch;
      const uint32_t sel_out = insert_selector(ch);
      float Y[M * M];
      output_transform_2d<M, MODE>(p, [&](int i, float (&mrow)[T_]) {
#pragma unroll
        for (int j = 0; j < T_; ++j) {
          if constexpr (QM) {
            mrow[j] = byte_to_float_sel(wd[i * T_ + j], sel_in, 8388736.0f);
          } else {
            const int* Mi = reinterpret_cast<const int*>(mbuf);
            mrow[j] = __int2float_rn(__ldg(Mi + ((long)(i * T_ + j) * p.T + tau) * p.K + k));
          }
        }
      }, Y);
      const float b_real = bias != nullptr ? __ldg(bias + k) : 0.0f;
      const float mult_Y = chan_or(chan, p.K, kChMultY, k, p.mult_Y);
      const float s_acc = chan_or(chan, p.K, kChSAcc, k, p.s_acc);
      float b_scaled = 0.0f;
      if (p.out_dtype == 0 && bias != nullptr)
        b_scaled = (float)((double)b_real / (double)chan_or(chan, p.K, kChSY, k, s_Y));
#pragma unroll
      for (int ip = 0; ip < M; ++ip)
#pragma unroll
        for (int jp = 0; jp < M; ++jp) {
          const float acc = Y[ip * M + jp];
          const int h = th * M + ip, wv = tw * M + jp;
          if constexpr (STATS) {
            ymax = fmaxf(ymax, fabsf(acc));
            if (h < p.H && wv < p.W) fmax_ = fmaxf(fmax_, fabsf(__fmaf_rn(acc, s_acc, b_real)));
          }
          if (p.out_dtype == 0) {
            const float yf = __fmaf_rn(acc, mult_Y, b_scaled);
            const float r = __fadd_rn(fminf(fmaxf(yf, p.lo_Y), p.hi_Y), kMagic);
            const uint32_t code = (uint32_t)(magic_to_int(r) + p.z_Y);
            outw[ip * M + jp] = CPT == 1 ? code : __byte_perm(outw[ip * M + jp], code, sel_out);
          } else if (y != nullptr && h < p.H && wv < p.W) {
            reinterpret_cast<float*>(y)[(((long)n * p.H + h) * p.W + wv) * p.K + k] =
                __fmaf_rn(acc, s_acc, b_real);
          }
        }
    }
    if (p.out_dtype == 0 && y != nullptr) {
      PT* yp = reinterpret_cast<PT*>(y) + (((long)n * p.H + th * M) * p.W + tw * M) * KG + kg;
      const int rstep = p.W * KG;
#pragma unroll
      for (int ip = 0; ip < M; ++ip)
#pragma unroll
        for (int jp = 0; jp < M; ++jp)
          if (th * M + ip < p.H && tw * M + jp < p.W) yp[ip * rstep + jp * KG] = (PT)outw[ip * M + jp];
    }
  }
  if constexpr (STATS) {
    atomic_absmax(absmax2 + 0, ymax);
    atomic_absmax(absmax2 + 1, fmax_);
  }
}

// ---------------------------------------------------------------------------
// Launchers.
// ---------------------------------------------------------------------------
namespace {

// Channels per thread: the widest element that still gives every SM several
// warps of work (148 SMs x 1024 threads as the target).
int pick_cpt(long items_times_channels) {
  const long target = 148l * 1024;
  if (items_times_channels / 4 >= target) return 4;
  if (items_times_channels / 2 >= target) return 2;
  return 1;
}

template <int M, int CPT>
int weight_cpt(const Params& p, const float* chan, const int8_t* w, int8_t* Uq, unsigned* absmax,
               unsigned* absmax_K, cudaStream_t st) {
  const long total = (long)p.K * (p.C / CPT);
  return launch_kernel(k_weight_transform<M, CPT>, dim3((unsigned)((total + 127) / 128)), dim3(128),
                       0, st, false, p, chan, w, Uq, absmax, absmax_K);
}
template <int M>
int weight_m(const Params& p, const float* chan, const int8_t* w, int8_t* Uq, unsigned* absmax,
             unsigned* absmax_K, cudaStream_t st) {
  const int cpt = pick_cpt((long)p.K * p.C);
  return cpt == 4 ? weight_cpt<M, 4>(p, chan, w, Uq, absmax, absmax_K, st)
       : cpt == 2 ? weight_cpt<M, 2>(p, chan, w, Uq, absmax, absmax_K, st)
                  : weight_cpt<M, 1>(p, chan, w, Uq, absmax, absmax_K, st);
}

template <int M, int MODE, int CPT>
int input_cpt(const Params& p, bool pdl, const int8_t* x, int8_t* Vq, unsigned* absmax,
              cudaStream_t st) {
  const long total = (long)p.T * (p.C / CPT);
  const dim3 grid((unsigned)((total + 127) / 128));
  if constexpr (CPT == 4) {   // the statistics variant exists for one width only
    if (absmax != nullptr)
      return launch_kernel(k_input_transform<M, MODE, 4, true>, grid, dim3(128), 0, st, pdl, p, x,
                           Vq, absmax);
  }
  return launch_kernel(k_input_transform<M, MODE, CPT, false>, grid, dim3(128), 0, st, pdl, p, x, Vq,
                       absmax);
}
template <int M, int MODE>
int input_mode(const Params& p, bool pdl, const int8_t* x, int8_t* Vq, unsigned* absmax,
               cudaStream_t st) {
  const int cpt = absmax != nullptr ? 4 : pick_cpt((long)p.T * p.C);
  return cpt == 4 ? input_cpt<M, MODE, 4>(p, pdl, x, Vq, absmax, st)
       : cpt == 2 ? input_cpt<M, MODE, 2>(p, pdl, x, Vq, absmax, st)
                  : input_cpt<M, MODE, 1>(p, pdl, x, Vq, absmax, st);
}
template <int M>
int input_m(const Params& p, const LaunchOpt& o, const int8_t* x, int8_t* Vq, unsigned* absmax,
            cudaStream_t st) {
  if (!o.std_mats) return input_mode<M, kDense>(p, o.pdl, x, Vq, absmax, st);
  // Cook-Toom B^T on integer codes is exact for m = 2, 4, 6: factored forms throughout.
  return input_mode<M, kExact>(p, o.pdl, x, Vq, absmax, st);
}

template <int M, int MODE, bool QM, int CPT>
int output_cpt(const Params& p, bool pdl, float s_Y, const void* mbuf, const float* bias, void* y,
               unsigned* absmax2, const float* chan, cudaStream_t st) {
  const long total = (long)p.T * (p.K / CPT);
  const dim3 grid((unsigned)((total + 127) / 128));
  if constexpr (CPT == 4) {
    if (absmax2 != nullptr)
      return launch_kernel(k_output_transform<M, MODE, QM, 4, true>, grid, dim3(128), 0, st, pdl, p,
                           mbuf, bias, y, s_Y, absmax2, chan);
  }
  return launch_kernel(k_output_transform<M, MODE, QM, CPT, false>, grid, dim3(128), 0, st, pdl, p,
                       mbuf, bias, y, s_Y, absmax2, chan);
}
template <int M, int MODE, bool QM>
int output_mode(const Params& p, bool pdl, float s_Y, const void* mbuf, const float* bias, void* y,
                unsigned* absmax2, const float* chan, cudaStream_t st) {
  const int cpt = absmax2 != nullptr ? 4 : pick_cpt((long)p.T * p.K);
  return cpt == 4 ? output_cpt<M, MODE, QM, 4>(p, pdl, s_Y, mbuf, bias, y, absmax2, chan, st)
       : cpt == 2 ? output_cpt<M, MODE, QM, 2>(p, pdl, s_Y, mbuf, bias, y, absmax2, chan, st)
                  : output_cpt<M, MODE, QM, 1>(p, pdl, s_Y, mbuf, bias, y, absmax2, chan, st);
}
template <int M>
int output_m(const Params& p, const LaunchOpt& o, float s_Y, const void* mbuf, const float* bias,
             void* y, unsigned* absmax2, cudaStream_t st) {
  const bool qm = p.qM_enabled != 0;
  if (!o.std_mats) {
    return qm ? output_mode<M, kDense, true>(p, o.pdl, s_Y, mbuf, bias, y, absmax2, o.chan, st)
              : output_mode<M, kDense, false>(p, o.pdl, s_Y, mbuf, bias, y, absmax2, o.chan, st);
  }
  // With Q_M on, the F4 output transform works on integers in [-128, 127]:
  // every intermediate is an integer below 2^24, so the factored form is exact.
  if (M != 6 && qm) return output_mode<M, kExact, true>(p, o.pdl, s_Y, mbuf, bias, y, absmax2, o.chan, st);
  return qm ? output_mode<M, kSparse, true>(p, o.pdl, s_Y, mbuf, bias, y, absmax2, o.chan, st)
            : output_mode<M, kSparse, false>(p, o.pdl, s_Y, mbuf, bias, y, absmax2, o.chan, st);
}

}  // namespace

// Entry points for this translation unit's tile size (one unit per m keeps the
// build parallel).
int WINO_CAT(launch_weight_transform_m, WINO_M)(const Params& p, const float* chan, const int8_t* w,
                                                 int8_t* Uq, unsigned* absmax, unsigned* absmax_K,
                                                 cudaStream_t st) {
  return weight_m<WINO_M>(p, chan, w, Uq, absmax, absmax_K, st);
}
int WINO_CAT(launch_input_transform_m, WINO_M)(const Params& p, const LaunchOpt& o,
                                                const int8_t* x, int8_t* Vq, unsigned* absmax,
                                                cudaStream_t st) {
  return input_m<WINO_M>(p, o, x, Vq, absmax, st);
}
int WINO_CAT(launch_output_transform_m, WINO_M)(const Params& p, const LaunchOpt& o, float s_Y,
                                                 const void* mbuf, const float* bias, void* y,
                                                 unsigned* absmax2, cudaStream_t st) {
  return output_m<WINO_M>(p, o, s_Y, mbuf, bias, y, absmax2, st);
}

}  // namespace wino
