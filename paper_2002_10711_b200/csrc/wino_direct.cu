// Direct int8 3x3 convolution (cross-correlation, zero padding 1, stride 1 or 2)
// with int32 accumulation: the lossless candidate the paper compares the
// Winograd-aware layers with (Sections 4 and 5.3), and the layer type of the
// network's strided convolutions, for which no Winograd form exists (Section 5.1).
// Integer dot products on the ALUs; thread = (output pixel, 4 or 8 output channels).
#include "wino_launch.h"

namespace wino {

struct DirectParams {
  int N, C, H, W, K, stride, Ho, Wo;
  int z_x, z_w, z_Y;
  float mult, s_in, s_Y, lo_Y, hi_Y;
  int out_dtype;
  // per-output-channel scales (device arrays of K floats, nullable) and the per-layer scales
  const float* s_w_K;
  const float* s_Y_K;
  float s_x, s_w;
};

// Channel k's output arithmetic: the multiplier on the accumulator (s_x * s_w[k] / s_Y[k] for
// integer output, s_x * s_w[k] for float output; the product of the two scales is exact in
// double) and the output scale the bias is divided by.
__device__ __forceinline__ void channel_scales(const DirectParams& p, int k, float& mult, float& s_in,
                                               float& s_Y) {
  mult = p.mult; s_in = p.s_in; s_Y = p.s_Y;
  if (p.s_w_K != nullptr || p.s_Y_K != nullptr) {
    const double s_in_k = (double)p.s_x * (double)(p.s_w_K != nullptr ? __ldg(p.s_w_K + k) : p.s_w);
    if (p.s_Y_K != nullptr) s_Y = __ldg(p.s_Y_K + k);
    mult = (float)(s_in_k / (double)s_Y);
    s_in = (float)s_in_k;
  }
}

// KPT output channels per thread.  Consecutive lanes take consecutive output
// pixels, so a weight word is one broadcast load for the warp and every lane
// walks the contiguous channels of its own input pixel.
template <int KPT>
__global__ void __launch_bounds__(128)
k_direct_conv(const DirectParams p, const int8_t* __restrict__ x, const int8_t* __restrict__ w,
              const float* __restrict__ bias, void* __restrict__ y) {
  const int KG = p.K / KPT, C4 = p.C >> 2;
  const long npix = (long)p.N * p.Ho * p.Wo;
  const long idx = blockIdx.x * (long)blockDim.x + threadIdx.x;
  griddep_launch();
  griddep_wait();
  if (idx >= npix * KG) return;
  const int kg = (int)(idx / npix);          // slow index: a warp shares its output channels
  long pix = idx - (long)kg * npix;
  const int wo = (int)(pix % p.Wo); pix /= p.Wo;
  const int ho = (int)(pix % p.Ho);
  const int n = (int)(pix / p.Ho);
  const int* x32 = reinterpret_cast<const int*>(x);
  const int* w32 = reinterpret_cast<const int*>(w);
  int acc[KPT];
#pragma unroll
  for (int j = 0; j < KPT; ++j) acc[j] = 0;
  const bool plain = p.z_x == 0 && p.z_w == 0;
#pragma unroll
  for (int a = 0; a < 3; ++a) {
    const int h = ho * p.stride - 1 + a;
    if (h < 0 || h >= p.H) continue;
#pragma unroll
    for (int b = 0; b < 3; ++b) {
      const int wv = wo * p.stride - 1 + b;
      if (wv < 0 || wv >= p.W) continue;          // padding is the real value zero
      const int* xp = x32 + (((long)n * p.H + h) * p.W + wv) * C4;
      const int* wp = w32 + (((long)(kg * KPT) * 3 + a) * 3 + b) * C4;
      for (int c4 = 0; c4 < C4; ++c4) {
        const int xv = __ldg(xp + c4);
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
          const int wv4 = __ldg(wp + (long)j * 9 * C4 + c4);
          if (plain) {
            acc[j] = __dp4a(xv, wv4, acc[j]);
          } else {
#pragma unroll
            for (int q = 0; q < 4; ++q)
              acc[j] += ((int)(int8_t)(xv >> (8 * q)) - p.z_x) * ((int)(int8_t)(wv4 >> (8 * q)) - p.z_w);
          }
        }
      }
    }
  }
  const long o = (((long)n * p.Ho + ho) * p.Wo + wo) * p.K + kg * KPT;
#pragma unroll
  for (int j4 = 0; j4 < KPT; j4 += 4) {
    if (p.out_dtype == 0) {
      uint32_t word = 0u;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int k = kg * KPT + j4 + j;
        float mult, s_in, s_Y;
        channel_scales(p, k, mult, s_in, s_Y);
        const float b = bias != nullptr ? (float)((double)__ldg(bias + k) / (double)s_Y) : 0.0f;
        const float yf = __fmaf_rn(__int2float_rn(acc[j4 + j]), mult, b);
        const float r = __fadd_rn(fminf(fmaxf(yf, p.lo_Y), p.hi_Y), kMagic);
        word |= ((uint32_t)(magic_to_int(r) + p.z_Y) & 0xFFu) << (8 * j);
      }
      *reinterpret_cast<uint32_t*>(reinterpret_cast<int8_t*>(y) + o + j4) = word;
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float b = bias != nullptr ? __ldg(bias + kg * KPT + j4 + j) : 0.0f;
        float mult, s_in, s_Y;
        channel_scales(p, kg * KPT + j4 + j, mult, s_in, s_Y);
        reinterpret_cast<float*>(y)[o + j4 + j] = __fmaf_rn(__int2float_rn(acc[j4 + j]), s_in, b);
      }
    }
  }
}

// Any channel counts (the network's three-channel first layer, Section 5.1): thread =
// (output pixel, output channel), byte loads.  Small layers only; nothing here is tuned.
__global__ void __launch_bounds__(128)
k_direct_conv_bytes(const DirectParams p, const int8_t* __restrict__ x, const int8_t* __restrict__ w,
                    const float* __restrict__ bias, void* __restrict__ y) {
  const long npix = (long)p.N * p.Ho * p.Wo;
  const long idx = blockIdx.x * (long)blockDim.x + threadIdx.x;
  griddep_launch();
  griddep_wait();
  if (idx >= npix * p.K) return;
  const int k = (int)(idx % p.K);             // consecutive lanes: consecutive output channels
  long pix = idx / p.K;
  const int wo = (int)(pix % p.Wo); pix /= p.Wo;
  const int ho = (int)(pix % p.Ho);
  const int n = (int)(pix / p.Ho);
  int acc = 0;
  for (int a = 0; a < 3; ++a) {
    const int h = ho * p.stride - 1 + a;
    if (h < 0 || h >= p.H) continue;
    for (int b = 0; b < 3; ++b) {
      const int wv = wo * p.stride - 1 + b;
      if (wv < 0 || wv >= p.W) continue;      // padding is the real value zero
      const int8_t* xp = x + (((long)n * p.H + h) * p.W + wv) * p.C;
      const int8_t* wp = w + (((long)k * 3 + a) * 3 + b) * p.C;
      for (int c = 0; c < p.C; ++c) acc += ((int)__ldg(xp + c) - p.z_x) * ((int)__ldg(wp + c) - p.z_w);
    }
  }
  const long o = (((long)n * p.Ho + ho) * p.Wo + wo) * p.K + k;
  float mult, s_in, s_Y;
  channel_scales(p, k, mult, s_in, s_Y);
  if (p.out_dtype == 0) {
    const float b = bias != nullptr ? (float)((double)__ldg(bias + k) / (double)s_Y) : 0.0f;
    const float yf = __fmaf_rn(__int2float_rn(acc), mult, b);
    const float r = __fadd_rn(fminf(fmaxf(yf, p.lo_Y), p.hi_Y), kMagic);
    reinterpret_cast<int8_t*>(y)[o] = (int8_t)(magic_to_int(r) + p.z_Y);
  } else {
    const float b = bias != nullptr ? __ldg(bias + k) : 0.0f;
    reinterpret_cast<float*>(y)[o] = __fmaf_rn(__int2float_rn(acc), s_in, b);
  }
}

int launch_direct_conv(int N, int C, int H, int W, int K, int stride, int z_x, int z_w, int z_Y,
                       float mult, float s_in, float s_Y, float lo_Y, float hi_Y, int out_dtype,
                       const int8_t* x, const int8_t* w, const float* bias, void* y,
                       const float* s_w_K, const float* s_Y_K, float s_x, float s_w, cudaStream_t st) {
  DirectParams p;
  p.s_w_K = s_w_K; p.s_Y_K = s_Y_K; p.s_x = s_x; p.s_w = s_w;
  p.N = N; p.C = C; p.H = H; p.W = W; p.K = K; p.stride = stride;
  p.Ho = (H - 1) / stride + 1; p.Wo = (W - 1) / stride + 1;
  p.z_x = z_x; p.z_w = z_w; p.z_Y = z_Y;
  p.mult = mult; p.s_in = s_in; p.s_Y = s_Y; p.lo_Y = lo_Y; p.hi_Y = hi_Y;
  p.out_dtype = out_dtype;
  const long npix = (long)N * p.Ho * p.Wo;
  if (C % 4 != 0 || K % 4 != 0) {
    const long blocks = (npix * K + 127) / 128;
    if (blocks > 0x7fffffffl) return -2;   // WINO_ERR_UNSUPPORTED: more blocks than a grid holds
    return launch_kernel(k_direct_conv_bytes, dim3((unsigned)blocks), dim3(128), 0, st, true, p, x, w,
                         bias, y);
  }
  if (K % 8 == 0)
    return launch_kernel(k_direct_conv<8>, dim3((unsigned)((npix * (K / 8) + 127) / 128)), dim3(128),
                         0, st, true, p, x, w, bias, y);
  return launch_kernel(k_direct_conv<4>, dim3((unsigned)((npix * (K / 4) + 127) / 128)), dim3(128), 0,
                       st, true, p, x, w, bias, y);
}

}  // namespace wino
