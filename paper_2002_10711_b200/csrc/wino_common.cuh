// Shared device-side definitions for the Winograd-aware quantized convolution
// kernels (sm_100a).  Notation follows the paper's Eq. 1: B^T, G, A^T are the
// input, filter and output transform matrices; t = m + 2.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace wino {

constexpr int kMaxT = 8;

// Everything a kernel needs to know about one layer; passed by value as a
// __grid_constant__ kernel parameter so that matrix entries are constant-bank
// operands.
struct Params {
  int N, C, H, W, K, m, t, TH, TW;
  int T;                       // tiles: N * TH * TW
  float BT[kMaxT * kMaxT];     // [t][t]
  float G[kMaxT * 3];          // [t][3]
  float AT[6 * kMaxT];         // [m][t]
  float mult_V, mult_U, mult_M, mult_Y, s_acc;
  float lo_V, hi_V, lo_U, hi_U, lo_M, hi_M, lo_Y, hi_Y;  // clamp bounds minus zero point
  int z_x, z_w, z_Y;
  int qM_enabled;
  int out_dtype;               // 0 int8, 1 float
};
// Per-output-channel scales travel beside Params as a device array `chan` [5][K] (null: the
// per-layer values of Params): row kChMultU = s_w[k]/s_U[k], kChMultM = s_U[k]*s_V/s_M[k],
// kChMultY = s_acc[k]/s_Y[k], kChSAcc = s_acc[k] (s_M[k] with Q_M, else s_U[k]*s_V),
// kChSY = s_Y[k].
enum { kChMultU = 0, kChMultM = 1, kChMultY = 2, kChSAcc = 3, kChSY = 4 };

// 1.5 * 2^23: adding it to a float of magnitude < 2^22 leaves the
// round-half-to-even integer in the low mantissa bits.
constexpr float kMagic = 12582912.0f;
constexpr int kMagicBits = 0x4B400000;

// Quantizer core: round_half_even(v * mult) of the exact product, then clamp.
// fmaf(v, mult, kMagic) rounds the exact value v*mult + kMagic once; for
// |v*mult| < 2^22 the result lies in [2^23, 2^24) where floats are the integers,
// so it equals kMagic + round_half_even(v*mult) (kMagic is even: ties agree).
// Larger products stay monotone and are caught by the clamp.  Returns
// kMagic + code; the low byte of the bit pattern is the two's-complement code.
__device__ __forceinline__ float quant_magic(float v, float mult, float lo, float hi) {
  const float r = __fmaf_rn(v, mult, kMagic);
  return fminf(fmaxf(r, __fadd_rn(lo, kMagic)), __fadd_rn(hi, kMagic));
}
__device__ __forceinline__ int magic_to_int(float r) { return __float_as_int(r) - kMagicBits; }
// Channel k's value of row `row` of the per-channel table, or the per-layer value.
__device__ __forceinline__ float chan_or(const float* chan, int K, int row, int k,
                                         float layer_value) {
  return chan != nullptr ? __ldg(chan + (long)row * K + k) : layer_value;
}

// Saturating pack of two 32-bit integers to signed bytes (cvt.pack.sat): byte 1 = sat(a),
// byte 0 = sat(b), upper half = lower half of c.
__device__ __forceinline__ uint32_t pack_sat_s8(int a, int b, uint32_t c) {
  uint32_t d;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// Four codes of one row as a little-endian packed word.  HI127: the upper bound of the
// quantizer is +127 and is applied by the saturating pack (which also covers products too
// large for the rounding constant: their bit patterns stay above it); the lower bound, any
// code >= -128, is applied on the float.  Otherwise both bounds are applied on the float.
template <bool HI127>
__device__ __forceinline__ uint32_t quant_pack4(float v0, float v1, float v2, float v3, float mult,
                                                float lo_magic, float hi_magic) {
  if constexpr (HI127) {
    const int c0 = magic_to_int(fmaxf(__fmaf_rn(v0, mult, kMagic), lo_magic));
    const int c1 = magic_to_int(fmaxf(__fmaf_rn(v1, mult, kMagic), lo_magic));
    const int c2 = magic_to_int(fmaxf(__fmaf_rn(v2, mult, kMagic), lo_magic));
    const int c3 = magic_to_int(fmaxf(__fmaf_rn(v3, mult, kMagic), lo_magic));
    return pack_sat_s8(c1, c0, pack_sat_s8(c3, c2, 0u));
  } else {
    const uint32_t r0 = __float_as_uint(fminf(fmaxf(__fmaf_rn(v0, mult, kMagic), lo_magic), hi_magic));
    const uint32_t r1 = __float_as_uint(fminf(fmaxf(__fmaf_rn(v1, mult, kMagic), lo_magic), hi_magic));
    const uint32_t r2 = __float_as_uint(fminf(fmaxf(__fmaf_rn(v2, mult, kMagic), lo_magic), hi_magic));
    const uint32_t r3 = __float_as_uint(fminf(fmaxf(__fmaf_rn(v3, mult, kMagic), lo_magic), hi_magic));
    return __byte_perm(__byte_perm(r0, r1, 0x0040u), __byte_perm(r2, r3, 0x0040u), 0x5410u);
  }
}
__device__ __forceinline__ float magic_to_float(float r) { return __fsub_rn(r, kMagic); }

// int8 byte `sel` (0..3) of a packed word, minus zero point z, as an exact float:
// flip the sign bit (value + 128 as unsigned), splice into the mantissa of 2^23,
// subtract 2^23 + 128 + z.
// `bias` is the float 8388608 + 128 + z (an exact integer).
__device__ __forceinline__ float byte_to_float(uint32_t word_flipped, int sel, float bias) {
  uint32_t b = __byte_perm(word_flipped, 0x4B000000u, 0x7440u | (uint32_t)sel);
  return __fsub_rn(__uint_as_float(b), bias);
}
// Same with a precomputed permute selector (0x7440 | byte index).
__device__ __forceinline__ float byte_to_float_sel(uint32_t word_flipped, uint32_t selector,
                                                   float bias) {
  return __fsub_rn(__uint_as_float(__byte_perm(word_flipped, 0x4B000000u, selector)), bias);
}
// Permute selector that inserts byte 0 of the second operand at byte `ch` of the first.
__device__ __forceinline__ uint32_t insert_selector(int ch) {
  return (0x3210u & ~(0xFu << (4 * ch))) | (4u << (4 * ch));
}

// Programmatic dependent launch: wait for the preceding kernel on the stream to
// finish (no-op when the kernel was launched normally); allow the following
// kernel to be scheduled early.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// int32 -> float (exact below 2^24).  On this architecture the conversion issues
// at the rate of an ordinary fp32 instruction, so it beats the two-instruction
// integer-add / float-subtract trick.
__device__ __forceinline__ float small_int_to_float(int v) { return __int2float_rn(v); }

__device__ __forceinline__ void atomic_absmax(unsigned* addr, float v) {
  // non-negative floats order like their bit patterns
  float m = v;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) atomicMax(addr, __float_as_uint(m));
}

// ---------------------------------------------------------------------------
// Cook-Toom matrices for the standard points {0, +-1}, {0, +-1, +-2},
// {0, +-1, +-2, +-1/2} (monic B^T rows, 1/N_j carried by G).  When a plan's
// matrices equal these bit for bit, kernels are instantiated with the entries
// as compile-time constants, so zero entries cost nothing.  Skipping a zero
// coefficient leaves a fused-multiply-add chain's value unchanged.
// ---------------------------------------------------------------------------
template <int M> __host__ __device__ constexpr float std_bt(int i, int k);
template <int M> __host__ __device__ constexpr float std_at(int i, int k);

template <> __host__ __device__ constexpr float std_bt<2>(int i, int k) {
  constexpr float a[4][4] = {{1, 0, -1, 0}, {0, 1, 1, 0}, {0, -1, 1, 0}, {0, -1, 0, 1}};
  return a[i][k];
}
template <> __host__ __device__ constexpr float std_at<2>(int i, int k) {
  constexpr float a[2][4] = {{1, 1, 1, 0}, {0, 1, -1, 1}};
  return a[i][k];
}
template <> __host__ __device__ constexpr float std_bt<4>(int i, int k) {
  constexpr float a[6][6] = {{4, 0, -5, 0, 1, 0},  {0, 4, 4, -1, -1, 0}, {0, -4, 4, 1, -1, 0},
                             {0, -2, -1, 2, 1, 0}, {0, 2, -1, -2, 1, 0}, {0, 4, 0, -5, 0, 1}};
  return a[i][k];
}
template <> __host__ __device__ constexpr float std_at<4>(int i, int k) {
  constexpr float a[4][6] = {{1, 1, 1, 1, 1, 0}, {0, 1, -1, 2, -2, 0}, {0, 1, 1, 4, 4, 0},
                             {0, 1, -1, 8, -8, 1}};
  return a[i][k];
}
template <> __host__ __device__ constexpr float std_bt<6>(int i, int k) {
  constexpr float a[8][8] = {{1, 0, -5.25f, 0, 5.25f, 0, -1, 0},
                             {0, -1, -1, 4.25f, 4.25f, -1, -1, 0},
                             {0, 1, -1, -4.25f, 4.25f, 1, -1, 0},
                             {0, 0.5f, 0.25f, -2.5f, -1.25f, 2, 1, 0},
                             {0, -0.5f, 0.25f, 2.5f, -1.25f, -2, 1, 0},
                             {0, 2, 4, -2.5f, -5, 0.5f, 1, 0},
                             {0, -2, 4, 2.5f, -5, -0.5f, 1, 0},
                             {0, -1, 0, 5.25f, 0, -5.25f, 0, 1}};
  return a[i][k];
}
template <> __host__ __device__ constexpr float std_at<6>(int i, int k) {
  constexpr float a[6][8] = {{1, 1, 1, 1, 1, 1, 1, 0},
                             {0, 1, -1, 2, -2, 0.5f, -0.5f, 0},
                             {0, 1, 1, 4, 4, 0.25f, 0.25f, 0},
                             {0, 1, -1, 8, -8, 0.125f, -0.125f, 0},
                             {0, 1, 1, 16, 16, 0.0625f, 0.0625f, 0},
                             {0, 1, -1, 32, -32, 0.03125f, -0.03125f, 1}};
  return a[i][k];
}

template <int M, bool STD>
struct Mat {
  static constexpr int T = M + 2;
  __device__ __forceinline__ static float bt(const Params& p, int i, int k) {
    if constexpr (STD) return std_bt<M>(i, k);
    else return p.BT[i * T + k];
  }
  __device__ __forceinline__ static float at(const Params& p, int i, int k) {
    if constexpr (STD) return std_at<M>(i, k);
    else return p.AT[i * T + k];
  }
};

// One step of a fused-multiply-add chain; with a compile-time zero coefficient
// the step disappears (the chain's value is unchanged by it).
template <bool STD>
__device__ __forceinline__ float chain(float coef, float x, float acc) {
  if constexpr (STD) {
    if (coef == 0.0f) return acc;
  }
  return __fmaf_rn(coef, x, acc);
}

}  // namespace wino
