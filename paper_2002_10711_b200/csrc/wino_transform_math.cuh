// Transform arithmetic shared by every kernel that applies B^T d B or A^T m A
// (paper: Eq. 1): the two-sided transforms as fused-multiply-add chains in the
// contract's order, with compile-time Cook-Toom constants (zero entries vanish)
// and the factored exact forms for F4.
//
// Transform modes:
//   kDense  : matrices are data (learnt "flex" transforms); every entry is used.
//   kSparse : the built-in Cook-Toom matrices as compile-time constants.
//   kExact  : Cook-Toom matrices on integer codes where every intermediate is
//             exactly representable (input stage for m = 2, 4, 6; output stage for
//             m = 2, 4 on int8 codes), so any summation order gives the same bits;
//             shared sub-expressions are factored out.  The F6 output stage falls
//             back to the ordered chains.
#pragma once
#include "wino_common.cuh"

namespace wino {

enum { kDense = 0, kSparse = 1, kExact = 2 };

template <int CPT> struct Pack;
template <> struct Pack<1> { typedef uint8_t type; };
template <> struct Pack<2> { typedef uint16_t type; };
template <> struct Pack<4> { typedef uint32_t type; };

__device__ __forceinline__ uint32_t insert_byte(uint32_t word, uint32_t bits, int ch) {
  const uint32_t sel = ch == 0 ? 0x3214u : ch == 1 ? 0x3240u : ch == 2 ? 0x3410u : 0x4210u;
  return __byte_perm(word, bits, sel);
}

// 1-D B^T, factored (exact mode only: every intermediate is a multiple of 1/16 below 2^20,
// so the order of the sums does not change the bits).
__device__ __forceinline__ void bt_exact(const float (&d)[4], float (&r)[4]) {
  r[0] = __fsub_rn(d[0], d[2]);
  r[1] = __fadd_rn(d[1], d[2]);
  r[2] = __fsub_rn(d[2], d[1]);
  r[3] = __fsub_rn(d[3], d[1]);
}
__device__ __forceinline__ void bt_exact(const float (&d)[8], float (&r)[8]) {
  const float e1 = __fmaf_rn(4.25f, d[4], -__fadd_rn(d[2], d[6]));
  const float o1 = __fmaf_rn(4.25f, d[3], -__fadd_rn(d[1], d[5]));
  const float e2 = __fmaf_rn(0.25f, d[2], __fmaf_rn(-1.25f, d[4], d[6]));
  const float o2 = __fmaf_rn(0.5f, d[1], __fmaf_rn(-2.5f, d[3], __fmul_rn(2.0f, d[5])));
  const float e3 = __fmaf_rn(4.0f, d[2], __fmaf_rn(-5.0f, d[4], d[6]));
  const float o3 = __fmaf_rn(2.0f, d[1], __fmaf_rn(-2.5f, d[3], __fmul_rn(0.5f, d[5])));
  r[0] = __fmaf_rn(5.25f, __fsub_rn(d[4], d[2]), __fsub_rn(d[0], d[6]));
  r[1] = __fadd_rn(e1, o1);
  r[2] = __fsub_rn(e1, o1);
  r[3] = __fadd_rn(e2, o2);
  r[4] = __fsub_rn(e2, o2);
  r[5] = __fadd_rn(e3, o3);
  r[6] = __fsub_rn(e3, o3);
  r[7] = __fmaf_rn(5.25f, __fsub_rn(d[3], d[5]), __fsub_rn(d[7], d[1]));
}
__device__ __forceinline__ void bt_exact(const float (&d)[6], float (&r)[6]) {
  const float t1 = __fsub_rn(d[3], d[1]);
  const float t2 = __fsub_rn(d[4], d[2]);
  const float u = __fmaf_rn(4.0f, d[2], -d[4]);
  const float v = __fmaf_rn(4.0f, d[1], -d[3]);
  r[0] = __fmaf_rn(4.0f, d[0], __fmaf_rn(-5.0f, d[2], d[4]));
  r[1] = __fadd_rn(u, v);
  r[2] = __fsub_rn(u, v);
  r[3] = __fmaf_rn(2.0f, t1, t2);
  r[4] = __fmaf_rn(-2.0f, t1, t2);
  r[5] = __fmaf_rn(4.0f, d[1], __fmaf_rn(-5.0f, d[3], d[5]));
}
// 1-D A^T, factored (exact mode only: integer codes in, integers below 2^24 throughout).
__device__ __forceinline__ void at_exact(const float (&m)[4], float (&y)[2]) {
  y[0] = __fadd_rn(__fadd_rn(m[0], m[1]), m[2]);
  y[1] = __fadd_rn(__fsub_rn(m[1], m[2]), m[3]);
}
__device__ __forceinline__ void at_exact(const float (&m)[6], float (&y)[4]) {
  const float a = __fadd_rn(m[1], m[2]);
  const float b = __fsub_rn(m[1], m[2]);
  const float c = __fadd_rn(m[3], m[4]);
  const float d = __fsub_rn(m[3], m[4]);
  y[0] = __fadd_rn(__fadd_rn(m[0], a), c);
  y[1] = __fmaf_rn(2.0f, d, b);
  y[2] = __fmaf_rn(4.0f, c, a);
  y[3] = __fadd_rn(__fmaf_rn(8.0f, d, b), m[5]);
}

// V = (B^T d) B for one channel.  d is given column-wise through `col(l, out)`.
template <int M, int MODE, typename ColFn>
__device__ __forceinline__ void input_transform_2d(const Params& p, ColFn col,
                                                   float (&V)[(M + 2) * (M + 2)]) {
  constexpr int T_ = M + 2;
  constexpr bool STD = MODE != kDense;
  using MT = Mat<M, STD>;
  float P[T_][T_];
#pragma unroll
  for (int l = 0; l < T_; ++l) {
    float dcol[T_];
    col(l, dcol);
    if constexpr (MODE == kExact) {
      float r[T_];
      bt_exact(dcol, r);
#pragma unroll
      for (int i = 0; i < T_; ++i) P[i][l] = r[i];
    } else {
#pragma unroll
      for (int i = 0; i < T_; ++i) {
        float acc = 0.0f;
#pragma unroll
        for (int k = 0; k < T_; ++k) acc = chain<STD>(MT::bt(p, i, k), dcol[k], acc);
        P[i][l] = acc;
      }
    }
  }
#pragma unroll
  for (int i = 0; i < T_; ++i) {
    if constexpr (MODE == kExact) {
      float r[T_];
      bt_exact(P[i], r);
#pragma unroll
      for (int j = 0; j < T_; ++j) V[i * T_ + j] = r[j];
    } else {
#pragma unroll
      for (int j = 0; j < T_; ++j) {
        float acc = 0.0f;
#pragma unroll
        for (int l = 0; l < T_; ++l) acc = chain<STD>(MT::bt(p, j, l), P[i][l], acc);
        V[i * T_ + j] = acc;
      }
    }
  }
}

// Y = A^T (m A) for one channel: right factor first.  m row-wise via `row(i, out)`.
template <int M, int MODE, typename RowFn>
__device__ __forceinline__ void output_transform_2d(const Params& p, RowFn row,
                                                    float (&Y)[M * M]) {
  constexpr int T_ = M + 2;
  constexpr bool STD = MODE != kDense;
  using MT = Mat<M, STD>;
  float R[T_][M];
#pragma unroll
  for (int i = 0; i < T_; ++i) {
    float mrow[T_];
    row(i, mrow);
    if constexpr (MODE == kExact && M != 6) {
      at_exact(mrow, R[i]);
    } else {
#pragma unroll
      for (int jp = 0; jp < M; ++jp) {
        float acc = 0.0f;
#pragma unroll
        for (int j = 0; j < T_; ++j) acc = chain<STD>(MT::at(p, jp, j), mrow[j], acc);
        R[i][jp] = acc;
      }
    }
  }
#pragma unroll
  for (int jp = 0; jp < M; ++jp) {
    if constexpr (MODE == kExact && M != 6) {
      float c[T_], y4[M];
#pragma unroll
      for (int i = 0; i < T_; ++i) c[i] = R[i][jp];
      at_exact(c, y4);
#pragma unroll
      for (int ip = 0; ip < M; ++ip) Y[ip * M + jp] = y4[ip];
    } else {
#pragma unroll
      for (int ip = 0; ip < M; ++ip) {
        float acc = 0.0f;
#pragma unroll
        for (int i = 0; i < T_; ++i) acc = chain<STD>(MT::at(p, ip, i), R[i][jp], acc);
        Y[ip * M + jp] = acc;
      }
    }
  }
}

}  // namespace wino
