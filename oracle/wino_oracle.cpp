// CPU oracle for the Winograd-aware quantized 3x3 convolution forward pass.
//
// THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, step-by-step statement of
// what the layer computes, written from the paper (Section 3.1 Eq. 1, Fig. 2,
// Section 3.2, Section 5.1).  It shares no code with the CUDA library and must
// never be called from the product path: only the tests, the smoke check and
// the benchmark's cpu_baseline / reference legs use it.
//
// Parity status of each part (what pins it to something other than itself):
//   cook_toom            : exact-rational FIR identity, printed zero fractions
//                          (Appendix A.2), weight expansion t^2/9 (Section 3.1)
//   winograd_f64         : equals direct convolution to 1e-10; multiply counts
//                          9 / 4 / 2.25 per output and 8100 vs 3600 (Sections 1, 3.1)
//   quantize             : rounding table, second implementation via lrintf
//   staged int8 pipeline : F2 lossless special case == integer direct conv;
//                          exact-rational recomputation on tiny layers
//   per-channel scales   : equal scales == per-layer pipeline; every output channel ==
//                          the per-layer pipeline on that channel alone
//   flex (perturbed) transforms: parity unpinned beyond the rational
//                          recomputation within its error bound (no external
//                          truth exists for a perturbed transform)
//
// Conventions (all tensors dense, row-major in the index order written):
//   t = m + 2, xi = i*t + j, TH = ceil(H/m), TW = ceil(W/m), T = N*TH*TW,
//   tau = (n*TH + th)*TW + tw, padding 1, stride 1.
//   x_q [N][H][W][C] int8      w_q [K][3][3][C] int8     U_q [t*t][K][C] int8
//   V_q [t*t][T][C] int8       M   [t*t][T][K] int32     m_q [t*t][T][K] int8
//   y   [N][H][W][K] int8 or float
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------------------
// Exact rationals (Cook-Toom construction, Section 3.1).
// ---------------------------------------------------------------------------
typedef __int128 i128;

i128 gcd128(i128 a, i128 b) {
  if (a < 0) a = -a;
  if (b < 0) b = -b;
  while (b != 0) { i128 r = a % b; a = b; b = r; }
  return a;
}

struct Rat {
  i128 n, d;  // d > 0, gcd(n, d) == 1
  Rat() : n(0), d(1) {}
  Rat(i128 nn, i128 dd) : n(nn), d(dd) { norm(); }
  void norm() {
    if (d < 0) { n = -n; d = -d; }
    i128 g = gcd128(n, d);
    if (g > 1) { n /= g; d /= g; }
    if (n == 0) d = 1;
  }
};
Rat operator+(const Rat& a, const Rat& b) { return Rat(a.n * b.d + b.n * a.d, a.d * b.d); }
Rat operator-(const Rat& a, const Rat& b) { return Rat(a.n * b.d - b.n * a.d, a.d * b.d); }
Rat operator*(const Rat& a, const Rat& b) { return Rat(a.n * b.n, a.d * b.d); }
Rat operator/(const Rat& a, const Rat& b) { return Rat(a.n * b.d, a.d * b.n); }
Rat neg(const Rat& a) { return Rat(-a.n, a.d); }

// Multiply polynomial p (ascending coefficients) by (x - a).
std::vector<Rat> mul_linear(const std::vector<Rat>& p, const Rat& a) {
  std::vector<Rat> q(p.size() + 1);
  for (size_t i = 0; i < p.size(); ++i) {
    q[i + 1] = q[i + 1] + p[i];
    q[i] = q[i] - p[i] * a;
  }
  return q;
}

// Correctly rounded (nearest, ties to even) conversion of n/d to binary32.
float rat_to_f32(const Rat& r) {
  if (r.n == 0) return 0.0f;
  double approx = (double)r.n / (double)r.d;
  float c0 = (float)approx;
  float cand[3] = {c0, std::nextafterf(c0, INFINITY), std::nextafterf(c0, -INFINITY)};
  // |n/d - c| compared exactly: c = mant * 2^e with integer mant.
  int best = -1;
  i128 best_num = 0, best_den = 1;  // error as a rational best_num / best_den
  for (int i = 0; i < 3; ++i) {
    int e;
    double fr = std::frexp((double)cand[i], &e);   // cand = fr * 2^e, 0.5 <= |fr| < 1
    i128 mant = (i128)std::ldexp(fr, 24);          // exact: 24-bit significand
    int ee = e - 24;                               // cand = mant * 2^ee
    Rat c = (ee >= 0) ? Rat(mant * ((i128)1 << ee), 1) : Rat(mant, (i128)1 << (-ee));
    Rat err = r - c;
    if (err.n < 0) err.n = -err.n;
    bool better;
    if (best < 0) better = true;
    else {
      i128 lhs = err.n * best_den, rhs = best_num * err.d;
      if (lhs < rhs) better = true;
      else if (lhs > rhs) better = false;
      else {  // tie: even significand wins
        uint32_t bits; std::memcpy(&bits, &cand[i], 4);
        better = (bits & 1u) == 0;
      }
    }
    if (better) { best = i; best_num = err.n; best_den = err.d; }
  }
  return cand[best];
}

// Cook-Toom matrices for F(m, 3) from t-1 finite points plus the point at
// infinity.  Rows of BT are monic polynomial coefficients, G carries 1/N_j.
void cook_toom_rat(int m, const Rat* pts, std::vector<Rat>& BT, std::vector<Rat>& G,
                   std::vector<Rat>& AT) {
  const int t = m + 2;
  BT.assign(t * t, Rat());
  G.assign(t * 3, Rat());
  AT.assign(m * t, Rat());
  for (int j = 0; j < t - 1; ++j) {
    std::vector<Rat> p(1, Rat(1, 1));
    Rat Nj(1, 1);
    for (int k = 0; k < t - 1; ++k) {
      if (k == j) continue;
      p = mul_linear(p, pts[k]);
      Nj = Nj * (pts[j] - pts[k]);
    }
    for (size_t c = 0; c < p.size(); ++c) BT[j * t + c] = p[c];
    Rat pw(1, 1);
    for (int k = 0; k < 3; ++k) { G[j * 3 + k] = pw / Nj; pw = pw * pts[j]; }
    pw = Rat(1, 1);
    for (int i = 0; i < m; ++i) { AT[i * t + j] = pw; pw = pw * pts[j]; }
    if (G[j * 3 + 0].n < 0) {
      for (int k = 0; k < 3; ++k) G[j * 3 + k] = neg(G[j * 3 + k]);
      for (int c = 0; c < t; ++c) BT[j * t + c] = neg(BT[j * t + c]);
    }
  }
  std::vector<Rat> p(1, Rat(1, 1));
  for (int k = 0; k < t - 1; ++k) p = mul_linear(p, pts[k]);
  for (int c = 0; c < t; ++c) BT[(t - 1) * t + c] = p[c];
  G[(t - 1) * 3 + 2] = Rat(1, 1);
  AT[(m - 1) * t + (t - 1)] = Rat(1, 1);
}

// ---------------------------------------------------------------------------
// Uniform quantizer (Section 5.1: per-layer symmetric uniform quantization):
// code = clamp(round_half_even(v * mult) + z), the rounding applied to the exact
// product of the fp32 value and the fixed fp32 multiplier.
// ---------------------------------------------------------------------------
inline int32_t quantize(float v, float mult, int32_t z, int32_t qmin, int32_t qmax) {
  // the product of two binary32 numbers is exact in binary64, so this rounds the
  // exact real product once, ties to even (default rounding mode)
  double r = std::nearbyint((double)v * (double)mult);
  double lo = (double)(qmin - z), hi = (double)(qmax - z);
  if (r < lo) r = lo;
  if (r > hi) r = hi;
  return (int32_t)r + z;
}

struct Quant { float scale; int32_t zero_point, qmin, qmax, enabled; };
struct Desc {
  int32_t N, C, H, W, K, m;
  const float *BT, *G, *AT;
  Quant q_x, q_w, q_V, q_U, q_M, q_Y;
  int32_t out_dtype;  // 0 = int8, 1 = float
  // Per-output-channel scales (Section 7 names per-channel quantization as the next
  // step beyond the per-layer scales of Section 5.1): K floats each, or null for the
  // per-layer scale of q_w / q_U / q_M / q_Y: the four tensors that carry the output-channel
  // axis (the input side is summed over its channels by the Hadamard stage and keeps one
  // scale).  Zero points and code ranges stay per layer.
  const float *s_w_K, *s_U_K, *s_M_K, *s_Y_K;
};
inline double scale_w(const Desc& d, int k) { return d.s_w_K ? (double)d.s_w_K[k] : (double)d.q_w.scale; }
inline double scale_U(const Desc& d, int k) { return d.s_U_K ? (double)d.s_U_K[k] : (double)d.q_U.scale; }
inline double scale_M(const Desc& d, int k) { return d.s_M_K ? (double)d.s_M_K[k] : (double)d.q_M.scale; }
inline double scale_Y(const Desc& d, int k) { return d.s_Y_K ? (double)d.s_Y_K[k] : (double)d.q_Y.scale; }

struct Geo {
  int m, t, TH, TW; long T;
  explicit Geo(const Desc& d) {
    m = d.m; t = m + 2;
    TH = (d.H + m - 1) / m; TW = (d.W + m - 1) / m;
    T = (long)d.N * TH * TW;
  }
};

inline float ratio_f32(double num, double den) { return (float)(num / den); }

// Two-sided transform Z = (L X) L^T with L of shape [p][q], X [q][q]:
// left pass then right pass, each a fused-multiply-add chain that starts from
// 0.0f and runs over the contracted index in ascending order.
void two_sided(const float* L, int p, int q, const float* X, float* Z) {
  float P[8 * 8];
  for (int i = 0; i < p; ++i)
    for (int l = 0; l < q; ++l) {
      float acc = 0.0f;
      for (int k = 0; k < q; ++k) acc = std::fmaf(L[i * q + k], X[k * q + l], acc);
      P[i * q + l] = acc;
    }
  for (int i = 0; i < p; ++i)
    for (int j = 0; j < p; ++j) {
      float acc = 0.0f;
      for (int l = 0; l < q; ++l) acc = std::fmaf(P[i * q + l], L[j * q + l], acc);
      Z[i * p + j] = acc;
    }
}

}  // namespace

extern "C" {

typedef Quant orc_quant_t;
typedef Desc orc_desc_t;

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void orc_set_num_threads(int n) {
#ifdef _OPENMP
  omp_set_num_threads(n);
#else
  (void)n;
#endif
}

// Section 3.1 (Cook-Toom construction).  Points are pts_num[i]/pts_den[i],
// i < m+1, in the order given.  Outputs: exact numerators/denominators
// (int64) and the correctly rounded fp32 / fp64 values.  Returns 0, or -1 on
// bad arguments.
int orc_cook_toom(int m, const int64_t* pts_num, const int64_t* pts_den,
                  int64_t* BT_num, int64_t* BT_den, int64_t* G_num, int64_t* G_den,
                  int64_t* AT_num, int64_t* AT_den,
                  float* BT_f32, float* G_f32, float* AT_f32,
                  double* BT_f64, double* G_f64, double* AT_f64) {
  if (m < 1 || m > 6) return -1;
  const int t = m + 2;
  std::vector<Rat> pts(t - 1);
  for (int i = 0; i < t - 1; ++i) {
    if (pts_den[i] == 0) return -1;
    pts[i] = Rat(pts_num[i], pts_den[i]);
  }
  std::vector<Rat> BT, G, AT;
  cook_toom_rat(m, pts.data(), BT, G, AT);
  for (int i = 0; i < t * t; ++i) {
    BT_num[i] = (int64_t)BT[i].n; BT_den[i] = (int64_t)BT[i].d;
    BT_f32[i] = rat_to_f32(BT[i]); BT_f64[i] = (double)BT[i].n / (double)BT[i].d;
  }
  for (int i = 0; i < t * 3; ++i) {
    G_num[i] = (int64_t)G[i].n; G_den[i] = (int64_t)G[i].d;
    G_f32[i] = rat_to_f32(G[i]); G_f64[i] = (double)G[i].n / (double)G[i].d;
  }
  for (int i = 0; i < m * t; ++i) {
    AT_num[i] = (int64_t)AT[i].n; AT_den[i] = (int64_t)AT[i].d;
    AT_f32[i] = rat_to_f32(AT[i]); AT_f64[i] = (double)AT[i].n / (double)AT[i].d;
  }
  return 0;
}

int32_t orc_quantize(float v, float mult, int32_t z, int32_t qmin, int32_t qmax) {
  return quantize(v, mult, z, qmin, qmax);
}

// The five fixed multipliers of the pipeline, each rounded once to fp32 from a
// double-precision ratio of the stage scales.
// out[0] = s_x/s_V, out[1] = s_w/s_U, out[2] = s_U*s_V/s_M,
// out[3] = s_acc/s_Y, out[4] = s_acc, where s_acc = s_M when Q_M is enabled and
// s_U*s_V otherwise.  Per-layer scales only (per-channel scales, when given, replace
// s_w, s_U, s_M and s_Y by their channel's value in the same formulas).
void orc_multipliers(const orc_desc_t* d, float* out) {
  double sUV = (double)d->q_U.scale * (double)d->q_V.scale;
  double s_acc = d->q_M.enabled ? (double)d->q_M.scale : sUV;
  out[0] = ratio_f32(d->q_x.scale, d->q_V.scale);
  out[1] = ratio_f32(d->q_w.scale, d->q_U.scale);
  out[2] = ratio_f32(sUV, d->q_M.scale);
  out[3] = ratio_f32(s_acc, d->q_Y.scale);
  out[4] = (float)s_acc;
}

// Stage (1): V = B^T d B on every (tile, channel) patch, then Q_V
// (Eq. 1, Fig. 2).  V_f32 (nullable) receives the un-quantized transform,
// V_q (nullable) the int8 codes.
int orc_input_stage(const orc_desc_t* d, const int8_t* x_q, float* V_f32, int8_t* V_q) {
  Geo g(*d);
  const int t = g.t, C = d->C, H = d->H, W = d->W;
  const float mult_V = ratio_f32(d->q_x.scale, d->q_V.scale);
#pragma omp parallel for schedule(static)
  for (long tau = 0; tau < g.T; ++tau) {
    int tw = (int)(tau % g.TW);
    int th = (int)((tau / g.TW) % g.TH);
    int n = (int)(tau / ((long)g.TW * g.TH));
    float patch[64], V[64];
    for (int c = 0; c < C; ++c) {
      for (int a = 0; a < t; ++a)
        for (int b = 0; b < t; ++b) {
          int h = th * g.m - 1 + a, w = tw * g.m - 1 + b;
          float v = 0.0f;
          if (h >= 0 && h < H && w >= 0 && w < W)
            v = (float)((int32_t)x_q[(((long)n * H + h) * W + w) * C + c] - d->q_x.zero_point);
          patch[a * t + b] = v;
        }
      two_sided(d->BT, t, t, patch, V);
      for (int xi = 0; xi < t * t; ++xi) {
        long o = ((long)xi * g.T + tau) * C + c;
        if (V_f32) V_f32[o] = V[xi];
        if (V_q)
          V_q[o] = (int8_t)quantize(V[xi], mult_V, d->q_V.zero_point, d->q_V.qmin, d->q_V.qmax);
      }
    }
  }
  return 0;
}

// Stage (2): U = G g G^T for every (k, c) filter, then Q_U (Eq. 1, Fig. 2).
int orc_weight_stage(const orc_desc_t* d, const int8_t* w_q, float* U_f32, int8_t* U_q) {
  const int t = d->m + 2, C = d->C, K = d->K;
#pragma omp parallel for schedule(static)
  for (int k = 0; k < K; ++k) {
    float gk[9], P[8 * 3], U[64];
    const float mult_U = ratio_f32(scale_w(*d, k), scale_U(*d, k));
    for (int c = 0; c < C; ++c) {
      for (int a = 0; a < 3; ++a)
        for (int b = 0; b < 3; ++b)
          gk[a * 3 + b] =
              (float)((int32_t)w_q[(((long)k * 3 + a) * 3 + b) * C + c] - d->q_w.zero_point);
      // left pass P = G g  ([t][3]), right pass U = P G^T ([t][t])
      for (int i = 0; i < t; ++i)
        for (int l = 0; l < 3; ++l) {
          float acc = 0.0f;
          for (int kk = 0; kk < 3; ++kk) acc = std::fmaf(d->G[i * 3 + kk], gk[kk * 3 + l], acc);
          P[i * 3 + l] = acc;
        }
      for (int i = 0; i < t; ++i)
        for (int j = 0; j < t; ++j) {
          float acc = 0.0f;
          for (int l = 0; l < 3; ++l) acc = std::fmaf(P[i * 3 + l], d->G[j * 3 + l], acc);
          U[i * t + j] = acc;
        }
      for (int xi = 0; xi < t * t; ++xi) {
        long o = ((long)xi * K + k) * C + c;
        if (U_f32) U_f32[o] = U[xi];
        if (U_q)
          U_q[o] = (int8_t)quantize(U[xi], mult_U, d->q_U.zero_point, d->q_U.qmin, d->q_U.qmax);
      }
    }
  }
  return 0;
}

// Stage (3): the Hadamard product summed over channels, i.e. t*t independent
// integer matrix products M[xi] = V_q[xi] * U_q[xi]^T (Sections 1 and 5.3).
int orc_hadamard(const orc_desc_t* d, const int8_t* V_q, const int8_t* U_q, int32_t* M) {
  Geo g(*d);
  const int t2 = g.t * g.t, C = d->C, K = d->K;
  const int zV = d->q_V.zero_point, zU = d->q_U.zero_point;
#pragma omp parallel for collapse(2) schedule(static)
  for (int xi = 0; xi < t2; ++xi)
    for (long tau = 0; tau < g.T; ++tau) {
      const int8_t* v = V_q + ((long)xi * g.T + tau) * C;
      for (int k = 0; k < K; ++k) {
        const int8_t* u = U_q + ((long)xi * K + k) * C;
        int32_t acc = 0;
        for (int c = 0; c < C; ++c) acc += ((int32_t)v[c] - zV) * ((int32_t)u[c] - zU);
        M[((long)xi * g.T + tau) * K + k] = acc;
      }
    }
  return 0;
}

// Q_M: quantize the Hadamard-stage output (Fig. 2: every intermediate is
// quantized to the level of the inputs and weights).
int orc_quantize_M(const orc_desc_t* d, const int32_t* M, int8_t* m_q) {
  Geo g(*d);
  const long total = (long)g.t * g.t * g.T * d->K;
  std::vector<float> mult_M((size_t)d->K);   // the accumulator of channel k carries s_U[k] * s_V
  for (int k = 0; k < d->K; ++k)
    mult_M[k] = ratio_f32(scale_U(*d, k) * (double)d->q_V.scale, scale_M(*d, k));
#pragma omp parallel for schedule(static)
  for (long i = 0; i < total; ++i)
    m_q[i] = (int8_t)quantize((float)M[i], mult_M[i % d->K], d->q_M.zero_point, d->q_M.qmin,
                              d->q_M.qmax);
  return 0;
}

// Stage (4): Y = A^T m A per (tile, k), plus bias, then Q_Y or a float output
// (Eq. 1, Fig. 2).  The right factor is applied first (R = m A), then the
// left one (Y = A^T R).  m is (float)m_q when Q_M is enabled, (float)M
// otherwise.  Y_f32 (nullable) receives the transform before the output
// scaling, laid out [T][K][m][m].  y is int8 or float per out_dtype.
int orc_output_stage(const orc_desc_t* d, const int32_t* M, const int8_t* m_q,
                     const float* bias, float* Y_f32, void* y) {
  Geo g(*d);
  const int t = g.t, m = g.m, K = d->K, H = d->H, W = d->W;
  // per output channel: s_acc = s_M[k] when Q_M is enabled and s_U[k] * s_V otherwise;
  // mult_Y = s_acc / s_Y[k]; the bias enters the integer output as bias / s_Y[k]
  std::vector<float> mult_Y_k((size_t)K), s_acc_k((size_t)K), bias_k((size_t)K);
  for (int k = 0; k < K; ++k) {
    const double s_acc_d =
        d->q_M.enabled ? scale_M(*d, k) : scale_U(*d, k) * (double)d->q_V.scale;
    mult_Y_k[k] = ratio_f32(s_acc_d, scale_Y(*d, k));
    s_acc_k[k] = (float)s_acc_d;
    bias_k[k] = bias ? (float)((double)bias[k] / scale_Y(*d, k)) : 0.0f;
  }
#pragma omp parallel for schedule(static)
  for (long tau = 0; tau < g.T; ++tau) {
    int tw = (int)(tau % g.TW);
    int th = (int)((tau / g.TW) % g.TH);
    int n = (int)(tau / ((long)g.TW * g.TH));
    float mf[64], R[8 * 6], Y[36];
    for (int k = 0; k < K; ++k) {
      for (int xi = 0; xi < t * t; ++xi) {
        long o = ((long)xi * g.T + tau) * K + k;
        mf[xi] = d->q_M.enabled ? (float)((int32_t)m_q[o] - d->q_M.zero_point) : (float)M[o];
      }
      for (int i = 0; i < t; ++i)
        for (int jp = 0; jp < m; ++jp) {
          float acc = 0.0f;
          for (int j = 0; j < t; ++j) acc = std::fmaf(mf[i * t + j], d->AT[jp * t + j], acc);
          R[i * m + jp] = acc;
        }
      for (int ip = 0; ip < m; ++ip)
        for (int jp = 0; jp < m; ++jp) {
          float acc = 0.0f;
          for (int i = 0; i < t; ++i) acc = std::fmaf(d->AT[ip * t + i], R[i * m + jp], acc);
          Y[ip * m + jp] = acc;
        }
      for (int ip = 0; ip < m; ++ip)
        for (int jp = 0; jp < m; ++jp) {
          float Yv = Y[ip * m + jp];
          if (Y_f32) Y_f32[((tau * K + k) * m + ip) * m + jp] = Yv;
          int h = th * m + ip, w = tw * m + jp;
          if (h >= H || w >= W) continue;
          long o = (((long)n * H + h) * W + w) * K + k;
          if (d->out_dtype == 1) {
            ((float*)y)[o] = std::fmaf(Yv, s_acc_k[k], bias ? bias[k] : 0.0f);
          } else {
            float yf = std::fmaf(Yv, mult_Y_k[k], bias_k[k]);
            ((int8_t*)y)[o] =
                (int8_t)quantize(yf, 1.0f, d->q_Y.zero_point, d->q_Y.qmin, d->q_Y.qmax);
          }
        }
    }
  }
  return 0;
}

// The whole forward pass, stage by stage.  Any of the dump pointers may be
// null.  U_q_in (nullable): pre-transformed weights; when null, w_q is
// transformed first.
int orc_forward(const orc_desc_t* d, const int8_t* x_q, const int8_t* w_q, const int8_t* U_q_in,
                const float* bias, void* y, int8_t* V_q_out, int8_t* U_q_out, int32_t* M_out,
                int8_t* m_q_out) {
  Geo g(*d);
  const long t2 = (long)g.t * g.t;
  std::vector<int8_t> Vq((size_t)(t2 * g.T * d->C));
  std::vector<int8_t> Uq;
  const int8_t* Uq_p = U_q_in;
  if (!Uq_p) {
    if (!w_q) return -1;
    Uq.resize((size_t)(t2 * d->K * d->C));
    orc_weight_stage(d, w_q, nullptr, Uq.data());
    Uq_p = Uq.data();
  }
  std::vector<int32_t> M((size_t)(t2 * g.T * d->K));
  std::vector<int8_t> mq;
  orc_input_stage(d, x_q, nullptr, Vq.data());
  orc_hadamard(d, Vq.data(), Uq_p, M.data());
  if (d->q_M.enabled) {
    mq.resize(M.size());
    orc_quantize_M(d, M.data(), mq.data());
  }
  orc_output_stage(d, M.data(), d->q_M.enabled ? mq.data() : nullptr, bias, nullptr, y);
  if (V_q_out) std::memcpy(V_q_out, Vq.data(), Vq.size());
  if (U_q_out) std::memcpy(U_q_out, Uq_p, (size_t)(t2 * d->K * d->C));
  if (M_out) std::memcpy(M_out, M.data(), M.size() * sizeof(int32_t));
  if (m_q_out && d->q_M.enabled) std::memcpy(m_q_out, mq.data(), mq.size());
  return 0;
}

// Direct 3x3 convolution (cross-correlation, padding 1) on integer codes with
// int32 accumulation; the reference any Winograd form must reproduce when no
// rounding intervenes.  stride 1 or 2.  acc: [N][Ho][Wo][K] with
// Ho = (H - 1)/stride + 1.
int orc_direct_conv_i32(int N, int C, int H, int W, int K, int stride, const int8_t* x_q,
                        int z_x, const int8_t* w_q, int z_w, int32_t* acc) {
  const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int ho = 0; ho < Ho; ++ho)
      for (int wo = 0; wo < Wo; ++wo)
        for (int k = 0; k < K; ++k) {
          int32_t s = 0;
          for (int a = 0; a < 3; ++a)
            for (int b = 0; b < 3; ++b) {
              int h = ho * stride - 1 + a, w = wo * stride - 1 + b;
              if (h < 0 || h >= H || w < 0 || w >= W) continue;
              const int8_t* xp = x_q + (((long)n * H + h) * W + w) * C;
              const int8_t* wp = w_q + (((long)k * 3 + a) * 3 + b) * C;
              for (int c = 0; c < C; ++c) s += ((int32_t)xp[c] - z_x) * ((int32_t)wp[c] - z_w);
            }
          acc[(((long)n * Ho + ho) * Wo + wo) * K + k] = s;
        }
  return 0;
}

// Output quantizer applied to a direct-convolution accumulator:
// y = Q(fmaf(acc, s_x*s_w/s_Y, bias/s_Y)).
int orc_requantize_acc(long count, int K, const int32_t* acc, double s_in, const float* bias,
                       const orc_quant_t* q_Y, int8_t* y) {
  const float mult = (float)(s_in / (double)q_Y->scale);
#pragma omp parallel for schedule(static)
  for (long i = 0; i < count; ++i) {
    int k = (int)(i % K);
    float bs = bias ? (float)((double)bias[k] / (double)q_Y->scale) : 0.0f;
    float yf = std::fmaf((float)acc[i], mult, bs);
    y[i] = (int8_t)quantize(yf, 1.0f, q_Y->zero_point, q_Y->qmin, q_Y->qmax);
  }
  return 0;
}

// The same with per-output-channel scales (Section 7): s_in_K[k] (nullable) replaces s_in
// and s_Y_K[k] (nullable) replaces q_Y->scale for channel k.
int orc_requantize_acc_channels(long count, int K, const int32_t* acc, double s_in,
                                const double* s_in_K, const float* bias, const orc_quant_t* q_Y,
                                const float* s_Y_K, int8_t* y) {
#pragma omp parallel for schedule(static)
  for (long i = 0; i < count; ++i) {
    int k = (int)(i % K);
    const double s_in_k = s_in_K ? s_in_K[k] : s_in;
    const double s_Y_k = s_Y_K ? (double)s_Y_K[k] : (double)q_Y->scale;
    const float mult = (float)(s_in_k / s_Y_k);
    float bs = bias ? (float)((double)bias[k] / s_Y_k) : 0.0f;
    float yf = std::fmaf((float)acc[i], mult, bs);
    y[i] = (int8_t)quantize(yf, 1.0f, q_Y->zero_point, q_Y->qmin, q_Y->qmax);
  }
  return 0;
}

// Un-quantized double-precision Winograd convolution (Eq. 1) and direct
// convolution on real-valued tensors; pad is 0 ("valid") or 1.  Both return
// the number of general multiplications they performed per (input channel,
// output channel) pair, i.e. the count Sections 1 and 3.1 quote.
// x [N][H][W][C], w [K][3][3][C], y [N][Ho][Wo][K], Ho = H + 2*pad - 2.
long orc_winograd_f64(int N, int C, int H, int W, int K, int m, int pad, const double* BT,
                      const double* G, const double* AT, const double* x, const double* w,
                      double* y) {
  const int t = m + 2;
  const int Ho = H + 2 * pad - 2, Wo = W + 2 * pad - 2;
  const int TH = (Ho + m - 1) / m, TW = (Wo + m - 1) / m;
  std::vector<double> U((size_t)t * t * K * C);
  for (int k = 0; k < K; ++k)
    for (int c = 0; c < C; ++c) {
      double P[8 * 3];
      for (int i = 0; i < t; ++i)
        for (int l = 0; l < 3; ++l) {
          double acc = 0;
          for (int kk = 0; kk < 3; ++kk)
            acc += G[i * 3 + kk] * w[(((long)k * 3 + kk) * 3 + l) * C + c];
          P[i * 3 + l] = acc;
        }
      for (int i = 0; i < t; ++i)
        for (int j = 0; j < t; ++j) {
          double acc = 0;
          for (int l = 0; l < 3; ++l) acc += P[i * 3 + l] * G[j * 3 + l];
          U[((long)(i * t + j) * K + k) * C + c] = acc;
        }
    }
  long mults = 0;
  for (int n = 0; n < N; ++n)
    for (int th = 0; th < TH; ++th)
      for (int tw = 0; tw < TW; ++tw) {
        std::vector<double> V((size_t)t * t * C);
        for (int c = 0; c < C; ++c) {
          double dd[64], P[64];
          for (int a = 0; a < t; ++a)
            for (int b = 0; b < t; ++b) {
              int h = th * m - pad + a, ww = tw * m - pad + b;
              dd[a * t + b] = (h >= 0 && h < H && ww >= 0 && ww < W)
                                  ? x[(((long)n * H + h) * W + ww) * C + c] : 0.0;
            }
          for (int i = 0; i < t; ++i)
            for (int l = 0; l < t; ++l) {
              double acc = 0;
              for (int k = 0; k < t; ++k) acc += BT[i * t + k] * dd[k * t + l];
              P[i * t + l] = acc;
            }
          for (int i = 0; i < t; ++i)
            for (int j = 0; j < t; ++j) {
              double acc = 0;
              for (int l = 0; l < t; ++l) acc += P[i * t + l] * BT[j * t + l];
              V[(long)(i * t + j) * C + c] = acc;
            }
        }
        for (int k = 0; k < K; ++k) {
          double Mx[64], R[8 * 6];
          for (int xi = 0; xi < t * t; ++xi) {
            double acc = 0;
            for (int c = 0; c < C; ++c) acc += V[(long)xi * C + c] * U[((long)xi * K + k) * C + c];
            Mx[xi] = acc;
          }
          if (k == 0) mults += (long)t * t;  // one product per xi per (c, k) pair
          for (int i = 0; i < t; ++i)
            for (int jp = 0; jp < m; ++jp) {
              double acc = 0;
              for (int j = 0; j < t; ++j) acc += Mx[i * t + j] * AT[jp * t + j];
              R[i * m + jp] = acc;
            }
          for (int ip = 0; ip < m; ++ip)
            for (int jp = 0; jp < m; ++jp) {
              double acc = 0;
              for (int i = 0; i < t; ++i) acc += AT[ip * t + i] * R[i * m + jp];
              int h = th * m + ip, ww = tw * m + jp;
              if (h < Ho && ww < Wo) y[(((long)n * Ho + h) * Wo + ww) * K + k] = acc;
            }
        }
      }
  return mults;
}

long orc_direct_f64(int N, int C, int H, int W, int K, int pad, const double* x, const double* w,
                    double* y) {
  const int Ho = H + 2 * pad - 2, Wo = W + 2 * pad - 2;
  long mults = 0;
  for (int n = 0; n < N; ++n)
    for (int ho = 0; ho < Ho; ++ho)
      for (int wo = 0; wo < Wo; ++wo) {
        mults += 9;  // nine products per output per (c, k) pair, padded taps included
        for (int k = 0; k < K; ++k) {
          double s = 0;
          for (int a = 0; a < 3; ++a)
            for (int b = 0; b < 3; ++b) {
              int h = ho - pad + a, ww = wo - pad + b;
              if (h < 0 || h >= H || ww < 0 || ww >= W) continue;
              for (int c = 0; c < C; ++c)
                s += x[(((long)n * H + h) * W + ww) * C + c] * w[(((long)k * 3 + a) * 3 + b) * C + c];
            }
          y[(((long)n * Ho + ho) * Wo + wo) * K + k] = s;
        }
      }
  return mults;
}

}  // extern "C"
