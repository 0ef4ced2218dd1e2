// Host side of the C ABI declared in include/wino.h: plan construction,
// argument checks, path choice, TMA descriptor encoding and kernel launches.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include <cuda.h>
#include <cuda_runtime.h>

#include "wino.h"
#include "wino_common.cuh"
#include "wino_gemm.cuh"
#include "wino_smallc.cuh"
#include "wino_transforms.cuh"

using namespace wino;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct wino_plan {
  wino_desc_t d;
  Params p;
  float s_Y;
  bool std_mats;        // BT and AT equal the built-in Cook-Toom matrices bit for bit
  int path;
  int* status_dev;      // device status word (may be null when no GPU is present)
  bool tc_attr_set;
  // memo of the last encoded tensor maps
  mutable const void* map_vq_ptr;
  mutable const void* map_uq_ptr;
  mutable CUtensorMap mapV, mapU;
  // last forward call, for wino_debug_dump_stage
  mutable const int8_t* last_uq;
  mutable void* last_ws;
  mutable cudaStream_t last_stream;
  mutable long launches;
  cudaEvent_t stage_ev[4];  // caller-owned; recorded around the three staged kernels when set
  bool stage_ev_on;
};

namespace {

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) ==
            cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

inline bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

bool quant_ok(const wino_quant_t& q) {
  return std::isfinite(q.scale) && q.scale > 0.0f && q.qmin >= -128 && q.qmax <= 127 &&
         q.qmin <= q.qmax;
}

template <int M>
bool is_std(const float* BT, const float* AT) {
  constexpr int T_ = M + 2;
  for (int i = 0; i < T_; ++i)
    for (int k = 0; k < T_; ++k)
      if (BT[i * T_ + k] != std_bt<M>(i, k)) return false;
  for (int i = 0; i < M; ++i)
    for (int k = 0; k < T_; ++k)
      if (AT[i * T_ + k] != std_at<M>(i, k)) return false;
  return true;
}

bool path_supported(const wino_plan_t* pl, int path) {
  const int C = pl->d.C, K = pl->d.K;
  switch (path) {
    case WINO_PATH_STAGED_TC: return C % 16 == 0 && K % 16 == 0;
    case WINO_PATH_STAGED_DP4A: return C % 4 == 0 && K % 4 == 0;
    case WINO_PATH_SMALLC: return C % 4 == 0 && K % 4 == 0 && C <= 32 && K <= 32;
    default: return false;
  }
}

size_t vq_bytes(const wino_plan_t* pl) { return (size_t)pl->p.t * pl->p.t * pl->p.T * pl->p.C; }
size_t m_elems(const wino_plan_t* pl) { return (size_t)pl->p.t * pl->p.t * pl->p.T * pl->p.K; }
size_t mbuf_bytes(const wino_plan_t* pl) { return m_elems(pl) * (pl->p.qM_enabled ? 1 : 4); }

int check_launch(const wino_plan_t* pl) {
  pl->launches++;
  return cudaGetLastError() == cudaSuccess ? WINO_OK : WINO_ERR_CUDA;
}

// --- launches -------------------------------------------------------------
template <int M>
int launch_weight(const wino_plan_t* pl, const int8_t* w, int8_t* Uq, unsigned* absmax,
                  cudaStream_t st) {
  const long total = (long)pl->p.K * (pl->p.C / 4);
  const int grid = (int)((total + 127) / 128);
  k_weight_transform<M><<<grid, 128, 0, st>>>(pl->p, w, Uq, absmax);
  return check_launch(pl);
}

template <int M>
int launch_input(const wino_plan_t* pl, const int8_t* x, int8_t* Vq, unsigned* absmax,
                 cudaStream_t st) {
  const long total = (long)pl->p.T * (pl->p.C / 4);
  const int grid = (int)((total + 127) / 128);
  if (pl->std_mats)
    k_input_transform<M, true><<<grid, 128, 0, st>>>(pl->p, x, Vq, absmax);
  else
    k_input_transform<M, false><<<grid, 128, 0, st>>>(pl->p, x, Vq, absmax);
  return check_launch(pl);
}

template <int M>
int launch_output(const wino_plan_t* pl, const void* mbuf, const float* bias, void* y,
                  unsigned* absmax2, cudaStream_t st) {
  const long total = (long)pl->p.T * (pl->p.K / 4);
  const int grid = (int)((total + 127) / 128);
  const bool qm = pl->p.qM_enabled != 0;
  if (pl->std_mats) {
    if (qm) k_output_transform<M, true, true><<<grid, 128, 0, st>>>(pl->p, mbuf, bias, y, pl->s_Y, absmax2);
    else k_output_transform<M, true, false><<<grid, 128, 0, st>>>(pl->p, mbuf, bias, y, pl->s_Y, absmax2);
  } else {
    if (qm) k_output_transform<M, false, true><<<grid, 128, 0, st>>>(pl->p, mbuf, bias, y, pl->s_Y, absmax2);
    else k_output_transform<M, false, false><<<grid, 128, 0, st>>>(pl->p, mbuf, bias, y, pl->s_Y, absmax2);
  }
  return check_launch(pl);
}

#define DISPATCH_M(pl, call)                         \
  ((pl)->p.m == 2 ? call<2> : (pl)->p.m == 4 ? call<4> : call<6>)

int encode_map(CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows, uint64_t mats,
               uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return WINO_ERR_CUDA;
  cuuint64_t dims[3] = {inner, rows, mats};
  cuuint64_t strides[2] = {inner, inner * rows};  // bytes (int8 elements)
  cuuint32_t box[3] = {(cuuint32_t)kStageK, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides,
                  box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? WINO_OK : WINO_ERR_CUDA;
}

struct TcGeom { int BN, stages, tmem_cols; size_t smem; };

TcGeom tc_geom(const wino_plan_t* pl) {
  TcGeom g;
  const int K = pl->p.K;
  g.BN = K >= 256 ? 256 : (int)round_up((size_t)K, 16);
  const int KB = (pl->p.C + kStageK - 1) / kStageK;
  g.stages = KB < 4 ? KB : 4;
  const size_t per_stage = (size_t)kBM * kStageK + (size_t)g.BN * kStageK;
  while (g.stages > 1 && g.stages * per_stage > 200 * 1024) --g.stages;
  g.tmem_cols = 32;
  while (g.tmem_cols < g.BN) g.tmem_cols *= 2;
  g.smem = 1024 + g.stages * per_stage + 16 * g.stages + 64;
  return g;
}

int launch_gemm(const wino_plan_t* pl, const int8_t* Vq, const int8_t* Uq, void* out, int out_mode,
                unsigned* absmaxM, cudaStream_t st) {
  const Params& p = pl->p;
  const int t2 = p.t * p.t;
  if (pl->path == WINO_PATH_STAGED_DP4A) {
    const long total = (long)p.T * (p.K / 4);
    dim3 grid((unsigned)((total + 127) / 128), 1, (unsigned)t2);
    k_gemm_dp4a<<<grid, 128, 0, st>>>(p, Vq, Uq, out, out_mode, absmaxM);
    return check_launch(pl);
  }
  TcGeom g = tc_geom(pl);
  if (pl->map_vq_ptr != Vq) {
    int rc = encode_map(&pl->mapV, Vq, (uint64_t)p.C, (uint64_t)p.T, (uint64_t)t2, kBM);
    if (rc != WINO_OK) return rc;
    pl->map_vq_ptr = Vq;
  }
  if (pl->map_uq_ptr != Uq) {
    int rc = encode_map(&pl->mapU, Uq, (uint64_t)p.C, (uint64_t)p.K, (uint64_t)t2, (uint32_t)g.BN);
    if (rc != WINO_OK) return rc;
    pl->map_uq_ptr = Uq;
  }
  if (!pl->tc_attr_set) {
    if (cudaFuncSetAttribute(k_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) !=
        cudaSuccess)
      return WINO_ERR_CUDA;
    const_cast<wino_plan_t*>(pl)->tc_attr_set = true;
  }
  GemmTcArgs a;
  a.BN = g.BN; a.stages = g.stages; a.tmem_cols = g.tmem_cols; a.out_mode = out_mode;
  dim3 grid((unsigned)((p.T + kBM - 1) / kBM), (unsigned)((p.K + g.BN - 1) / g.BN), (unsigned)t2);
  k_gemm_tc<<<grid, 128, g.smem, st>>>(p, pl->mapV, pl->mapU, a, out, absmaxM, pl->status_dev);
  return check_launch(pl);
}

int forward_impl(const wino_plan_t* pl, const int8_t* x, const int8_t* Uq, const float* bias, void* y,
                 void* ws, unsigned* absmax4, cudaStream_t st) {
  if (pl->status_dev == nullptr) return WINO_ERR_CUDA;
  const bool calib = absmax4 != nullptr;
  if (pl->path == WINO_PATH_SMALLC && !calib) {
    int rc = launch_smallc(pl->p, pl->std_mats, x, Uq, bias, y, pl->s_Y, st);
    pl->launches++;
    return rc == 0 && cudaGetLastError() == cudaSuccess ? WINO_OK : WINO_ERR_CUDA;
  }
  if (ws == nullptr) return WINO_ERR_WORKSPACE;
  if (!aligned16(ws)) return WINO_ERR_ALIGNMENT;
  int8_t* Vq = reinterpret_cast<int8_t*>(ws);
  void* mbuf = reinterpret_cast<uint8_t*>(ws) + round_up(vq_bytes(pl), 1024);
  // calibration on a small-channel plan uses the dp4a kernels for the middle stage
  wino_plan_t tmp_holder;
  const wino_plan_t* run = pl;
  if (pl->path == WINO_PATH_SMALLC) {
    tmp_holder = *pl;
    tmp_holder.path = WINO_PATH_STAGED_DP4A;
    run = &tmp_holder;
  }
  const bool ev = pl->stage_ev_on;
  if (ev) cudaEventRecord(pl->stage_ev[0], st);
  int rc = DISPATCH_M(pl, launch_input)(pl, x, Vq, calib ? absmax4 + 0 : nullptr, st);
  if (rc != WINO_OK) return rc;
  if (ev) cudaEventRecord(pl->stage_ev[1], st);
  rc = launch_gemm(run, Vq, Uq, mbuf, pl->p.qM_enabled ? kOutMq : kOutI32,
                   calib ? absmax4 + 1 : nullptr, st);
  if (run != pl) pl->launches++;
  if (rc != WINO_OK) return rc;
  if (ev) cudaEventRecord(pl->stage_ev[2], st);
  rc = DISPATCH_M(pl, launch_output)(pl, mbuf, bias, y, calib ? absmax4 + 2 : nullptr, st);
  if (rc != WINO_OK) return rc;
  if (ev) cudaEventRecord(pl->stage_ev[3], st);
  pl->last_uq = Uq;
  pl->last_ws = ws;
  pl->last_stream = st;
  return WINO_OK;
}

}  // namespace

extern "C" {

int wino_plan(const wino_desc_t* desc, wino_plan_t** out) {
  if (desc == nullptr || out == nullptr) return WINO_ERR_INVALID;
  *out = nullptr;
  const wino_desc_t& d = *desc;
  if (d.BT == nullptr || d.G == nullptr || d.AT == nullptr) return WINO_ERR_INVALID;
  if (d.N < 1 || d.C < 1 || d.H < 1 || d.W < 1 || d.K < 1) return WINO_ERR_INVALID;
  if (d.out_dtype != 0 && d.out_dtype != 1) return WINO_ERR_INVALID;
  if (!quant_ok(d.q_x) || !quant_ok(d.q_w) || !quant_ok(d.q_V) || !quant_ok(d.q_U) ||
      !quant_ok(d.q_Y))
    return WINO_ERR_INVALID;
  if (d.q_M.enabled && !quant_ok(d.q_M)) return WINO_ERR_INVALID;
  if (d.m != 2 && d.m != 4 && d.m != 6) return WINO_ERR_UNSUPPORTED;
  if (d.q_V.zero_point != 0 || d.q_U.zero_point != 0 || (d.q_M.enabled && d.q_M.zero_point != 0))
    return WINO_ERR_UNSUPPORTED;
  if (d.q_x.zero_point < -128 || d.q_x.zero_point > 127 || d.q_w.zero_point < -128 ||
      d.q_w.zero_point > 127 || d.q_Y.zero_point < -128 || d.q_Y.zero_point > 127)
    return WINO_ERR_INVALID;
  if (d.C > 1040) return WINO_ERR_UNSUPPORTED;
  const int t = d.m + 2;
  const long TH = (d.H + d.m - 1) / d.m, TW = (d.W + d.m - 1) / d.m;
  const long T = (long)d.N * TH * TW;
  if (T > (1l << 30) || (long)d.N * d.H * d.W * (long)(d.C > d.K ? d.C : d.K) > (1l << 40))
    return WINO_ERR_INVALID;
  for (int i = 0; i < t * t; ++i) if (!std::isfinite(d.BT[i])) return WINO_ERR_INVALID;
  for (int i = 0; i < t * 3; ++i) if (!std::isfinite(d.G[i])) return WINO_ERR_INVALID;
  for (int i = 0; i < d.m * t; ++i) if (!std::isfinite(d.AT[i])) return WINO_ERR_INVALID;

  wino_plan_t* pl = new (std::nothrow) wino_plan_t();
  if (pl == nullptr) return WINO_ERR_INVALID;
  std::memset(pl, 0, sizeof(*pl));
  pl->d = d;
  Params& p = pl->p;
  p.N = d.N; p.C = d.C; p.H = d.H; p.W = d.W; p.K = d.K; p.m = d.m; p.t = t;
  p.TH = (int)TH; p.TW = (int)TW; p.T = (int)T;
  std::memcpy(p.BT, d.BT, sizeof(float) * t * t);
  std::memcpy(p.G, d.G, sizeof(float) * t * 3);
  std::memcpy(p.AT, d.AT, sizeof(float) * d.m * t);
  pl->d.BT = p.BT; pl->d.G = p.G; pl->d.AT = p.AT;
  const double sUV = (double)d.q_U.scale * (double)d.q_V.scale;
  const double s_acc = d.q_M.enabled ? (double)d.q_M.scale : sUV;
  p.mult_V = (float)((double)d.q_x.scale / (double)d.q_V.scale);
  p.mult_U = (float)((double)d.q_w.scale / (double)d.q_U.scale);
  p.mult_M = d.q_M.enabled ? (float)(sUV / (double)d.q_M.scale) : 1.0f;
  p.mult_Y = (float)(s_acc / (double)d.q_Y.scale);
  p.s_acc = (float)s_acc;
  pl->s_Y = d.q_Y.scale;
  p.lo_V = (float)d.q_V.qmin; p.hi_V = (float)d.q_V.qmax;
  p.lo_U = (float)d.q_U.qmin; p.hi_U = (float)d.q_U.qmax;
  p.lo_M = (float)d.q_M.qmin; p.hi_M = (float)d.q_M.qmax;
  p.lo_Y = (float)(d.q_Y.qmin - d.q_Y.zero_point);
  p.hi_Y = (float)(d.q_Y.qmax - d.q_Y.zero_point);
  p.z_x = d.q_x.zero_point; p.z_w = d.q_w.zero_point; p.z_Y = d.q_Y.zero_point;
  p.qM_enabled = d.q_M.enabled ? 1 : 0;
  p.out_dtype = d.out_dtype;
  pl->std_mats = d.m == 2 ? is_std<2>(p.BT, p.AT) : d.m == 4 ? is_std<4>(p.BT, p.AT)
                                                               : is_std<6>(p.BT, p.AT);
  if (path_supported(pl, WINO_PATH_SMALLC)) pl->path = WINO_PATH_SMALLC;
  else if (path_supported(pl, WINO_PATH_STAGED_TC)) pl->path = WINO_PATH_STAGED_TC;
  else if (path_supported(pl, WINO_PATH_STAGED_DP4A)) pl->path = WINO_PATH_STAGED_DP4A;
  else { delete pl; return WINO_ERR_UNSUPPORTED; }
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) == cudaSuccess && ndev > 0) {
    if (cudaMalloc(&pl->status_dev, 256) == cudaSuccess) {
      cudaMemset(pl->status_dev, 0, 256);
    } else {
      pl->status_dev = nullptr;
    }
  }
  cudaGetLastError();
  *out = pl;
  return WINO_OK;
}

size_t wino_weight_bytes(const wino_plan_t* pl) {
  return pl ? (size_t)pl->p.t * pl->p.t * pl->p.K * pl->p.C : 0;
}

size_t wino_workspace_bytes(const wino_plan_t* pl) {
  if (pl == nullptr) return 0;
  // the fused small-channel path needs none; calibration on such a plan still does
  return round_up(vq_bytes(pl), 1024) + round_up(mbuf_bytes(pl), 1024);
}

int wino_plan_path(const wino_plan_t* pl) { return pl ? pl->path : WINO_ERR_INVALID; }

int wino_plan_force_path(wino_plan_t* pl, int path) {
  if (pl == nullptr) return WINO_ERR_INVALID;
  if (path < WINO_PATH_STAGED_TC || path > WINO_PATH_SMALLC) return WINO_ERR_INVALID;
  if (!path_supported(pl, path)) return WINO_ERR_UNSUPPORTED;
  pl->path = path;
  return WINO_OK;
}

int wino_plan_multipliers(const wino_plan_t* pl, float out[5]) {
  if (pl == nullptr || out == nullptr) return WINO_ERR_INVALID;
  out[0] = pl->p.mult_V; out[1] = pl->p.mult_U;
  out[2] = (float)((double)pl->d.q_U.scale * (double)pl->d.q_V.scale / (double)pl->d.q_M.scale);
  out[3] = pl->p.mult_Y; out[4] = pl->p.s_acc;
  return WINO_OK;
}

int wino_transform_weights(const wino_plan_t* pl, const int8_t* w, int8_t* Uq, uint32_t* absmax,
                           void* stream) {
  if (pl == nullptr || w == nullptr || Uq == nullptr) return WINO_ERR_INVALID;
  if (!aligned16(w) || !aligned16(Uq)) return WINO_ERR_ALIGNMENT;
  if (pl->status_dev == nullptr) return WINO_ERR_CUDA;
  return DISPATCH_M(pl, launch_weight)(pl, w, Uq, absmax, (cudaStream_t)stream);
}

int wino_conv_forward(const wino_plan_t* pl, const int8_t* x, const int8_t* Uq, const float* bias,
                      void* y, void* ws, void* stream) {
  if (pl == nullptr || x == nullptr || Uq == nullptr || y == nullptr) return WINO_ERR_INVALID;
  if (!aligned16(x) || !aligned16(Uq) || !aligned16(y) || (bias && !aligned16(bias)))
    return WINO_ERR_ALIGNMENT;
  return forward_impl(pl, x, Uq, bias, y, ws, nullptr, (cudaStream_t)stream);
}

int wino_calibrate_forward(const wino_plan_t* pl, const int8_t* x, const int8_t* Uq,
                           const float* bias, void* y, void* ws, uint32_t* absmax4, void* stream) {
  if (pl == nullptr || x == nullptr || Uq == nullptr || absmax4 == nullptr) return WINO_ERR_INVALID;
  if (!aligned16(x) || !aligned16(Uq) || (y && !aligned16(y)) || (bias && !aligned16(bias)))
    return WINO_ERR_ALIGNMENT;
  return forward_impl(pl, x, Uq, bias, y, ws, absmax4, (cudaStream_t)stream);
}

int wino_last_status(const wino_plan_t* pl, void* stream) {
  if (pl == nullptr) return WINO_ERR_INVALID;
  if (pl->status_dev == nullptr) return WINO_ERR_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return WINO_ERR_CUDA;
  int v = 0;
  if (cudaMemcpy(&v, pl->status_dev, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
    return WINO_ERR_CUDA;
  return v;
}

int wino_debug_dump_stage(const wino_plan_t* pl, int stage, void* dst, size_t bytes) {
  if (pl == nullptr || dst == nullptr) return WINO_ERR_INVALID;
  if (pl->last_ws == nullptr) return WINO_ERR_UNSUPPORTED;
  if (!aligned16(dst)) return WINO_ERR_ALIGNMENT;
  const uint8_t* ws = reinterpret_cast<const uint8_t*>(pl->last_ws);
  cudaStream_t st = pl->last_stream;
  if (stage == WINO_STAGE_VQ) {
    if (bytes != vq_bytes(pl)) return WINO_ERR_INVALID;
    return cudaMemcpyAsync(dst, ws, bytes, cudaMemcpyDeviceToDevice, st) == cudaSuccess ? WINO_OK
                                                                                        : WINO_ERR_CUDA;
  }
  if (stage == WINO_STAGE_MQ) {
    if (!pl->p.qM_enabled) return WINO_ERR_UNSUPPORTED;
    if (bytes != m_elems(pl)) return WINO_ERR_INVALID;
    return cudaMemcpyAsync(dst, ws + round_up(vq_bytes(pl), 1024), bytes, cudaMemcpyDeviceToDevice,
                           st) == cudaSuccess ? WINO_OK : WINO_ERR_CUDA;
  }
  if (stage == WINO_STAGE_M_I32) {
    if (bytes != m_elems(pl) * 4) return WINO_ERR_INVALID;
    wino_plan_t tmp = *pl;
    if (tmp.path == WINO_PATH_SMALLC) tmp.path = WINO_PATH_STAGED_DP4A;
    int rc = launch_gemm(&tmp, reinterpret_cast<const int8_t*>(ws), pl->last_uq, dst, kOutI32,
                         nullptr, st);
    pl->launches++;
    pl->map_vq_ptr = tmp.map_vq_ptr; pl->map_uq_ptr = tmp.map_uq_ptr;
    pl->mapV = tmp.mapV; pl->mapU = tmp.mapU;
    const_cast<wino_plan_t*>(pl)->tc_attr_set = tmp.tc_attr_set;
    return rc;
  }
  return WINO_ERR_INVALID;
}

long wino_launch_count(const wino_plan_t* pl) { return pl ? pl->launches : 0; }

int wino_plan_set_stage_events(wino_plan_t* pl, void* const events[4]) {
  if (pl == nullptr) return WINO_ERR_INVALID;
  if (events == nullptr) { pl->stage_ev_on = false; return WINO_OK; }
  for (int i = 0; i < 4; ++i) {
    if (events[i] == nullptr) return WINO_ERR_INVALID;
    pl->stage_ev[i] = (cudaEvent_t)events[i];
  }
  pl->stage_ev_on = true;
  return WINO_OK;
}

void wino_destroy(wino_plan_t* pl) {
  if (pl == nullptr) return;
  if (pl->status_dev) cudaFree(pl->status_dev);
  delete pl;
}

const char* wino_strerror(int code) {
  switch (code) {
    case WINO_OK: return "ok";
    case WINO_ERR_INVALID: return "invalid argument";
    case WINO_ERR_UNSUPPORTED: return "unsupported configuration";
    case WINO_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
    case WINO_ERR_WORKSPACE: return "workspace missing";
    case WINO_ERR_CUDA: return "CUDA call failed";
    case WINO_ERR_TIMEOUT: return "bounded device wait expired";
    default: return "unknown error";
  }
}

}  // extern "C"
