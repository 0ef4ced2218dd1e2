// Host side of the C ABI declared in include/wino.h: plan construction,
// argument checks, path choice, TMA descriptor encoding and kernel launches.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include <cuda.h>
#include <cuda_runtime.h>

#include "wino.h"
#include "wino_launch.h"

using namespace wino;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Small round-robin memo of encoded tensor maps keyed by the buffer address.
struct MapCache {
  static constexpr int kN = 32;
  const void* key[kN];
  CUtensorMap map[kN];
  int next;
  const CUtensorMap* find(const void* k) const {
    for (int i = 0; i < kN; ++i)
      if (key[i] == k) return &map[i];
    return nullptr;
  }
  CUtensorMap* slot(const void* k) {
    const int i = next;
    next = (next + 1) % kN;
    key[i] = k;
    return &map[i];
  }
};

struct wino_plan {
  wino_desc_t d;
  Params p;
  float s_Y;
  bool std_mats;        // BT and AT equal the built-in Cook-Toom matrices bit for bit
  int path;
  int* status_dev;      // device status word (may be null when no GPU is present)
  float* chan_dev;      // per-output-channel multipliers [5][K] (null: per-layer scales)
  void* kron_dev;       // Kronecker tables of the tensor-core transforms (same allocation)
  unsigned* counters_dev;  // progress counters of the single-launch layer kernel (same allocation)
  CUtensorMap fmapV, fmapU;   // GEMM operand maps of the single-launch kernel
  const void* fmap_vq_ptr;
  const void* fmap_uq_ptr;
  int num_sms;
  int device;           // the device that was current when the plan was made
  bool pdl;             // programmatic dependent launch between the stages
  // memo of the last encoded tensor maps
  const void* map_vq_ptr;
  const void* map_uq_ptr;
  CUtensorMap mapV, mapU;
  // maps of the TMA-staged transform kernels, keyed by buffer address
  MapCache cache_x, cache_vst, cache_mld, cache_y, cache_uf, cache_x_sw, cache_m_sw;
  // last forward call, for wino_debug_dump_stage
  const int8_t* last_uq;
  void* last_ws;
  cudaStream_t last_stream;
  long launches;
};

// Scratch of wino_conv_forward_static: V_q and m_q of one layer call.  A plain
// file-scope device array, so every GPU that loads this library holds these
// bytes from module load until the process exits.  In host code the name below
// is only a handle; the device address is looked up once per device with
// cudaGetSymbolAddress and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[WINO_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_static_scratch_mutex;

// Device address of the static scratch on the current device (looked up on the
// first call for that device, with that device current).
int static_scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return WINO_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (g_static_scratch_addr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
      cudaGetLastError();
      return WINO_ERR_CUDA;
    }
    g_static_scratch_addr[dev] = ptr;
  }
  *out = g_static_scratch_addr[dev];
  return WINO_OK;
}

EncodeTiledFn lookup_encode_fn() {
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) ==
          cudaSuccess &&
      q == cudaDriverEntryPointSuccess)
    return reinterpret_cast<EncodeTiledFn>(ptr);
  cudaGetLastError();
  return nullptr;
}
EncodeTiledFn get_encode_fn() {
  static const EncodeTiledFn fn = lookup_encode_fn();   // initialised once, thread-safe
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
  // per-output-channel scales are built into the staged kernels only
  if (pl->chan_dev != nullptr && path != WINO_PATH_STAGED_TC && path != WINO_PATH_STAGED_TC_PTR &&
      path != WINO_PATH_STAGED_DP4A)
    return false;
  switch (path) {
    case WINO_PATH_STAGED_TC:
    case WINO_PATH_STAGED_TC_MMA:
    case WINO_PATH_STAGED_TC_PTR: return C % 16 == 0 && K % 16 == 0;
    case WINO_PATH_STAGED_DP4A: return C % 4 == 0 && K % 4 == 0;
    case WINO_PATH_SMALLC: return C % 4 == 0 && K % 4 == 0 && C <= 32 && K <= 32;
    case WINO_PATH_FUSED_F2: return fused_f2_supported(pl->p, pl->std_mats);
    case WINO_PATH_FUSED_LAYER:
      return layer_fused_supported(pl->p, pl->std_mats) &&
             layer_fused_geometry(pl->p, pl->num_sms).stages >= 2;
    default: return false;
  }
}

size_t vq_bytes(const wino_plan_t* pl) { return (size_t)pl->p.t * pl->p.t * pl->p.T * pl->p.C; }
size_t m_elems(const wino_plan_t* pl) { return (size_t)pl->p.t * pl->p.t * pl->p.T * pl->p.K; }
size_t mbuf_bytes(const wino_plan_t* pl) { return m_elems(pl) * (pl->p.qM_enabled ? 1 : 4); }

LaunchOpt opt_of(const wino_plan_t* pl, bool pdl) {
  LaunchOpt o;
  o.std_mats = pl->std_mats;
  o.pdl = pdl;
  o.device = pl->device;
  o.num_sms = pl->num_sms;
  o.chan = pl->chan_dev;
  return o;
}

int encode_tiled(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                 const uint32_t* box, CUtensorMapSwizzle swz) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return WINO_ERR_CUDA;
  cuuint64_t d[5], strides[4];
  cuuint32_t b[5], estr[5] = {1, 1, 1, 1, 1};
  uint64_t stride = 1;
  for (int i = 0; i < rank; ++i) {
    d[i] = dims[i];
    b[i] = box[i];
    stride *= dims[i];
    if (i < rank - 1) strides[i] = stride;  // bytes: int8 elements
  }
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)rank, const_cast<void*>(base), d,
                  strides, b, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? WINO_OK : WINO_ERR_CUDA;
}

int encode_map(CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows, uint64_t mats,
               uint32_t box_rows) {
  const uint64_t dims[3] = {inner, rows, mats};
  const uint32_t box[3] = {(uint32_t)kStageK, box_rows, 1};
  return encode_tiled(map, base, 3, dims, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

// Tensor maps of the TMA-staged transform kernels (no swizzle).
const CUtensorMap* map_x(wino_plan_t* pl, const void* x) {
  if (const CUtensorMap* m = pl->cache_x.find(x)) return m;
  const Params& p = pl->p;
  const uint64_t dims[4] = {(uint64_t)p.C, (uint64_t)p.W, (uint64_t)p.H, (uint64_t)p.N};
  const uint32_t box[4] = {(uint32_t)tma_chunk(p.C), (uint32_t)p.t, (uint32_t)p.t, 1};
  CUtensorMap* m = pl->cache_x.slot(x);
  if (encode_tiled(m, x, 4, dims, box, CU_TENSOR_MAP_SWIZZLE_NONE) != WINO_OK) {
    pl->cache_x.key[(pl->cache_x.next + MapCache::kN - 1) % MapCache::kN] = nullptr;
    return nullptr;
  }
  return m;
}
const CUtensorMap* map_y(wino_plan_t* pl, const void* y) {
  if (const CUtensorMap* m = pl->cache_y.find(y)) return m;
  const Params& p = pl->p;
  const uint64_t dims[4] = {(uint64_t)p.K, (uint64_t)p.W, (uint64_t)p.H, (uint64_t)p.N};
  const uint32_t box[4] = {(uint32_t)tma_chunk(p.K), (uint32_t)p.m, (uint32_t)p.m, 1};
  CUtensorMap* m = pl->cache_y.slot(y);
  if (encode_tiled(m, y, 4, dims, box, CU_TENSOR_MAP_SWIZZLE_NONE) != WINO_OK) {
    pl->cache_y.key[(pl->cache_y.next + MapCache::kN - 1) % MapCache::kN] = nullptr;
    return nullptr;
  }
  return m;
}
// V_q (store side) and m_q (load side): [t*t][T][channels], box {chunk, G, t*t}
const CUtensorMap* map_stage(wino_plan_t* pl, MapCache& cache, const void* buf, int channels) {
  if (const CUtensorMap* m = cache.find(buf)) return m;
  const Params& p = pl->p;
  const int chunk = tma_chunk(channels);
  const uint64_t dims[3] = {(uint64_t)channels, (uint64_t)p.T, (uint64_t)(p.t * p.t)};
  const uint32_t box[3] = {(uint32_t)chunk, (uint32_t)tma_group(chunk), (uint32_t)(p.t * p.t)};
  CUtensorMap* m = cache.slot(buf);
  if (encode_tiled(m, buf, 3, dims, box, CU_TENSOR_MAP_SWIZZLE_NONE) != WINO_OK) {
    cache.key[(cache.next + MapCache::kN - 1) % MapCache::kN] = nullptr;
    return nullptr;
  }
  return m;
}

// Swizzled maps of the tensor-core transform kernels: x as [N][H][W][C] with box
// {128, t, t, 1}; m_q as [t*t][T][K] with box {128, 1, t*t}.
const CUtensorMap* map_x_sw(wino_plan_t* pl, const void* x) {
  if (const CUtensorMap* m = pl->cache_x_sw.find(x)) return m;
  const Params& p = pl->p;
  const uint64_t dims[4] = {(uint64_t)p.C, (uint64_t)p.W, (uint64_t)p.H, (uint64_t)p.N};
  const uint32_t box[4] = {128, (uint32_t)p.t, (uint32_t)p.t, 1};
  CUtensorMap* m = pl->cache_x_sw.slot(x);
  if (encode_tiled(m, x, 4, dims, box, CU_TENSOR_MAP_SWIZZLE_128B) != WINO_OK) {
    pl->cache_x_sw.key[(pl->cache_x_sw.next + MapCache::kN - 1) % MapCache::kN] = nullptr;
    return nullptr;
  }
  return m;
}
const CUtensorMap* map_m_sw(wino_plan_t* pl, const void* mbuf) {
  if (const CUtensorMap* m = pl->cache_m_sw.find(mbuf)) return m;
  const Params& p = pl->p;
  const uint64_t dims[3] = {(uint64_t)p.K, (uint64_t)p.T, (uint64_t)(p.t * p.t)};
  const uint32_t box[3] = {128, 1, (uint32_t)(p.t * p.t)};
  CUtensorMap* m = pl->cache_m_sw.slot(mbuf);
  if (encode_tiled(m, mbuf, 3, dims, box, CU_TENSOR_MAP_SWIZZLE_128B) != WINO_OK) {
    pl->cache_m_sw.key[(pl->cache_m_sw.next + MapCache::kN - 1) % MapCache::kN] = nullptr;
    return nullptr;
  }
  return m;
}

// U_q for the fused F2 kernel: [16][K][C], box {64, 64, 1}, 64-byte swizzle
const CUtensorMap* map_u_fused(wino_plan_t* pl, const void* Uq) {
  if (const CUtensorMap* m = pl->cache_uf.find(Uq)) return m;
  const Params& p = pl->p;
  const uint64_t dims[3] = {(uint64_t)p.C, (uint64_t)p.K, 16};
  const uint32_t box[3] = {64, 64, 1};
  CUtensorMap* m = pl->cache_uf.slot(Uq);
  if (encode_tiled(m, Uq, 3, dims, box, CU_TENSOR_MAP_SWIZZLE_64B) != WINO_OK) {
    pl->cache_uf.key[(pl->cache_uf.next + MapCache::kN - 1) % MapCache::kN] = nullptr;
    return nullptr;
  }
  return m;
}

int launch_gemm(wino_plan_t* pl, const int8_t* Vq, const int8_t* Uq, void* out, int out_mode,
                unsigned* absmaxM, bool pdl, cudaStream_t st) {
  const Params& p = pl->p;
  const int t2 = p.t * p.t;
  pl->launches++;
  if (pl->path == WINO_PATH_STAGED_DP4A)
    return launch_gemm_dp4a(p, opt_of(pl, pdl), Vq, Uq, out, out_mode, absmaxM, st);
  const TcGeom g = tc_geometry(p, pl->num_sms);
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
  return launch_gemm_tc(p, opt_of(pl, pdl), g, pl->mapV, pl->mapU, out, out_mode, absmaxM,
                        pl->status_dev, st);
}

// stage_mask: bit 0 input transform, bit 1 Hadamard GEMMs, bit 2 output transform.
// dbgM (single-kernel paths only): receives the int32 Hadamard sums M[xi][tau][k].
int forward_impl(wino_plan_t* pl, const int8_t* x, const int8_t* Uq, const float* bias, void* y,
                 void* ws, unsigned* absmax4, cudaStream_t st, int stage_mask = 7,
                 int* dbgM = nullptr) {
  if (pl->status_dev == nullptr) return WINO_ERR_CUDA;
  const bool calib = absmax4 != nullptr;
  const bool pdl = pl->pdl && !calib;
  if (pl->path == WINO_PATH_SMALLC && !calib) {
    pl->launches++;
    return launch_smallc(pl->p, opt_of(pl, pdl), x, Uq, bias, y, pl->s_Y, dbgM, st);
  }
  if (pl->path == WINO_PATH_FUSED_F2 && !calib && stage_mask == 7) {
    const CUtensorMap* mu = map_u_fused(pl, Uq);
    if (mu == nullptr) return WINO_ERR_CUDA;
    pl->launches++;
    return launch_fused_f2(pl->p, opt_of(pl, pdl), *mu, x, bias, y, pl->s_Y, pl->num_sms,
                           pl->status_dev, dbgM, st);
  }
  if (ws == nullptr) return WINO_ERR_WORKSPACE;
  if (!aligned16(ws)) return WINO_ERR_ALIGNMENT;
  int8_t* Vq = reinterpret_cast<int8_t*>(ws);
  void* mbuf = reinterpret_cast<uint8_t*>(ws) + round_up(vq_bytes(pl), 1024);
  if (pl->path == WINO_PATH_FUSED_LAYER && !calib && stage_mask == 7) {
    const Params& p = pl->p;
    const FusedGeom g = layer_fused_geometry(p, pl->num_sms);
    const int t2 = p.t * p.t;
    if (pl->fmap_vq_ptr != Vq) {
      int rc = encode_map(&pl->fmapV, Vq, (uint64_t)p.C, (uint64_t)p.T, (uint64_t)t2, kBM);
      if (rc != WINO_OK) return rc;
      pl->fmap_vq_ptr = Vq;
    }
    if (pl->fmap_uq_ptr != Uq) {
      int rc = encode_map(&pl->fmapU, Uq, (uint64_t)p.C, (uint64_t)p.K, (uint64_t)t2, (uint32_t)g.BN);
      if (rc != WINO_OK) return rc;
      pl->fmap_uq_ptr = Uq;
    }
    FusedMaps m;
    m.x = map_x_sw(pl, x);
    m.v_store = map_stage(pl, pl->cache_vst, Vq, p.C);
    m.v_load = &pl->fmapV;
    m.u = &pl->fmapU;
    m.m_load = map_m_sw(pl, mbuf);
    m.y = map_y(pl, y);
    if (m.x == nullptr || m.v_store == nullptr || m.m_load == nullptr || m.y == nullptr)
      return WINO_ERR_CUDA;
    pl->launches++;
    const int rc = launch_layer_fused(p, opt_of(pl, pdl), g, m, pl->kron_dev, pl->counters_dev,
                                      reinterpret_cast<int8_t*>(mbuf), bias, pl->s_Y,
                                      pl->status_dev, st);
    if (rc != WINO_OK) return rc;
    pl->last_uq = Uq;
    pl->last_ws = ws;
    pl->last_stream = st;
    return WINO_OK;
  }
  // calibration on a single-kernel plan runs the staged kernels (dp4a or tcgen05 middle stage)
  const int saved_path = pl->path;
  int gemm_path = pl->path;
  if (pl->path == WINO_PATH_SMALLC) gemm_path = WINO_PATH_STAGED_DP4A;
  if (pl->path == WINO_PATH_FUSED_F2) gemm_path = WINO_PATH_STAGED_TC_PTR;
  if (pl->path == WINO_PATH_FUSED_LAYER) gemm_path = WINO_PATH_STAGED_TC;
  const bool tma_ok = (pl->path == WINO_PATH_STAGED_TC || pl->path == WINO_PATH_STAGED_TC_MMA) && !calib;
  const bool mma_ok = pl->path == WINO_PATH_STAGED_TC_MMA && !calib;
  int rc = WINO_OK;
  if (!(stage_mask & 1)) {
  } else if (pl->launches++, mma_ok && pl->p.z_x == 0 &&
             transform_mma_supported(pl->p, pl->std_mats, pl->p.C)) {
    const CUtensorMap* mx = map_x_sw(pl, x);
    const CUtensorMap* mv = map_stage(pl, pl->cache_vst, Vq, pl->p.C);
    if (mx == nullptr || mv == nullptr) return WINO_ERR_CUDA;
    rc = launch_input_transform_mma(pl->p, opt_of(pl, pdl), *mx, *mv, pl->kron_dev, pl->num_sms,
                                    pl->status_dev, st);
  } else if (tma_ok && pl->p.z_x == 0 && tma_chunk(pl->p.C) != 0) {
    const CUtensorMap* mx = map_x(pl, x);
    const CUtensorMap* mv = map_stage(pl, pl->cache_vst, Vq, pl->p.C);
    if (mx == nullptr || mv == nullptr) return WINO_ERR_CUDA;
    LaunchOpt o = opt_of(pl, pdl);
    if ((stage_mask & 2) && !calib) {   // the GEMMs that follow read U_q, which no kernel of this call writes
      o.l2_hint = Uq;
      o.l2_hint_bytes = (size_t)pl->p.t * pl->p.t * pl->p.K * pl->p.C;
    }
    rc = launch_input_transform_tma(pl->p, o, *mx, *mv, pl->status_dev, st);
  } else {
    rc = launch_input_transform(pl->p, opt_of(pl, pdl), x, Vq, calib ? absmax4 + 0 : nullptr, st);
  }
  if (rc != WINO_OK) return rc;
  if (stage_mask & 2) {
    pl->path = gemm_path;
    rc = launch_gemm(pl, Vq, Uq, mbuf, pl->p.qM_enabled ? kOutMq : kOutI32,
                     calib ? absmax4 + 1 : nullptr, pdl, st);
    pl->path = saved_path;
  }
  if (rc != WINO_OK) return rc;
  if (!(stage_mask & 4)) {
  } else if (pl->launches++, mma_ok && pl->p.qM_enabled && pl->p.out_dtype == 0 &&
             transform_mma_supported(pl->p, pl->std_mats, pl->p.K)) {
    const CUtensorMap* mm = map_m_sw(pl, mbuf);
    const CUtensorMap* my = map_y(pl, y);
    if (mm == nullptr || my == nullptr) return WINO_ERR_CUDA;
    rc = launch_output_transform_mma(pl->p, opt_of(pl, pdl), *mm, *my, pl->kron_dev, bias, pl->s_Y,
                                     pl->num_sms, pl->status_dev, st);
  } else if (tma_ok && pl->p.qM_enabled && pl->p.out_dtype == 0 && tma_chunk(pl->p.K) != 0) {
    const CUtensorMap* mm = map_stage(pl, pl->cache_mld, mbuf, pl->p.K);
    const CUtensorMap* my = map_y(pl, y);
    if (mm == nullptr || my == nullptr) return WINO_ERR_CUDA;
    rc = launch_output_transform_tma(pl->p, opt_of(pl, pdl), *mm, *my, bias, pl->s_Y,
                                     pl->status_dev, st);
  } else {
    rc = launch_output_transform(pl->p, opt_of(pl, pdl), pl->s_Y, mbuf, bias, y,
                                 calib ? absmax4 + 2 : nullptr, st);
  }
  if (rc != WINO_OK) return rc;
  pl->last_uq = Uq;
  pl->last_ws = ws;
  pl->last_stream = st;
  return WINO_OK;
}

bool path_uses_scratch(const wino_plan_t* pl) {
  return pl->path != WINO_PATH_SMALLC && pl->path != WINO_PATH_FUSED_F2;
}

DeviceOnce g_once_selftest;

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
  // Automatic choice, by measurement on B200: the fused F2 kernel where it applies; for
  // layers of at most 16 channels in and out the staged path with integer dot products on the
  // ALUs (a 16-wide GEMM leaves the tensor-core pipeline mostly empty: 54 against 73 us at
  // 16 channels, 32x32, batch 256, F2); else the staged tcgen05 path, else the staged dp4a
  // path.  The warp-shuffle small-channel kernel stays selectable (wino_plan_force_path) but
  // a staged path was faster on every layer size tried, tiny batches included.
  if (path_supported(pl, WINO_PATH_FUSED_F2)) pl->path = WINO_PATH_FUSED_F2;
  else if (d.C <= 16 && d.K <= 16 && path_supported(pl, WINO_PATH_STAGED_DP4A))
    pl->path = WINO_PATH_STAGED_DP4A;
  else if (path_supported(pl, WINO_PATH_STAGED_TC)) pl->path = WINO_PATH_STAGED_TC;
  else if (path_supported(pl, WINO_PATH_STAGED_DP4A)) pl->path = WINO_PATH_STAGED_DP4A;
  else { delete pl; return WINO_ERR_UNSUPPORTED; }
  pl->num_sms = 148;
  pl->pdl = true;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) == cudaSuccess && ndev > 0) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) pl->device = dev;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, pl->device) == cudaSuccess &&
        sms > 0)
      pl->num_sms = sms;
    // one small allocation: the status word, then (256 bytes in) the Kronecker tables
    const size_t dev_bytes = 256 + kKronBytes + sizeof(unsigned) * kFusedCounterWords;
    if (cudaMalloc(&pl->status_dev, dev_bytes) == cudaSuccess) {
      cudaMemset(pl->status_dev, 0, dev_bytes);
      pl->kron_dev = reinterpret_cast<uint8_t*>(pl->status_dev) + 256;
      pl->counters_dev = reinterpret_cast<unsigned*>(reinterpret_cast<uint8_t*>(pl->kron_dev) + kKronBytes);
      if (pl->std_mats && (d.m == 2 || d.m == 4)) {
        int8_t tables[kKronBytes];
        fill_kronecker_tables(d.m, tables);
        if (cudaMemcpy(pl->kron_dev, tables, kKronBytes, cudaMemcpyHostToDevice) != cudaSuccess) {
          cudaFree(pl->status_dev);
          pl->status_dev = nullptr;
        }
      }
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
  if (path < WINO_PATH_STAGED_TC || path > WINO_PATH_FUSED_LAYER) return WINO_ERR_INVALID;
  if (!path_supported(pl, path)) return WINO_ERR_UNSUPPORTED;
  pl->path = path;
  return WINO_OK;
}

int wino_plan_set_channel_scales(wino_plan_t* pl, const float* s_w_K, const float* s_U_K,
                                 const float* s_M_K, const float* s_Y_K) {
  if (pl == nullptr) return WINO_ERR_INVALID;
  const int K = pl->d.K;
  if (s_w_K == nullptr && s_U_K == nullptr && s_M_K == nullptr && s_Y_K == nullptr) {   // per-layer scales again
    if (pl->chan_dev) cudaFree(pl->chan_dev);
    pl->chan_dev = nullptr;
    return WINO_OK;
  }
  for (const float* a : {s_w_K, s_U_K, s_M_K, s_Y_K})
    if (a != nullptr)
      for (int k = 0; k < K; ++k)
        if (!std::isfinite(a[k]) || !(a[k] > 0.0f)) return WINO_ERR_INVALID;
  if (pl->status_dev == nullptr) return WINO_ERR_CUDA;
  std::vector<float> tab((size_t)5 * K);
  const wino_desc_t& d = pl->d;
  for (int k = 0; k < K; ++k) {
    const double s_w = s_w_K ? (double)s_w_K[k] : (double)d.q_w.scale;
    const double s_U = s_U_K ? (double)s_U_K[k] : (double)d.q_U.scale;
    const double s_Y = s_Y_K ? (double)s_Y_K[k] : (double)d.q_Y.scale;
    const double s_M = s_M_K ? (double)s_M_K[k] : (double)d.q_M.scale;
    const double sUV = s_U * (double)d.q_V.scale;
    const double s_acc = d.q_M.enabled ? s_M : sUV;
    tab[(size_t)kChMultU * K + k] = (float)(s_w / s_U);
    tab[(size_t)kChMultM * K + k] = d.q_M.enabled ? (float)(sUV / s_M) : 1.0f;
    tab[(size_t)kChMultY * K + k] = (float)(s_acc / s_Y);
    tab[(size_t)kChSAcc * K + k] = (float)s_acc;
    tab[(size_t)kChSY * K + k] = (float)s_Y;
  }
  float* fresh = pl->chan_dev;
  if (fresh == nullptr && cudaMalloc(&fresh, tab.size() * sizeof(float)) != cudaSuccess) {
    cudaGetLastError();
    return WINO_ERR_CUDA;
  }
  if (cudaMemcpy(fresh, tab.data(), tab.size() * sizeof(float), cudaMemcpyHostToDevice) !=
      cudaSuccess) {
    cudaGetLastError();
    if (pl->chan_dev == nullptr) cudaFree(fresh);
    return WINO_ERR_CUDA;
  }
  pl->chan_dev = fresh;
  if (!path_supported(pl, pl->path)) {   // every shape the library plans has a staged path
    if (path_supported(pl, WINO_PATH_STAGED_TC)) pl->path = WINO_PATH_STAGED_TC;
    else pl->path = WINO_PATH_STAGED_DP4A;
  }
  return WINO_OK;
}

int wino_plan_multipliers(const wino_plan_t* pl, float out[5]) {
  if (pl == nullptr || out == nullptr) return WINO_ERR_INVALID;
  out[0] = pl->p.mult_V; out[1] = pl->p.mult_U;
  out[2] = (float)((double)pl->d.q_U.scale * (double)pl->d.q_V.scale / (double)pl->d.q_M.scale);
  out[3] = pl->p.mult_Y; out[4] = pl->p.s_acc;
  return WINO_OK;
}

int wino_transform_weights(wino_plan_t* pl, const int8_t* w, int8_t* Uq, uint32_t* absmax,
                           void* stream) {
  if (pl == nullptr || w == nullptr || Uq == nullptr) return WINO_ERR_INVALID;
  if (!aligned16(w) || !aligned16(Uq)) return WINO_ERR_ALIGNMENT;
  if (pl->status_dev == nullptr) return WINO_ERR_CUDA;
  pl->launches++;
  return launch_weight_transform(pl->p, pl->chan_dev, w, Uq, absmax, nullptr, (cudaStream_t)stream);
}

int wino_transform_weights_channel_stats(wino_plan_t* pl, const int8_t* w, int8_t* Uq,
                                         uint32_t* absmax_K, void* stream) {
  if (pl == nullptr || w == nullptr || Uq == nullptr || absmax_K == nullptr) return WINO_ERR_INVALID;
  if (!aligned16(w) || !aligned16(Uq)) return WINO_ERR_ALIGNMENT;
  if (pl->status_dev == nullptr) return WINO_ERR_CUDA;
  pl->launches++;
  return launch_weight_transform(pl->p, pl->chan_dev, w, Uq, nullptr, absmax_K, (cudaStream_t)stream);
}

int wino_conv_forward(wino_plan_t* pl, const int8_t* x, const int8_t* Uq, const float* bias,
                      void* y, void* ws, void* stream) {
  if (pl == nullptr || x == nullptr || Uq == nullptr || y == nullptr) return WINO_ERR_INVALID;
  if (!aligned16(x) || !aligned16(Uq) || !aligned16(y) || (bias && !aligned16(bias)))
    return WINO_ERR_ALIGNMENT;
  return forward_impl(pl, x, Uq, bias, y, ws, nullptr, (cudaStream_t)stream);
}

int wino_conv_forward_static(wino_plan_t* pl, const int8_t* x, const int8_t* Uq,
                             const float* bias, void* y, void* stream) {
  if (pl == nullptr || x == nullptr || Uq == nullptr || y == nullptr) return WINO_ERR_INVALID;
  if (!aligned16(x) || !aligned16(Uq) || !aligned16(y) || (bias && !aligned16(bias)))
    return WINO_ERR_ALIGNMENT;
  void* scratch = nullptr;
  if (path_uses_scratch(pl)) {   // the single-kernel paths keep V_q and m_q on the SM
    if (wino_workspace_bytes(pl) > (size_t)WINO_STATIC_SCRATCH_BYTES) return WINO_ERR_WORKSPACE;
    const int rc = static_scratch_address(&scratch);
    if (rc != WINO_OK) return rc;
  }
  return forward_impl(pl, x, Uq, bias, y, scratch, nullptr, (cudaStream_t)stream);
}

int wino_calibrate_forward(wino_plan_t* pl, const int8_t* x, const int8_t* Uq,
                           const float* bias, void* y, void* ws, uint32_t* absmax4, void* stream) {
  if (pl == nullptr || x == nullptr || Uq == nullptr || absmax4 == nullptr) return WINO_ERR_INVALID;
  if (!aligned16(x) || !aligned16(Uq) || (y && !aligned16(y)) || (bias && !aligned16(bias)))
    return WINO_ERR_ALIGNMENT;
  return forward_impl(pl, x, Uq, bias, y, ws, absmax4, (cudaStream_t)stream);
}

int wino_debug_run_stages(wino_plan_t* pl, int stage_mask, const int8_t* x, const int8_t* Uq,
                          const float* bias, void* y, void* ws, void* stream) {
  if (pl == nullptr || x == nullptr || Uq == nullptr || y == nullptr) return WINO_ERR_INVALID;
  if (stage_mask < 1 || stage_mask > 7) return WINO_ERR_INVALID;
  if ((pl->path == WINO_PATH_SMALLC || pl->path == WINO_PATH_FUSED_F2) && stage_mask != 7)
    return WINO_ERR_UNSUPPORTED;   // the fused paths have no separate stages
  if (!aligned16(x) || !aligned16(Uq) || !aligned16(y) || (bias && !aligned16(bias)))
    return WINO_ERR_ALIGNMENT;
  return forward_impl(pl, x, Uq, bias, y, ws, nullptr, (cudaStream_t)stream, stage_mask);
}

int wino_direct_conv_forward(const wino_direct_desc_t* d, const int8_t* x, const int8_t* w,
                             const float* bias, void* y, void* stream) {
  if (d == nullptr || x == nullptr || w == nullptr || y == nullptr) return WINO_ERR_INVALID;
  if (d->N < 1 || d->C < 1 || d->H < 1 || d->W < 1 || d->K < 1) return WINO_ERR_INVALID;
  if (d->stride != 1 && d->stride != 2) return WINO_ERR_INVALID;
  if (d->out_dtype != 0 && d->out_dtype != 1) return WINO_ERR_INVALID;
  if (!quant_ok(d->q_x) || !quant_ok(d->q_w) || !quant_ok(d->q_Y)) return WINO_ERR_INVALID;
  if (!aligned16(x) || !aligned16(w) || !aligned16(y) || (bias && !aligned16(bias)))
    return WINO_ERR_ALIGNMENT;
  if ((reinterpret_cast<uintptr_t>(d->s_w_K_dev) & 3u) != 0 || (reinterpret_cast<uintptr_t>(d->s_Y_K_dev) & 3u) != 0)
    return WINO_ERR_ALIGNMENT;
  const double s_in = (double)d->q_x.scale * (double)d->q_w.scale;
  if (direct_tc_supported(d->C, d->K, d->H, d->W, d->stride, d->q_x.zero_point, d->q_w.zero_point) &&
      (reinterpret_cast<uintptr_t>(y) & 31u) == 0) {
    // implicit GEMM on the tensor cores: x as [N][H][W][C] boxes of one output tile, w as
    // [K][9][C] slices of one tap
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) return WINO_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
      sms = 148;
    DirectTcArgs a = direct_tc_geometry(d->N, d->C, d->H, d->W, d->K, d->stride, sms);
    a.mult = (float)(s_in / (double)d->q_Y.scale);
    a.s_in = (float)s_in;
    a.s_Y = d->q_Y.scale;
    a.s_w_K = d->s_w_K_dev; a.s_Y_K = d->s_Y_K_dev;
    a.s_x = d->q_x.scale; a.s_w = d->q_w.scale;
    a.lo_Y = (float)(d->q_Y.qmin - d->q_Y.zero_point);
    a.hi_Y = (float)(d->q_Y.qmax - d->q_Y.zero_point);
    a.z_Y = d->q_Y.zero_point;
    a.out_dtype = d->out_dtype;
    const CUtensorMapSwizzle swz = a.cB == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
    CUtensorMap mapX, mapW;
    int rcx;
    if (d->stride == 1) {
      const uint64_t xd[4] = {(uint64_t)d->C, (uint64_t)d->W, (uint64_t)d->H, (uint64_t)d->N};
      const uint32_t xb[4] = {(uint32_t)a.cB, (uint32_t)a.BW, (uint32_t)a.BH, (uint32_t)a.BI};
      rcx = encode_tiled(&mapX, x, 4, xd, xb, swz);
    } else {
      // stride 2 (H and W even): x as [N][H/2][2][W/2][2*C], so that the pixels an output tile
      // needs for one tap (every other row and column) are a dense box with the row and column
      // parities as coordinates
      const uint64_t xd[5] = {(uint64_t)(2 * d->C), (uint64_t)(d->W / 2), 2, (uint64_t)(d->H / 2),
                              (uint64_t)d->N};
      const uint32_t xb[5] = {(uint32_t)a.cB, (uint32_t)a.BW, 1, (uint32_t)a.BH, (uint32_t)a.BI};
      rcx = encode_tiled(&mapX, x, 5, xd, xb, swz);
    }
    const uint64_t wd[3] = {(uint64_t)d->C, 9, (uint64_t)d->K};
    const uint32_t wb[3] = {(uint32_t)a.cB, 1, (uint32_t)a.BN};
    if (rcx != WINO_OK || encode_tiled(&mapW, w, 3, wd, wb, swz) != WINO_OK) return WINO_ERR_CUDA;
    return launch_direct_conv_tc(a, dev, sms, mapX, mapW, bias, y, (cudaStream_t)stream) == 0
               ? WINO_OK : WINO_ERR_CUDA;
  }
  return launch_direct_conv(d->N, d->C, d->H, d->W, d->K, d->stride, d->q_x.zero_point,
                            d->q_w.zero_point, d->q_Y.zero_point,
                            (float)(s_in / (double)d->q_Y.scale), (float)s_in, d->q_Y.scale,
                            (float)(d->q_Y.qmin - d->q_Y.zero_point),
                            (float)(d->q_Y.qmax - d->q_Y.zero_point), d->out_dtype, x, w, bias, y,
                            d->s_w_K_dev, d->s_Y_K_dev, d->q_x.scale, d->q_w.scale,
                            (cudaStream_t)stream);
}

int wino_direct_last_status(void* stream) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return WINO_ERR_CUDA;
  int* word = direct_tc_status_word(dev);
  if (word == nullptr) return WINO_ERR_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return WINO_ERR_CUDA;
  int v = 0;
  if (cudaMemcpy(&v, word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return WINO_ERR_CUDA;
  if (v != 0 && cudaMemset(word, 0, sizeof(int)) != cudaSuccess) return WINO_ERR_CUDA;
  return v;
}

int wino_debug_mma_probe(wino_plan_t* pl, int iters, void* stream) {
  if (pl == nullptr || iters < 1 || iters > (1 << 22)) return WINO_ERR_INVALID;
  if (pl->status_dev == nullptr) return WINO_ERR_CUDA;
  pl->launches++;
  return launch_mma_peak(iters, pl->num_sms, pl->device, pl->status_dev, (cudaStream_t)stream);
}

int wino_debug_wait_probe(wino_plan_t* pl, long long limit_cycles, void* stream) {
  if (pl == nullptr || limit_cycles < 1 || limit_cycles > 100000000ll) return WINO_ERR_INVALID;
  if (pl->status_dev == nullptr) return WINO_ERR_CUDA;
  pl->launches++;
  return launch_wait_probe(limit_cycles, pl->status_dev, (cudaStream_t)stream);
}

int wino_debug_forward_accumulators(wino_plan_t* pl, const int8_t* x, const int8_t* Uq,
                                    const float* bias, void* y, int32_t* M_dev, size_t bytes,
                                    void* stream) {
  if (pl == nullptr || x == nullptr || Uq == nullptr || y == nullptr || M_dev == nullptr)
    return WINO_ERR_INVALID;
  if (path_uses_scratch(pl)) return WINO_ERR_UNSUPPORTED;   // staged paths: wino_debug_dump_stage
  if (bytes != m_elems(pl) * 4) return WINO_ERR_INVALID;
  if (!aligned16(x) || !aligned16(Uq) || !aligned16(y) || !aligned16(M_dev) ||
      (bias && !aligned16(bias)))
    return WINO_ERR_ALIGNMENT;
  return forward_impl(pl, x, Uq, bias, y, nullptr, nullptr, (cudaStream_t)stream, 7, M_dev);
}

int wino_debug_once_per_device(int device) {
  if (device < 0 || device >= DeviceOnce::kMaxDevices) return WINO_ERR_INVALID;
  int ran = 0;
  g_once_selftest.run(device, [&]() -> int { ran = 1; return 0; });
  return ran;
}

int wino_last_status(wino_plan_t* pl, void* stream) {
  if (pl == nullptr) return WINO_ERR_INVALID;
  if (pl->status_dev == nullptr) return WINO_ERR_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return WINO_ERR_CUDA;
  int v = 0;
  if (cudaMemcpy(&v, pl->status_dev, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
    return WINO_ERR_CUDA;
  // read and clear: the word is sticky on the device, the next read starts afresh
  if (v != 0 && cudaMemset(pl->status_dev, 0, sizeof(int)) != cudaSuccess) return WINO_ERR_CUDA;
  return v;
}

int wino_debug_dump_stage(wino_plan_t* pl, int stage, void* dst, size_t bytes) {
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
    const int saved_path = pl->path;
    if (pl->path == WINO_PATH_SMALLC) pl->path = WINO_PATH_STAGED_DP4A;
    if (pl->path == WINO_PATH_FUSED_F2) pl->path = WINO_PATH_STAGED_TC_PTR;
    if (pl->path == WINO_PATH_FUSED_LAYER) pl->path = WINO_PATH_STAGED_TC;
    const int rc = launch_gemm(pl, reinterpret_cast<const int8_t*>(ws), pl->last_uq, dst, kOutI32,
                               nullptr, false, st);
    pl->path = saved_path;
    return rc;
  }
  return WINO_ERR_INVALID;
}

long wino_launch_count(const wino_plan_t* pl) { return pl ? pl->launches : 0; }

void wino_destroy(wino_plan_t* pl) {
  if (pl == nullptr) return;
  if (pl->status_dev) cudaFree(pl->status_dev);
  if (pl->chan_dev) cudaFree(pl->chan_dev);
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
