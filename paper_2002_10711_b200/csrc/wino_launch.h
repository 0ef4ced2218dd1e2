// Internal interface between the host planner (wino_host.cu) and the kernel
// translation units.  Every function enqueues work on `st` and returns 0 or a
// negative WINO_ERR_* code; none allocates or synchronizes.
#pragma once
#include <cstdio>
#include <mutex>

#include <cuda.h>
#include <cuda_runtime.h>
#include "wino_common.cuh"

namespace wino {

// Launch options shared by all kernels.
struct LaunchOpt {
  bool std_mats = false;      // B^T and A^T are the built-in Cook-Toom matrices
  bool pdl = false;           // programmatic dependent launch on the stream
  int device = 0;             // the plan's device (current when the launcher runs)
  int num_sms = 148;          // its SM count
  // A buffer a later kernel of the same call will read and that no kernel of the call
  // writes (the transformed weights): the input transform's blocks ask for it to be brought
  // into L2 while they run.  A hint only; null: none.
  const void* l2_hint = nullptr;
  size_t l2_hint_bytes = 0;   // a multiple of 16
  // Per-output-channel multipliers, device array [5][K] (rows kChMultU ... kChSY), or null
  // for the per-layer values of Params.  Read by the weight transform, the GEMM epilogues
  // and the output transforms.
  const float* chan = nullptr;
};

// "Done once per device" bookkeeping.  cudaFuncSetAttribute applies to the device
// that is current when it is called, so the opt-in to more than 48 KB of dynamic
// shared memory has to be repeated on every device a kernel is launched on.
// run(dev, fn) calls fn() the first time it sees `dev` (and again if fn failed)
// under a lock, so concurrent first launches from several host threads are safe.
// Device indices beyond the table always run fn.
class DeviceOnce {
 public:
  static constexpr int kMaxDevices = 64;
  template <typename Fn>
  int run(int dev, Fn fn) {
    if (dev < 0 || dev >= kMaxDevices) return fn();
    std::lock_guard<std::mutex> lock(mu_);
    if (done_[dev]) return 0;
    const int rc = fn();
    if (rc == 0) done_[dev] = true;
    return rc;
  }
 private:
  std::mutex mu_;
  bool done_[kMaxDevices] = {};
};

// Opt a kernel in to `smem` bytes of dynamic shared memory on device `dev`.
template <typename Kern>
int set_max_smem(DeviceOnce& once, int dev, Kern kernel, size_t smem) {
  return once.run(dev, [&]() -> int {
    const cudaError_t e =
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
#ifdef WINO_TRACE
    if (e != cudaSuccess)
      std::fprintf(stderr, "shared-memory attribute failed: %s (%zu bytes)\n", cudaGetErrorString(e), smem);
#endif
    return e == cudaSuccess ? 0 : -5;
  });
}

// absmax (nullable): one word, max |U| of the layer; absmax_K (nullable): K words, max |U| of
// each filter; both as float bits, caller-zeroed.
int launch_weight_transform(const Params& p, const float* chan, const int8_t* w, int8_t* Uq,
                            unsigned* absmax, unsigned* absmax_K, cudaStream_t st);
int launch_input_transform(const Params& p, const LaunchOpt& o, const int8_t* x, int8_t* Vq,
                           unsigned* absmax, cudaStream_t st);
int launch_output_transform(const Params& p, const LaunchOpt& o, float s_Y, const void* mbuf,
                            const float* bias, void* y, unsigned* absmax2, cudaStream_t st);
int launch_gemm_dp4a(const Params& p, const LaunchOpt& o, const int8_t* Vq, const int8_t* Uq,
                     void* out, int out_mode, unsigned* absmaxM, cudaStream_t st);

// TMA-staged transform kernels (input needs z_x == 0 and C % 16 == 0; output needs
// Q_M on, int8 output and K % 16 == 0).  Channel chunk per block:
// (128 channels x 1 tile per block measured best on 256-channel layers: twice the
// blocks of a 256-channel chunk, so the single wave balances over the SMs)
inline int tma_chunk(int channels) {
  return channels % 128 == 0 ? 128 : channels % 64 == 0 ? 64 : channels % 32 == 0 ? 32
       : channels % 16 == 0 ? 16 : 0;
}
inline int tma_group(int chunk) { return chunk == 128 ? 1 : chunk == 64 ? 4 : chunk == 32 ? 4 : 8; }
int launch_input_transform_tma(const Params& p, const LaunchOpt& o, const CUtensorMap& mapX,
                               const CUtensorMap& mapV, int* status, cudaStream_t st);
int launch_output_transform_tma(const Params& p, const LaunchOpt& o, const CUtensorMap& mapM,
                                const CUtensorMap& mapY, const float* bias, float s_Y, int* status,
                                cudaStream_t st);

// Tensor-core transforms (Cook-Toom F2 / F4, channel count a multiple of 128; input
// needs z_x == 0, output needs Q_M on and an int8 output).  mapX and mapM carry the
// 128-byte swizzle; mapV and mapY are the plain maps of the kernels above.
// `kron`: device copy of the plan's Kronecker tables (fill_kronecker_tables).
constexpr int kKronInRows = 48, kKronOutRows = 16;
constexpr int kKronBytes = (kKronInRows + kKronOutRows) * 64;
bool transform_mma_supported(const Params& p, bool std_mats, int channels);
void fill_kronecker_tables(int m, int8_t* dst_host);
int launch_input_transform_mma(const Params& p, const LaunchOpt& o, const CUtensorMap& mapX,
                               const CUtensorMap& mapV, const void* kron, int num_sms, int* status,
                               cudaStream_t st);
int launch_output_transform_mma(const Params& p, const LaunchOpt& o, const CUtensorMap& mapM,
                                const CUtensorMap& mapY, const void* kron, const float* bias,
                                float s_Y, int num_sms, int* status, cudaStream_t st);

// The whole layer in one persistent launch (Cook-Toom F2 / F4, C and K multiples of
// 128, input zero point 0, Q_M on, int8 output).  `counters`: plan-owned device words,
// zero between launches (the kernel clears them when it finishes):
// [kFusedMaxMblk] cnt_in, [kFusedMaxMblk] cnt_m, then the exit ticket.
constexpr int kFusedMaxMblk = 1024;
constexpr int kFusedCounterWords = 2 * kFusedMaxMblk + 16;
struct FusedGeom { int BN, stages, n_mblk, n_nblk, n_items, grid; size_t smem; };
struct FusedMaps { const CUtensorMap *x, *v_store, *v_load, *u, *m_load, *y; };
bool layer_fused_supported(const Params& p, bool std_mats);
FusedGeom layer_fused_geometry(const Params& p, int num_sms);
int launch_layer_fused(const Params& p, const LaunchOpt& o, const FusedGeom& g, const FusedMaps& m,
                       const void* kron, unsigned* counters, int8_t* mq, const float* bias,
                       float s_Y, int* status, cudaStream_t st);

struct TcGeom { int BN, MB, stages, tmem_cols, grid; size_t smem; };
TcGeom tc_geometry(const Params& p, int num_sms);
int launch_gemm_tc(const Params& p, const LaunchOpt& o, const TcGeom& g, const CUtensorMap& mapV,
                   const CUtensorMap& mapU, void* out, int out_mode, unsigned* absmaxM,
                   int* status, cudaStream_t st);
int launch_smallc(const Params& p, const LaunchOpt& o, const int8_t* x, const int8_t* Uq,
                  const float* bias, void* y, float s_Y, int* dbgM, cudaStream_t st);

// Fully fused F2 kernel for narrow layers (C in {32, 64}, K <= 64, Cook-Toom matrices).
bool fused_f2_supported(const Params& p, bool std_mats);
int launch_fused_f2(const Params& p, const LaunchOpt& o, const CUtensorMap& mapU, const int8_t* x,
                    const float* bias, void* y, float s_Y, int num_sms, int* status, int* dbgM,
                    cudaStream_t st);

// Direct int8 3x3 convolution (stride 1 or 2) on the ALUs.
// Tensor-core direct convolution (no zero points on x and w, C % 64 == 0, K % 32 == 0; stride 2
// with even H and W).
struct DirectTcArgs {
  int N, C, H, W, K;       // H, W: output height and width
  int stride;
  int BW, BH, BI;          // output tile: BW x BH pixels of BI images, BW * BH * BI = 128
  int nW, nH, nI;          // tiles along width, height, batch
  int BN, n_nblk;          // output-channel block and their number
  int cB, KB;              // channel bytes per stage (64 or 128) and stages per tap
  int stages, tmem_cols, acc_stride;
  int n_items;
  // Narrow layers whose whole weight tensor fits beside the input ring: the weights are
  // fetched once per block and stay in shared memory (w_resident), and a stage then holds the
  // input boxes of `taps_per_stage` = 3 taps, one row of the filter (1 otherwise).
  int w_resident, taps_per_stage;
  float mult, s_in, s_Y, lo_Y, hi_Y;
  int z_Y, out_dtype;
  // per-output-channel scales (device arrays of K floats, nullable) and the per-layer scales
  // they replace
  const float* s_w_K;
  const float* s_Y_K;
  float s_x, s_w;
};
bool direct_tc_supported(int C, int K, int H, int W, int stride, int z_x, int z_w);
DirectTcArgs direct_tc_geometry(int N, int C, int H, int W, int K, int stride, int num_sms);
int* direct_tc_status_word(int device);
int launch_direct_conv_tc(const DirectTcArgs& a, int device, int num_sms, const CUtensorMap& mapX,
                          const CUtensorMap& mapW, const float* bias, void* y, cudaStream_t st);
// s_w_K, s_Y_K (nullable device arrays of K floats): per-output-channel scales replacing s_w
// and s_Y; s_x, s_w: the per-layer scales behind mult and s_in.
int launch_direct_conv(int N, int C, int H, int W, int K, int stride, int z_x, int z_w, int z_Y,
                       float mult, float s_in, float s_Y, float lo_Y, float hi_Y, int out_dtype,
                       const int8_t* x, const int8_t* w, const float* bias, void* y,
                       const float* s_w_K, const float* s_Y_K, float s_x, float s_w, cudaStream_t st);

// Tensor-pipe probe: `iters` back-to-back 128x256x32 int8 MMAs on every SM.
int launch_mma_peak(int iters, int num_sms, int device, int* status, cudaStream_t st);

// Bounded-wait probe: one block waits, with the given cycle limit, on a barrier
// that nothing arrives at, records WINO_ERR_TIMEOUT in *status and exits normally.
int launch_wait_probe(long long limit_cycles, int* status, cudaStream_t st);

enum { kOutMq = 0, kOutI32 = 1 };
constexpr int kBM = 128;      // tiles per GEMM block (MMA M)
constexpr int kStageK = 128;  // channels (bytes) per shared-memory stage

// Generic launcher: plain <<<>>> or cudaLaunchKernelEx with the programmatic
// stream serialization attribute (the kernel then calls griddep_wait()).
template <typename... KArgs, typename... Args>
int launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                  bool pdl, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
#ifdef WINO_TRACE
  if (e != cudaSuccess)
    std::fprintf(stderr, "launch failed: %s (grid %u block %u smem %zu)\n", cudaGetErrorString(e), grid.x,
                 block.x, smem);
#endif
  return e == cudaSuccess ? 0 : -5;
}

}  // namespace wino
