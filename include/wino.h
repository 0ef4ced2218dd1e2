/*
 * wino.h - C ABI of the B200 (sm_100a) Winograd-aware quantized 3x3 convolution
 * forward pass.
 *
 * The layer computes, for every (m+2)x(m+2) input patch d and 3x3 filter g,
 *     Y = A^T [ (G g G^T) (.) (B^T d B) ] A            (paper: Section 3.1, Eq. 1)
 * with a uniform quantizer after every stage (paper: Fig. 2 and Section 3.2:
 * transformed weights, transformed input, Hadamard product, output) using
 * per-layer symmetric quantization (paper: Section 5.1).  The transform
 * matrices B^T, G, A^T are data: either the Cook-Toom ones or relaxed, learnt
 * ("flex") ones (paper: Sections 3.1, 3.2).
 *
 * Notation.  t = m + 2; xi = i*t + j indexes the t*t Winograd-domain positions;
 * TH = ceil(H/m), TW = ceil(W/m), T = N*TH*TW tiles; tile index
 * tau = (n*TH + th)*TW + tw.  Filters are 3x3, stride 1, zero padding 1.
 *
 * Tensor layouts (dense, row-major in the index order written, DEVICE memory):
 *   x    int8  [N][H][W][C]      activations (codes)
 *   w    int8  [K][3][3][C]      filters (codes)
 *   U_q  int8  [t*t][K][C]       transformed, quantized filters
 *   y    int8 or float [N][H][W][K]
 *   bias float [K]               in real units (optional)
 *
 * Arithmetic contract (what "the same result" means, bit for bit):
 *   - quantizer  Q(v; mult, z, qmin, qmax) = clamp(rne(v * mult) + z, qmin, qmax):
 *     the exact product of the fp32 value v and the fp32 multiplier is rounded
 *     once, half to even; mult is precomputed,
 *     mult = (float)((double)s_src / (double)s_dst);
 *   - a transform  Z = (L X) L^T  is evaluated as a left pass then a right pass,
 *     each entry one fused-multiply-add chain starting from 0.0f and running
 *     over the contracted index in ascending order, in fp32;
 *   - input stage   V = B^T d B on d = (float)(x - z_x) (0 outside the image),
 *                   V_q = Q(V; s_x/s_V);
 *   - weight stage  U = G g G^T on g = (float)(w - z_w), U_q = Q(U; s_w/s_U);
 *   - Hadamard stage M[xi][tau][k] = sum_c V_q * U_q in int32 (exact),
 *                   m_q = Q((float)M; s_U*s_V/s_M) when q_M.enabled;
 *   - output stage  right factor first: R = m A, then Y = A^T R (same chain
 *                   rule), m = (float)m_q, or (float)M when q_M is disabled;
 *                   int8 output: Q(fmaf(Y, s_acc/s_Y, bias/s_Y); 1) with
 *                   s_acc = s_M (or s_U*s_V when q_M is disabled);
 *                   float output: fmaf(Y, (float)s_acc, bias).
 *
 * Ownership.  The caller owns every device buffer and the stream.  A plan owns
 * only its copy of the descriptor and matrices plus one small device status
 * word.  No entry point below allocates device memory except wino_plan.
 *
 * Errors.  Every function returns WINO_OK (0) or a negative code; nothing
 * throws, aborts or traps.  Launches are asynchronous on the given stream.
 *
 * Devices and threads.  A plan belongs to the device that was current when
 * wino_plan ran (its status word lives there); use it with that device current.
 * Plans on several devices may coexist in one process.  A plan is not
 * thread-safe: every call that launches work updates the plan (caches of
 * tensor maps, launch counter), which is why those calls take a non-const
 * plan; calls on one plan must not overlap in time on the host.  Different
 * plans may be used from different threads.
 */
#ifndef WINO_H_
#define WINO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  WINO_OK = 0,
  WINO_ERR_INVALID = -1,     /* null pointer, size out of range, bad enum */
  WINO_ERR_UNSUPPORTED = -2, /* valid request this build does not implement */
  WINO_ERR_ALIGNMENT = -3,   /* a device pointer is not 16-byte aligned */
  WINO_ERR_WORKSPACE = -4,   /* workspace missing */
  WINO_ERR_CUDA = -5,        /* a CUDA runtime / driver call failed */
  WINO_ERR_TIMEOUT = -6      /* a bounded device-side wait expired */
};

/* Execution paths a plan can use (see wino_plan_path / wino_plan_force_path).  The automatic
 * choice is 5 where it applies, else 2 for layers of at most 16 channels in and out, else 1
 * where C and K are multiples of 16, else 2. */
enum {
  WINO_PATH_AUTO = 0,
  WINO_PATH_STAGED_TC = 1,   /* transform kernels (TMA-staged where the shape allows) + tcgen05 int8 GEMMs */
  WINO_PATH_STAGED_DP4A = 2, /* transform kernels + integer-dot-product GEMMs on the ALUs */
  WINO_PATH_SMALLC = 3,      /* one fused warp-shuffle kernel, C <= 32 and K <= 32 (never chosen automatically) */
  WINO_PATH_STAGED_TC_PTR = 4, /* as 1, but always the pointer-based transform kernels */
  WINO_PATH_FUSED_F2 = 5,    /* one fused tcgen05 kernel: m = 2, Cook-Toom matrices, C in {32, 64}, K <= 64 */
  WINO_PATH_STAGED_TC_MMA = 6, /* as 1, with the transforms themselves on the tensor cores where that is
                                 exact: Cook-Toom F2 / F4, channel counts multiples of 128 */
  WINO_PATH_FUSED_LAYER = 7   /* the whole layer in one persistent launch (tensor-core transforms and
                                 GEMMs; V_q and m_q pass through the workspace in L2): Cook-Toom F2 / F4,
                                 C and K multiples of 128, input zero point 0, Q_M on, int8 output */
};

/* Stages that wino_debug_dump_stage can copy out (staged paths only). */
enum { WINO_STAGE_VQ = 0, WINO_STAGE_M_I32 = 1, WINO_STAGE_MQ = 2 };

/* One uniform quantizer (paper: Section 5.1).  real = scale * (code - zero_point);
 * codes are clamped to [qmin, qmax], which must lie inside [-128, 127].
 * `enabled` is only read for q_M (0 = feed the int32 sums straight to the output
 * transform). */
typedef struct {
  float scale;
  int32_t zero_point;
  int32_t qmin, qmax;
  int32_t enabled;
} wino_quant_t;

/* Problem statement of one layer.  BT, G, AT are HOST pointers to row-major
 * fp32 matrices BT[t][t], G[t][3], AT[m][t]; they are copied by wino_plan.
 * transforms_exact is advisory: the library itself recognises the Cook-Toom
 * matrices for the standard points (bit-for-bit comparison) and only then uses
 * kernels that rely on their products with integer codes being exact in fp32.
 * out_dtype: 0 = int8 codes, 1 = float real values.
 * Restrictions (WINO_ERR_UNSUPPORTED otherwise): m in {2, 4, 6};
 * zero_point == 0 for q_V, q_U, q_M; C <= 1040 (so that (float)M is exact). */
typedef struct {
  int32_t N, C, H, W, K, m;
  const float* BT;
  const float* G;
  const float* AT;
  int32_t transforms_exact;
  wino_quant_t q_x, q_w, q_V, q_U, q_M, q_Y;
  int32_t out_dtype;
} wino_desc_t;

typedef struct wino_plan wino_plan_t; /* opaque */

/* Validates the descriptor, copies it, precomputes the fixed multipliers and
 * picks an execution path (paper: Eq. 1 / Fig. 2 define what is planned).
 * *out receives a new plan (free with wino_destroy).  Works without a GPU for
 * size queries; launches then fail with WINO_ERR_CUDA. */
int wino_plan(const wino_desc_t* desc, wino_plan_t** out);

/* Bytes of U_q: t*t*K*C (paper: Section 3.1 "Memory": 1.78x / 4x the filters). */
size_t wino_weight_bytes(const wino_plan_t* plan);

/* Bytes of scratch for the staged paths and for wino_calibrate_forward: V_q plus
 * m_q (or M in int32 when q_M is disabled).  On the fused small-channel path
 * wino_conv_forward itself needs none and accepts a NULL workspace. */
size_t wino_workspace_bytes(const wino_plan_t* plan);

/* The path the plan will run (one of WINO_PATH_*), and a way to pin it.
 * Forcing a path the shape cannot use returns WINO_ERR_UNSUPPORTED. */
int wino_plan_path(const wino_plan_t* plan);
int wino_plan_force_path(wino_plan_t* plan, int path);

/* Per-output-channel scales (paper: Section 7 names per-channel quantization as the step
 * beyond the per-layer scales of Section 5.1).  Each argument is a HOST array of K positive
 * finite floats, copied by the call, or NULL to keep the descriptor's per-layer scale, for
 * the four tensors that carry the output-channel axis: s_w_K[k] replaces q_w.scale for
 * filter k, s_U_K[k] replaces q_U.scale for the transformed filter k (so the Hadamard sums
 * of channel k carry s_U_K[k] * q_V.scale), s_M_K[k] replaces q_M.scale for channel k of the
 * quantized Hadamard sums (ignored when q_M is disabled), s_Y_K[k] replaces q_Y.scale for
 * output channel k (the bias enters the integer output as bias[k] / s_Y_K[k]).  The input
 * side (x, V) is summed over its channels and keeps one scale; zero points and code ranges
 * stay per layer.  All four NULL returns the plan to per-layer scales.  Call before
 * wino_transform_weights; U_q made under other scales is stale.  The staged paths
 * (WINO_PATH_STAGED_TC, WINO_PATH_STAGED_TC_PTR, WINO_PATH_STAGED_DP4A) implement it: a
 * plan on another path moves to the staged tcgen05 path (or the staged dp4a path), forcing
 * another path afterwards returns WINO_ERR_UNSUPPORTED, and wino_plan_multipliers keeps
 * reporting the per-layer values.  Synchronous (one small host-to-device copy);
 * WINO_ERR_INVALID for a bad scale, WINO_ERR_CUDA without a device. */
int wino_plan_set_channel_scales(wino_plan_t* plan, const float* s_w_K, const float* s_U_K,
                                 const float* s_M_K, const float* s_Y_K);

/* The five fixed multipliers the plan uses, for inspection:
 * out[0]=s_x/s_V, out[1]=s_w/s_U, out[2]=s_U*s_V/s_M, out[3]=s_acc/s_Y, out[4]=s_acc. */
int wino_plan_multipliers(const wino_plan_t* plan, float out[5]);

/* Weight transform U_q = Q(G g G^T) (paper: Eq. 1; done once per layer, so its
 * cost is spread over every later inference: Section 3.1).  w_KRSC_dev: int8 [K][3][3][C]; Uq_dev:
 * int8 [t*t][K][C]; both device pointers, 16-byte aligned.  absmax_dev
 * (nullable, device, one uint32 holding float bits, caller-zeroed) receives
 * max |U| before quantization, for calibration. */
int wino_transform_weights(wino_plan_t* plan, const int8_t* w_KRSC_dev, int8_t* Uq_dev,
                           uint32_t* absmax_dev, void* stream);

/* The same transform, recording max |U| of every filter (before quantization, in units of
 * the weight codes) in absmax_K_dev[k] as float bits (device, uint32[K], caller-zeroed): the
 * statistic a per-output-channel scale for the transformed weights is set from (see
 * wino_plan_set_channel_scales).  Uq_dev is written as by wino_transform_weights. */
int wino_transform_weights_channel_stats(wino_plan_t* plan, const int8_t* w_KRSC_dev,
                                         int8_t* Uq_dev, uint32_t* absmax_K_dev, void* stream);

/* The forward pass (paper: Eq. 1 with the quantizers of Fig. 2): input
 * transform, Hadamard stage as t*t int8 GEMMs over channels with int32
 * accumulation, output transform, bias, output quantizer.
 * x_NHWC_dev int8 [N][H][W][C]; Uq_dev from wino_transform_weights; bias_K_dev
 * float [K] or NULL; y_NHWK_dev int8 or float [N][H][W][K] per out_dtype;
 * workspace_dev at least wino_workspace_bytes (may be NULL when that is 0).
 * All device pointers 16-byte aligned. */
int wino_conv_forward(wino_plan_t* plan, const int8_t* x_NHWC_dev, const int8_t* Uq_dev,
                      const float* bias_K_dev, void* y_NHWK_dev, void* workspace_dev,
                      void* stream);

/* Largest workspace wino_conv_forward_static can serve, in bytes. */
#define WINO_STATIC_SCRATCH_BYTES (20u * 1024u * 1024u)

/* wino_conv_forward for callers that cannot hand over a workspace because they
 * cannot allocate device memory at this point.  (The paper has no counterpart:
 * this is a deployment convenience of this library.)  Typical cases: a plug-in
 * inside a host framework that owns all device memory through its own pool and
 * does not let plug-ins call the CUDA allocator; a latency-critical serving
 * loop, where cudaMalloc may block on the whole device and can fail late under
 * a fixed memory budget; start-up code that runs before the application's
 * allocator exists.
 *
 * Same arguments, results and errors as wino_conv_forward, minus the workspace:
 * V_q and m_q live in a static device array of WINO_STATIC_SCRATCH_BYTES built
 * into the library (every GPU that loads the library holds those bytes until
 * the process exits).  A plan on a staged path whose wino_workspace_bytes
 * exceeds that size is refused with WINO_ERR_WORKSPACE and nothing is launched;
 * plans on a single-kernel path (WINO_PATH_SMALLC, WINO_PATH_FUSED_F2) need no
 * scratch and are accepted at any size.  The call makes no cudaMalloc /
 * cudaFree and uses no allocating library routine.
 *
 * First use on a device: the first call made with a given device current looks
 * up the array's device address (cudaGetSymbolAddress) and remembers it; make
 * that first call before starting any stream capture on that device.
 * Sharing: all calls on a device, from every plan and stream, use the same
 * array, and it keeps whatever the last call left there.  Nothing in it has to
 * start at zero (each call overwrites every byte it later reads).  Two calls
 * whose kernels overlap on the GPU (different streams, no ordering between
 * them) race on the array and corrupt each other's result: order them. */
int wino_conv_forward_static(wino_plan_t* plan, const int8_t* x_NHWC_dev,
                             const int8_t* Uq_dev, const float* bias_K_dev, void* y_NHWK_dev,
                             void* stream);

/* Calibration pass (paper: Table 1 caption, range "warmup"; here a one-shot
 * max-abs): runs the forward pass on a staged path and records, as float bits
 * in absmax4_dev[0..3] (device, caller-zeroed uint32[4]), the max-abs of
 * V (before Q_V), of M (as a float), of Y before the output scaling, and of
 * the float-mode output fmaf(Y, s_acc, bias).  y_NHWK_dev may be NULL. */
int wino_calibrate_forward(wino_plan_t* plan, const int8_t* x_NHWC_dev,
                           const int8_t* Uq_dev, const float* bias_K_dev, void* y_NHWK_dev,
                           void* workspace_dev, uint32_t* absmax4_dev, void* stream);

/* Direct int8 3x3 convolution (cross-correlation, zero padding 1, stride 1 or 2), the
 * lossless candidate of the paper's search space (Section 4, "im2row") and the
 * layer type of its strided convolutions, which have no Winograd form (Section
 * 5.1).  acc = sum over the 3x3xC window of (x - z_x)(w - z_w) in int32 (padding
 * is the real value zero); int8 output Q(fmaf((float)acc, (float)(s_x*s_w/s_Y),
 * (float)(bias/s_Y)); 1), float output fmaf((float)acc, (float)(s_x*s_w), bias).
 * x int8 [N][H][W][C], w int8 [K][3][3][C], y [N][Ho][Wo][K] with
 * Ho = (H-1)/stride + 1; any C and K (a layer whose C or K is not a multiple of 4,
 * such as a three-channel first layer, runs on a simple byte-wise kernel); device
 * pointers 16-byte aligned.
 * Stateless: no plan, no workspace.  Without zero points on x and w, with C a
 * multiple of 64, K a multiple of 32 (at most 2048), y 32-byte aligned and, at
 * stride 2, even H and W, the layer runs as an implicit GEMM on the tensor cores;
 * everything else on the integer ALUs.
 * The results are the same bits either way. */
typedef struct {
  int32_t N, C, H, W, K, stride;
  wino_quant_t q_x, q_w, q_Y;
  int32_t out_dtype;
  /* Per-output-channel scales (paper: Section 7), DEVICE arrays of K positive floats or NULL:
   * s_w_K_dev[k] replaces q_w.scale for filter k, s_Y_K_dev[k] replaces q_Y.scale for output
   * channel k.  The kernels form, per channel, (float)((double)s_x * s_w[k] / s_Y[k]) and
   * (float)((double)bias[k] / s_Y[k]); the values are not validated (they live on the device). */
  const float* s_w_K_dev;
  const float* s_Y_K_dev;
} wino_direct_desc_t;
int wino_direct_conv_forward(const wino_direct_desc_t* desc, const int8_t* x_NHWC_dev,
                             const int8_t* w_KRSC_dev, const float* bias_K_dev, void* y_dev,
                             void* stream);
/* Status of the direct convolutions on the current device, which have no plan to keep
 * one in: synchronizes `stream`, returns WINO_OK, WINO_ERR_TIMEOUT (a bounded wait
 * inside the tensor-core kernel expired; its output is undefined) or WINO_ERR_CUDA,
 * and clears the word. */
int wino_direct_last_status(void* stream);

/* Synchronizes `stream` and returns the plan's device status word: WINO_OK, or
 * WINO_ERR_TIMEOUT if a bounded wait inside a kernel expired (the kernel then
 * stopped early and its output is undefined), or WINO_ERR_CUDA.  On the device
 * the word is sticky (a later successful launch does not reset it); this call
 * reads it and clears it, so the next call reports only what happened since. */
int wino_last_status(wino_plan_t* plan, void* stream);

/* Copies one intermediate of the most recent wino_conv_forward on this plan
 * (staged paths only) into dst_dev: V_q int8 [t*t][T][C], M int32 [t*t][T][K]
 * (recomputed from V_q and U_q with the plan's GEMM kernel), m_q int8
 * [t*t][T][K].  `bytes` must equal the stage size.  Asynchronous on the stream
 * of that forward call. */
int wino_debug_dump_stage(wino_plan_t* plan, int stage, void* dst_dev, size_t bytes);

/* The forward pass on a single-kernel path (WINO_PATH_SMALLC, WINO_PATH_FUSED_F2;
 * WINO_ERR_UNSUPPORTED on the staged paths, which have wino_debug_dump_stage)
 * that also writes the int32 Hadamard sums the kernel held in registers /
 * tensor memory (paper: Eq. 1, the product inside the brackets, summed over
 * channels) to M_dev, int32 [t*t][T][K]; `bytes` must equal that size. */
int wino_debug_forward_accumulators(wino_plan_t* plan, const int8_t* x_NHWC_dev,
                                    const int8_t* Uq_dev, const float* bias_K_dev,
                                    void* y_NHWK_dev, int32_t* M_dev, size_t bytes, void* stream);

/* Runs a subset of the three kernels of a staged path on the caller's buffers
 * (stages of the paper's Fig. 2): stage_mask bit 0 = input transform (x -> V_q in
 * the workspace), bit 1 = Hadamard GEMMs (V_q, U_q -> m_q in the workspace),
 * bit 2 = output transform (m_q -> y).  Stages left out read whatever an earlier
 * call left in the workspace.  For debugging and per-kernel timing. */
int wino_debug_run_stages(wino_plan_t* plan, int stage_mask, const int8_t* x_NHWC_dev,
                          const int8_t* Uq_dev, const float* bias_K_dev, void* y_NHWK_dev,
                          void* workspace_dev, void* stream);

/* Tensor-pipe probe for the roofline of the Hadamard stage (the stage the paper calls
 * the bulk of the computation, Section 1): launches, on every SM of the plan's device,
 * `iters` back-to-back tcgen05 int8 MMAs of 128x256x32 on operands held in shared
 * memory.  The work is iters * SMs * 2*128*256*32 operations; the caller times the
 * launch (CUDA events) to get the sustained int8 tensor rate of the device.
 * A bounded wait that expires is reported through wino_last_status. */
int wino_debug_mma_probe(wino_plan_t* plan, int iters, void* stream);

/* Shows what every kernel of this library does when a barrier it waits for never
 * completes (no counterpart in the paper).  Launches one small block that
 * waits, for at most limit_cycles SM clocks (1 .. 1e8), on a barrier nothing
 * arrives at, then records WINO_ERR_TIMEOUT in the plan's status word and exits
 * normally; wino_last_status reports it and clears it, and the plan stays
 * usable.  Production kernels use the same wait with a limit of about a second. */
int wino_debug_wait_probe(wino_plan_t* plan, long long limit_cycles, void* stream);

/* Host-side check of the library's once-per-device bookkeeping (kernel attributes
 * are set once on every device a kernel runs on): returns 1 the first time it is
 * called with a device index in [0, 64), 0 on later calls with the same index,
 * WINO_ERR_INVALID outside the range.  Touches no GPU. */
int wino_debug_once_per_device(int device);

/* Number of kernels launched by this plan since it was created. */
long wino_launch_count(const wino_plan_t* plan);

void wino_destroy(wino_plan_t* plan);
const char* wino_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* WINO_H_ */
