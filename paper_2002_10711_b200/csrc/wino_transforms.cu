// Dispatch of the transform launchers over the tile size m.
#include "wino_launch.h"

namespace wino {

#define WINO_DECL(m)                                                                              \
  int launch_weight_transform_m##m(const Params&, const float*, const int8_t*, int8_t*, unsigned*, \
                                   unsigned*, cudaStream_t);                                      \
  int launch_input_transform_m##m(const Params&, const LaunchOpt&, const int8_t*, int8_t*,        \
                                  unsigned*, cudaStream_t);                                       \
  int launch_output_transform_m##m(const Params&, const LaunchOpt&, float, const void*,           \
                                   const float*, void*, unsigned*, cudaStream_t);            \
  int launch_input_transform_tma_m##m(const Params&, const LaunchOpt&, const CUtensorMap&,        \
                                      const CUtensorMap&, int*, cudaStream_t);                    \
  int launch_output_transform_tma_m##m(const Params&, const LaunchOpt&, const CUtensorMap&,       \
                                       const CUtensorMap&, const float*, float, int*, cudaStream_t);
WINO_DECL(2)
WINO_DECL(4)
WINO_DECL(6)
#undef WINO_DECL

int launch_weight_transform(const Params& p, const float* chan, const int8_t* w, int8_t* Uq,
                            unsigned* absmax, unsigned* absmax_K, cudaStream_t st) {
  return p.m == 2 ? launch_weight_transform_m2(p, chan, w, Uq, absmax, absmax_K, st)
       : p.m == 4 ? launch_weight_transform_m4(p, chan, w, Uq, absmax, absmax_K, st)
                  : launch_weight_transform_m6(p, chan, w, Uq, absmax, absmax_K, st);
}
int launch_input_transform(const Params& p, const LaunchOpt& o, const int8_t* x, int8_t* Vq,
                           unsigned* absmax, cudaStream_t st) {
  return p.m == 2 ? launch_input_transform_m2(p, o, x, Vq, absmax, st)
       : p.m == 4 ? launch_input_transform_m4(p, o, x, Vq, absmax, st)
                  : launch_input_transform_m6(p, o, x, Vq, absmax, st);
}
int launch_output_transform(const Params& p, const LaunchOpt& o, float s_Y, const void* mbuf,
                            const float* bias, void* y, unsigned* absmax2, cudaStream_t st) {
  return p.m == 2 ? launch_output_transform_m2(p, o, s_Y, mbuf, bias, y, absmax2, st)
       : p.m == 4 ? launch_output_transform_m4(p, o, s_Y, mbuf, bias, y, absmax2, st)
                  : launch_output_transform_m6(p, o, s_Y, mbuf, bias, y, absmax2, st);
}

int launch_input_transform_tma(const Params& p, const LaunchOpt& o, const CUtensorMap& mapX,
                               const CUtensorMap& mapV, int* status, cudaStream_t st) {
  return p.m == 2 ? launch_input_transform_tma_m2(p, o, mapX, mapV, status, st)
       : p.m == 4 ? launch_input_transform_tma_m4(p, o, mapX, mapV, status, st)
                  : launch_input_transform_tma_m6(p, o, mapX, mapV, status, st);
}
int launch_output_transform_tma(const Params& p, const LaunchOpt& o, const CUtensorMap& mapM,
                                const CUtensorMap& mapY, const float* bias, float s_Y, int* status,
                                cudaStream_t st) {
  return p.m == 2 ? launch_output_transform_tma_m2(p, o, mapM, mapY, bias, s_Y, status, st)
       : p.m == 4 ? launch_output_transform_tma_m4(p, o, mapM, mapY, bias, s_Y, status, st)
                  : launch_output_transform_tma_m6(p, o, mapM, mapY, bias, s_Y, status, st);
}

}  // namespace wino
