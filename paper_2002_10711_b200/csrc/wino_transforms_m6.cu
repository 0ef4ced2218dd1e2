// Transform kernels instantiated for F(6x6, 3x3).
#define WINO_M 6
#include "wino_transforms_impl.cuh"
#include "wino_transforms_tma.cuh"
