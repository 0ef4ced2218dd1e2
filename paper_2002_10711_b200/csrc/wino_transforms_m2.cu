// Transform kernels instantiated for F(2x2, 3x3).
#define WINO_M 2
#include "wino_transforms_impl.cuh"
#include "wino_transforms_tma.cuh"
