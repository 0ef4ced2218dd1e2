// Transform kernels instantiated for F(4x4, 3x3).
#define WINO_M 4
#include "wino_transforms_impl.cuh"
#include "wino_transforms_tma.cuh"
