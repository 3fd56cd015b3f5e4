// Tensor-core convolution kernels (tcgen05 / TMEM / TMA).  Each entry returns false when it does
// not take the shape, and the caller then runs the fp32 kernel.
#include "common.cuh"

bool conv_fprop_tc(Exec &, const void *, Geom, const Layer &, Pair, Pair, int) { return false; }
bool conv_dgrad_tc(Exec &, const void *, Geom, const Layer &, float *) { return false; }
bool conv_wgrad_tc(Exec &, const void *, const void *, Geom, const Layer &, float *) { return false; }
