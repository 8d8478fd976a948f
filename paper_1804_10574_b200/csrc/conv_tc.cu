// Tensor-core convolution path (placeholder until the tcgen05 kernels land: nothing is routed here yet).
#include "conv_tc.h"

namespace ddg {
bool conv_tc_supported(int, int, int, int, int, int) { return false; }
int launch_conv_tc(int, const void *, const void *, void *, int, int, int, int, Shortcut, cudaStream_t) { return 0; }
bool wgrad_tc_supported(int, int, int, int, int, int) { return false; }
size_t wgrad_tc_scratch_elems() { return 0; }
int launch_wgrad_tc(const void *, const void *, float *, float *, int, int, int, int, cudaStream_t) { return 0; }
int conv_tc_init() { return 0; }
}  // namespace ddg
