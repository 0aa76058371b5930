// Tensor-core convolution kernels (tcgen05 + TMEM).  Placeholder until the kernels land: no shape is
// accepted, so every convolution runs on the CUDA-core family.
#include "internal.h"
namespace resist {
bool conv_tc_supported(const ConvProb&, int) { return false; }
void launch_conv_tc(const ConvProb*, int, int, int, cudaStream_t) {}
}  // namespace resist
