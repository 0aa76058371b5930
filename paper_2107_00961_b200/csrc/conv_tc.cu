// Tensor-core convolution kernels (tcgen05 + TMEM).  Placeholder until the kernels land: no shape is
// accepted, so every convolution runs on the CUDA-core family.
#include "internal.h"
namespace resist {
bool conv_tc_supported(const ConvProb&, int) { return false; }
void launch_conv_tc(const ConvProb*, int, int, int, cudaStream_t) {}
size_t conv_tc_scratch_bytes(const ConvProb&, int) { return 0; }
void conv_tc_prepare(ConvProb&, int, void*, int) {}
}  // namespace resist
