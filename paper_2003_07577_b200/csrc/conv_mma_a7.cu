// Warp-level tensor-pipe (int8 MMA on merged bit planes) convolution kernels for 7-bit activations.
#include "conv_mma.cuh"

namespace ebs {
static_assert(NUM_MMA_VARIANTS == NUM_CONV_MMA_VARIANTS && MMA_KTAB == CONV_MMA_MAX_KK, "tables out of sync");
EBS_DEFINE_MMA_ROW(7)
}  // namespace ebs
