// tcgen05 (int8 MMA on bit planes, accumulator in tensor memory) convolution kernels for 1-bit weights.
#include "conv_umma.cuh"

namespace ebs {
static_assert(NUM_UMMA_VARIANTS == NUM_CONV_UMMA_VARIANTS && UMMA_KTAB == CONV_MMA_MAX_KK, "tables out of sync");
EBS_DEFINE_UMMA_TABLE(1)
}  // namespace ebs
