// Persistent pipeline tcgen05 convolution kernels for 1-bit activations.
#include "conv_umma_pipe.cuh"

namespace ebs {
static_assert(NUM_UMMA_PIPE_VARIANTS == NUM_CONV_PIPE_VARIANTS, "tables out of sync");
EBS_DEFINE_PIPE_ROW(1)
}  // namespace ebs
