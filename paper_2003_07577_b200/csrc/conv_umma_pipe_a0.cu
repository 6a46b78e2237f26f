// Persistent pipeline tcgen05 convolution kernels for activations given as unpacked byte codes (the context path that
// skips the bit-plane expansion).
#include "conv_umma_pipe.cuh"

namespace ebs {
EBS_DEFINE_PIPE_ROW(0)
}  // namespace ebs
