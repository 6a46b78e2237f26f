// Popcount-path convolution kernels for 4-bit weights (all activation bitwidths, all tile families).
#include "conv_popc.cuh"

namespace ebs {
EBS_DEFINE_WB_TABLE(4)
}  // namespace ebs
