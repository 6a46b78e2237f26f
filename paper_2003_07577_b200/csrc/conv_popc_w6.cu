// Popcount-path convolution kernels for 6-bit weights (all activation bitwidths, all tile families).
#include "conv_popc.cuh"

namespace ebs {
EBS_DEFINE_WB_TABLE(6)
}  // namespace ebs
