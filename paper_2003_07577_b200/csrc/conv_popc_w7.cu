// Popcount-path convolution kernels for 7-bit weights (all activation bitwidths, all tile families).
#include "conv_popc.cuh"

namespace ebs {
EBS_DEFINE_WB_TABLE(7)
}  // namespace ebs
