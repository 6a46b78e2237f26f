// Instantiations of the warp-level strip kernel (activation bitwidth x channel tile).
#include "conv_mma_strip.cuh"

namespace ebs {

template <int AB, int VARIANT>
constexpr ConvVariant make_mma_strip_variant() {
    // tile_c 16: 8 warps x (32 pixels x 16 channels); 32: 4 warps x (16 x 32); 64: 4 x 2 warps of (16 x 32)
    if constexpr (VARIANT == 0) return ConvVariant{&launch_conv_mma_strip<AB, 2, 2, 8, 1>, 256, 16, 256};
    else if constexpr (VARIANT == 1) return ConvVariant{&launch_conv_mma_strip<AB, 1, 4, 4, 1>, 64, 32, 128};
    else return ConvVariant{&launch_conv_mma_strip<AB, 1, 4, 4, 2>, 64, 64, 256};
}

#define EBS_MS_ROW(AB) {make_mma_strip_variant<AB, 0>(), make_mma_strip_variant<AB, 1>(), make_mma_strip_variant<AB, 2>()}

const ConvVariant* conv_mma_strip_variant(int a_bits, int variant) {
    static const ConvVariant table[8][NUM_MMA_STRIP_VARIANTS] = {EBS_MS_ROW(1), EBS_MS_ROW(2), EBS_MS_ROW(3), EBS_MS_ROW(4),
                                                                 EBS_MS_ROW(5), EBS_MS_ROW(6), EBS_MS_ROW(7), EBS_MS_ROW(8)};
    if (a_bits < 1 || a_bits > 8 || variant < 0 || variant >= NUM_MMA_STRIP_VARIANTS) return nullptr;
    return &table[a_bits - 1][variant];
}

bool conv_mma_strip_applies(const ConvParams& p, int variant) {
    const ConvVariant* v = conv_mma_strip_variant(1, variant);
    return v && mma_strip_geometry(p, v->tile_p, v->tile_c).ok;
}

}  // namespace ebs
