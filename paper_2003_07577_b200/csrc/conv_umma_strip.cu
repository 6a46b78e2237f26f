// Instantiations of the stride-1 strip kernel: the weight operand is a byte image, so the kernel depends
// on the activation bitwidth and the channel tile only.
#include "conv_umma_strip.cuh"

namespace ebs {

template <int AB, int VARIANT>
constexpr ConvVariant make_strip_variant() {
    constexpr int TILE_N = 16 << VARIANT;
    return ConvVariant{&launch_conv_umma_strip<AB, TILE_N>, UMMA_M, TILE_N, UMMA_THREADS};
}

#define EBS_STRIP_ROW(AB)                                                                             \
    {make_strip_variant<AB, 0>(), make_strip_variant<AB, 1>(), make_strip_variant<AB, 2>(),           \
     make_strip_variant<AB, 3>(), make_strip_variant<AB, 4>()}

const ConvVariant* conv_umma_strip_variant(int a_bits, int variant) {
    static const ConvVariant table[8][NUM_UMMA_STRIP_VARIANTS] = {
        EBS_STRIP_ROW(1), EBS_STRIP_ROW(2), EBS_STRIP_ROW(3), EBS_STRIP_ROW(4),
        EBS_STRIP_ROW(5), EBS_STRIP_ROW(6), EBS_STRIP_ROW(7), EBS_STRIP_ROW(8)};
    if (a_bits < 1 || a_bits > 8 || variant < 0 || variant >= NUM_UMMA_STRIP_VARIANTS) return nullptr;
    return &table[a_bits - 1][variant];
}

bool conv_umma_strip_applies(const ConvParams& p, int variant) {
    return variant >= 0 && variant < NUM_UMMA_STRIP_VARIANTS && strip_geometry(p, 16 << variant).ok;
}

unsigned long long conv_umma_strip_timeouts() {
    unsigned long long v = 0;
    cudaMemcpyFromSymbol(&v, g_umma_timeouts, sizeof(v));
    return v;
}

}  // namespace ebs
