// Instantiations of the persistent, weight-resident strip kernel (activation bitwidth x channel tile).
#include "conv_umma_resident.cuh"

namespace ebs {

int resident_sm_count() {
    int dev = 0, n = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    return n > 0 ? n : 148;
}

template <int AB, int VARIANT>
constexpr ConvVariant make_resident_variant() {
    constexpr int TILE_N = 16 << VARIANT;
    return ConvVariant{&launch_conv_umma_resident<AB, TILE_N>, UMMA_M, TILE_N, RES_THREADS};
}

#define EBS_RES_ROW(AB)                                                                               \
    {make_resident_variant<AB, 0>(), make_resident_variant<AB, 1>(), make_resident_variant<AB, 2>(),  \
     make_resident_variant<AB, 3>(), make_resident_variant<AB, 4>()}

const ConvVariant* conv_umma_resident_variant(int a_bits, int variant) {
    static const ConvVariant table[8][NUM_UMMA_RESIDENT_VARIANTS] = {
        EBS_RES_ROW(1), EBS_RES_ROW(2), EBS_RES_ROW(3), EBS_RES_ROW(4),
        EBS_RES_ROW(5), EBS_RES_ROW(6), EBS_RES_ROW(7), EBS_RES_ROW(8)};
    if (a_bits < 1 || a_bits > 8 || variant < 0 || variant >= NUM_UMMA_RESIDENT_VARIANTS) return nullptr;
    return &table[a_bits - 1][variant];
}

bool conv_umma_resident_applies(const ConvParams& p, int variant) {
    return variant >= 0 && variant < NUM_UMMA_RESIDENT_VARIANTS &&
           resident_geometry(p, 16 << variant, resident_sm_count()).ok;
}

unsigned long long conv_umma_resident_timeouts() {
    unsigned long long v = 0;
    cudaMemcpyFromSymbol(&v, g_umma_timeouts, sizeof(v));
    return v;
}

}  // namespace ebs
