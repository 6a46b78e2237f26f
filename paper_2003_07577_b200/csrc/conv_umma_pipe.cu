// Dispatch over the activation bit count for the persistent pipeline kernel, and its host-side geometry check.
#include "conv_umma_pipe.cuh"

namespace ebs {

#define EBS_DECLARE_PIPE(AB)                                         \
    const ConvVariant* conv_umma_pipe_variant_a##AB(int variant);    \
    unsigned long long conv_umma_pipe_timeouts_a##AB();
EBS_DECLARE_PIPE(0) EBS_DECLARE_PIPE(1) EBS_DECLARE_PIPE(2) EBS_DECLARE_PIPE(3) EBS_DECLARE_PIPE(4)
EBS_DECLARE_PIPE(5) EBS_DECLARE_PIPE(6) EBS_DECLARE_PIPE(7) EBS_DECLARE_PIPE(8)
#undef EBS_DECLARE_PIPE

int pipe_sm_count() {
    int dev = 0, n = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    return n > 0 ? n : 148;
}

const ConvVariant* conv_umma_pipe_variant(int a_bits, int variant) {
    switch (a_bits) {
        case 0: return conv_umma_pipe_variant_a0(variant);      // activations as byte codes
        case 1: return conv_umma_pipe_variant_a1(variant);
        case 2: return conv_umma_pipe_variant_a2(variant);
        case 3: return conv_umma_pipe_variant_a3(variant);
        case 4: return conv_umma_pipe_variant_a4(variant);
        case 5: return conv_umma_pipe_variant_a5(variant);
        case 6: return conv_umma_pipe_variant_a6(variant);
        case 7: return conv_umma_pipe_variant_a7(variant);
        case 8: return conv_umma_pipe_variant_a8(variant);
        default: return nullptr;
    }
}

bool conv_umma_pipe_applies(const ConvParams& p, int variant) {
    if (variant == 3) return pipe_pair_request_ok(p) && pipe_geometry(p, 256, pipe_sm_count(), p.pipe_m_sub, true).ok;
    return variant >= 0 && variant < 3 && pipe_geometry(p, 64 << variant, pipe_sm_count(), p.pipe_m_sub).ok;
}

long long conv_umma_pipe_items(const ConvParams& p, int variant) {
    if (variant < 0 || variant >= NUM_UMMA_PIPE_VARIANTS) return -1;
    const PipeGeom g = variant == 3 ? pipe_geometry(p, 256, pipe_sm_count(), p.pipe_m_sub, true)
                                    : pipe_geometry(p, 64 << variant, pipe_sm_count(), p.pipe_m_sub);
    return g.ok ? (long long)g.n_ptiles * g.n_ctiles : -1;
}

unsigned long long conv_umma_pipe_timeouts() {
    return conv_umma_pipe_timeouts_a0() + conv_umma_pipe_timeouts_a1() + conv_umma_pipe_timeouts_a2() + conv_umma_pipe_timeouts_a3() +
           conv_umma_pipe_timeouts_a4() + conv_umma_pipe_timeouts_a5() + conv_umma_pipe_timeouts_a6() +
           conv_umma_pipe_timeouts_a7() + conv_umma_pipe_timeouts_a8();
}

}  // namespace ebs
