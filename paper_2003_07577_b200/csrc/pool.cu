// Max pooling on packed bit planes (the 3x3 stride-2 pooling between the first convolution and the first block of the
// ImageNet ResNets of Sec. 5), computed in the bit-plane domain: the codes are never unpacked.
//
// A thread owns one (output pixel, 32-channel word).  The maximum of two bit-sliced numbers, 32 channels at a time: walk
// the planes from the top; `gt` collects the channels where a is already known to be larger, `eq` those still equal:
//     gt |= eq & a_j & ~b_j;   eq &= ~(a_j ^ b_j);
// and the result takes a's planes where gt is set and b's elsewhere.  Window positions outside the image are skipped
// (codes are >= 0, so this equals padding with the zero code).
#include "ebs_internal.cuh"

namespace ebs {

template <int AB>
__global__ void __launch_bounds__(256) maxpool_packed_kernel(const uint32_t* __restrict__ x, int N, int H, int W, int CW,
                                                             int k, int stride, int pad, int Ho, int Wo,
                                                             uint32_t* __restrict__ out) {
    const long long items = (long long)N * Ho * Wo * CW;
    const long long step = (long long)gridDim.x * blockDim.x;
    for (long long item = (long long)blockIdx.x * blockDim.x + threadIdx.x; item < items; item += step) {
        const int cw = (int)(item % CW);
        long long pix = item / CW;
        const int wo = (int)(pix % Wo);
        pix /= Wo;
        const int ho = (int)(pix % Ho), n = (int)(pix / Ho);
        uint32_t best[AB];
#pragma unroll
        for (int j = 0; j < AB; ++j) best[j] = 0u;
        for (int r = 0; r < k; ++r) {
            const int h = ho * stride + r - pad;
            if ((unsigned)h >= (unsigned)H) continue;
            for (int s = 0; s < k; ++s) {
                const int w = wo * stride + s - pad;
                if ((unsigned)w >= (unsigned)W) continue;
                uint32_t a[AB];
                load_words_global<AB>(x + ((((long long)n * H + h) * W + w) * CW + cw) * AB, a);
                uint32_t gt = 0u, eq = 0xFFFFFFFFu;
#pragma unroll
                for (int j = AB - 1; j >= 0; --j) {
                    gt |= eq & a[j] & ~best[j];
                    eq &= ~(a[j] ^ best[j]);
                }
#pragma unroll
                for (int j = 0; j < AB; ++j) best[j] = (gt & a[j]) | (~gt & best[j]);
            }
        }
        uint32_t* dst = out + item * AB;
#pragma unroll
        for (int j = 0; j < AB; ++j) dst[j] = best[j];
    }
}

int launch_maxpool_packed(const uint32_t* x, int n, int h, int w, int c, int bits, int k, int stride, int pad, int ho,
                          int wo, uint32_t* out, cudaStream_t st) {
    const int CW = (c + 31) / 32;
    const long long items = (long long)n * ho * wo * CW;
    long long blocks = (items + 255) / 256;
    if (blocks > 148LL * 32) blocks = 148LL * 32;
    if (blocks < 1) blocks = 1;
#define EBS_POOL_CASE(B) case B: maxpool_packed_kernel<B><<<(int)blocks, 256, 0, st>>>(x, n, h, w, CW, k, stride, pad, ho, wo, out); break;
    switch (bits) {
        EBS_POOL_CASE(1) EBS_POOL_CASE(2) EBS_POOL_CASE(3) EBS_POOL_CASE(4)
        EBS_POOL_CASE(5) EBS_POOL_CASE(6) EBS_POOL_CASE(7) EBS_POOL_CASE(8)
        default: return EBS_ERR_INVALID_ARG;
    }
#undef EBS_POOL_CASE
    return check_cuda(cudaGetLastError());
}

}  // namespace ebs
