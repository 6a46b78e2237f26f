// Quantize + bit-plane packing kernels (Eq. 1b/1c quantizer; B_x and B_w of Eq. 12/15).
//
// A warp turns 32 consecutive channels of one pixel into a_bits words with one __ballot_sync per
// plane: lane = channel, so bit (c % 32) of a plane word is that plane's bit of channel c.  The
// kernels are pure streaming (HBM-bound): 4 bytes (fp32) or 1 byte (codes) read per element,
// a_bits/8 bytes written.
#include "ebs_internal.cuh"

namespace ebs {

template <typename T>
__device__ __forceinline__ uint32_t act_code(T v, float inv_scale, int qmax);
template <>
__device__ __forceinline__ uint32_t act_code<float>(float v, float inv_scale, int qmax) {
    return (uint32_t)quantize_code(v, inv_scale, 0, qmax);
}
template <>
__device__ __forceinline__ uint32_t act_code<uint8_t>(uint8_t v, float, int qmax) {
    return (uint32_t)v & (uint32_t)qmax;
}

// NHWC input: items are (pixel, channel word); one warp per item, grid-stride.
template <typename T>
__global__ void __launch_bounds__(256) pack_acts_nhwc_kernel(const T* __restrict__ x, long long pixels, int C,
                                                             int CW, int AB, float inv_scale,
                                                             uint32_t* __restrict__ out) {
    const int lane = threadIdx.x & 31;
    const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    const long long items = pixels * CW;
    const int qmax = (1 << AB) - 1;
    for (long long item = warp0; item < items; item += nwarps) {
        const long long pix = item / CW;
        const int cw = (int)(item - pix * CW);
        const int c = cw * 32 + lane;
        uint32_t code = 0u;
        if (c < C) code = act_code<T>(x[pix * C + c], inv_scale, qmax);
        uint32_t mine = 0u;
        for (int j = 0; j < AB; ++j) {
            const uint32_t word = __ballot_sync(0xffffffffu, (code >> j) & 1u);
            if (lane == j) mine = word;
        }
        if (lane < AB) out[item * AB + lane] = mine;
    }
}

// NHWC integer codes: one thread per (pixel, 32-channel word).  The thread reads its 32 code bytes
// as 16-byte vectors and gathers plane j of four codes at a time into a nibble with one multiply
// (((x >> j) & 0x01010101) * 0x01020408) >> 24, so no cross-lane traffic is needed and a warp moves
// 1 KB per load instruction.
__global__ void __launch_bounds__(256) pack_acts_nhwc_u8_kernel(const uint8_t* __restrict__ x, long long items, int C,
                                                                int CW, int AB, uint32_t* __restrict__ out) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    const bool vec16 = (C % 16) == 0;
    for (long long item = (long long)blockIdx.x * blockDim.x + threadIdx.x; item < items; item += stride) {
        const long long pix = item / CW;
        const int cw = (int)(item - pix * CW);
        const int c0 = cw * 32;
        const int nvalid = C - c0 < 32 ? C - c0 : 32;
        const uint8_t* src = x + pix * C + c0;
        uint32_t codes[8];
        if (vec16) {
            const uint4 lo = __ldg(reinterpret_cast<const uint4*>(src));
            codes[0] = lo.x; codes[1] = lo.y; codes[2] = lo.z; codes[3] = lo.w;
            if (nvalid > 16) {
                const uint4 hi = __ldg(reinterpret_cast<const uint4*>(src) + 1);
                codes[4] = hi.x; codes[5] = hi.y; codes[6] = hi.z; codes[7] = hi.w;
            } else {
                codes[4] = codes[5] = codes[6] = codes[7] = 0u;
            }
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                uint32_t wv = 0u;
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    if (4 * k + b < nvalid) wv |= (uint32_t)__ldg(src + 4 * k + b) << (8 * b);
                codes[k] = wv;
            }
        }
        uint32_t* dst = out + item * AB;
        for (int j = 0; j < AB; ++j) {
            uint32_t word = 0u;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t t = (codes[k] >> j) & 0x01010101u;
                word |= ((t * 0x01020408u) >> 24) << (4 * k);
            }
            dst[j] = word;
        }
    }
}

// NCHW input: a CTA transposes a [32 channels][32 pixels] tile through shared memory so that
// global reads run along the contiguous pixel axis and the ballot still sees lane = channel.
template <typename T>
__global__ void __launch_bounds__(256) pack_acts_nchw_kernel(const T* __restrict__ x, int N, int C, int HW,
                                                             int CW, int AB, float inv_scale,
                                                             uint32_t* __restrict__ out) {
    __shared__ uint32_t tile[32][33];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int ptiles = (HW + 31) / 32;
    const long long tiles = (long long)N * CW * ptiles;
    const int qmax = (1 << AB) - 1;
    for (long long tix = blockIdx.x; tix < tiles; tix += gridDim.x) {
        const int pt = (int)(tix % ptiles);
        const long long rest = tix / ptiles;
        const int cw = (int)(rest % CW), n = (int)(rest / CW);
        const int p0 = pt * 32;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int cl = warp * 4 + k, c = cw * 32 + cl, pp = p0 + lane;
            uint32_t code = 0u;
            if (c < C && pp < HW) code = act_code<T>(x[((long long)n * C + c) * HW + pp], inv_scale, qmax);
            tile[cl][lane] = code;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int pl = warp * 4 + k, pp = p0 + pl;
            const uint32_t code = tile[lane][pl];
            uint32_t mine = 0u;
            for (int j = 0; j < AB; ++j) {
                const uint32_t word = __ballot_sync(0xffffffffu, (code >> j) & 1u);
                if (lane == j) mine = word;
            }
            if (pp < HW && lane < AB) out[(((long long)n * HW + pp) * CW + cw) * AB + lane] = mine;
        }
        __syncthreads();
    }
}

// Weights: one warp per (tap, channel word, output channel); tiny and off the inference path.
template <typename T>
__global__ void __launch_bounds__(256) pack_weights_kernel(const T* __restrict__ wt, int layout, int Co, int C,
                                                           int kh, int kw, int CW, int WB, float inv_scale,
                                                           uint32_t* __restrict__ out) {
    const int lane = threadIdx.x & 31;
    const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    const long long items = (long long)kh * kw * CW * Co;
    const int lo = -(1 << (WB - 1)), hi = (1 << (WB - 1)) - 1;
    for (long long item = warp0; item < items; item += nwarps) {
        const int co = (int)(item % Co);
        long long rest = item / Co;
        const int cw = (int)(rest % CW);
        rest /= CW;
        const int s = (int)(rest % kw), r = (int)(rest / kw);
        const int c = cw * 32 + lane;
        uint32_t code = 0u;
        if (c < C) {
            const long long idx = layout == EBS_NCHW ? (((long long)co * C + c) * kh + r) * kw + s
                                                     : (((long long)co * kh + r) * kw + s) * C + c;
            int q;
            if constexpr (sizeof(T) == 4) q = quantize_code((float)wt[idx], inv_scale, lo, hi);
            else q = (int)wt[idx];
            code = (uint32_t)q & ((1u << WB) - 1u);      // two's-complement bit pattern
        }
        uint32_t mine = 0u;
        for (int m = 0; m < WB; ++m) {
            const uint32_t word = __ballot_sync(0xffffffffu, (code >> m) & 1u);
            if (lane == m) mine = word;
        }
        if (lane < WB) out[item * WB + lane] = mine;
    }
}

static int grid_for(long long warps_needed, int sm_count) {
    long long blocks = (warps_needed + 7) / 8;
    const long long cap = (long long)sm_count * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

static int sm_count() {
    int dev = 0, n = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    return n > 0 ? n : 148;
}

int launch_pack_acts(const void* x, int dtype, int layout, int n, int c, int h, int w, int a_bits,
                     float inv_scale, uint32_t* out, cudaStream_t st) {
    const int CW = (c + 31) / 32;
    const long long pixels = (long long)n * h * w;
    const int sms = sm_count();
    if (layout == EBS_NHWC) {
        const int grid = grid_for(pixels * CW, sms);
        if (dtype == EBS_F32)
            pack_acts_nhwc_kernel<float><<<grid, 256, 0, st>>>((const float*)x, pixels, c, CW, a_bits, inv_scale, out);
        else {
            const long long items = pixels * CW;
            long long blocks = (items + 255) / 256;
            if (blocks > (long long)sms * 32) blocks = (long long)sms * 32;
            pack_acts_nhwc_u8_kernel<<<(int)blocks, 256, 0, st>>>((const uint8_t*)x, items, c, CW, a_bits, out);
        }
    } else {
        const long long tiles = (long long)n * CW * ((h * w + 31) / 32);
        long long grid = tiles < (long long)sms * 16 ? tiles : (long long)sms * 16;
        if (grid < 1) grid = 1;
        if (dtype == EBS_F32)
            pack_acts_nchw_kernel<float><<<(int)grid, 256, 0, st>>>((const float*)x, n, c, h * w, CW, a_bits, inv_scale, out);
        else
            pack_acts_nchw_kernel<uint8_t><<<(int)grid, 256, 0, st>>>((const uint8_t*)x, n, c, h * w, CW, a_bits, inv_scale, out);
    }
    return check_cuda(cudaGetLastError());
}

int launch_pack_weights(const void* wt, int dtype, int layout, const ebs_conv_desc& d, float inv_scale,
                        uint32_t* out, cudaStream_t st) {
    const int CW = (d.c_in + 31) / 32;
    const long long items = (long long)d.kh * d.kw * CW * d.c_out;
    const int grid = grid_for(items, sm_count());
    if (dtype == EBS_F32)
        pack_weights_kernel<float><<<grid, 256, 0, st>>>((const float*)wt, layout, d.c_out, d.c_in, d.kh, d.kw, CW,
                                                         d.w_bits, inv_scale, out);
    else
        pack_weights_kernel<int8_t><<<grid, 256, 0, st>>>((const int8_t*)wt, layout, d.c_out, d.c_in, d.kh, d.kw, CW,
                                                          d.w_bits, inv_scale, out);
    return check_cuda(cudaGetLastError());
}

}  // namespace ebs
