// Quantize + bit-plane packing kernels (Eq. 1b/1c quantizer; B_x and B_w of Eq. 12/15).
//
// The activation kernels give one thread the 32 codes of a (pixel, 32-channel word), four code bytes
// to a register, and gather plane j of four codes into a nibble with one multiply; bit (c % 32) of a
// plane word is that plane's bit of channel c.  They are pure streaming (HBM-bound): 4 bytes (fp32)
// or 1 byte (codes) read per element, a_bits/8 bytes written.  The weight kernel (off the inference
// path) uses one warp per word and a __ballot_sync per plane.
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

__device__ __forceinline__ void store_planes(const uint32_t (&codes)[8], int AB, uint32_t* __restrict__ dst);

// Four activation codes as the bytes of one word (byte i = code of v_i), identical to quantize_code on each value but
// without the float -> int conversion, which issues at an eighth of the fp32 rate: t = fl(fl(v * inv) + 0.5) as two
// individually rounded operations; max(t, 0) (the maximum-number operation: a NaN gives 0, like quantize_code);
// floor(t) is then in the low mantissa bits of t + 2^23 added with rounding toward minus infinity, and the clamp at
// qmax is an integer minimum of the sum's bit pattern with bits(2^23) + qmax; the low bytes are the codes.
__device__ __forceinline__ uint32_t act_codes4(float v0, float v1, float v2, float v3, float inv_scale, int qmax) {
    const int m_hi = 0x4B000000 + qmax;
    auto pat = [&](float v) {
        const float t = fmaxf(__fadd_rn(__fmul_rn(v, inv_scale), 0.5f), 0.0f);
        return (uint32_t)min(__float_as_int(__fadd_rd(t, 8388608.0f)), m_hi);
    };
    return __byte_perm(__byte_perm(pat(v0), pat(v1), 0x0040), __byte_perm(pat(v2), pat(v3), 0x0040), 0x5410);
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
        store_planes(codes, AB, out + item * AB);
    }
}

// Plane words of 32 codes held as eight words of four code bytes each (word k = channels 4k .. 4k+3).
// The codes are first regrouped with byte permutes into registers c[bb] = channels {bb, 8 + bb, 16 + bb, 24 + bb}
// (byte i = channel 8i + bb, the spacing the plane words have); with each register rotated left by bb, plane j is then
// rotr(OR_bb c[bb] & (0x01010101 << ((bb + j) & 7)), j): one masked merge per register and plane instead of a
// shift, mask, multiply, shift and merge per four codes.
__device__ __forceinline__ void store_planes(const uint32_t (&codes)[8], int AB, uint32_t* __restrict__ dst) {
    uint32_t c[8];
#pragma unroll
    for (int bb = 0; bb < 8; ++bb) {
        const uint32_t sel = 0x0040u + 0x11u * (uint32_t)(bb & 3);                      // byte (bb & 3) of both operands
        const uint32_t lo = __byte_perm(codes[bb >> 2], codes[2 + (bb >> 2)], sel);
        const uint32_t hi = __byte_perm(codes[4 + (bb >> 2)], codes[6 + (bb >> 2)], sel);
        const uint32_t g = __byte_perm(lo, hi, 0x5410);
        c[bb] = __funnelshift_l(g, g, bb);
    }
    uint32_t w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        uint32_t word = 0u;
        if (j < AB) {
            uint32_t t = c[0] & (0x01010101u << j);
#pragma unroll
            for (int bb = 1; bb < 8; ++bb) t |= c[bb] & (0x01010101u << ((bb + j) & 7));
            word = __funnelshift_r(t, t, j);
        }
        w[j] = word;
    }
    if (AB == 4) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
    else if (AB == 8) {
        *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(dst + 4) = make_uint4(w[4], w[5], w[6], w[7]);
    } else if (AB == 2) *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
    else {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (j < AB) dst[j] = w[j];
    }
}

// NHWC, channels a multiple of 32: a warp takes 32 consecutive (pixel, 32-channel word) items, i.e.
// 1024 consecutive values.  Loads are fully coalesced (lane l reads 16-byte chunk i*32+l of the run),
// each chunk is quantized (fp32) and reduced to one word of four code bytes, the words are regrouped
// through shared memory so that lane l holds the eight code words of item l, and the lane builds the
// plane words with the multiply-gather.
__global__ void __launch_bounds__(256) pack_acts_nhwc_f32_coalesced_kernel(const float* __restrict__ x, long long items, int AB,
                                                                       float inv_scale, uint32_t* __restrict__ out) {
    __shared__ uint32_t regroup[8][32][9];                    // [warp][item][code word], padded
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    const int qmax = (1 << AB) - 1;
    const long long groups = (items + 31) / 32;
    for (long long grp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; grp < groups; grp += nwarps) {
        const long long item0 = grp * 32;
        const long long left = items - item0;
        const int nitems = left < 32 ? (int)left : 32;
        {
            const float4* src = reinterpret_cast<const float4*>(x + item0 * 32);
            float4 v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int chunk = i * 32 + lane;                  // 16-byte chunk of the run: item chunk/8, word chunk%8
                v[i] = (chunk >> 3) < nitems ? __ldg(src + chunk) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int chunk = i * 32 + lane;
                regroup[warp][chunk >> 3][chunk & 7] = act_codes4(v[i].x, v[i].y, v[i].z, v[i].w, inv_scale, qmax);
            }
        }
        __syncwarp();
        if (lane < nitems) {
            uint32_t codes[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) codes[k] = regroup[warp][lane][k];
            store_planes(codes, AB, out + (item0 + lane) * AB);
        }
        __syncwarp();
    }
}

// Integer codes, channels a multiple of 32, 32-byte aligned tensor: a thread reads the 32 code bytes of its items with one
// 256-bit load each (a warp instruction reads 1 KB of consecutive memory: no regrouping through shared memory is needed)
// and builds the plane words.  UNROLL items per thread are loaded before any is used.
template <int UNROLL>
__global__ void __launch_bounds__(256) pack_acts_nhwc_u8_v8_kernel(const uint8_t* __restrict__ x, long long items, int AB,
                                                                   uint32_t* __restrict__ out) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long item0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; item0 < items; item0 += stride * UNROLL) {
        uint32_t codes[UNROLL][8];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long item = item0 + u * stride;
            if (item < items) {
                asm volatile("ld.global.nc.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                             : "=r"(codes[u][0]), "=r"(codes[u][1]), "=r"(codes[u][2]), "=r"(codes[u][3]), "=r"(codes[u][4]),
                               "=r"(codes[u][5]), "=r"(codes[u][6]), "=r"(codes[u][7])
                             : "l"(x + item * 32));
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long item = item0 + u * stride;
            if (item < items) store_planes(codes[u], AB, out + item * AB);
        }
    }
}

// Same for integer codes; a warp takes 128 items (4 KB) per iteration so that enough loads are in flight.
__global__ void __launch_bounds__(256) pack_acts_nhwc_u8_coalesced_kernel(const uint8_t* __restrict__ x, long long items,
                                                                          int AB, uint32_t* __restrict__ out) {
    constexpr int G = 4;                                       // groups of 32 items per warp iteration
    __shared__ uint32_t regroup[8][G * 32][9];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    const long long groups = (items + G * 32 - 1) / (G * 32);
    for (long long grp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; grp < groups; grp += nwarps) {
        const long long item0 = grp * (G * 32);
        const long long left = items - item0;
        const int nitems = left < G * 32 ? (int)left : G * 32;
        const uint4* src = reinterpret_cast<const uint4*>(x + item0 * 32);
        uint4 v[2 * G];
#pragma unroll
        for (int i = 0; i < 2 * G; ++i) {
            const int chunk = i * 32 + lane;                      // 16-byte chunk: item chunk/2, code words 4*(chunk%2)..
            v[i] = (chunk >> 1) < nitems ? __ldg(src + chunk) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int i = 0; i < 2 * G; ++i) {
            const int chunk = i * 32 + lane;
            uint32_t* dst = &regroup[warp][chunk >> 1][(chunk & 1) * 4];
            dst[0] = v[i].x; dst[1] = v[i].y; dst[2] = v[i].z; dst[3] = v[i].w;
        }
        __syncwarp();
#pragma unroll
        for (int gq = 0; gq < G; ++gq) {
            const int it = gq * 32 + lane;
            if (it < nitems) {
                uint32_t codes[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) codes[k] = regroup[warp][it][k];
                store_planes(codes, AB, out + (item0 + it) * AB);
            }
        }
        __syncwarp();
    }
}

// NHWC fp32, any channel count: one thread per (pixel, 32-channel word).
__global__ void __launch_bounds__(256) pack_acts_nhwc_f32_kernel(const float* __restrict__ x, long long items, int C,
                                                                 int CW, int AB, float inv_scale,
                                                                 uint32_t* __restrict__ out) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    const int qmax = (1 << AB) - 1;
    const bool vec = (C % 4) == 0;
    for (long long item = (long long)blockIdx.x * blockDim.x + threadIdx.x; item < items; item += stride) {
        const long long pix = item / CW;
        const int cw = (int)(item - pix * CW);
        const int c0 = cw * 32;
        const int nvalid = C - c0 < 32 ? C - c0 : 32;
        const float* src = x + pix * C + c0;
        uint32_t codes[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            uint32_t wv = 0u;
            if (vec) {
                if (4 * k < nvalid) {
                    const float4 v = __ldg(reinterpret_cast<const float4*>(src) + k);
                    wv = act_codes4(v.x, v.y, v.z, v.w, inv_scale, qmax);
                }
            } else {
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    if (4 * k + b < nvalid)
                        wv |= (uint32_t)quantize_act_code(__ldg(src + 4 * k + b), inv_scale, qmax) << (8 * b);
            }
            codes[k] = wv;
        }
        store_planes(codes, AB, out + item * AB);
    }
}

// NCHW input (fp32 or codes): a CTA takes 32 channels x 128 pixels; global reads run along the
// contiguous pixel axis, the codes are transposed through shared memory (one byte each), then one
// thread per pixel gathers its 32 codes and builds the plane words.
template <typename T>
__global__ void __launch_bounds__(128) pack_acts_nchw_kernel(const T* __restrict__ x, int N, int C, int HW,
                                                             int CW, int AB, float inv_scale,
                                                             uint32_t* __restrict__ out) {
    constexpr int PT = 128, ROWB = 36;                       // pixels per tile; bytes per pixel row (32 codes + pad)
    __shared__ __align__(16) uint8_t tile[PT * ROWB];
    const int ptiles = (HW + PT - 1) / PT;
    const long long tiles = (long long)N * CW * ptiles;
    const int qmax = (1 << AB) - 1;
    for (long long tix = blockIdx.x; tix < tiles; tix += gridDim.x) {
        const int pt = (int)(tix % ptiles);
        const long long rest = tix / ptiles;
        const int cw = (int)(rest % CW), n = (int)(rest / CW);
        const int p0 = pt * PT;
        for (int e = threadIdx.x; e < 32 * PT; e += 128) {   // e -> (channel, pixel): consecutive threads, consecutive pixels
            const int cl = e / PT, pl = e - cl * PT;
            const int c = cw * 32 + cl, pp = p0 + pl;
            uint32_t code = 0u;
            if (c < C && pp < HW) code = act_code<T>(x[((long long)n * C + c) * HW + pp], inv_scale, qmax);
            tile[pl * ROWB + cl] = (uint8_t)code;
        }
        __syncthreads();
        const int pp = p0 + threadIdx.x;
        if (pp < HW) {
            const uint32_t* row = reinterpret_cast<const uint32_t*>(tile + threadIdx.x * ROWB);
            uint32_t codes[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) codes[k] = row[k];
            store_planes(codes, AB, out + (((long long)n * HW + pp) * CW + cw) * AB);
        }
        __syncthreads();
    }
}

// NCHW fp32 with a pixel count that is a multiple of four: a CTA of 256 threads takes 32 channels x 256 pixels.  Every
// thread issues its eight 16-byte loads (four pixels of one channel each, consecutive threads consecutive pixel quads, so
// a warp reads 512 contiguous bytes of a channel row) before it uses any of them, quantizes four channels of a pixel
// into one word of a pixel-major tile in shared memory; one thread per pixel then builds the plane words.
__global__ void __launch_bounds__(256) pack_acts_nchw_f32_vec_kernel(const float* __restrict__ x, int N, int C, int HW,
                                                                     int CW, int AB, float inv_scale,
                                                                     uint32_t* __restrict__ out) {
    // A thread takes 4 consecutive pixels of 8 channels: the two groups of four consecutive channels 4 cg .. 4 cg + 3
    // and 16 + 4 cg ..  Per pixel and group its four codes are one word of the pixel's row of eight code words; the row of
    // pixel 4 quad + j sits at word 9 quad + 584 j, which makes both the stores (lanes along quad, stride 9 words) and
    // the row reads (lanes along pixels: 9 (t / 4) + 584 (t % 4), and 584 = 8 mod 32) free of bank conflicts.
    constexpr int PT = 256, QP = 9, JP = 584;                // pixels per tile; word pitch along quad and along j
    __shared__ __align__(16) uint32_t tile[4 * JP];
    const int ptiles = (HW + PT - 1) / PT;
    const long long tiles = (long long)N * CW * ptiles;
    const int qmax = (1 << AB) - 1;
    const int quad = threadIdx.x & 63, cg = threadIdx.x >> 6;            // pixel quad 0..63, channel group 0..3
    for (long long tix = blockIdx.x; tix < tiles; tix += gridDim.x) {
        const int pt = (int)(tix % ptiles);
        const long long rest = tix / ptiles;
        const int cw = (int)(rest % CW), n = (int)(rest / CW);
        const int p0 = pt * PT, pp4 = p0 + 4 * quad;
        float4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int c = cw * 32 + (i >> 2) * 16 + 4 * cg + (i & 3);
            v[i] = (c < C && pp4 < HW) ? __ldg(reinterpret_cast<const float4*>(x + ((long long)n * C + c) * HW + pp4))
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int gq = 0; gq < 2; ++gq) {
            uint32_t* dst = tile + quad * QP + gq * 4 + cg;
            dst[0] = act_codes4(v[4 * gq].x, v[4 * gq + 1].x, v[4 * gq + 2].x, v[4 * gq + 3].x, inv_scale, qmax);
            dst[JP] = act_codes4(v[4 * gq].y, v[4 * gq + 1].y, v[4 * gq + 2].y, v[4 * gq + 3].y, inv_scale, qmax);
            dst[2 * JP] = act_codes4(v[4 * gq].z, v[4 * gq + 1].z, v[4 * gq + 2].z, v[4 * gq + 3].z, inv_scale, qmax);
            dst[3 * JP] = act_codes4(v[4 * gq].w, v[4 * gq + 1].w, v[4 * gq + 2].w, v[4 * gq + 3].w, inv_scale, qmax);
        }
        __syncthreads();
        const int pp = p0 + threadIdx.x;
        if (pp < HW) {
            const uint32_t* row = tile + (threadIdx.x >> 2) * QP + (threadIdx.x & 3) * JP;
            uint32_t codes[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) codes[k] = row[k];
            store_planes(codes, AB, out + (((long long)n * HW + pp) * CW + cw) * AB);
        }
        __syncthreads();
    }
}

// Space-to-depth packing for a stride-2 first layer with few channels (u8 NHWC codes, 4 * C <= 32): output pixel (i, j)
// of the [N][Hs][Ws] tensor holds the 2 x 2 block of input pixels (2i - off + dy, 2j - off + dx), channel slot
// (2 dy + dx) * C + c, zero outside the image; off = 1 shifts the blocks by one pixel so that an odd padding of the
// original convolution becomes a whole number of blocks.  A k x k stride-2 convolution over the image is then a
// ceil(k/2) x ceil(k/2) stride-1 convolution over this tensor with the weights regrouped the same way: its reduction
// words are a quarter as many and four times as full.  One thread per output pixel.
__global__ void __launch_bounds__(256) pack_acts_s2d_u8_kernel(const uint8_t* __restrict__ x, int N, int C, int H, int W, int Hs,
                                                               int Ws, int off, int AB, uint32_t* __restrict__ out) {
    const long long total = (long long)N * Hs * Ws;
    const long long stride = (long long)gridDim.x * blockDim.x;
    const uint32_t code_mask = (1u << AB) - 1u;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += stride) {
        const int j = (int)(t % Ws);
        const long long r = t / Ws;
        const int i = (int)(r % Hs), n = (int)(r / Hs);
        uint32_t codes[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
        for (int dy = 0; dy < 2; ++dy) {
            const int h = 2 * i - off + dy;
            if ((unsigned)h >= (unsigned)H) continue;
#pragma unroll
            for (int dx = 0; dx < 2; ++dx) {
                const int w = 2 * j - off + dx;
                if ((unsigned)w >= (unsigned)W) continue;
                const uint8_t* src = x + (((long long)n * H + h) * W + w) * C;
                for (int c = 0; c < C; ++c) {
                    const int slot = (2 * dy + dx) * C + c;
                    codes[slot >> 2] |= ((uint32_t)__ldg(src + c) & code_mask) << (8 * (slot & 3));
                }
            }
        }
        store_planes(codes, AB, out + t * AB);
    }
}

// Weights: one warp per (tap, channel word, output channel); tiny and off the inference path.
template <typename T>
__global__ void __launch_bounds__(256) pack_weights_kernel(const T* __restrict__ wt, int layout, int Co, int C,
                                                           int kh, int kw, int CW, int WB, float inv_scale,
                                                           int w_levels, uint32_t* __restrict__ out) {
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
            if constexpr (sizeof(T) == 4)
                q = w_levels ? quantize_weight_level((float)wt[idx], inv_scale, WB) : quantize_code((float)wt[idx], inv_scale, lo, hi);
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

int launch_pack_acts_s2d(const void* x, int n, int c, int h, int w, int off, int a_bits, uint32_t* out, cudaStream_t st) {
    const int Hs = (h + off) / 2 + off, Ws = (w + off) / 2 + off;
    const long long total = (long long)n * Hs * Ws;
    long long blocks = (total + 255) / 256;
    const long long cap = (long long)sm_count() * 32;
    if (blocks > cap) blocks = cap;
    pack_acts_s2d_u8_kernel<<<(int)blocks, 256, 0, st>>>((const uint8_t*)x, n, c, h, w, Hs, Ws, off, a_bits, out);
    return check_cuda(cudaGetLastError());
}


int launch_pack_acts(const void* x, int dtype, int layout, int n, int c, int h, int w, int a_bits,
                     float inv_scale, uint32_t* out, cudaStream_t st) {
    const int CW = (c + 31) / 32;
    const long long pixels = (long long)n * h * w;
    const int sms = sm_count();
    if (layout == EBS_NHWC) {
        const int grid = grid_for(pixels * CW, sms);
        const long long items = pixels * CW;
        long long blocks = (items + 255) / 256;
        if (blocks > (long long)sms * 32) blocks = (long long)sms * 32;
        (void)grid;
        if (c % 32 == 0 && (dtype == EBS_F32 || items >= (1LL << 20))) {   // full, aligned runs of 32 values; small
                                                                             // code tensors are latency-bound and
                                                                             // do better with a thread per word
            long long wblocks = ((items + 31) / 32 + 7) / 8;
            if (wblocks > (long long)sms * 32) wblocks = (long long)sms * 32;
            if (dtype == EBS_F32)
                pack_acts_nhwc_f32_coalesced_kernel<<<(int)wblocks, 256, 0, st>>>((const float*)x, items, a_bits, inv_scale, out);
            else if ((reinterpret_cast<uintptr_t>(x) & 31u) == 0) {
                long long vblocks = (items + 256 * 4 - 1) / (256 * 4);
                if (vblocks > (long long)sms * 16) vblocks = (long long)sms * 16;
                pack_acts_nhwc_u8_v8_kernel<4><<<(int)vblocks, 256, 0, st>>>((const uint8_t*)x, items, a_bits, out);
            } else {
                long long ublocks = ((items + 127) / 128 + 7) / 8;
                if (ublocks > (long long)sms * 16) ublocks = (long long)sms * 16;
                pack_acts_nhwc_u8_coalesced_kernel<<<(int)ublocks, 256, 0, st>>>((const uint8_t*)x, items, a_bits, out);
            }
        } else if (dtype == EBS_F32)
            pack_acts_nhwc_f32_kernel<<<(int)blocks, 256, 0, st>>>((const float*)x, items, c, CW, a_bits, inv_scale, out);
        else
            pack_acts_nhwc_u8_kernel<<<(int)blocks, 256, 0, st>>>((const uint8_t*)x, items, c, CW, a_bits, out);
    } else {
        const long long tiles = (long long)n * CW * ((h * w + 127) / 128);
        long long grid = tiles < (long long)sms * 16 ? tiles : (long long)sms * 16;
        if (grid < 1) grid = 1;
        if (dtype == EBS_F32 && (h * w) % 4 == 0) {
            const long long vtiles = (long long)n * CW * ((h * w + 255) / 256);
            long long vgrid = vtiles < (long long)sms * 16 ? vtiles : (long long)sms * 16;
            pack_acts_nchw_f32_vec_kernel<<<(int)vgrid, 256, 0, st>>>((const float*)x, n, c, h * w, CW, a_bits, inv_scale, out);
        } else if (dtype == EBS_F32)
            pack_acts_nchw_kernel<float><<<(int)grid, 128, 0, st>>>((const float*)x, n, c, h * w, CW, a_bits, inv_scale, out);
        else
            pack_acts_nchw_kernel<uint8_t><<<(int)grid, 128, 0, st>>>((const uint8_t*)x, n, c, h * w, CW, a_bits, inv_scale, out);
    }
    return check_cuda(cudaGetLastError());
}

// Byte image of the packed weights for the tcgen05 strip kernel: per reduction word kk = tap * CW + cw
// and output channel co one 32-byte row of two's-complement codes (the planes merged, top plane as sign
// extension), laid out [kk][Co16][32] with Co16 = c_out rounded up to 16.  Byte 4b + i of a row is
// channel 8i + b of the word and the two 16-byte halves of row co are swapped when (co >> 2) & 1: the
// order and the 32-byte swizzle the kernel's shared-memory operand tiles use, so that a tile is one
// contiguous copy.  Rows co >= c_out are zero.
__global__ void __launch_bounds__(256) weight_byte_image_kernel(const uint32_t* __restrict__ planes, long long rows,
                                                                int Co, int Co16, int WB, uint4* __restrict__ out) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x; r < rows; r += stride) {
        const long long kk = r / Co16;
        const int co = (int)(r - kk * Co16);
        uint32_t reg[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
        if (co < Co) {
            const uint32_t* src = planes + ((size_t)kk * Co + co) * WB;
            for (int m = 0; m < WB; ++m) {
                const uint32_t w = __ldg(src + m);
                const uint32_t mask = 0x01010101u << m;
                const uint32_t scale = (m == WB - 1 && WB < 8) ? ((1u << (9 - WB)) - 1u) : 1u;
#pragma unroll
                for (int b = 0; b < 8; ++b) reg[b] |= (__funnelshift_r(w, w, b - m) & mask) * scale;
            }
        }
        const int sw = (co >> 2) & 1;
        out[r * 2 + sw] = make_uint4(reg[0], reg[1], reg[2], reg[3]);
        out[r * 2 + (sw ^ 1)] = make_uint4(reg[4], reg[5], reg[6], reg[7]);
    }
}

size_t packed_weight_plane_bytes(const ebs_conv_desc& d) {
    const size_t raw = (size_t)d.kh * d.kw * ((d.c_in + 31) / 32) * d.c_out * d.w_bits * sizeof(uint32_t);
    return (raw + 255) & ~(size_t)255;
}
size_t packed_weight_image_bytes(const ebs_conv_desc& d) {
    const size_t co16 = ((size_t)d.c_out + 15) & ~(size_t)15;
    return (size_t)d.kh * d.kw * ((d.c_in + 31) / 32) * co16 * 32;
}

int launch_pack_weights(const void* wt, int dtype, int layout, const ebs_conv_desc& d, float inv_scale,
                        uint32_t* out, cudaStream_t st) {
    const int CW = (d.c_in + 31) / 32;
    const long long items = (long long)d.kh * d.kw * CW * d.c_out;
    const int grid = grid_for(items, sm_count());
    if (dtype == EBS_F32)
        pack_weights_kernel<float><<<grid, 256, 0, st>>>((const float*)wt, layout, d.c_out, d.c_in, d.kh, d.kw, CW,
                                                         d.w_bits, inv_scale, d.w_levels, out);
    else
        pack_weights_kernel<int8_t><<<grid, 256, 0, st>>>((const int8_t*)wt, layout, d.c_out, d.c_in, d.kh, d.kw, CW,
                                                          d.w_bits, inv_scale, d.w_levels, out);
    if (check_cuda(cudaGetLastError())) return EBS_ERR_CUDA;
    // second part of the buffer: the byte image, built from the plane words just written
    const int Co16 = (d.c_out + 15) & ~15;
    const long long rows = (long long)d.kh * d.kw * CW * Co16;
    uint4* image = reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(out) + packed_weight_plane_bytes(d));
    weight_byte_image_kernel<<<grid_for(rows, sm_count()), 256, 0, st>>>(out, rows, d.c_out, Co16, d.w_bits, image);
    return check_cuda(cudaGetLastError());
}

}  // namespace ebs
