// Stand-alone de-quantization of int32 accumulators (the scaling back to real values that Eq. 1c
// folds into the quantizer, and the scale merge of Sec. 4.3).  Pure streaming: 4 bytes read + 4 bytes written per element.
#include "ebs_internal.cuh"

namespace ebs {

__device__ __forceinline__ float dequant_one(int a, int co, float scale, const float* __restrict__ ch_scale,
                                             const float* __restrict__ ch_bias, int relu) {
    float y = __fmul_rn((float)a, scale);
    if (ch_scale) y = __fmul_rn(y, __ldg(ch_scale + co));
    if (ch_bias) y = __fadd_rn(y, __ldg(ch_bias + co));
    if (relu && !(y > 0.0f)) y = 0.0f;
    return y;
}

// VEC = 4: c_out % 4 == 0, so a 16-byte vector never straddles a pixel and its channels are co..co+3.
template <int VEC>
__global__ void __launch_bounds__(256) dequant_kernel(const int32_t* __restrict__ acc, size_t total, int c_out,
                                                      float scale, const float* __restrict__ ch_scale,
                                                      const float* __restrict__ ch_bias, int relu,
                                                      float* __restrict__ y) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    if constexpr (VEC == 4) {
        const size_t nvec = total / 4;
        constexpr int U = 4;                                   // independent 16-byte loads in flight per thread
        for (size_t v0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x; v0 < nvec; v0 += stride * U) {
            int4 a[U];
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (v0 + u * stride < nvec) a[u] = __ldg(reinterpret_cast<const int4*>(acc) + v0 + u * stride);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const size_t v = v0 + u * stride;
                if (v < nvec) {
                    const int co = (int)((v * 4) % (size_t)c_out);
                    float4 o;
                    o.x = dequant_one(a[u].x, co, scale, ch_scale, ch_bias, relu);
                    o.y = dequant_one(a[u].y, co + 1, scale, ch_scale, ch_bias, relu);
                    o.z = dequant_one(a[u].z, co + 2, scale, ch_scale, ch_bias, relu);
                    o.w = dequant_one(a[u].w, co + 3, scale, ch_scale, ch_bias, relu);
                    reinterpret_cast<float4*>(y)[v] = o;
                }
            }
        }
    } else {
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride)
            y[i] = dequant_one(acc[i], (int)(i % (size_t)c_out), scale, ch_scale, ch_bias, relu);
    }
}

// Global average pooling of an NHWC fp32 tensor: one thread per (image, channel) adds the pixels in
// order p = 0 .. hw-1 (a fixed order, so the result is reproducible bit for bit) and multiplies by
// fl(1/hw).  Consecutive threads read consecutive channels, so every load is coalesced.
__global__ void __launch_bounds__(256) avgpool_kernel(const float* __restrict__ y, int n, int hw, int c, float inv_hw,
                                                      float* __restrict__ out) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n * c) return;
    const int img = idx / c, ch = idx - img * c;
    const float* src = y + (size_t)img * hw * c + ch;
    float acc = 0.0f;
    for (int p = 0; p < hw; ++p) acc = __fadd_rn(acc, __ldg(src + (size_t)p * c));
    out[idx] = __fmul_rn(acc, inv_hw);
}

int launch_avgpool(const float* y, int n, int hw, int c, float* out, cudaStream_t st) {
    const int total = n * c;
    avgpool_kernel<<<(total + 255) / 256, 256, 0, st>>>(y, n, hw, c, 1.0f / (float)hw, out);
    return check_cuda(cudaGetLastError());
}

int launch_dequant(const int32_t* acc, size_t n_pixels, int c_out, float scale, const float* ch_scale,
                   const float* ch_bias, int relu, float* y, cudaStream_t st) {
    const size_t total = n_pixels * (size_t)c_out;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const bool vec = (c_out % 4) == 0;
    const size_t work = vec ? total / 4 : total;
    size_t blocks = (work + 255) / 256;
    const size_t cap = (size_t)sms * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (vec) dequant_kernel<4><<<(int)blocks, 256, 0, st>>>(acc, total, c_out, scale, ch_scale, ch_bias, relu, y);
    else dequant_kernel<1><<<(int)blocks, 256, 0, st>>>(acc, total, c_out, scale, ch_scale, ch_bias, relu, y);
    return check_cuda(cudaGetLastError());
}

}  // namespace ebs
