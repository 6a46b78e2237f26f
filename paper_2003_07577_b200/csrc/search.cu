// Search-stage forward of the bitwidth search (Eq. 6-7): the meta tensor is quantized at every
// candidate bitwidth and the results are blended with the given coefficients, in one pass.
// Element-wise and HBM-bound: 4 bytes in, 4 bytes out per value, candidates looped in registers.
#include "ebs_internal.cuh"

namespace ebs {

struct SearchParams {
    float coeff[EBS_MAX_CANDIDATES];   // blend coefficients (softmax of the strengths, or Gumbel-softmax)
    float levels[EBS_MAX_CANDIDATES];  // 2^b - 1 as float
    float inv_levels[EBS_MAX_CANDIDATES];  // fl32(1 / (2^b - 1))
    float w_gain[EBS_MAX_CANDIDATES];  // weights: fl32(2 coeff / (2^b - 1)), the weight of one code step in the blend
    float w_offset;                    // weights: -sum of the coefficients
    int n_cand;
};

// quantize_b of Eq. 1c on a value in [0, 1]: round half up to one of 2^b integer codes, scaled by 1/(2^b - 1).
__device__ __forceinline__ float quantize_unit(float u, float levels, float inv_levels) {
    // u is in [0, 1] up to one rounding, so the code is in 0 .. 2^b - 1 without a clamp (b <= 16)
    const float code = floorf(__fadd_rn(__fmul_rn(u, levels), 0.5f));
    return __fmul_rn(inv_levels, code);
}

// max |w| over the tensor as raw float bits (non-negative floats order like unsigned integers)
__global__ void __launch_bounds__(256) abs_max_kernel(const float* __restrict__ w, size_t n, unsigned* __restrict__ out) {
    float m = 0.0f;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t n4 = n / 4;
    const float4* w4 = reinterpret_cast<const float4*>(w);
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n4; i += 4 * stride) {                 // four independent 16-byte loads in flight per thread
        const float4 a = __ldg(w4 + i), b = __ldg(w4 + i + stride), c = __ldg(w4 + i + 2 * stride), d = __ldg(w4 + i + 3 * stride);
        const float ma = fmaxf(fmaxf(fabsf(a.x), fabsf(a.y)), fmaxf(fabsf(a.z), fabsf(a.w)));
        const float mb = fmaxf(fmaxf(fabsf(b.x), fabsf(b.y)), fmaxf(fabsf(b.z), fabsf(b.w)));
        const float mc = fmaxf(fmaxf(fabsf(c.x), fabsf(c.y)), fmaxf(fabsf(c.z), fabsf(c.w)));
        const float md = fmaxf(fmaxf(fabsf(d.x), fabsf(d.y)), fmaxf(fabsf(d.z), fabsf(d.w)));
        m = fmaxf(m, fmaxf(fmaxf(ma, mb), fmaxf(mc, md)));
    }
    for (; i < n4; i += stride) {
        const float4 v = __ldg(w4 + i);
        m = fmaxf(fmaxf(fmaxf(m, fabsf(v.x)), fmaxf(fabsf(v.y), fabsf(v.z))), fabsf(v.w));
    }
    for (size_t t = n4 * 4 + (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < n; t += stride) m = fmaxf(m, fabsf(__ldg(w + t)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0 && m > 0.0f) atomicMax(out, __float_as_uint(m));
}

// tanh(w) = sign(w) (1 - 2 / (exp(2|w|) + 1)) with the hardware exponential and reciprocal: absolute error below 3e-7
// (the cancellation for small |w| costs relative, not absolute accuracy, and the blend needs the latter); tanhf spends
// twice the instructions on a relative bound.
__device__ __forceinline__ float tanh_fast(float w) {
    const float e = __expf(2.0f * fabsf(w));                   // +inf for large |w|: 2 / inf = 0, tanh = 1
    return copysignf(1.0f - __fdividef(2.0f, e + 1.0f), w);
}

// Eq. 1a per candidate, blended (Eq. 6): w_hat = sum_i coeff_i * (2 * quantize_b_i(tanh(w) / (2 max|tanh|) + 1/2) - 1),
// evaluated as sum_i (2 coeff_i / L_i) * code_i - sum_i coeff_i with code_i = floor(L_i u + 1/2): a multiply-add, a
// floor and a multiply-add per candidate.  The floor is taken on the fp32 pipe (u L + 1/2 is in [0.5, 2^16), so adding
// 2^23 with rounding toward -inf leaves it in the low mantissa bits): the conversion pipe, which tanhf already loads
// with an exponential and a reciprocal, retires 16 results per clock and SM and bounded this kernel.
template <int NC>
__device__ __forceinline__ float blend_weight(float w, float inv_2max, const SearchParams& sp) {
    const float u = fmaf(tanh_fast(w), inv_2max, 0.5f);
    float acc = sp.w_offset;
#pragma unroll
    for (int i = 0; i < NC; ++i) {
        const float code = __fadd_rn(__fadd_rd(fmaf(u, sp.levels[i], 0.5f), 8388608.0f), -8388608.0f);
        acc = fmaf(sp.w_gain[i], code, acc);
    }
    return acc;
}

// Eq. 1b per candidate, blended (Eq. 7): x_hat = alpha * sum_j coeff_j * quantize_b_j(clip(x, 0, alpha) * (1/alpha))
template <int NC>
__device__ __forceinline__ float blend_act(float x, float alpha, float inv_alpha, const SearchParams& sp) {
    const float u = __fmul_rn(fminf(fmaxf(x, 0.0f), alpha), inv_alpha);
    float acc = 0.0f;
#pragma unroll
    for (int j = 0; j < NC; ++j) acc = __fadd_rn(acc, __fmul_rn(sp.coeff[j], quantize_unit(u, sp.levels[j], sp.inv_levels[j])));
    return __fmul_rn(alpha, acc);
}

template <bool WEIGHTS, int NC>
__global__ void __launch_bounds__(256) search_forward_kernel(const float* __restrict__ src, size_t n, float alpha,
                                                             const unsigned* __restrict__ abs_max_bits,
                                                             const SearchParams sp, float* __restrict__ dst) {
    float k = 1.0f / alpha;                      // fl32(1 / alpha), one rounded division
    if (WEIGHTS) {                               // 1 / (2 max|tanh(w)|); tanh is monotonic, so max|tanh(w)| = tanh(max|w|)
        const float mt = tanh_fast(__uint_as_float(__ldg(abs_max_bits)));   // the same tanh as the elements: u <= 1
        k = mt > 0.0f ? __fdiv_rn(1.0f, __fmul_rn(2.0f, mt)) : 0.0f;
    }
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t n4 = n / 4;
    const float4* s4 = reinterpret_cast<const float4*>(src);
    float4* d4 = reinterpret_cast<float4*>(dst);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        const float4 v = __ldg(s4 + i);
        float4 o;
        if (WEIGHTS) { o.x = blend_weight<NC>(v.x, k, sp); o.y = blend_weight<NC>(v.y, k, sp); o.z = blend_weight<NC>(v.z, k, sp); o.w = blend_weight<NC>(v.w, k, sp); }
        else { o.x = blend_act<NC>(v.x, alpha, k, sp); o.y = blend_act<NC>(v.y, alpha, k, sp); o.z = blend_act<NC>(v.z, alpha, k, sp); o.w = blend_act<NC>(v.w, alpha, k, sp); }
        d4[i] = o;
    }
    for (size_t i = n4 * 4 + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        dst[i] = WEIGHTS ? blend_weight<NC>(__ldg(src + i), k, sp) : blend_act<NC>(__ldg(src + i), alpha, k, sp);
}

static int sm_count() {
    int dev = 0, n = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    return n > 0 ? n : 148;
}

template <bool WEIGHTS>
static void launch_forward(int n_cand, int grid, cudaStream_t st, const float* src, size_t n, float alpha, const unsigned* mx,
                           const SearchParams& sp, float* dst) {
    switch (n_cand) {
#define EBS_SEARCH_CASE(NC) case NC: search_forward_kernel<WEIGHTS, NC><<<grid, 256, 0, st>>>(src, n, alpha, mx, sp, dst); break;
        EBS_SEARCH_CASE(1) EBS_SEARCH_CASE(2) EBS_SEARCH_CASE(3) EBS_SEARCH_CASE(4)
        EBS_SEARCH_CASE(5) EBS_SEARCH_CASE(6) EBS_SEARCH_CASE(7) EBS_SEARCH_CASE(8)
#undef EBS_SEARCH_CASE
        default: break;
    }
}

static int fill_params(SearchParams& sp, const int* bits, const float* coeff, int n_cand) {
    if (!bits || !coeff || n_cand < 1 || n_cand > EBS_MAX_CANDIDATES) return EBS_ERR_INVALID_ARG;
    sp.n_cand = n_cand;
    for (int i = 0; i < n_cand; ++i) {
        if (bits[i] < 1 || bits[i] > 16 || !(coeff[i] == coeff[i])) return EBS_ERR_INVALID_ARG;
        sp.coeff[i] = coeff[i];
        sp.levels[i] = (float)((1 << bits[i]) - 1);
        sp.inv_levels[i] = 1.0f / sp.levels[i];
        sp.w_gain[i] = (float)(2.0 * (double)coeff[i] / (double)sp.levels[i]);
    }
    double csum = 0.0;
    for (int i = 0; i < n_cand; ++i) csum += (double)coeff[i];
    sp.w_offset = (float)-csum;
    return EBS_OK;
}

static int grid_size(size_t n) {
    const size_t want = (n / 4 + 255) / 256 + 1;
    const size_t cap = (size_t)sm_count() * 16;
    return (int)(want < cap ? want : cap);
}

int launch_search_weights(const float* w, size_t n, const int* bits, const float* coeff, int n_cand, float* w_hat,
                          void* scratch, cudaStream_t st) {
    SearchParams sp;
    const int rc = fill_params(sp, bits, coeff, n_cand);
    if (rc) return rc;
    unsigned* mx = static_cast<unsigned*>(scratch);
    if (check_cuda(cudaMemsetAsync(mx, 0, sizeof(unsigned), st))) return EBS_ERR_CUDA;
    abs_max_kernel<<<grid_size(n), 256, 0, st>>>(w, n, mx);
    launch_forward<true>(n_cand, grid_size(n), st, w, n, 1.0f, mx, sp, w_hat);
    return check_cuda(cudaGetLastError());
}

int launch_search_acts(const float* x, size_t n, float alpha, const int* bits, const float* coeff, int n_cand, float* x_hat,
                       cudaStream_t st) {
    SearchParams sp;
    const int rc = fill_params(sp, bits, coeff, n_cand);
    if (rc) return rc;
    launch_forward<false>(n_cand, grid_size(n), st, x, n, alpha, nullptr, sp, x_hat);
    return check_cuda(cudaGetLastError());
}

}  // namespace ebs
