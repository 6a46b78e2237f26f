// Register-resident throughput probes for the pipes the convolution can use.  Their measured
// rate is the denominator of the arithmetic roofline the benchmark reports.
#include "ebs_internal.cuh"

namespace ebs {

constexpr int PROBE_CHAINS = 16;
constexpr int PROBE_UNROLL = 8;

// kind 0: acc += popc(x & w)  (LOP3 + POPC + IADD per 32 bit pairs);  kind 2: POPC alone.
template <int KIND>
__global__ void __launch_bounds__(256) probe_popc_kernel(uint32_t* out, int iters, uint32_t seed) {
    uint32_t x[PROBE_CHAINS];
#pragma unroll
    for (int k = 0; k < PROBE_CHAINS; ++k) x[k] = seed * (k + 1) + threadIdx.x * 2654435761u;
    const uint32_t b = seed ^ 0x5bd1e995u;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < PROBE_UNROLL; ++u) {
#pragma unroll
            for (int k = 0; k < PROBE_CHAINS; ++k) {
                if (KIND == 0)
                    asm volatile("{.reg .b32 t; and.b32 t, %0, %1; popc.b32 t, t; add.u32 %0, %0, t;}"
                                 : "+r"(x[k]) : "r"(b));
                else
                    asm volatile("popc.b32 %0, %0;" : "+r"(x[k]));
            }
        }
    }
    uint32_t s = 0;
#pragma unroll
    for (int k = 0; k < PROBE_CHAINS; ++k) s ^= x[k];
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

// kind 1: warp-level binary MMA, 16 x 8 outputs x 256 bits per instruction.
__global__ void __launch_bounds__(256) probe_bmma_kernel(uint32_t* out, int iters, uint32_t seed) {
    constexpr int SETS = 4;
    int c[SETS][4];
#pragma unroll
    for (int k = 0; k < SETS; ++k)
#pragma unroll
        for (int j = 0; j < 4; ++j) c[k][j] = 0;
    const uint32_t a0 = seed * threadIdx.x, a1 = a0 * 3u + 1u, a2 = a0 * 5u + 2u, a3 = a0 * 7u + 3u;
    const uint32_t b0 = seed ^ threadIdx.x, b1 = b0 * 11u;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < PROBE_UNROLL; ++u) {
#pragma unroll
            for (int k = 0; k < SETS; ++k)
                asm volatile(
                    "mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc "
                    "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                    : "+r"(c[k][0]), "+r"(c[k][1]), "+r"(c[k][2]), "+r"(c[k][3])
                    : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
        }
    }
    int s = 0;
#pragma unroll
    for (int k = 0; k < SETS; ++k)
#pragma unroll
        for (int j = 0; j < 4; ++j) s ^= c[k][j];
    out[blockIdx.x * blockDim.x + threadIdx.x] = (uint32_t)s;
}

// kind 3: warp-level int8 MMA, 16 x 8 outputs x 32 bytes per instruction (the pipe conv_mma_kernel uses).
__global__ void __launch_bounds__(256) probe_imma_kernel(uint32_t* out, int iters, uint32_t seed) {
    constexpr int SETS = 4;
    int c[SETS][4];
#pragma unroll
    for (int k = 0; k < SETS; ++k)
#pragma unroll
        for (int j = 0; j < 4; ++j) c[k][j] = 0;
    const uint32_t a0 = seed * threadIdx.x, a1 = a0 * 3u + 1u, a2 = a0 * 5u + 2u, a3 = a0 * 7u + 3u;
    const uint32_t b0 = seed ^ threadIdx.x, b1 = b0 * 11u;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < PROBE_UNROLL; ++u) {
#pragma unroll
            for (int k = 0; k < SETS; ++k)
                asm volatile(
                    "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 "
                    "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                    : "+r"(c[k][0]), "+r"(c[k][1]), "+r"(c[k][2]), "+r"(c[k][3])
                    : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
        }
    }
    int s = 0;
#pragma unroll
    for (int k = 0; k < SETS; ++k)
#pragma unroll
        for (int j = 0; j < 4; ++j) s ^= c[k][j];
    out[blockIdx.x * blockDim.x + threadIdx.x] = (uint32_t)s;
}

int probe_umma_i8(int iters, double* macs_per_second, int n_cols);     // probe_umma.cu

}  // namespace ebs

extern "C" int ebs_probe_pipe(int kind, int iters, double* bit_ops_per_second) {
    using namespace ebs;
    if (kind < 0 || kind > 5 || iters < 1 || iters > (1 << 22) || !bit_ops_per_second) return EBS_ERR_INVALID_ARG;
    if (kind >= 4) return iters > (1 << 14) ? EBS_ERR_INVALID_ARG : probe_umma_i8(iters, bit_ops_per_second, kind == 4 ? 256 : 64);
    int dev = 0, sms = 0;
    if (check_cuda(cudaGetDevice(&dev))) return EBS_ERR_CUDA;
    if (check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev))) return EBS_ERR_CUDA;
    const int blocks = sms * 4;
    uint32_t* out = nullptr;
    if (check_cuda(cudaMalloc(&out, (size_t)blocks * 256 * sizeof(uint32_t)))) return EBS_ERR_CUDA;
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    auto launch = [&](int n) {
        if (kind == 0) probe_popc_kernel<0><<<blocks, 256>>>(out, n, 12345u);
        else if (kind == 2) probe_popc_kernel<2><<<blocks, 256>>>(out, n, 12345u);
        else if (kind == 3) probe_imma_kernel<<<blocks, 256>>>(out, n, 77u);
        else probe_bmma_kernel<<<blocks, 256>>>(out, n, 77u);
    };
    launch(iters);                          // warm-up (also lets the clocks ramp)
    cudaEventRecord(e0);
    launch(iters);
    cudaEventRecord(e1);
    int rc = check_cuda(cudaDeviceSynchronize());
    float ms = 0.f;
    cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(out);
    if (rc) return rc;
    double per_thread_iter = kind == 1   ? 4.0 * PROBE_UNROLL * (16.0 * 8 * 256 / 32.0)
                             : kind == 3 ? 4.0 * PROBE_UNROLL * (16.0 * 8 * 32 / 32.0)
                                         : (double)PROBE_CHAINS * PROBE_UNROLL * 32.0;
    *bit_ops_per_second = per_thread_iter * iters * 256.0 * blocks / (ms * 1e-3);
    return EBS_OK;
}
