// Throughput probe of the 5th-generation tensor core for the instruction the convolution kernels issue:
// tcgen05.mma kind::i8, M = 128, N = 256, K = 32, both operands from shared memory, accumulators in tensor memory.
// One CTA per SM; one thread issues `iters` rounds of 16 MMAs over eight different operand tiles and two accumulators
// and waits (bounded) for a single commit at the end.  The operands are zero bytes: the rate does not depend on the data.
// Measurement support: the paper has no counterpart.
#include "conv_umma_strip.cuh"

namespace ebs {

constexpr int PROBE_UMMA_TILES = 8;
constexpr int PROBE_UMMA_A_BYTES = 128 * 32, PROBE_UMMA_B_BYTES = 256 * 32;
constexpr int PROBE_UMMA_SMEM = PROBE_UMMA_TILES * (PROBE_UMMA_A_BYTES + PROBE_UMMA_B_BYTES) + 1024;

template <int N>
__global__ void __launch_bounds__(128, 1) probe_umma_i8_kernel(int iters, unsigned wait_limit, unsigned* gave_up) {
    extern __shared__ uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t done_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    uint8_t* base = dyn_smem + ((1024u - (smem_u32(dyn_smem) & 1023u)) & 1023u);
    uint8_t* a_tiles = base;                                             // [tile][2 halves][128 rows][16 bytes]
    uint8_t* b_tiles = base + PROBE_UMMA_TILES * PROBE_UMMA_A_BYTES;     // [tile][256 rows][32 bytes], 32-byte swizzle
    const int tid = threadIdx.x, warp = tid >> 5;
    for (int i = tid; i < PROBE_UMMA_TILES * (PROBE_UMMA_A_BYTES + PROBE_UMMA_B_BYTES) / 16; i += blockDim.x)
        reinterpret_cast<uint4*>(base)[i] = make_uint4(0u, 0u, 0u, 0u);
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    if (tid == 0) {
        abort_flag = 0;
        mbar_init(&done_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_slot)), "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const uint32_t tmem_base = tmem_slot;
    if (tid == 0) {
        constexpr uint32_t IDESC = umma_idesc_i8(N);
        const uint64_t da0 = umma_desc_interleaved(smem_u32(a_tiles), 128u * 16u);
        const uint64_t db0 = umma_desc_sw32(smem_u32(b_tiles));
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (int u = 0; u < 2 * PROBE_UMMA_TILES; ++u) {
                const int t = u % PROBE_UMMA_TILES;
                umma_i8(tmem_base + (uint32_t)((u & 1) * 256), da0 + (uint64_t)(t * (PROBE_UMMA_A_BYTES >> 4)),
                        db0 + (uint64_t)(t * (PROBE_UMMA_B_BYTES >> 4)), IDESC, (it | u) > 1 ? 1u : 0u);
            }
        }
        umma_commit(&done_bar);
        if (!mbar_wait_bounded(&done_bar, 0u, &abort_flag, wait_limit)) atomicAdd(gave_up, 1u);
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(512u) : "memory");
}

// Byte multiply-accumulates per second over all SMs; EBS_ERR_TIMEOUT if a CTA's wait ran out.
template <int N>
static int probe_umma_i8_n(int iters, double* macs_per_second) {
    int dev = 0, sms = 0;
    if (check_cuda(cudaGetDevice(&dev))) return EBS_ERR_CUDA;
    if (check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev))) return EBS_ERR_CUDA;
    if (check_cuda(cudaFuncSetAttribute(probe_umma_i8_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, PROBE_UMMA_SMEM)))
        return EBS_ERR_CUDA;
    unsigned* gave_up = nullptr;
    if (check_cuda(cudaMalloc(&gave_up, sizeof(unsigned)))) return EBS_ERR_CUDA;
    cudaMemset(gave_up, 0, sizeof(unsigned));
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    // the wait covers the whole run: 16 * iters MMAs of at least 128 clocks, polled every 40-200 ns
    const unsigned limit = 1u << 22;
    probe_umma_i8_kernel<N><<<sms, 128, PROBE_UMMA_SMEM>>>(iters, limit, gave_up);     // warm-up
    cudaEventRecord(e0);
    probe_umma_i8_kernel<N><<<sms, 128, PROBE_UMMA_SMEM>>>(iters, limit, gave_up);
    cudaEventRecord(e1);
    int rc = check_cuda(cudaDeviceSynchronize());
    float ms = 0.f;
    cudaEventElapsedTime(&ms, e0, e1);
    unsigned n_gave_up = 0;
    cudaMemcpy(&n_gave_up, gave_up, sizeof(unsigned), cudaMemcpyDeviceToHost);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(gave_up);
    if (rc) return rc;
    if (n_gave_up) return EBS_ERR_TIMEOUT;
    *macs_per_second = 2.0 * PROBE_UMMA_TILES * iters * (128.0 * N * 32.0) * sms / (ms * 1e-3);
    return EBS_OK;
}

// n_cols: 256 (the widest channel tile) or 64 (the narrowest: the same instruction count at a quarter of the work, which
// shows what one issuing thread can sustain)
int probe_umma_i8(int iters, double* macs_per_second, int n_cols) {
    return n_cols == 64 ? probe_umma_i8_n<64>(iters, macs_per_second) : probe_umma_i8_n<256>(iters, macs_per_second);
}

}  // namespace ebs
