// ebs_conv2d_mixed_host_noalloc: the host-buffer layer call for callers that cannot allocate
// device memory.  Its device scratch is a fixed array that is part of the library image.
#include <mutex>

#include "ebs_internal.cuh"

namespace {

constexpr size_t kScratchBytes = (size_t)EBS_NOALLOC_SCRATCH_BYTES;

// Lives in every CUDA context that loads this library, from load until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address a kernel can
// use; the device address is looked up once per device, with that device current.
int scratch_for_current_device(void** out) {
    int dev = -1;
    if (ebs::check_cuda(cudaGetDevice(&dev))) return EBS_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return EBS_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        if (ebs::check_cuda(cudaGetSymbolAddress(&p, g_noalloc_scratch))) return EBS_ERR_CUDA;
        if (!p) return EBS_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return EBS_OK;
}

}  // namespace

extern "C" {

size_t ebs_noalloc_scratch_bytes(void) { return kScratchBytes; }

int ebs_conv2d_mixed_host_noalloc(const void* x_host, int dtype, int layout, int n, int h, int w,
                                  const void* packed_w_dev, const ebs_conv_desc* desc, const ebs_epilogue* epi,
                                  int32_t* acc_out_host, float* y_out_host, void* packed_next_host, void* stream) {
    if (!desc) return EBS_ERR_INVALID_ARG;
    if (packed_next_host && !epi) return EBS_ERR_INVALID_ARG;
    const int next_bits = packed_next_host ? epi->next_a_bits : 0;
    const size_t need = ebs_host_workspace_bytes(desc, n, h, w, dtype, next_bits);
    if (need == 0) return EBS_ERR_INVALID_ARG;
    if (need > kScratchBytes) return EBS_ERR_SCRATCH_TOO_SMALL;
    void* scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch);
    if (rc) return rc;
    return ebs_conv2d_mixed_host(x_host, dtype, layout, n, h, w, packed_w_dev, desc, epi, scratch, kScratchBytes,
                                 acc_out_host, y_out_host, packed_next_host, stream);
}

}  // extern "C"
