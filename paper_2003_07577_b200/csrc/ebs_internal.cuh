// Internal declarations shared by the translation units of libebs (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ebs.h"

namespace ebs {

constexpr int PIPE_ZERO_WORDS = 8192;   // words of the zero page (ConvParams::zero_words): >= CW * planes of a layer on the pipeline kernel

// Everything the convolution kernels need, passed by value as a kernel argument.
struct ConvParams {
    const uint32_t* __restrict__ x;   // packed activations [N][H][W][CW][AB]
    const uint32_t* __restrict__ w;   // packed weights     [kh][kw][CW][Co][WB]
    const uint8_t* __restrict__ w8;   // byte image of the weights [kh*kw*CW][Co16][32] (second part of the buffer)
    int Co16;                         // c_out rounded up to 16
    int N, H, W, CW;
    int Co, Ho, Wo, CWo;              // CWo = ceil(Co/32)
    int kh, kw, sh, sw, ph, pw;
    int KK;                           // kh*kw*CW reduction words per plane pair
    int P;                            // N*Ho*Wo output pixels
    int32_t* __restrict__ acc;        // nullable, [P][Co]
    float* __restrict__ y;            // nullable
    uint32_t* __restrict__ packed_next;  // nullable, [P][CWo][next_bits]
    float S;                          // fl32(w_scale * a_scale)
    const float* __restrict__ ch_scale;
    const float* __restrict__ ch_bias;
    const float* __restrict__ residual;
    const uint32_t* __restrict__ res_packed;   // nullable: shortcut as packed planes [P][CWo][res_bits]
    int res_bits;
    float res_scale;
    int relu;
    int next_bits;
    float inv_next;
    int y_nchw;
    int w_levels;                     // 1: accumulator = 2 * plane sum + window sum of the activation codes
    int fold;                         // taps OR-ed into one reduction word by the tensor-pipe kernels: 1, 2, 4, 8
    int fold_bits;                    // 32 / fold: bits each folded tap occupies (>= c_in)
    int strip_pix, strip_ks;          // strip kernel only (set by its launcher): pixels of a strip, words per stage
    unsigned wait_limit;              // polls a bounded device-side wait makes before the CTA gives up
    int test_flags;                   // bit 0 (tests only): the MMA issuer issues nothing, so that waits run out
    int pipe_m_sub;                   // persistent pipeline kernel: accumulators per super-tile (0 = chosen by the library)
    int acc_small;                    // 1: every accumulator of the layer is below 2^22 in magnitude (worst case of its sizes and bit counts)
    // Extents of the buffers, for the range-checked build (EBS_CHECKED); filled in every build.
    long long lim_x, lim_w;           // 32-bit words of the packed activations (bytes / 4 on the byte-code path) and of the weight plane words
    long long lim_w8;                 // bytes of the weight byte image
    long long lim_out, lim_pn;        // elements of acc / y; 32-bit words of packed_next
    const uint32_t* zero_words;       // device page of zero words (pipeline kernel: what its expanders read for padding)
    unsigned long long* check_status; // EBS_CHECKED: device words {site << 48 | 1, index, limit}; else null
};

// Range-checked build (-DEBS_CHECKED, a second library beside the normal one): the indices the kernels compute from the
// run-time geometry -- offsets into the operand and result buffers, into the shared-memory rings and tables -- pass
// through EBS_IN_RANGE before the access.  A violation is recorded (the first one wins: site, index, limit) and the
// access is skipped; nothing traps or asserts, the kernel runs to its end and the host reads the record with
// ebs_checked_status.  In the normal build the macro is the constant `true` and costs nothing.
#ifdef EBS_CHECKED
__device__ __forceinline__ bool check_in_range(unsigned long long* st, unsigned site, long long idx, long long limit) {
    if (idx >= 0 && idx < limit) return true;
    if (st && atomicCAS(&st[0], 0ull, ((unsigned long long)site << 48) | 1ull) == 0ull) {
        st[1] = (unsigned long long)idx;
        st[2] = (unsigned long long)limit;
    }
    return false;
}
#define EBS_IN_RANGE(p, site, idx, limit) ::ebs::check_in_range((p).check_status, (site), (long long)(idx), (long long)(limit))
#else
#define EBS_IN_RANGE(p, site, idx, limit) true
#endif
// Sites (kernel family * 16 + access): 1x pipeline kernel, 2x warp-level strip kernel, 3x warp-level per-tap kernel,
// 4x integer-pipe kernel, 5x shared epilogue helpers.
enum CheckSite {
    CHK_PIPE_X = 0x10, CHK_PIPE_STAGE = 0x11, CHK_PIPE_TAB = 0x12, CHK_PIPE_ACC = 0x13, CHK_PIPE_Y = 0x14, CHK_PIPE_PN = 0x15,
    CHK_PIPE_W8 = 0x16,
    CHK_MS_X = 0x20, CHK_MS_STRIP = 0x21, CHK_MS_W8 = 0x22, CHK_MS_ACC = 0x23, CHK_MS_Y = 0x24, CHK_MS_PN = 0x25, CHK_MS_WS = 0x26,
    CHK_MMA_X = 0x30, CHK_MMA_W8 = 0x31, CHK_MMA_ACC = 0x32, CHK_MMA_Y = 0x33, CHK_MMA_STAGE = 0x34,
    CHK_POPC_X = 0x40, CHK_POPC_W = 0x41, CHK_POPC_ACC = 0x42, CHK_POPC_Y = 0x43, CHK_POPC_SMEM = 0x44,
    CHK_TILE_PN = 0x50, CHK_TILE_CODES = 0x51,
};

// One instantiation of the popcount kernel: launch function + its tile geometry.
struct ConvVariant {
    int (*launch)(const ConvParams&, dim3 grid, cudaStream_t);   // EBS_OK once the kernel is enqueued
    int tile_p, tile_c, threads;
};

// Number of tile variants per (w_bits, a_bits); see VariantGeom in conv_popc.cuh.
enum { NUM_CONV_VARIANTS = 10, CONV_VARIANT_SMALL = 9 };

// Filled by the per-bitwidth translation units (conv_popc_w1.cu .. conv_popc_w8.cu).
const ConvVariant* conv_popc_variant(int w_bits, int a_bits, int variant);
#define EBS_DECLARE_WB(WB) const ConvVariant* conv_popc_variant_w##WB(int a_bits, int variant);
EBS_DECLARE_WB(1) EBS_DECLARE_WB(2) EBS_DECLARE_WB(3) EBS_DECLARE_WB(4)
EBS_DECLARE_WB(5) EBS_DECLARE_WB(6) EBS_DECLARE_WB(7) EBS_DECLARE_WB(8)
#undef EBS_DECLARE_WB

// Warp-level tensor-pipe kernels (conv_mma_a1.cu .. conv_mma_a8.cu, one per activation bit count; the weights come
// as bytes, so the kernel does not depend on their bit count); variant 0 .. NUM_CONV_MMA_VARIANTS-1.
enum { NUM_CONV_MMA_VARIANTS = 9, CONV_MMA_MAX_KK = 256 };
const ConvVariant* conv_mma_variant(int w_bits, int a_bits, int variant);
#define EBS_DECLARE_AB(AB) const ConvVariant* conv_mma_variant_a##AB(int variant);
EBS_DECLARE_AB(1) EBS_DECLARE_AB(2) EBS_DECLARE_AB(3) EBS_DECLARE_AB(4)
EBS_DECLARE_AB(5) EBS_DECLARE_AB(6) EBS_DECLARE_AB(7) EBS_DECLARE_AB(8)
#undef EBS_DECLARE_AB

// 5th-generation tensor-core kernels (conv_umma_w1.cu .. conv_umma_w8.cu); variant = log2(tile_n / 16).
enum { NUM_CONV_UMMA_VARIANTS = 5, NUM_CONV_STRIP_VARIANTS = 5, NUM_CONV_RESIDENT_VARIANTS = 5, NUM_CONV_MMA_STRIP_VARIANTS = 3,
       NUM_CONV_PIPE_VARIANTS = 4 };
// Persistent pipeline kernel for any stride (conv_umma_pipe.cu): variants 0-2 by channel tile 64 << variant, variant 3 the
// 256-channel tile on a pair of CTAs (a cluster of two sharing every MMA).
const ConvVariant* conv_umma_pipe_variant(int a_bits, int variant);
bool conv_umma_pipe_applies(const ConvParams& p, int variant);
unsigned long long conv_umma_pipe_timeouts();
long long conv_umma_pipe_items(const ConvParams& p, int variant);   // (pixel super-tile, channel tile) work items, -1 if it does not apply
// Warp-level strip kernel for small stride-1 layers (conv_mma_strip.cu): channel tile 16 / 32 / 64.
const ConvVariant* conv_mma_strip_variant(int a_bits, int variant);
bool conv_mma_strip_applies(const ConvParams& p, int variant);
// Persistent weight-resident strip kernel (conv_umma_resident.cu): variants by channel tile 16 << variant.
const ConvVariant* conv_umma_resident_variant(int a_bits, int variant);
bool conv_umma_resident_applies(const ConvParams& p, int variant);
unsigned long long conv_umma_resident_timeouts();
// Stride-1 strip kernel (conv_umma_strip.cu): variants by channel tile 16 << variant.
const ConvVariant* conv_umma_strip_variant(int a_bits, int variant);
bool conv_umma_strip_applies(const ConvParams& p, int variant);
unsigned long long conv_umma_strip_timeouts();
const ConvVariant* conv_umma_variant(int w_bits, int a_bits, int variant);
unsigned long long conv_umma_timeouts();
#define EBS_DECLARE_WB(WB)                                                   \
    const ConvVariant* conv_umma_variant_w##WB(int a_bits, int variant);     \
    unsigned long long conv_umma_timeouts_w##WB();
EBS_DECLARE_WB(1) EBS_DECLARE_WB(2) EBS_DECLARE_WB(3) EBS_DECLARE_WB(4)
EBS_DECLARE_WB(5) EBS_DECLARE_WB(6) EBS_DECLARE_WB(7) EBS_DECLARE_WB(8)
#undef EBS_DECLARE_WB

// pack.cu
int launch_pack_acts_s2d(const void* x, int n, int c, int h, int w, int off, int a_bits, uint32_t* out, cudaStream_t st);
int launch_pack_acts(const void* x, int dtype, int layout, int n, int c, int h, int w, int a_bits,
                     float inv_scale, uint32_t* out, cudaStream_t st);
int launch_pack_weights(const void* wt, int dtype, int layout, const ebs_conv_desc& d, float inv_scale,
                        uint32_t* out, cudaStream_t st);
// dequant.cu
int launch_dequant(const int32_t* acc, size_t n_pixels, int c_out, float scale, const float* ch_scale,
                   const float* ch_bias, int relu, float* y, cudaStream_t st);

size_t packed_weight_plane_bytes(const ebs_conv_desc& d);   // bit-plane words, rounded up to 256 bytes
size_t packed_weight_image_bytes(const ebs_conv_desc& d);   // byte image that follows them
int launch_search_weights(const float* w, size_t n, const int* bits, const float* coeff, int n_cand, float* w_hat,
                          void* scratch, cudaStream_t st);
int launch_search_acts(const float* x, size_t n, float alpha, const int* bits, const float* coeff, int n_cand,
                       float* x_hat, cudaStream_t st);
int fused_plan_upload(const void* layers_host, int n_layers, void* layers_dev, cudaStream_t st);
int launch_fused_resnet(const uint8_t* images, int n, int img_h, int img_w, const void* layers_dev, int n_layers,
                        const void* head_host, float* logits, uint8_t* trace, long long trace_stride, cudaStream_t st);
unsigned long long fused_net_timeouts();
int launch_avgpool(const float* y, int n, int hw, int c, float* out, cudaStream_t st);
int launch_maxpool_packed(const uint32_t* x, int n, int h, int w, int c, int bits, int k, int stride, int pad, int ho,
                          int wo, uint32_t* out, cudaStream_t st);

// Records a CUDA error for ebs_last_cuda_error() and returns EBS_ERR_CUDA (or EBS_OK).
int check_cuda(cudaError_t e);

// Reads NWORDS consecutive packed words from global memory through the read-only path.
template <int NWORDS>
__device__ __forceinline__ void load_words_global(const uint32_t* __restrict__ src, uint32_t (&dst)[NWORDS]) {
    // src is aligned to 4*NWORDS bytes when NWORDS is a power of two (plane-minor layout).
    if constexpr (NWORDS % 4 == 0) {
#pragma unroll
        for (int v = 0; v < NWORDS / 4; ++v) {
            uint4 t = __ldg(reinterpret_cast<const uint4*>(src) + v);
            dst[4 * v] = t.x; dst[4 * v + 1] = t.y; dst[4 * v + 2] = t.z; dst[4 * v + 3] = t.w;
        }
    } else if constexpr (NWORDS % 2 == 0) {
#pragma unroll
        for (int v = 0; v < NWORDS / 2; ++v) {
            uint2 t = __ldg(reinterpret_cast<const uint2*>(src) + v);
            dst[2 * v] = t.x; dst[2 * v + 1] = t.y;
        }
    } else {
#pragma unroll
        for (int v = 0; v < NWORDS; ++v) dst[v] = __ldg(src + v);
    }
}

// quantize_b of Eq. 1c in code form: round half up, every fp32 operation rounded on its own.
__device__ __forceinline__ int quantize_code(float x, float inv_scale, int lo, int hi) {
    float v = __fmul_rn(x, inv_scale);
    float f = floorf(__fadd_rn(v, 0.5f));
    int q;
    if (!(f >= (float)lo)) q = lo;       // NaN lands here too
    else if (f > (float)hi) q = hi;
    else q = (int)f;
    return q;
}

// Nearest of the paper's weight levels w_scale * (2 q_u - (2^b - 1)), q_u = 0 .. 2^b-1 (Eq. 1a), returned
// as the signed code q_u - 2^(b-1).  (v + L)/2 is exact in fp32 for the magnitudes that survive the clamp.
__device__ __forceinline__ int quantize_weight_level(float w, float inv_scale, int bits) {
    const int L = (1 << bits) - 1;
    const float v = __fmul_rn(w, inv_scale);
    const float u = __fmul_rn(__fadd_rn(v, (float)L), 0.5f);
    const float f = floorf(__fadd_rn(u, 0.5f));
    int qu;
    if (!(f >= 0.0f)) qu = 0;
    else if (f > (float)L) qu = L;
    else qu = (int)f;
    return qu - (1 << (bits - 1));
}

// The same quantizer for activation codes (lo = 0): floor and float->int in one conversion
// (round toward -inf, saturating; NaN converts to 0), then an integer clamp.
__device__ __forceinline__ int quantize_act_code(float y, float inv_scale, int qmax) {
    const float r = __fadd_rn(__fmul_rn(y, inv_scale), 0.5f);
    return min(max(__float2int_rd(r), 0), qmax);
}

// Shortcut of a residual block kept as packed planes: real value res_scale * code of channel co at
// output pixel gp (one rounded multiply).  Deliberately not inlined: only the epilogue of a layer
// with such a shortcut calls it, and inlining it raised the register count of every kernel (and so
// lowered the occupancy of layers that never take this path).  Arguments are scalars so that the
// kernel parameter block is not copied to local memory.
static __device__ __noinline__ float packed_residual_at(const uint32_t* __restrict__ res_packed, int CWo, int res_bits,
                                                 float res_scale, int gp, int co) {
    const uint32_t* w = res_packed + ((size_t)gp * CWo + (co >> 5)) * res_bits;
    uint32_t code = 0u;
    for (int j = 0; j < res_bits; ++j) code |= ((__ldg(w + j) >> (co & 31)) & 1u) << j;
    return __fmul_rn(res_scale, (float)code);
}
__device__ __forceinline__ float packed_residual(const ConvParams& p, int gp, int co) {
    return packed_residual_at(p.res_packed, p.CWo, p.res_bits, p.res_scale, gp, co);
}

// Row pitch (bytes) of the tile of requantized codes kept in shared memory: 4 bytes of padding make
// consecutive pixels start in different banks.
__host__ __device__ constexpr int code_row_bytes(int tile_c) { return tile_c + 4; }

// Packs a CTA's tile of requantized codes (one byte per output, [TILE_P][code_row_bytes(TILE_C)] in
// shared memory) into the next layer's bit-plane words.  One thread per (pixel, 32-channel word):
// four code bytes at a time, plane j of the four codes is gathered into a nibble with one multiply
// ((x >> j) & 0x01010101) * 0x01020408 >> 24.
template <int TILE_P, int TILE_C, int NTHREADS>
__device__ __forceinline__ void pack_code_tile(const uint8_t* out_s, const ConvParams& p, int tile_p0, int co0) {
    constexpr int ROWB = code_row_bytes(TILE_C);
    constexpr int CWL = (TILE_C + 31) / 32;
    constexpr int NW = TILE_C >= 32 ? 8 : TILE_C / 4;           // code words per 32-channel group
#pragma unroll 1
    for (int item = threadIdx.x; item < TILE_P * CWL; item += NTHREADS) {
        const int cwl = item / TILE_P, pl = item - cwl * TILE_P;
        const int gp = tile_p0 + pl, cwg = (co0 >> 5) + cwl;
        if (gp >= p.P || cwg >= p.CWo) continue;
        const uint32_t* row = reinterpret_cast<const uint32_t*>(out_s + pl * ROWB + cwl * 32);
        uint32_t codes[NW];
#pragma unroll
        for (int k = 0; k < NW; ++k) codes[k] = row[k];
        uint32_t* dst = p.packed_next + ((size_t)gp * p.CWo + cwg) * p.next_bits;
        if (!EBS_IN_RANGE(p, CHK_TILE_PN, ((size_t)gp * p.CWo + cwg) * p.next_bits + p.next_bits - 1, p.lim_pn)) continue;
#pragma unroll 1
        for (int j = 0; j < p.next_bits; ++j) {
            uint32_t word = 0u;
#pragma unroll
            for (int k = 0; k < NW; ++k) {
                const uint32_t t = (codes[k] >> j) & 0x01010101u;
                word |= ((t * 0x01020408u) >> 24) << (4 * k);
            }
            dst[j] = word;
        }
    }
}

}  // namespace ebs
