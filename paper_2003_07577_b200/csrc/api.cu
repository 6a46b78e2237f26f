// C ABI of libebs: host-side validation, kernel selection, launches.  See include/ebs.h.
#include <string.h>

#include "ebs_internal.cuh"

namespace ebs {

static thread_local char g_cuda_error[256] = "";

int check_cuda(cudaError_t e) {
    if (e == cudaSuccess) return EBS_OK;
    strncpy(g_cuda_error, cudaGetErrorString(e), sizeof(g_cuda_error) - 1);
    g_cuda_error[sizeof(g_cuda_error) - 1] = '\0';
    return EBS_ERR_CUDA;
}

const ConvVariant* conv_popc_variant(int w_bits, int a_bits, int variant) {
    switch (w_bits) {
        case 1: return conv_popc_variant_w1(a_bits, variant);
        case 2: return conv_popc_variant_w2(a_bits, variant);
        case 3: return conv_popc_variant_w3(a_bits, variant);
        case 4: return conv_popc_variant_w4(a_bits, variant);
        case 5: return conv_popc_variant_w5(a_bits, variant);
        case 6: return conv_popc_variant_w6(a_bits, variant);
        case 7: return conv_popc_variant_w7(a_bits, variant);
        case 8: return conv_popc_variant_w8(a_bits, variant);
        default: return nullptr;
    }
}

const ConvVariant* conv_mma_variant(int w_bits, int a_bits, int variant) {
    if (w_bits < 1 || w_bits > 8) return nullptr;
    switch (a_bits) {
        case 1: return conv_mma_variant_a1(variant);
        case 2: return conv_mma_variant_a2(variant);
        case 3: return conv_mma_variant_a3(variant);
        case 4: return conv_mma_variant_a4(variant);
        case 5: return conv_mma_variant_a5(variant);
        case 6: return conv_mma_variant_a6(variant);
        case 7: return conv_mma_variant_a7(variant);
        case 8: return conv_mma_variant_a8(variant);
        default: return nullptr;
    }
}

const ConvVariant* conv_umma_variant(int w_bits, int a_bits, int variant) {
    switch (w_bits) {
        case 1: return conv_umma_variant_w1(a_bits, variant);
        case 2: return conv_umma_variant_w2(a_bits, variant);
        case 3: return conv_umma_variant_w3(a_bits, variant);
        case 4: return conv_umma_variant_w4(a_bits, variant);
        case 5: return conv_umma_variant_w5(a_bits, variant);
        case 6: return conv_umma_variant_w6(a_bits, variant);
        case 7: return conv_umma_variant_w7(a_bits, variant);
        case 8: return conv_umma_variant_w8(a_bits, variant);
        default: return nullptr;
    }
}

unsigned long long conv_umma_timeouts() {
    return conv_umma_timeouts_w1() + conv_umma_timeouts_w2() + conv_umma_timeouts_w3() + conv_umma_timeouts_w4() +
           conv_umma_timeouts_w5() + conv_umma_timeouts_w6() + conv_umma_timeouts_w7() + conv_umma_timeouts_w8() +
           conv_umma_strip_timeouts() + conv_umma_resident_timeouts() + conv_umma_pipe_timeouts() + fused_net_timeouts();
}

// Polls a bounded device-side wait makes before it gives up (about 40 ns each), and test flags; process-wide,
// changed only by ebs_test_set_device_wait.
static unsigned g_wait_limit = 1u << 20;
static int g_test_flags = 0;
static long long g_check_shrink = 0;      // range-checked build, tests only: result extents declared this much too short

// Range-checked build only: the device words the kernels record their first out-of-range index in.
#ifdef EBS_CHECKED
static __device__ unsigned long long g_check_words[4];
static unsigned long long* check_status_words() {
    void* ptr = nullptr;
    return cudaGetSymbolAddress(&ptr, g_check_words) == cudaSuccess ? static_cast<unsigned long long*>(ptr) : nullptr;
}
#else
static unsigned long long* check_status_words() { return nullptr; }
#endif

// A page of zero words on the device (what the pipeline kernel's expanders read where a layer pads); its address is
// looked up once per device.
static __device__ __align__(256) uint32_t g_zero_words[PIPE_ZERO_WORDS];
static const uint32_t* zero_words_ptr() {
    static const uint32_t* cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cached[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_zero_words) == cudaSuccess) cached[dev] = static_cast<const uint32_t*>(ptr);
    }
    return cached[dev];
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int out_dim(int in, int pad, int k, int stride) {
    const int span = in + 2 * pad - k;
    return span < 0 ? 0 : span / stride + 1;
}

static int validate_desc(const ebs_conv_desc* d) {
    if (!d) return EBS_ERR_INVALID_ARG;
    if (d->c_in <= 0 || d->c_out <= 0 || d->kh <= 0 || d->kw <= 0 || d->stride_h <= 0 || d->stride_w <= 0 ||
        d->pad_h < 0 || d->pad_w < 0)
        return EBS_ERR_INVALID_ARG;
    if (d->w_bits < 1 || d->w_bits > 8 || d->a_bits < 1 || d->a_bits > 8) return EBS_ERR_INVALID_ARG;
    if (d->kh > 255 || d->kw > 255 || d->c_in > (1 << 20) || d->c_out > (1 << 20)) return EBS_ERR_UNSUPPORTED;
    if (!(d->w_scale > 0.0f) || !(d->a_scale > 0.0f)) return EBS_ERR_INVALID_ARG;
    // largest |acc| = c_in*kh*kw * 2^(w_bits-1) * (2^a_bits - 1) must fit int32
    const long long s = (long long)d->c_in * d->kh * d->kw;
    if (d->w_levels != 0 && d->w_levels != 1) return EBS_ERR_INVALID_ARG;
    const long long wmax = d->w_levels ? (1LL << d->w_bits) - 1 : (1LL << (d->w_bits - 1));   // largest |weight level|
    const long long worst = s * wmax * ((1LL << d->a_bits) - 1);
    if (worst >= (1LL << 31)) return EBS_ERR_OVERFLOW;
    return EBS_OK;
}

static int sm_count() {
    int dev = 0, n = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    return n > 0 ? n : 148;
}

// Picks the tile variant: tile_c from c_out, then the largest pixel tile that still gives every SM
// about two CTAs; problems too small for that use the small tile.
static int choose_variant(int w_bits, int a_bits, int P, int Co, bool want_packed, int sms) {
    const int tc_idx = Co <= 16 ? 0 : (Co <= 32 ? 1 : 2);
    for (int tp_idx = 2; tp_idx >= 0; --tp_idx) {
        const ConvVariant* v = conv_popc_variant(w_bits, a_bits, tc_idx * 3 + tp_idx);
        const long long ctas = (long long)((P + v->tile_p - 1) / v->tile_p) * ((Co + v->tile_c - 1) / v->tile_c);
        if (ctas >= 2LL * sms) return tc_idx * 3 + tp_idx;
    }
    const ConvVariant* v1 = conv_popc_variant(w_bits, a_bits, tc_idx * 3);
    const long long ctas1 = (long long)((P + v1->tile_p - 1) / v1->tile_p) * ((Co + v1->tile_c - 1) / v1->tile_c);
    if (ctas1 >= sms) return tc_idx * 3;
    // the small tile has 16 channels: a packed output word needs all 32 channels of a word in one CTA
    if (want_packed && Co > 16) return tc_idx * 3;
    return CONV_VARIANT_SMALL;
}

// The tensor-pipe kernels keep a table of the reduction words in shared memory, masks of valid taps
// in 32-bit words and word offsets in int: layers outside those limits use the popcount kernels.
static bool mma_path_supported(const ConvParams& p, const ebs_conv_desc* d) {
    const long long x_words = (long long)p.N * p.H * p.W * p.CW * d->a_bits;
    return p.KK <= CONV_MMA_MAX_KK && d->kh <= 32 && d->kw <= 32 && x_words < (1LL << 31);
}

// Tensor-pipe variant: tile_c from c_out; the largest warp tile that still gives every SM about a
// dozen warps (smaller layers need more, smaller tiles to hide latency).
static int choose_mma_variant(int w_bits, int a_bits, int P, int Co, int sms) {
    const int tc_idx = Co <= 16 ? 0 : (Co <= 32 ? 1 : 2);
    for (int cls = 0; cls < 2; ++cls) {
        const ConvVariant* v = conv_mma_variant(w_bits, a_bits, cls * 3 + tc_idx);
        const long long ctas = (long long)((P + v->tile_p - 1) / v->tile_p) * ((Co + v->tile_c - 1) / v->tile_c);
        if (ctas * (v->threads / 32) >= 12LL * sms) return cls * 3 + tc_idx;
    }
    return 6 + tc_idx;
}

// Stride-1 layers with at least 64 output channels and enough outputs to fill the GPU run on the strip
// kernel (every input pixel expanded once per CTA, weights fetched as bytes).  The channel tile is the
// largest of 256/128/64 that divides c_out, so that every tile is whole and takes the straight-line
// epilogue; failing that the largest not above c_out.  (Rule fitted to per-variant timings of the
// ResNet-18/20/50 layer shapes.)  Returns the strip variant or -1.
static int choose_strip_variant(const ConvParams& p) {
    if (p.Co < 64 || (long long)p.P * p.Co < (1LL << 20)) return -1;
    int pick = -1;
    for (int v = 4; v >= 2; --v)
        if (p.Co % (16 << v) == 0) { pick = v; break; }
    if (pick < 0) pick = p.Co >= 256 ? 4 : (p.Co >= 128 ? 3 : 2);
    for (; pick >= 2; --pick)
        if (conv_umma_strip_applies(p, pick)) return pick;
    return -1;
}

// The per-tap tcgen05 kernels (any stride) pay off when a CTA's 128 x tile_n accumulator sees a deep
// reduction, the channel tile is wide enough to amortise the activation expansion, and the layer has
// enough output tiles; smaller layers run faster on the warp-level kernels.  Returns the variant or -1.
// The persistent pipeline kernel covers stride-1 and strided k x k layers and 1x1 layers at any stride.  It pays off
// when the layer has at least 64 output channels and enough outputs to fill the GPU.  Channel tile: the widest of
// 256/128/64 that divides c_out (every tile whole: straight-line epilogue; the fewer channel tiles, the less often an
// input pixel is expanded and the less weight traffic per multiply -- measured faster even where it leaves some SMs
// without a tile).  Returns the pipeline variant (0..2) or -1.
static int choose_pipe_variant(const ConvParams& p, int sms) {
    (void)sms;
    // (layers with few input channels too: the kernel spends a whole 32-channel word per tap on them, and is still
    // six times faster on an ImageNet stem, 3 -> 64 channels 7x7 stride 2, than the tap-folding per-tap kernels)
    if (p.Co < 64 || (long long)p.P * p.Co < (1LL << 20) || p.w_levels) return -1;
    for (int v = 2; v >= 0; --v) {
        if (p.Co % (64 << v) != 0 && v != 0) continue;
        if (conv_umma_pipe_applies(p, v)) return v;
    }
    return -1;
}

static int choose_umma_variant(const ConvParams& p, const ebs_conv_desc* d) {
    const int kwords = (p.KK + p.fold - 1) / p.fold;
    const long long outputs = (long long)p.P * p.Co;
    (void)d;
    if (p.Co < 64 || kwords < 8) return -1;
    if (outputs < (1LL << 20) && kwords < 72) return -1;
    return p.Co >= 128 ? 3 : 2;             // tile_n 128 or 64
}

// A validated, fully decided launch: nothing has been enqueued when conv_plan returns.
struct ConvPlan {
    ConvParams p;
    const ConvVariant* v;
    dim3 grid;
};

// byte_acts: packed_x holds the activations as unpacked u8 NHWC codes instead of bit planes (ebs_conv2d_i8).
static int conv_plan(const void* packed_x, int n, int h, int w, const void* packed_w, const ebs_conv_desc* d,
                     const ebs_epilogue* epi, int32_t* acc_out, float* y_out, void* packed_next, int variant,
                     ConvPlan* plan, bool byte_acts = false) {
    int rc = validate_desc(d);
    if (rc) return rc;
    if (!packed_x || !packed_w || n <= 0 || h <= 0 || w <= 0) return EBS_ERR_INVALID_ARG;
    if (!acc_out && !y_out && !packed_next) return EBS_ERR_INVALID_ARG;
    if (!aligned16(packed_x) || !aligned16(packed_w) || !aligned16(acc_out) || !aligned16(y_out) ||
        !aligned16(packed_next))
        return EBS_ERR_INVALID_ARG;
    if (h > 32000 || w > 32000) return EBS_ERR_UNSUPPORTED;
    const int Ho = out_dim(h, d->pad_h, d->kh, d->stride_h), Wo = out_dim(w, d->pad_w, d->kw, d->stride_w);
    if (Ho <= 0 || Wo <= 0) return EBS_ERR_INVALID_ARG;
    const long long P = (long long)n * Ho * Wo, in_pixels = (long long)n * h * w;
    if (P >= (1LL << 31) || in_pixels >= (1LL << 31) || P * d->c_out >= (1LL << 40)) return EBS_ERR_OVERFLOW;
    if (packed_next) {
        if (!epi || epi->next_a_bits < 1 || epi->next_a_bits > 8 || !(epi->next_a_scale > 0.0f))
            return EBS_ERR_INVALID_ARG;
    }
    if (epi) {
        if (epi->y_layout != EBS_NCHW && epi->y_layout != EBS_NHWC) return EBS_ERR_INVALID_ARG;
        if (!aligned16(epi->residual_dev) || !aligned16(epi->res_packed_dev)) return EBS_ERR_INVALID_ARG;
        if (epi->res_packed_dev && (epi->res_bits < 1 || epi->res_bits > 8)) return EBS_ERR_INVALID_ARG;
    }
    constexpr int STRIP_BASE = NUM_CONV_VARIANTS + NUM_CONV_MMA_VARIANTS + NUM_CONV_UMMA_VARIANTS;
    constexpr int RES_BASE = STRIP_BASE + NUM_CONV_STRIP_VARIANTS;
    constexpr int MS_BASE = RES_BASE + NUM_CONV_RESIDENT_VARIANTS;
    constexpr int PIPE_BASE = MS_BASE + NUM_CONV_MMA_STRIP_VARIANTS;
    if (variant >= PIPE_BASE + NUM_CONV_PIPE_VARIANTS) return EBS_ERR_INVALID_ARG;

    ConvParams& p = plan->p;
    memset(&p, 0, sizeof(p));
    p.x = static_cast<const uint32_t*>(packed_x);
    p.w = static_cast<const uint32_t*>(packed_w);
    p.w8 = static_cast<const uint8_t*>(packed_w) + packed_weight_plane_bytes(*d);
    p.Co16 = (d->c_out + 15) & ~15;
    p.N = n; p.H = h; p.W = w; p.CW = (d->c_in + 31) / 32;
    p.Co = d->c_out; p.Ho = Ho; p.Wo = Wo; p.CWo = (d->c_out + 31) / 32;
    p.kh = d->kh; p.kw = d->kw; p.sh = d->stride_h; p.sw = d->stride_w; p.ph = d->pad_h; p.pw = d->pad_w;
    p.KK = d->kh * d->kw * p.CW;
    p.P = (int)P;
    p.acc = acc_out; p.y = y_out; p.packed_next = static_cast<uint32_t*>(packed_next);
    p.S = d->w_scale * d->a_scale;       // one rounded fp32 multiply
    p.next_bits = 1;
    p.w_levels = d->w_levels;
    p.fold = d->c_in <= 4 ? 8 : (d->c_in <= 8 ? 4 : (d->c_in <= 16 ? 2 : 1));
    p.fold_bits = 32 / p.fold;
    {
        const long long wmax = d->w_levels ? (1LL << d->w_bits) - 1 : (1LL << (d->w_bits - 1));
        p.acc_small = (long long)d->c_in * d->kh * d->kw * wmax * ((1LL << d->a_bits) - 1) < (1LL << 22) ? 1 : 0;
    }
    p.wait_limit = g_wait_limit;
    p.test_flags = g_test_flags;
    p.lim_x = byte_acts ? in_pixels * p.CW * 8 : in_pixels * p.CW * d->a_bits;
    p.lim_w = (long long)(packed_weight_plane_bytes(*d) / 4);
    p.lim_w8 = (long long)d->kh * d->kw * p.CW * p.Co16 * 32;
    p.lim_out = P * d->c_out - g_check_shrink;
    p.lim_pn = packed_next && epi ? P * p.CWo * epi->next_a_bits : 0;
    p.check_status = check_status_words();
    p.zero_words = zero_words_ptr();
    if (epi) {
        p.ch_scale = epi->ch_scale_dev; p.ch_bias = epi->ch_bias_dev; p.residual = epi->residual_dev;
        p.res_packed = static_cast<const uint32_t*>(epi->res_packed_dev); p.res_bits = epi->res_bits; p.res_scale = epi->res_scale;
        p.relu = epi->relu ? 1 : 0;
        p.y_nchw = epi->y_layout == EBS_NCHW;
        if (packed_next) { p.next_bits = epi->next_a_bits; p.inv_next = 1.0f / epi->next_a_scale; }
    }
    const bool mma_ok = mma_path_supported(p, d);
    if (byte_acts) {
        // the context path exists in the persistent pipeline kernels only: whole 32-channel words of byte codes
        if ((d->c_in & 31) != 0 || d->w_levels || !mma_ok) return EBS_ERR_UNSUPPORTED;
        int pick = -1;
        for (int v = 2; v >= 0 && pick < 0; --v)
            if ((p.Co % (64 << v) == 0 || v == 0) && conv_umma_pipe_applies(p, v)) pick = v;
        if (pick < 0) return EBS_ERR_UNSUPPORTED;
        const ConvVariant* bv = conv_umma_pipe_variant(0, pick);
        if (!bv) return EBS_ERR_UNSUPPORTED;
        plan->v = bv;
        plan->grid = dim3(1, 1, 1);
        return EBS_OK;
    }
    if (variant == -2) {
        variant = choose_variant(d->w_bits, d->a_bits, p.P, p.Co, packed_next != nullptr, sm_count());
    } else if (variant < 0) {
        const int pipe = mma_ok ? choose_pipe_variant(p, sm_count()) : -1;
        const int strip = (mma_ok && pipe < 0) ? choose_strip_variant(p) : -1;
        const int umma = (mma_ok && strip < 0 && pipe < 0) ? choose_umma_variant(p, d) : -1;
        // deep reductions whose weight tiles fit in shared memory: the persistent form of the same tile
        if (pipe >= 0) variant = PIPE_BASE + pipe;
        else if (strip >= 0 && p.CW * d->kh * d->kw >= 8 && conv_umma_resident_applies(p, strip)) variant = RES_BASE + strip;
        else if (strip >= 0) variant = STRIP_BASE + strip;
        else if (umma >= 0) variant = NUM_CONV_VARIANTS + NUM_CONV_MMA_VARIANTS + umma;
        // small stride-1 k x k layers with up to 64 output channels: the warp-level strip kernel (it expands every input
        // pixel once instead of once per tap, and its time does not grow with the plane count) at any batch size --
        // measured against every other variant on 16-, 32- and 64-channel layers from 1 to 64 images it is 15-45%
        // faster; 1x1 layers have nothing to save there and stay on the per-tap kernel.  33-64 channels: the
        // 32-channel tile (two CTAs per pixel tile) below 2^13 output pixels, the 64-channel tile from there.
        else if (mma_ok && p.Co <= 16 && d->kh * d->kw > 1 && conv_mma_strip_applies(p, 0)) variant = MS_BASE;
        else if (mma_ok && p.Co > 16 && p.Co <= 32 && d->kh * d->kw > 1 && conv_mma_strip_applies(p, 1)) variant = MS_BASE + 1;
        else if (mma_ok && p.Co > 32 && p.Co <= 64 && d->kh * d->kw > 1 && p.P < (1 << 13) && conv_mma_strip_applies(p, 1))
            variant = MS_BASE + 1;
        else if (mma_ok && p.Co > 32 && p.Co <= 64 && d->kh * d->kw > 1 && conv_mma_strip_applies(p, 2))
            variant = MS_BASE + 2;
        else variant = mma_ok ? NUM_CONV_VARIANTS + choose_mma_variant(d->w_bits, d->a_bits, p.P, p.Co, sm_count())
                              : choose_variant(d->w_bits, d->a_bits, p.P, p.Co, packed_next != nullptr, sm_count());
    }
    if (variant >= NUM_CONV_VARIANTS && !mma_ok) return EBS_ERR_UNSUPPORTED;
    if (variant >= PIPE_BASE) {
        if (!conv_umma_pipe_applies(p, variant - PIPE_BASE)) return EBS_ERR_UNSUPPORTED;
    } else if (variant >= MS_BASE) {
        if (!conv_mma_strip_applies(p, variant - MS_BASE)) return EBS_ERR_UNSUPPORTED;
    } else if (variant >= RES_BASE) {
        if (!conv_umma_resident_applies(p, variant - RES_BASE)) return EBS_ERR_UNSUPPORTED;
    } else if (variant >= STRIP_BASE && !conv_umma_strip_applies(p, variant - STRIP_BASE)) {
        return EBS_ERR_UNSUPPORTED;
    }
    const ConvVariant* v =
        variant >= PIPE_BASE ? conv_umma_pipe_variant(d->a_bits, variant - PIPE_BASE) :
        variant >= MS_BASE ? conv_mma_strip_variant(d->a_bits, variant - MS_BASE) :
        variant >= RES_BASE ? conv_umma_resident_variant(d->a_bits, variant - RES_BASE) :
        variant >= STRIP_BASE ? conv_umma_strip_variant(d->a_bits, variant - STRIP_BASE) :
        variant >= NUM_CONV_VARIANTS + NUM_CONV_MMA_VARIANTS
            ? conv_umma_variant(d->w_bits, d->a_bits, variant - NUM_CONV_VARIANTS - NUM_CONV_MMA_VARIANTS)
            : (variant >= NUM_CONV_VARIANTS ? conv_mma_variant(d->w_bits, d->a_bits, variant - NUM_CONV_VARIANTS)
                                            : conv_popc_variant(d->w_bits, d->a_bits, variant));
    if (!v) return EBS_ERR_UNSUPPORTED;
    if (packed_next && (v->tile_c % 32) != 0 && v->tile_c < p.Co) return EBS_ERR_UNSUPPORTED;
    const long long gx = (P + v->tile_p - 1) / v->tile_p, gy = (p.Co + v->tile_c - 1) / v->tile_c;
    if (gy > 65535) return EBS_ERR_UNSUPPORTED;
    plan->v = v;
    plan->grid = dim3((unsigned)gx, (unsigned)gy, 1);
    return EBS_OK;
}

static int conv_launch(const ConvPlan& plan, void* stream) {
    const int rc = plan.v->launch(plan.p, plan.grid, static_cast<cudaStream_t>(stream));
    if (rc) return rc;
    return check_cuda(cudaGetLastError());
}

static int conv_impl(const void* packed_x, int n, int h, int w, const void* packed_w, const ebs_conv_desc* d,
                     const ebs_epilogue* epi, int32_t* acc_out, float* y_out, void* packed_next, void* stream,
                     int variant) {
    ConvPlan plan;
    const int rc = conv_plan(packed_x, n, h, w, packed_w, d, epi, acc_out, y_out, packed_next, variant, &plan);
    if (rc) return rc;
    return conv_launch(plan, stream);
}

}  // namespace ebs

using namespace ebs;

extern "C" {

int ebs_version(void) { return 100; }

const char* ebs_status_string(int status) {
    switch (status) {
        case EBS_OK: return "ok";
        case EBS_ERR_INVALID_ARG: return "invalid argument";
        case EBS_ERR_UNSUPPORTED: return "unsupported configuration";
        case EBS_ERR_OVERFLOW: return "accumulator or index would overflow";
        case EBS_ERR_CUDA: return "CUDA runtime error";
        case EBS_ERR_TIMEOUT: return "device-side wait timed out";
        case EBS_ERR_SCRATCH_TOO_SMALL: return "request exceeds the built-in scratch of the no-allocation call";
        default: return "unknown status";
    }
}

const char* ebs_last_cuda_error(void) { return g_cuda_error; }

int ebs_conv_out_shape(const ebs_conv_desc* d, int h, int w, int* h_out, int* w_out) {
    int rc = validate_desc(d);
    if (rc) return rc;
    if (h <= 0 || w <= 0 || !h_out || !w_out) return EBS_ERR_INVALID_ARG;
    const int Ho = out_dim(h, d->pad_h, d->kh, d->stride_h), Wo = out_dim(w, d->pad_w, d->kw, d->stride_w);
    if (Ho <= 0 || Wo <= 0) return EBS_ERR_INVALID_ARG;
    *h_out = Ho;
    *w_out = Wo;
    return EBS_OK;
}

size_t ebs_packed_weight_bytes(const ebs_conv_desc* d) {
    if (validate_desc(d)) return 0;
    return packed_weight_plane_bytes(*d) + packed_weight_image_bytes(*d);
}

size_t ebs_packed_weight_plane_bytes(const ebs_conv_desc* d) {
    if (validate_desc(d)) return 0;
    return packed_weight_plane_bytes(*d);
}

size_t ebs_packed_act_bytes(int n, int h, int w, int c, int a_bits) {
    if (n <= 0 || h <= 0 || w <= 0 || c <= 0 || a_bits < 1 || a_bits > 8) return 0;
    return (size_t)n * h * w * ((c + 31) / 32) * a_bits * sizeof(uint32_t);
}

int ebs_pack_weights(const void* w_dev, int dtype, int layout, const ebs_conv_desc* d, void* packed_w_dev,
                     void* stream) {
    int rc = validate_desc(d);
    if (rc) return rc;
    if (!w_dev || !packed_w_dev || !aligned16(w_dev) || !aligned16(packed_w_dev)) return EBS_ERR_INVALID_ARG;
    if (dtype != EBS_F32 && dtype != EBS_I8_CODES) return EBS_ERR_INVALID_ARG;
    if (layout != EBS_NCHW && layout != EBS_NHWC) return EBS_ERR_INVALID_ARG;
    return launch_pack_weights(w_dev, dtype, layout, *d, 1.0f / d->w_scale, static_cast<uint32_t*>(packed_w_dev),
                               static_cast<cudaStream_t>(stream));
}

static int validate_pack_acts(const void* x_dev, int dtype, int layout, int n, int c, int h, int w, int a_bits,
                              float a_scale, const void* packed_x_dev) {
    if (!x_dev || !packed_x_dev || n <= 0 || c <= 0 || h <= 0 || w <= 0) return EBS_ERR_INVALID_ARG;
    if (a_bits < 1 || a_bits > 8) return EBS_ERR_INVALID_ARG;
    if (dtype != EBS_F32 && dtype != EBS_U8_CODES) return EBS_ERR_INVALID_ARG;
    if (layout != EBS_NCHW && layout != EBS_NHWC) return EBS_ERR_INVALID_ARG;
    if (dtype == EBS_F32 && !(a_scale > 0.0f)) return EBS_ERR_INVALID_ARG;
    if (!aligned16(x_dev) || !aligned16(packed_x_dev)) return EBS_ERR_INVALID_ARG;
    if ((long long)n * h * w >= (1LL << 31)) return EBS_ERR_OVERFLOW;
    return EBS_OK;
}

int ebs_pack_acts(const void* x_dev, int dtype, int layout, int n, int c, int h, int w, int a_bits, float a_scale,
                  void* packed_x_dev, void* stream) {
    const int rc = validate_pack_acts(x_dev, dtype, layout, n, c, h, w, a_bits, a_scale, packed_x_dev);
    if (rc) return rc;
    const float inv = dtype == EBS_F32 ? 1.0f / a_scale : 1.0f;
    return launch_pack_acts(x_dev, dtype, layout, n, c, h, w, a_bits, inv, static_cast<uint32_t*>(packed_x_dev),
                            static_cast<cudaStream_t>(stream));
}

int ebs_pack_acts_s2d(const void* x_dev, int n, int c, int h, int w, int offset, int a_bits, void* packed_x_dev,
                      void* stream) {
    if (!x_dev || !packed_x_dev || n <= 0 || c <= 0 || h <= 0 || w <= 0) return EBS_ERR_INVALID_ARG;
    if (a_bits < 1 || a_bits > 8 || (offset != 0 && offset != 1)) return EBS_ERR_INVALID_ARG;
    if (4 * c > 32 || (h & 1) || (w & 1)) return EBS_ERR_UNSUPPORTED;
    if (!aligned16(packed_x_dev)) return EBS_ERR_INVALID_ARG;
    if (h > 32000 || w > 32000 || (long long)n * h * w >= (1LL << 31)) return EBS_ERR_OVERFLOW;
    return launch_pack_acts_s2d(x_dev, n, c, h, w, offset, a_bits, static_cast<uint32_t*>(packed_x_dev),
                                static_cast<cudaStream_t>(stream));
}

int ebs_conv2d_mixed(const void* packed_x_dev, int n, int h, int w, const void* packed_w_dev,
                     const ebs_conv_desc* desc, const ebs_epilogue* epi, int32_t* acc_out_dev, float* y_out_dev,
                     void* packed_next_dev, void* stream) {
    return conv_impl(packed_x_dev, n, h, w, packed_w_dev, desc, epi, acc_out_dev, y_out_dev, packed_next_dev,
                     stream, -1);
}

int ebs_conv2d_i8(const void* x_codes_dev, int n, int h, int w, const void* packed_w_dev, const ebs_conv_desc* desc,
                  const ebs_epilogue* epi, int32_t* acc_out_dev, float* y_out_dev, void* packed_next_dev, void* stream) {
    ConvPlan plan;
    const int rc = conv_plan(x_codes_dev, n, h, w, packed_w_dev, desc, epi, acc_out_dev, y_out_dev, packed_next_dev, -1,
                             &plan, true);
    if (rc) return rc;
    return conv_launch(plan, stream);
}

int ebs_num_conv_variants(void) {
    return NUM_CONV_VARIANTS + NUM_CONV_MMA_VARIANTS + NUM_CONV_UMMA_VARIANTS + NUM_CONV_STRIP_VARIANTS +
           NUM_CONV_RESIDENT_VARIANTS + NUM_CONV_MMA_STRIP_VARIANTS + NUM_CONV_PIPE_VARIANTS;
}

const char* ebs_conv_variant_family(int variant) {
    int v = variant;
    if (v < 0) return "";
    if (v < NUM_CONV_VARIANTS) return "popc";
    v -= NUM_CONV_VARIANTS;
    if (v < NUM_CONV_MMA_VARIANTS) return "mma";
    v -= NUM_CONV_MMA_VARIANTS;
    if (v < NUM_CONV_UMMA_VARIANTS) return "umma";
    v -= NUM_CONV_UMMA_VARIANTS;
    if (v < NUM_CONV_STRIP_VARIANTS) return "umma_strip";
    v -= NUM_CONV_STRIP_VARIANTS;
    if (v < NUM_CONV_RESIDENT_VARIANTS) return "umma_resident";
    v -= NUM_CONV_RESIDENT_VARIANTS;
    if (v < NUM_CONV_MMA_STRIP_VARIANTS) return "mma_strip";
    v -= NUM_CONV_MMA_STRIP_VARIANTS;
    if (v < NUM_CONV_PIPE_VARIANTS) return "umma_pipe";
    return "";
}

int ebs_conv_variant_applies(const ebs_conv_desc* desc, int n, int h, int w, const ebs_epilogue* epi, int want_acc,
                             int want_y, int want_packed_next, int variant) {
    // the validation and selection of a launch with stand-in buffers (aligned, never dereferenced): nothing is enqueued
    void* fake = reinterpret_cast<void*>(static_cast<uintptr_t>(256));
    ConvPlan plan;
    return conv_plan(fake, n, h, w, fake, desc, epi, want_acc ? static_cast<int32_t*>(fake) : nullptr,
                     want_y ? static_cast<float*>(fake) : nullptr, want_packed_next ? fake : nullptr, variant, &plan);
}

int ebs_test_set_device_wait(unsigned int limit, int skip_mma) {
    g_wait_limit = limit == 0 ? (1u << 20) : limit;
    g_test_flags = skip_mma ? 1 : 0;
    return EBS_OK;
}

int ebs_check_device_status(void) {
    static long long seen = 0;
    const long long now = (long long)conv_umma_timeouts();
    const bool fresh = now > seen;
    seen = now;
    return fresh ? EBS_ERR_TIMEOUT : EBS_OK;
}

int ebs_checked_build(void) {
#ifdef EBS_CHECKED
    return 1;
#else
    return 0;
#endif
}

int ebs_checked_status(int* site, long long* index, long long* limit, int clear) {
#ifdef EBS_CHECKED
    unsigned long long w[4] = {0, 0, 0, 0};
    if (cudaDeviceSynchronize() != cudaSuccess) return EBS_ERR_CUDA;
    if (cudaMemcpyFromSymbol(w, g_check_words, sizeof(w)) != cudaSuccess) return EBS_ERR_CUDA;
    if (site) *site = (int)(w[0] >> 48);
    if (index) *index = (long long)w[1];
    if (limit) *limit = (long long)w[2];
    if (clear) {
        const unsigned long long z[4] = {0, 0, 0, 0};
        if (cudaMemcpyToSymbol(g_check_words, z, sizeof(z)) != cudaSuccess) return EBS_ERR_CUDA;
    }
    return w[0] ? 1 : 0;
#else
    (void)site; (void)index; (void)limit; (void)clear;
    return EBS_ERR_UNSUPPORTED;
#endif
}

int ebs_test_checked_shrink(long long elements) {
#ifdef EBS_CHECKED
    if (elements < 0) return EBS_ERR_INVALID_ARG;
    g_check_shrink = elements;
    return EBS_OK;
#else
    (void)elements;
    return EBS_ERR_UNSUPPORTED;
#endif
}

long long ebs_device_wait_timeouts(void) { return (long long)conv_umma_timeouts(); }

int ebs_conv2d_mixed_variant(const void* packed_x_dev, int n, int h, int w, const void* packed_w_dev,
                             const ebs_conv_desc* desc, const ebs_epilogue* epi, int32_t* acc_out_dev,
                             float* y_out_dev, void* packed_next_dev, void* stream, int variant) {
    return conv_impl(packed_x_dev, n, h, w, packed_w_dev, desc, epi, acc_out_dev, y_out_dev, packed_next_dev,
                     stream, variant);
}

int ebs_dequant(const int32_t* acc_dev, size_t n_pixels, int c_out, float scale, const float* ch_scale_dev,
                const float* ch_bias_dev, int relu, float* y_dev, void* stream) {
    if (!acc_dev || !y_dev || n_pixels == 0 || c_out <= 0) return EBS_ERR_INVALID_ARG;
    if (!aligned16(acc_dev) || !aligned16(y_dev)) return EBS_ERR_INVALID_ARG;
    if (n_pixels >= ((size_t)1 << 40) / (size_t)c_out) return EBS_ERR_OVERFLOW;
    return launch_dequant(acc_dev, n_pixels, c_out, scale, ch_scale_dev, ch_bias_dev, relu ? 1 : 0, y_dev,
                          static_cast<cudaStream_t>(stream));
}

int ebs_search_weight_forward(const float* w_dev, size_t n, const int* bits, const float* coeff, int n_cand,
                              float* w_hat_dev, void* scratch_dev, void* stream) {
    if (!w_dev || !w_hat_dev || !scratch_dev || n == 0) return EBS_ERR_INVALID_ARG;
    if (!aligned16(w_dev) || !aligned16(w_hat_dev) || !aligned16(scratch_dev)) return EBS_ERR_INVALID_ARG;
    return launch_search_weights(w_dev, n, bits, coeff, n_cand, w_hat_dev, scratch_dev, static_cast<cudaStream_t>(stream));
}

int ebs_search_act_forward(const float* x_dev, size_t n, float alpha, const int* bits, const float* coeff, int n_cand,
                           float* x_hat_dev, void* stream) {
    if (!x_dev || !x_hat_dev || n == 0 || !(alpha > 0.0f)) return EBS_ERR_INVALID_ARG;
    if (!aligned16(x_dev) || !aligned16(x_hat_dev)) return EBS_ERR_INVALID_ARG;
    return launch_search_acts(x_dev, n, alpha, bits, coeff, n_cand, x_hat_dev, static_cast<cudaStream_t>(stream));
}

float ebs_combined_scale(float w_scale, float a_scale) { return w_scale * a_scale; }        // one rounded fp32 multiply
float ebs_reciprocal_step(float step) { return 1.0f / step; }                               // one rounded fp32 division

double ebs_expected_flops(double macs, const int* bits_w, const float* coeff_w, int n_w, const int* bits_x,
                          const float* coeff_x, int n_x) {
    if (!bits_w || !coeff_w || !bits_x || !coeff_x || n_w < 1 || n_x < 1 || !(macs >= 0.0)) return -1.0;
    double m = 0.0, k = 0.0;
    for (int i = 0; i < n_w; ++i) m += (double)coeff_w[i] * bits_w[i];
    for (int j = 0; j < n_x; ++j) k += (double)coeff_x[j] * bits_x[j];
    return macs * m * k;
}

int ebs_fused_plan_upload(const ebs_fused_layer* layers_host, int n_layers, void* layers_dev, void* stream) {
    if (!layers_host || !layers_dev || n_layers < 1 || n_layers > 4096) return EBS_ERR_INVALID_ARG;
    return fused_plan_upload(layers_host, n_layers, layers_dev, static_cast<cudaStream_t>(stream));
}

int ebs_resnet_cifar_forward(const unsigned char* images_dev, int n, int img_h, int img_w, const void* layers_dev,
                             int n_layers, const ebs_fused_head* head_host, float* logits_dev, unsigned char* trace_dev,
                             long long trace_stride, void* stream) {
    if (!images_dev || !layers_dev || !head_host || !logits_dev || n < 1 || n_layers < 1) return EBS_ERR_INVALID_ARG;
    if (img_h < 1 || img_w < 1 || (img_h + 2) * (img_w + 2) > 1156) return EBS_ERR_UNSUPPORTED;
    if (!head_host->w8 || head_host->c_in < 1 || head_host->c_in > 64 || head_host->c_out < 1 || head_host->c_out > 256)
        return EBS_ERR_INVALID_ARG;
    return launch_fused_resnet(images_dev, n, img_h, img_w, layers_dev, n_layers, head_host, logits_dev, trace_dev,
                               trace_stride, static_cast<cudaStream_t>(stream));
}

int ebs_global_avgpool(const float* y_dev, int n, int hw, int c, float* out_dev, void* stream) {
    if (!y_dev || !out_dev || n <= 0 || hw <= 0 || c <= 0) return EBS_ERR_INVALID_ARG;
    if ((long long)n * c >= (1LL << 31)) return EBS_ERR_OVERFLOW;
    return launch_avgpool(y_dev, n, hw, c, out_dev, static_cast<cudaStream_t>(stream));
}

int ebs_maxpool_packed(const void* packed_x_dev, int n, int h, int w, int c, int a_bits, int k, int stride, int pad,
                       void* packed_out_dev, void* stream) {
    if (!packed_x_dev || !packed_out_dev || n <= 0 || h <= 0 || w <= 0 || c <= 0) return EBS_ERR_INVALID_ARG;
    if (a_bits < 1 || a_bits > 8 || k < 1 || stride < 1 || pad < 0 || pad >= k) return EBS_ERR_INVALID_ARG;
    if (!aligned16(packed_x_dev) || !aligned16(packed_out_dev) || packed_x_dev == packed_out_dev) return EBS_ERR_INVALID_ARG;
    const int ho = out_dim(h, pad, k, stride), wo = out_dim(w, pad, k, stride);
    if (ho <= 0 || wo <= 0) return EBS_ERR_INVALID_ARG;
    if ((long long)n * h * w * ((c + 31) / 32) * a_bits >= (1LL << 31)) return EBS_ERR_OVERFLOW;
    return launch_maxpool_packed(static_cast<const uint32_t*>(packed_x_dev), n, h, w, c, a_bits, k, stride, pad, ho, wo,
                                 static_cast<uint32_t*>(packed_out_dev), static_cast<cudaStream_t>(stream));
}

static size_t round256(size_t v) { return (v + 255) & ~(size_t)255; }

size_t ebs_host_workspace_bytes(const ebs_conv_desc* d, int n, int h, int w, int dtype, int next_a_bits) {
    if (validate_desc(d) || n <= 0 || h <= 0 || w <= 0) return 0;
    const int Ho = out_dim(h, d->pad_h, d->kh, d->stride_h), Wo = out_dim(w, d->pad_w, d->kw, d->stride_w);
    if (Ho <= 0 || Wo <= 0) return 0;
    const size_t elems_in = (size_t)n * h * w * d->c_in, outs = (size_t)n * Ho * Wo * d->c_out;
    size_t total = round256(elems_in * (dtype == EBS_F32 ? 4 : 1));
    total += round256(ebs_packed_act_bytes(n, h, w, d->c_in, d->a_bits));
    total += round256(outs * 4) * 2;                                   // acc and y
    if (next_a_bits >= 1 && next_a_bits <= 8) total += round256(ebs_packed_act_bytes(n, Ho, Wo, d->c_out, next_a_bits));
    return total;
}

int ebs_conv2d_mixed_host(const void* x_host, int dtype, int layout, int n, int h, int w, const void* packed_w_dev,
                          const ebs_conv_desc* d, const ebs_epilogue* epi, void* workspace_dev, size_t workspace_bytes,
                          int32_t* acc_out_host, float* y_out_host, void* packed_next_host, void* stream) {
    int rc = validate_desc(d);
    if (rc) return rc;
    if (!x_host || !workspace_dev || !aligned16(workspace_dev) || n <= 0 || h <= 0 || w <= 0) return EBS_ERR_INVALID_ARG;
    if (dtype != EBS_F32 && dtype != EBS_U8_CODES) return EBS_ERR_INVALID_ARG;
    if (!acc_out_host && !y_out_host && !packed_next_host) return EBS_ERR_INVALID_ARG;
    if (packed_next_host && (!epi || epi->next_a_bits < 1 || epi->next_a_bits > 8)) return EBS_ERR_INVALID_ARG;
    const int next_bits = packed_next_host ? epi->next_a_bits : 0;
    const size_t need = ebs_host_workspace_bytes(d, n, h, w, dtype, next_bits);
    if (need == 0 || workspace_bytes < need) return EBS_ERR_INVALID_ARG;
    const int Ho = out_dim(h, d->pad_h, d->kh, d->stride_h), Wo = out_dim(w, d->pad_w, d->kw, d->stride_w);
    const size_t elems_in = (size_t)n * h * w * d->c_in, outs = (size_t)n * Ho * Wo * d->c_out;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    char* ws = static_cast<char*>(workspace_dev);
    void* x_dev = ws;                 ws += round256(elems_in * (dtype == EBS_F32 ? 4 : 1));
    void* px_dev = ws;                ws += round256(ebs_packed_act_bytes(n, h, w, d->c_in, d->a_bits));
    int32_t* acc_dev = (int32_t*)ws;  ws += round256(outs * 4);
    float* y_dev = (float*)ws;        ws += round256(outs * 4);
    void* pn_dev = ws;

    // every argument check of the two device calls comes first: an error return means nothing was enqueued
    // (and, for the caller that shares one scratch between calls, that the scratch was not touched)
    rc = validate_pack_acts(x_dev, dtype, layout, n, d->c_in, h, w, d->a_bits, d->a_scale, px_dev);
    if (rc) return rc;
    ConvPlan plan;
    rc = conv_plan(px_dev, n, h, w, packed_w_dev, d, epi, acc_out_host ? acc_dev : nullptr,
                   y_out_host ? y_dev : nullptr, packed_next_host ? pn_dev : nullptr, -1, &plan);
    if (rc) return rc;

    rc = check_cuda(cudaMemcpyAsync(x_dev, x_host, elems_in * (dtype == EBS_F32 ? 4 : 1), cudaMemcpyHostToDevice, st));
    if (rc) return rc;
    rc = ebs_pack_acts(x_dev, dtype, layout, n, d->c_in, h, w, d->a_bits, d->a_scale, px_dev, stream);
    if (rc) return rc;
    rc = conv_launch(plan, stream);
    if (rc) return rc;
    if (acc_out_host) {
        rc = check_cuda(cudaMemcpyAsync(acc_out_host, acc_dev, outs * 4, cudaMemcpyDeviceToHost, st));
        if (rc) return rc;
    }
    if (y_out_host) {
        rc = check_cuda(cudaMemcpyAsync(y_out_host, y_dev, outs * 4, cudaMemcpyDeviceToHost, st));
        if (rc) return rc;
    }
    if (packed_next_host) {
        rc = check_cuda(cudaMemcpyAsync(packed_next_host, pn_dev, ebs_packed_act_bytes(n, Ho, Wo, d->c_out, next_bits),
                                        cudaMemcpyDeviceToHost, st));
        if (rc) return rc;
    }
    return EBS_OK;
}

}  // extern "C"
