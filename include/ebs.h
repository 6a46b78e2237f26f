/*
 * ebs.h -- C ABI of the binary-decomposition (BD) mixed-precision convolution
 * library for NVIDIA B200 (sm_100a).
 *
 * The operation (paper Sec. 4.3, Eq. 12-15, built on Eq. 2): a convolution between
 * M-bit weights and K-bit activations is computed by splitting both operands into
 * binary bit-planes; stage 1 is a binary convolution (AND + bitcount) between every
 * weight plane m and activation plane k, stage 2 recombines the M*K partial results
 * with powers of two 2^(m+k).  Every layer may use its own (M, K).  In this header
 * M is `w_bits` and K is `a_bits`.
 *
 * Number formats.  Activation codes are unsigned, 0 .. 2^a_bits-1 (Eq. 1b: the
 * activation is a_scale * code with a_scale = alpha / (2^a_bits-1)).  Weight codes
 * are signed two's complement, -2^(w_bits-1) .. 2^(w_bits-1)-1, real value w_scale *
 * code; the top weight plane therefore carries the coefficient -2^(w_bits-1).
 * Rounding is "round half up" (text after Eq. 1c): code = floor(x * (1/scale) + 0.5),
 * evaluated in fp32 with 1/scale rounded once and every operation rounded on its own.
 *
 * Conventions for every entry point
 *  - Pointers named *_dev are DEVICE pointers on the current CUDA device; pointers
 *    named *_host are host pointers.  All buffers are owned by the caller; the library
 *    keeps no state between calls and allocates nothing (the one exception is the
 *    measurement helper ebs_probe_pipe, which allocates and frees a small scratch).
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *    Work is enqueued on it and the call returns without waiting.
 *  - Device buffers must be 16-byte aligned (buffers from cudaMalloc / torch are).
 *  - Return value: an ebs_status (0 = success, negative = error).  Arguments are
 *    validated on the host before anything is launched; on error nothing has been
 *    enqueued.  No call aborts, throws or traps.
 *
 * Packed bit-plane layouts (little-endian 32-bit words, CW = ceil(C/32)):
 *  - activations  u32 [N][H][W][CW][a_bits]: bit (c % 32) of word [n][h][w][c/32][k]
 *    is bit k of the code of channel c at pixel (n,h,w);
 *  - weights      u32 [kh][kw][CW][C_out][w_bits]: bit (c % 32) of word
 *    [r][s][c/32][co][m] is bit m of the two's-complement code of W[co][c][r][s];
 *  - bits of channels >= C are zero in both.
 */
#ifndef EBS_H_
#define EBS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum ebs_status {
    EBS_OK = 0,
    EBS_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, bitwidth outside 1..8, misalignment */
    EBS_ERR_UNSUPPORTED = -2, /* valid request this build has no kernel for */
    EBS_ERR_OVERFLOW = -3,    /* c_in*kh*kw*2^(w_bits-1)*(2^a_bits-1) >= 2^31 (w_levels = 1: c_in*kh*kw*(2^w_bits-1)*
                                 (2^a_bits-1)), or an index would overflow */
    EBS_ERR_CUDA = -4,        /* a CUDA runtime call failed (launch error, bad device pointer, ...) */
    EBS_ERR_TIMEOUT = -5,     /* a bounded device-side wait gave up (reported by ebs_check_device_status) */
    EBS_ERR_SCRATCH_TOO_SMALL = -6 /* the request needs more than the built-in scratch of the no-allocation call */
} ebs_status;

typedef enum ebs_layout {
    EBS_NCHW = 0, /* activations [N][C][H][W]; weights [C_out][C_in][kh][kw] */
    EBS_NHWC = 1  /* activations [N][H][W][C]; weights [C_out][kh][kw][C_in] */
} ebs_layout;

typedef enum ebs_dtype {
    EBS_F32 = 0,      /* real values; quantized inside the call (Eq. 1b / 1c) */
    EBS_I8_CODES = 1, /* signed 8-bit integer codes (weights) */
    EBS_U8_CODES = 2  /* unsigned 8-bit integer codes (activations) */
} ebs_dtype;

/* One convolution layer (Sec. 3: weight tensor c_i x c_o x k x k; Sec. 4.3: per-layer M and K). */
typedef struct ebs_conv_desc {
    int c_in, c_out;
    int kh, kw;
    int stride_h, stride_w;
    int pad_h, pad_w;   /* zero padding: a padded tap is the real value 0 */
    int w_bits, a_bits; /* M and K of the paper, 1..8 each */
    float w_scale;      /* real weight  = w_scale * code (w_levels = 0) or w_scale * (2*code + 1) (w_levels = 1) */
    float a_scale;      /* real input   = a_scale * code */
    int w_levels;       /* 0: two's-complement weights, real weight = w_scale * code.
                           1: the paper's own weight levels (Eq. 1a): the 2^b levels 2*q_u - (2^b - 1), q_u = 0 .. 2^b-1,
                              symmetric about zero; stored as the signed code q_u - 2^(b-1), so the level is
                              2*code + 1 and w_scale = 1/(2^b - 1) gives the paper's range [-1, 1].  The accumulator
                              is then sum (2*code + 1) * activation code = 2 * (bit-plane sum) + (sum of the
                              activation codes under the filter window); the window sum is taken from the
                              activation planes inside the same kernel. */
} ebs_conv_desc;

/*
 * Optional epilogue after the integer accumulator (scale merge of Sec. 4.3, clip and
 * round of Eq. 1b-1c / Eq. 16a-16c), each step a separately rounded fp32 operation:
 *   y = float(acc) * S                 S = fl32(w_scale * a_scale)
 *   y = y * ch_scale[co]               if ch_scale_dev
 *   y = y + ch_bias[co]                if ch_bias_dev
 *   y = y + residual[n][ho][wo][co]    if residual_dev   (fp32, NHWC, output shape)
 *   y = y + res_scale * code           if res_packed_dev (the shortcut of a residual block given as packed
 *                                      activation planes u32 [N][Ho][Wo][ceil(C_out/32)][res_bits], e.g. the block's
 *                                      own packed input: it is de-quantized on the fly, one rounded multiply)
 *   y = max(y, 0)                      if relu
 *   q = clamp(floor(y * (1/next_a_scale) + 0.5), 0, 2^next_a_bits - 1)   (packed output only)
 * A NULL epilogue means: no per-channel terms, no residual, no ReLU, y in NHWC.
 */
typedef struct ebs_epilogue {
    const float *ch_scale_dev; /* nullable, length c_out */
    const float *ch_bias_dev;  /* nullable, length c_out */
    const float *residual_dev; /* nullable */
    int relu;                  /* 0 / 1 */
    int next_a_bits;           /* bitwidth of packed_next (1..8); ignored if packed_next is NULL */
    float next_a_scale;        /* step of the next layer's activation quantizer */
    int y_layout;              /* ebs_layout of y_out */
    const void *res_packed_dev; /* nullable; packed planes with the output's pixel grid and c_out channels */
    int res_bits;              /* planes of res_packed_dev (1..8) */
    float res_scale;           /* real value of a residual code */
} ebs_epilogue;

/* Library version (major*10000 + minor*100 + patch). */
int ebs_version(void);

/* Human-readable text for an ebs_status; never NULL. */
const char *ebs_status_string(int status);

/* Text of the last CUDA error seen by this thread's failing call ("" if none). */
const char *ebs_last_cuda_error(void);

/* Output height/width of the img2col convolution (Sec. 4.3): floor((in + 2 pad - k)/stride) + 1.
 * Returns EBS_ERR_INVALID_ARG if the kernel is larger than the padded input. */
int ebs_conv_out_shape(const ebs_conv_desc *desc, int h, int w, int *h_out, int *w_out);

/* Size in bytes of the packed weight buffer of a layer.  It has two parts:
 *   1. the bit planes B_w, kh*kw*ceil(c_in/32)*c_out*w_bits 32-bit words laid out
 *      [kh][kw][ceil(c_in/32)][c_out][w_bits], the same memory as the weights before decomposition
 *      (Sec. 4.3, complexity), rounded up to a multiple of 256 bytes
 *      (ebs_packed_weight_plane_bytes);
 *   2. the same codes once more as one signed byte per (tap, channel, output channel) in the
 *      order the tensor-core kernels read them, kh*kw*ceil(c_in/32)*roundup(c_out,16)*32 bytes.
 *      The paper has no counterpart for part 2: it is a prepared copy of a static operand, written
 *      once by ebs_pack_weights, so that those kernels do not rebuild it in every thread block.
 * 0 on bad input. */
size_t ebs_packed_weight_bytes(const ebs_conv_desc *desc);
size_t ebs_packed_weight_plane_bytes(const ebs_conv_desc *desc);

/* Size in bytes of packed activation planes: n*h*w*ceil(c/32)*a_bits*4.  0 on bad input. */
size_t ebs_packed_act_bytes(int n, int h, int w, int c, int a_bits);

/*
 * Weight quantization and bit-plane expansion B_w (Eq. 12, Eq. 15; quantizer Eq. 1c).
 *   w_dev       c_out*c_in*kh*kw values in `layout`; EBS_F32 (quantized with desc->w_scale to
 *               signed desc->w_bits codes: code = floor(w/w_scale + 0.5), or with w_levels = 1 the
 *               nearest level, code = floor((w/w_scale + 2^b - 1)/2 + 0.5) - 2^(b-1), clamped) or
 *               EBS_I8_CODES (signed codes taken as they are; must be in range).
 *   packed_w_dev  ebs_packed_weight_bytes(desc) bytes, fully overwritten.
 * Done once per layer, off the inference path.
 */
int ebs_pack_weights(const void *w_dev, int dtype, int layout, const ebs_conv_desc *desc,
                     void *packed_w_dev, void *stream);

/*
 * Activation quantization (Eq. 1b: clip to [0, alpha], round half up) and bit-plane expansion B_x
 * (Sec. 4.3).  x_dev holds n*c*h*w values in `layout`; EBS_F32 (quantized with a_scale) or
 * EBS_U8_CODES (only the low a_bits bits of each code are used).  packed_x_dev receives
 * ebs_packed_act_bytes(n,h,w,c,a_bits) bytes, fully overwritten.
 */
int ebs_pack_acts(const void *x_dev, int dtype, int layout, int n, int c, int h, int w, int a_bits,
                  float a_scale, void *packed_x_dev, void *stream);

/*
 * Space-to-depth packing for a stride-2 first layer with few input channels (the paper has no counterpart: it leaves
 * the first layer unquantized; networks run it at 8 bits through this library).  x_dev: u8 codes, NHWC [n][h][w][c],
 * device memory, 4 * c <= 32, h and w even.  Output: bit planes in the packed activation layout of a tensor
 * [n][hs][ws] with 4 * c channels, hs = (h + offset) / 2 + offset (likewise ws): pixel (i, j) holds the 2 x 2 block of
 * input pixels (2 i - offset + dy, 2 j - offset + dx), dy, dx in {0, 1}, as channel (2 dy + dx) * c + ch; positions
 * outside the image are code 0.  A k x k, stride-2, pad-p convolution (k odd) over x equals a ((k + 1) / 2)-square,
 * stride-1, pad-((p - offset) / 2) convolution over this tensor with offset = p mod 2 and the weights regrouped as
 * w2[co][(2 dy + dx) * c + ch][bi][bj] = w[co][ch][2 bi + dy][2 bj + dx] (zero where 2 bi + dy or 2 bj + dx reaches
 * k): a quarter of the reduction words, four times as full.  packed_x_dev: ebs_packed_act_bytes(n, hs, ws, 4 * c,
 * a_bits) bytes, 16-byte aligned, caller-owned.  Asynchronous on `stream`.  Returns EBS_ERR_UNSUPPORTED for 4 * c > 32
 * or odd h / w, EBS_ERR_INVALID_ARG for null pointers, sizes <= 0, a_bits outside 1..8, offset outside {0, 1}.
 */
int ebs_pack_acts_s2d(const void* x_dev, int n, int c, int h, int w, int offset, int a_bits, void* packed_x_dev,
                      void* stream);

/*
 * The mixed-precision convolution by binary decomposition (Eq. 13-14): for every output
 * (n, ho, wo, co)
 *   acc = sum_{m<M} sum_{k<K} c_m 2^(m+k) * sum_{taps, channel words} popcount(A_k AND W_m),
 *   c_m = -1 for m = M-1 (signed weights), +1 otherwise,
 * with taps outside the image contributing zero; with desc->w_levels = 1 the accumulator is
 * 2 * acc + sum_{k<K} 2^k * sum_{taps, channel words} popcount(A_k) (see ebs_conv_desc).  The M*K partial sums (the paper's matrix P)
 * never leave the chip.  Any subset of the three outputs may be requested (at least one):
 *   acc_out_dev     int32 [N][Ho][Wo][C_out]                      exact accumulators
 *   y_out_dev       fp32, epilogue applied, layout epi->y_layout  (NHWC if epi is NULL)
 *   packed_next_dev u32 [N][Ho][Wo][ceil(C_out/32)][next_a_bits]  requantized, ready to be the
 *                   packed_x_dev of the next layer (requires epi)
 * packed_x_dev: activations [n][h][w] with desc->c_in channels and desc->a_bits planes;
 * packed_w_dev: weights of `desc`.  Both as produced by the pack calls (or a previous layer).
 */
int ebs_conv2d_mixed(const void *packed_x_dev, int n, int h, int w, const void *packed_w_dev,
                     const ebs_conv_desc *desc, const ebs_epilogue *epi, int32_t *acc_out_dev,
                     float *y_out_dev, void *packed_next_dev, void *stream);

/*
 * The same call with the kernel variant forced (0 .. ebs_num_conv_variants()-1) instead of chosen by
 * the built-in heuristic (-1); the result is identical for every variant, only the speed differs.
 *   0..9    integer-pipe kernels: the plane-pair double sum of Eq. 13-14 evaluated literally
 *           (AND + POPC + shift-add per plane pair);
 *   10..18  warp-level tensor-pipe kernels (int8 mma.sync; the planes of a channel merged into
 *           its byte in registers, one MMA per 32 channels of a tap);
 *   19..23  tcgen05 kernels, any stride (same product, 128 pixels x 16/32/64/128/256 channels
 *           per CTA, accumulator in tensor memory);
 *   24..28  tcgen05 strip kernels for stride-1 layers and strided 1x1 layers (every input
 *           pixel expanded once per CTA; weights read from the byte image);
 *   29..33  the same as persistent CTAs that keep the weight bytes of their channel tile in
 *           shared memory and overlap expansion, MMAs and epilogue of consecutive pixel tiles
 *           (layers whose weight tiles fit in 150 KB, w_levels = 0);
 *   34..36  warp-level kernels for small stride-1 layers (c_in 5..128, even c_out, NHWC
 *           output): the strip of input pixels expanded to bytes once per thread block,
 *           fragments loaded from shared memory, weights from the byte image; channel tile
 *           16 / 32 / 64;
 *   37..39  persistent pipeline tcgen05 kernels for stride-1 and strided k x k layers and 1x1 layers
 *           at any stride (stride <= 2, w_levels = 0): every input pixel expanded once per thread
 *           block and tile, several 128-pixel accumulators per weight tile, weights resident in
 *           shared memory or streamed, expansion / MMAs / epilogue of consecutive tiles overlapped;
 *           channel tile 64 / 128 / 256.
 * variant = -2 lets the library choose among the integer-pipe kernels only (the literal
 * bit-plane evaluation), for comparison runs.
 * For tuning and for tests that must cover every kernel instantiation.  Returns
 * EBS_ERR_UNSUPPORTED if the variant does not apply to the layer or cannot produce the requested
 * packed output.
 */
int ebs_num_conv_variants(void);
int ebs_conv2d_mixed_variant(const void *packed_x_dev, int n, int h, int w, const void *packed_w_dev,
                             const ebs_conv_desc *desc, const ebs_epilogue *epi, int32_t *acc_out_dev,
                             float *y_out_dev, void *packed_next_dev, void *stream, int variant);

/*
 * Context kernel, NOT the paper's method: the same convolution with the activations given as unpacked 8-bit codes
 * (u8, NHWC [n][h][w][c_in], c_in a multiple of 32) instead of bit planes.  The codes go straight into the int8
 * tensor-core operand (no bit-plane expansion); weights, epilogue, outputs and results are those of
 * ebs_conv2d_mixed (desc->a_bits only documents the code range; the result is exact for any u8 codes within the
 * overflow bound of desc).  It exists to measure what keeping the activations as bit planes in memory costs or
 * saves on this machine: a_bits/8 of the activation traffic against the expansion work (the paper motivates the
 * decomposition by hardware that has only INT8/INT4/binary operations, Sec. 1).  Runs on the persistent pipeline
 * kernels; EBS_ERR_UNSUPPORTED where they do not apply (c_in not a multiple of 32, stride above 2, w_levels = 1).
 */
int ebs_conv2d_i8(const void *x_codes_dev, int n, int h, int w, const void *packed_w_dev, const ebs_conv_desc *desc,
                  const ebs_epilogue *epi, int32_t *acc_out_dev, float *y_out_dev, void *packed_next_dev,
                  void *stream);

/*
 * Which kernel family a variant number belongs to ("popc", "mma", "umma", "umma_strip", "umma_resident",
 * "mma_strip", "umma_pipe"; "" if out of range), and whether a variant can run a layer: the full validation and
 * kernel selection of ebs_conv2d_mixed_variant for a request with the given outputs (want_* are 0 / 1), without
 * touching any buffer and without launching anything.  Returns EBS_OK, EBS_ERR_UNSUPPORTED, or the error the real
 * call would return.  For tests and tuning tools that have to enumerate the variants of a layer.
 */
const char *ebs_conv_variant_family(int variant);
int ebs_conv_variant_applies(const ebs_conv_desc *desc, int n, int h, int w, const ebs_epilogue *epi, int want_acc,
                             int want_y, int want_packed_next, int variant);

/*
 * Number of thread blocks that gave up a bounded device-side wait (on the tensor core's completion
 * barrier) since the library was loaded; such a block skips its outputs.  0 in a healthy run.
 * Synchronizes the device.  The paper has no counterpart.
 */
long long ebs_device_wait_timeouts(void);

/*
 * EBS_ERR_TIMEOUT if thread blocks gave up a bounded wait since the previous call of this function (their
 * outputs are missing: run the layer again), else EBS_OK.  Synchronizes the device.  A launch itself cannot
 * report this: it returns before the kernel runs.  The paper has no counterpart.
 */
int ebs_check_device_status(void);

/*
 * The range-checked build (the paper has no counterpart).  The library is built twice from the same sources:
 * libebs.so, and libebs_checked.so with -DEBS_CHECKED, in which the convolution kernels pass the indices they
 * compute from the run-time geometry (offsets into the operand and result buffers, into their shared-memory rings
 * and tables) through a range test before the access.  A violation is recorded on the device -- the first one wins
 * -- and the access is skipped: nothing traps, the kernel runs to its end, results may be incomplete.
 * ebs_checked_build: 1 in the checked library, 0 in the normal one.
 * ebs_checked_status: synchronizes the device; returns 1 if a violation was recorded (and stores the site code --
 * kernel family * 16 + access, see CheckSite in csrc/ebs_internal.cuh --, the offending index and its limit in the
 * non-null host pointers), 0 if none, EBS_ERR_UNSUPPORTED in the normal build, EBS_ERR_CUDA if a runtime call failed;
 * clear != 0 resets the record afterwards.
 */
int ebs_checked_build(void);
int ebs_checked_status(int* site, long long* index, long long* limit, int clear);
/*
 * Test hook of the range-checked build (EBS_ERR_UNSUPPORTED in the normal one): the convolution launches made
 * afterwards take their accumulator / fp32 result buffers to be `elements` elements shorter than they are, so the
 * stores of the last elements are refused and recorded although the memory is there: it shows the record working
 * without any access out of bounds.  0 restores the true extents.  Process-wide.
 */
int ebs_test_checked_shrink(long long elements);

/*
 * Test hook for the give-up path of the tensor-core kernels (the paper has no counterpart).  `limit` = number of
 * polls a bounded wait makes before it gives up (0 restores the default, about 2^20 polls of >= 40 ns);
 * skip_mma = 1 makes the persistent pipeline kernel's issuing thread issue no tensor-core work at all, so that
 * every wait for it runs out with nothing in flight: each thread block then raises its abort flag, leaves its
 * loops, frees its tensor memory and returns, and ebs_device_wait_timeouts() rises.  Process-wide; affects the
 * launches made afterwards.  Nothing faults or hangs by construction.
 */
int ebs_test_set_device_wait(unsigned int limit, int skip_mma);

/*
 * Stand-alone de-quantization of accumulators: the scaling by 1/(2^b - 1) that Eq. 1c folds into
 * the quantizer (text after Eq. 1c), applied to integer results as one combined step
 * y = float(acc) * scale, then * ch_scale[co], + ch_bias[co], ReLU, each optional, over
 * n_pixels * c_out values stored pixel-major (NHWC).
 */
int ebs_dequant(const int32_t *acc_dev, size_t n_pixels, int c_out, float scale,
                const float *ch_scale_dev, const float *ch_bias_dev, int relu, float *y_dev,
                void *stream);

/*
 * Search-stage forward of the bitwidth search (Sec. 4.1; next-row kernels, not on the deployment
 * path).  The full-precision meta tensor is quantized at every candidate bitwidth and the results
 * are blended in one pass:
 *   weights (Eq. 1a, Eq. 6):  u = tanh(w) / (2 max|tanh(w)|) + 1/2,
 *                             w_hat = sum_i coeff[i] * (2 quantize_b[i](u) - 1)
 *   activations (Eq. 1b, Eq. 7):  u = clip(x, 0, alpha) * fl32(1/alpha),
 *                             x_hat = alpha * sum_j coeff[j] * quantize_b[j](u)
 *   quantize_b(u) = fl32(1/(2^b - 1)) * floor((2^b - 1) u + 0.5)   (Eq. 1c, round half up)
 * `bits` (each 1..16) and `coeff` are HOST arrays of n_cand <= EBS_MAX_CANDIDATES entries; coeff is
 * the softmax of the strengths (deterministic search) or the Gumbel-softmax sample (stochastic
 * search, Eq. 8), computed by the caller.  Activations: every fp32 operation is rounded on its own
 * and candidates are accumulated in array order (bit-exact against that chain).  Weights: fp32 with
 * tanhf, the blend evaluated as sum_i fl32(2 coeff[i] / (2^b[i] - 1)) * code_i - sum_i coeff[i] with
 * fused multiply-adds (within 1e-5 of the formula in double precision away from rounding ties of
 * the codes).  src/dst are device tensors of n floats (16-byte aligned; dst
 * may alias src); scratch_dev is 16 bytes of device memory the weight call uses for max|w|.
 */
#define EBS_MAX_CANDIDATES 8
int ebs_search_weight_forward(const float *w_dev, size_t n, const int *bits, const float *coeff, int n_cand,
                              float *w_hat_dev, void *scratch_dev, void *stream);
int ebs_search_act_forward(const float *x_dev, size_t n, float alpha, const int *bits, const float *coeff,
                           int n_cand, float *x_hat_dev, void *stream);

/*
 * Expected operation count of a layer during the search (Eq. 11):
 * FLOP(sum_i coeff_w[i] bits_w[i], sum_j coeff_x[j] bits_x[j]) with FLOP(M, K) = macs * M * K
 * (Sec. 4.3: s n c_o M K AND operations).  Host arithmetic in double; negative on bad arguments.
 */
double ebs_expected_flops(double macs, const int *bits_w, const float *coeff_w, int n_w, const int *bits_x,
                          const float *coeff_x, int n_x);

/*
 * The two host-side fp32 roundings of the scale handling, exactly as the entry points above apply them:
 * S = fl32(w_scale * a_scale) (scale merge of Sec. 4.3) and fl32(1 / step) (the quantizer multiplies by the
 * reciprocal of its step, Eq. 1b-1c).  For callers that fill ebs_fused_layer / ebs_fused_head records.
 */
float ebs_combined_scale(float w_scale, float a_scale);
float ebs_reciprocal_step(float step);

/*
 * Whole-network inference of a basic-block CIFAR ResNet (Sec. 5, Table 1) in ONE launch: a thread
 * block carries one image through every layer with its activation codes resident in shared memory
 * as bytes (no bit planes, no global traffic and no launch between layers); the arithmetic of every
 * layer is that of ebs_conv2d_mixed with a fused epilogue, so the logits equal those of the
 * layer-by-layer calls bit for bit.  The paper has no counterpart (it runs layer by layer).
 *
 * Layers are described by ebs_fused_layer records in execution order:
 *   w8         the byte image of the layer's weights: packed_w + ebs_packed_weight_plane_bytes(desc)
 *   k, stride  3x3 (stride 1 or 2, padding 1) or the 1x1 stride-2 projection shortcut (hold = 1)
 *   src, dst   activation strips 0..2 in shared memory; the image is loaded into strip 0; dst = -1
 *              on the last layer sends its fp32 result to pooling
 *   res        0 none; 1 identity shortcut: res_step * code read from strip res_buf; 2 projection:
 *              the previous record (hold = 1) kept its accumulators in tensor memory and this
 *              epilogue adds fl(fl(acc * S) * ch_scale + ch_bias) of that record
 *   zero_dst   clear strip dst first (set whenever the strip last held another geometry)
 *   S          fl32(w_scale * a_scale); out_inv_step = fl32(1 / step of the output codes)
 *   trace_off  byte offset of this layer's output codes (u8, [Ho][Wo][c_out]) inside each image's
 *              slice of the trace buffer, or -1
 * Limits: c_in, c_out <= 64, (h_in + 2) * (w_in + 2) <= 1156 frame pixels (32 x 32 images).
 * ebs_fused_plan_upload validates the records (host array) and copies them to layers_dev
 * (n_layers * sizeof(ebs_fused_layer) bytes of device memory); ebs_resnet_cifar_forward takes that
 * device array, u8 NHWC images [n][img_h][img_w][3] and writes fp32 logits [n][head.c_out].
 * The head is global average pooling (pixels added in order, times fl32(1/HW)), quantization of the
 * pooled features to 8 bits (a_inv_step = fl32(1 / a_scale)) and the classifier as an integer dot
 * product with its byte image, scaled by S and the per-channel terms.
 */
typedef struct ebs_fused_layer {
    const unsigned char *w8;
    const float *ch_scale;
    const float *ch_bias;
    int c_in, c_out, k, stride;
    int h_in, w_in;
    int src, dst;
    int res;
    int relu, out_bits, hold;
    int zero_dst;
    int trace_off;
    float S, out_inv_step, res_step;
    int res_buf;
} ebs_fused_layer;

typedef struct ebs_fused_head {
    const unsigned char *w8;
    const float *ch_scale;
    const float *ch_bias;
    int c_in, c_out;
    float a_inv_step, S;
} ebs_fused_head;

int ebs_fused_plan_upload(const ebs_fused_layer *layers_host, int n_layers, void *layers_dev, void *stream);
int ebs_resnet_cifar_forward(const unsigned char *images_dev, int n, int img_h, int img_w, const void *layers_dev,
                             int n_layers, const ebs_fused_head *head_host, float *logits_dev,
                             unsigned char *trace_dev, long long trace_stride, void *stream);

/*
 * Global average pooling between the last residual block and the classifier of the ResNets the
 * paper evaluates (Sec. 5); not part of the binary decomposition itself.  y_dev is fp32 NHWC
 * [n][hw][c]; out_dev receives [n][c]: the pixels are added in order 0 .. hw-1 in fp32 and the
 * sum is multiplied by fl(1/hw).
 */
int ebs_global_avgpool(const float *y_dev, int n, int hw, int c, float *out_dev, void *stream);

/*
 * Max pooling of packed activation planes (the 3x3 stride-2 pooling after the first convolution of the ImageNet
 * ResNets of Sec. 5; not part of the binary decomposition itself).  All codes of a tensor share one step, so the
 * maximum of the values is the maximum of the codes; it is taken in the bit-plane domain, 32 channels at a time.
 * Window positions outside the image are ignored (equivalent to padding with the zero code).
 *   packed_x_dev    u32 [n][h][w][ceil(c/32)][a_bits]
 *   packed_out_dev  u32 [n][ho][wo][ceil(c/32)][a_bits], ho = floor((h + 2 pad - k) / stride) + 1 (likewise wo);
 *                   must not alias the input.  pad < k.
 */
int ebs_maxpool_packed(const void *packed_x_dev, int n, int h, int w, int c, int a_bits, int k, int stride, int pad,
                       void *packed_out_dev, void *stream);

/*
 * One layer from HOST buffers, for callers whose data lives on the host: copies the activations
 * to the device, packs them, runs ebs_conv2d_mixed and copies the requested outputs back, all
 * enqueued on `stream` (host buffers should be pinned for the copies to be asynchronous; the
 * caller synchronizes the stream before reading the outputs).
 *   x_host            n*c_in*h*w values, dtype EBS_F32 or EBS_U8_CODES, in `layout`
 *   packed_w_dev      packed weights already on the device
 *   workspace_dev     caller-provided device scratch of at least ebs_host_workspace_bytes(...)
 *   acc_out_host / y_out_host / packed_next_host   any subset, same shapes as the device call
 * epi's pointers are still DEVICE pointers.
 */
size_t ebs_host_workspace_bytes(const ebs_conv_desc *desc, int n, int h, int w, int dtype, int next_a_bits);
int ebs_conv2d_mixed_host(const void *x_host, int dtype, int layout, int n, int h, int w,
                          const void *packed_w_dev, const ebs_conv_desc *desc, const ebs_epilogue *epi,
                          void *workspace_dev, size_t workspace_bytes, int32_t *acc_out_host,
                          float *y_out_host, void *packed_next_host, void *stream);

/*
 * ebs_conv2d_mixed_host for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this is an integration aid.)  Some hosts of this library are not allowed to call
 * cudaMalloc at all: code running inside a framework whose memory pool owns the whole device,
 * plug-ins that are handed a context with a fixed memory budget, real-time loops in which an
 * allocation could block or fail.  They cannot supply the `workspace_dev` scratch the ordinary
 * host call wants.  This variant takes the same arguments without the workspace and keeps the
 * scratch in a fixed array of EBS_NOALLOC_SCRATCH_BYTES (32 MiB) that is part of the library
 * image: every GPU context that loads the library holds those bytes until the process exits.
 *  - It calls no allocating routine (no cudaMalloc / cudaFree, no library that allocates).
 *  - A layer whose ebs_host_workspace_bytes(...) exceeds EBS_NOALLOC_SCRATCH_BYTES is rejected with
 *    EBS_ERR_SCRATCH_TOO_SMALL before anything is enqueued; ebs_noalloc_scratch_bytes() returns the limit.
 *  - The first call on each device looks up the device address of the array (a one-time,
 *    synchronous runtime query made with that device current); make that first call outside any
 *    stream capture.  Later calls on that device only enqueue work.  With lazy module loading that
 *    first query is also the moment the driver loads this library's device code and sets the 32 MiB
 *    aside; on a device whose memory is already fully claimed it fails and the call returns
 *    EBS_ERR_CUDA (nothing enqueued).  Callers inside a pool that owns the device should make one
 *    call early, before the pool takes everything, or load eagerly (CUDA_MODULE_LOADING=EAGER).
 *  - The address is remembered per device ordinal and belongs to that device's primary context.  It
 *    is wrong for a caller running on another (driver-API) context of the same device, and it is
 *    stale after cudaDeviceReset(): neither is supported by this entry point.
 *  - Every argument is checked before the first copy is enqueued: a call that returns an error has
 *    not touched the shared array.
 *  - All calls on a device share the one array, and it keeps whatever the previous call left in
 *    it.  Every byte the path reads is written earlier in the same call, so nothing needs to be
 *    cleared; but two calls whose GPU work overlaps (different streams, or the same stream from
 *    two threads) race on it.  Run them one after the other on one stream.
 * Inputs, outputs, epilogue and results are exactly those of ebs_conv2d_mixed_host.
 */
#define EBS_NOALLOC_SCRATCH_BYTES (32u << 20)
size_t ebs_noalloc_scratch_bytes(void);
int ebs_conv2d_mixed_host_noalloc(const void *x_host, int dtype, int layout, int n, int h, int w,
                                  const void *packed_w_dev, const ebs_conv_desc *desc, const ebs_epilogue *epi,
                                  int32_t *acc_out_host, float *y_out_host, void *packed_next_host,
                                  void *stream);

/*
 * Register-resident throughput probe of the execution pipes the convolution can use; the
 * measured rate is the denominator of the kernel's arithmetic roofline.  Runs `iters` loop
 * iterations on every SM, synchronizes the device, and writes the measured rate.
 *   kind 0: AND + POPC + accumulate on the integer pipes        -> bit-AND-popcounts per second
 *   kind 1: mma.sync m16n8k256 b1 AND.POPC                      -> bit-AND-popcounts per second
 *   kind 2: POPC alone                                          -> bit-popcounts per second
 *   kind 3: mma.sync m16n8k32 u8 x s8 (one byte per bit)        -> byte multiply-accumulates per second
 *   kind 4: tcgen05.mma kind::i8, M 128 x N 256 x K 32 from shared memory into tensor memory, 16 * iters
 *           instructions per SM issued by one thread (iters <= 16384)  -> byte multiply-accumulates per second;
 *           EBS_ERR_TIMEOUT if the bounded wait for their completion ran out
 *   kind 5: the same with N 64 (a quarter of the work per instruction: what one issuing thread sustains)
 * The paper has no counterpart; this is measurement support.
 */
int ebs_probe_pipe(int kind, int iters, double *bit_ops_per_second);

#ifdef __cplusplus
}
#endif
#endif /* EBS_H_ */
