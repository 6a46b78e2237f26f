/*
 * CPU oracle for the binary-decomposition mixed-precision convolution.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, obviously-correct
 * statement of what the GPU path must compute.  It shares no code with the CUDA
 * library, includes none of its headers, and must never be called from the
 * product path: only tests, the smoke check and the benchmark's CPU-baseline /
 * reference legs may use it.
 *
 * Every function works on HOST memory, in the paper's tensor order
 * (activations N,C,H,W; weights C_out,C_in,kh,kw) with one int32 per code.
 * Integer work is exact (int64 accumulation, checked to fit int32); the fp32
 * epilogue rounds every operation individually (build with -ffp-contract=off).
 *
 * Parallelism: one OpenMP "parallel for" over (image, output channel).  Nothing
 * is blocked, fused or reordered beyond that.
 *
 * Pins (see tests/): brute force on tiny inputs, the bit-plane identity (Eq. 2),
 * the matrix form B_w B_x with the power-of-two recombination (Eq. 12-15),
 * numpy int64 matmul for 1x1 kernels, float64 library convolution, closed forms.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG (-1)
#define ORACLE_ERR_OVERFLOW (-3)

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static int out_dim(int in, int pad, int k, int stride) {
    /* floor((in + 2 pad - k) / stride) + 1, the img2col output size (Sec. 4.3) */
    int span = in + 2 * pad - k;
    if (span < 0) return 0;
    return span / stride + 1;
}

int oracle_out_dim(int in, int pad, int k, int stride) { return out_dim(in, pad, k, stride); }

/*
 * quantize_b of Eq. 1c, integer-code form: round-half-up of x * inv_step, clamped
 * to [lo, hi].  "round half up" (text after Eq. 1c) is floor(v + 0.5), not
 * round-half-even.  x * inv_step and the + 0.5 are two separately rounded fp32
 * operations.  Activations (Eq. 1b): lo = 0, hi = 2^b - 1 (the clip to
 * [0, alpha] becomes the clamp of the code).  Signed weights: lo = -2^(b-1),
 * hi = 2^(b-1) - 1.
 */
void oracle_quantize(const float *x, size_t count, float inv_step, int lo, int hi, int32_t *q) {
    for (size_t t = 0; t < count; ++t) {
        volatile float v = x[t] * inv_step;
        volatile float r = v + 0.5f;
        float f = floorf(r);
        int32_t c;
        if (!(f >= (float)lo)) c = lo;           /* also catches NaN -> lo */
        else if (f > (float)hi) c = hi;
        else c = (int32_t)f;
        q[t] = c;
    }
}

/*
 * The definition: direct integer convolution of the codes (left-hand side of
 * Eq. 2 summed over the img2col window of Sec. 4.3).  Taps that fall outside the
 * image contribute nothing (a zero code is the real value 0).
 *   qa  [N][C][H][W]       activation codes
 *   qw  [Co][C][kh][kw]    weight codes (signed)
 *   acc [N][Co][Ho][Wo]    int32 accumulators
 */
int oracle_conv2d_codes(const int32_t *qa, const int32_t *qw, int N, int C, int H, int W, int Co,
                        int kh, int kw, int sh, int sw, int ph, int pw, int32_t *acc) {
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || Co <= 0 || kh <= 0 || kw <= 0 || sh <= 0 || sw <= 0 ||
        ph < 0 || pw < 0)
        return ORACLE_ERR_ARG;
    const int Ho = out_dim(H, ph, kh, sh), Wo = out_dim(W, pw, kw, sw);
    if (Ho <= 0 || Wo <= 0) return ORACLE_ERR_ARG;
    int overflow = 0;
#pragma omp parallel for collapse(2) schedule(static) reduction(| : overflow)
    for (int n = 0; n < N; ++n) {
        for (int co = 0; co < Co; ++co) {
            for (int ho = 0; ho < Ho; ++ho) {
                for (int wo = 0; wo < Wo; ++wo) {
                    int64_t sum = 0;
                    for (int ci = 0; ci < C; ++ci) {
                        for (int r = 0; r < kh; ++r) {
                            const int hi = ho * sh + r - ph;
                            if (hi < 0 || hi >= H) continue;
                            for (int s = 0; s < kw; ++s) {
                                const int wi = wo * sw + s - pw;
                                if (wi < 0 || wi >= W) continue;
                                const int64_t a = qa[(((size_t)n * C + ci) * H + hi) * W + wi];
                                const int64_t w = qw[(((size_t)co * C + ci) * kh + r) * kw + s];
                                sum += a * w;
                            }
                        }
                    }
                    if (sum > INT32_MAX || sum < INT32_MIN) overflow = 1;
                    acc[(((size_t)n * Co + co) * Ho + ho) * Wo + wo] = (int32_t)sum;
                }
            }
        }
    }
    return overflow ? ORACLE_ERR_OVERFLOW : ORACLE_OK;
}

/*
 * The paper's own weight format (Eq. 1a): b-bit weights take the 2^b levels 2*q_u - (2^b - 1),
 * q_u = 0 .. 2^b - 1 (times 1/(2^b - 1)).  With the signed code qw = q_u - 2^(b-1) the level is
 * 2*qw + 1, and the convolution of levels with activation codes is
 *   acc[n][co][ho][wo] = sum (2*qw + 1) * qa        (direct definition, taps outside the image skipped).
 */
int oracle_conv2d_levels(const int32_t *qa, const int32_t *qw, int N, int C, int H, int W, int Co,
                         int kh, int kw, int sh, int sw, int ph, int pw, int32_t *acc) {
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || Co <= 0 || kh <= 0 || kw <= 0 || sh <= 0 || sw <= 0 ||
        ph < 0 || pw < 0)
        return ORACLE_ERR_ARG;
    const int Ho = out_dim(H, ph, kh, sh), Wo = out_dim(W, pw, kw, sw);
    if (Ho <= 0 || Wo <= 0) return ORACLE_ERR_ARG;
    int overflow = 0;
#pragma omp parallel for collapse(2) schedule(static) reduction(| : overflow)
    for (int n = 0; n < N; ++n) {
        for (int co = 0; co < Co; ++co) {
            for (int ho = 0; ho < Ho; ++ho) {
                for (int wo = 0; wo < Wo; ++wo) {
                    int64_t sum = 0;
                    for (int ci = 0; ci < C; ++ci)
                        for (int r = 0; r < kh; ++r) {
                            const int hi = ho * sh + r - ph;
                            if (hi < 0 || hi >= H) continue;
                            for (int s = 0; s < kw; ++s) {
                                const int wi = wo * sw + s - pw;
                                if (wi < 0 || wi >= W) continue;
                                const int64_t a = qa[(((size_t)n * C + ci) * H + hi) * W + wi];
                                const int64_t level = 2 * (int64_t)qw[(((size_t)co * C + ci) * kh + r) * kw + s] + 1;
                                sum += a * level;
                            }
                        }
                    if (sum > INT32_MAX || sum < INT32_MIN) overflow = 1;
                    acc[(((size_t)n * Co + co) * Ho + ho) * Wo + wo] = (int32_t)sum;
                }
            }
        }
    }
    return overflow ? ORACLE_ERR_OVERFLOW : ORACLE_OK;
}

/*
 * Weight quantizer of Eq. 1a in code form: the nearest level w_step * (2*q_u - L), L = 2^b - 1,
 * round half up; returns the signed code q_u - 2^(b-1).
 *   v = fl(w * inv_step);  u = fl(fl(v + L) * 0.5);  q_u = clamp(floor(fl(u + 0.5)), 0, L).
 * With w = w_n (normalised to [-1, 1]) and w_step = 1/L this is q_u = round(L * (w_n/2 + 1/2)).
 */
void oracle_quantize_weight_levels(const float *w, size_t count, float inv_step, int bits, int32_t *q) {
    const int L = (1 << bits) - 1;
    for (size_t t = 0; t < count; ++t) {
        volatile float v = w[t] * inv_step;
        volatile float s = v + (float)L;
        volatile float u = s * 0.5f;
        volatile float r = u + 0.5f;
        float f = floorf(r);
        int32_t qu;
        if (!(f >= 0.0f)) qu = 0;
        else if (f > (float)L) qu = L;
        else qu = (int32_t)f;
        q[t] = qu - (1 << (bits - 1));
    }
}

/*
 * The same result by the bit-plane route of Eq. 2, one bit at a time and without
 * any packing:  sum_m sum_k c_m 2^(m+k) bitcount(AND(bit m of w, bit k of x)).
 * Weights are Wb-bit two's-complement codes, so the coefficient of the top
 * weight plane is -2^(Wb-1) when signed_w != 0 (with signed_w == 0 the codes are
 * the paper's unsigned ones and every coefficient is positive).  Activations are
 * unsigned Ab-bit codes.
 */
int oracle_conv2d_bitplanes(const int32_t *qa, const int32_t *qw, int N, int C, int H, int W, int Co,
                            int kh, int kw, int sh, int sw, int ph, int pw, int Wb, int Ab,
                            int signed_w, int32_t *acc) {
    if (Wb < 1 || Wb > 8 || Ab < 1 || Ab > 8) return ORACLE_ERR_ARG;
    const int Ho = out_dim(H, ph, kh, sh), Wo = out_dim(W, pw, kw, sw);
    if (Ho <= 0 || Wo <= 0) return ORACLE_ERR_ARG;
    const uint32_t wmask = (1u << Wb) - 1u;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int co = 0; co < Co; ++co) {
            for (int ho = 0; ho < Ho; ++ho) {
                for (int wo = 0; wo < Wo; ++wo) {
                    int64_t total = 0;
                    for (int m = 0; m < Wb; ++m) {
                        for (int k = 0; k < Ab; ++k) {
                            int64_t bitcount = 0;
                            for (int ci = 0; ci < C; ++ci)
                                for (int r = 0; r < kh; ++r) {
                                    const int hi = ho * sh + r - ph;
                                    if (hi < 0 || hi >= H) continue;
                                    for (int s = 0; s < kw; ++s) {
                                        const int wi = wo * sw + s - pw;
                                        if (wi < 0 || wi >= W) continue;
                                        const uint32_t a =
                                            (uint32_t)qa[(((size_t)n * C + ci) * H + hi) * W + wi];
                                        const uint32_t w =
                                            (uint32_t)qw[(((size_t)co * C + ci) * kh + r) * kw + s] & wmask;
                                        bitcount += ((a >> k) & 1u) & ((w >> m) & 1u);
                                    }
                                }
                            const int64_t coef = (int64_t)1 << (m + k);
                            if (signed_w && m == Wb - 1) total -= coef * bitcount;
                            else total += coef * bitcount;
                        }
                    }
                    acc[(((size_t)n * Co + co) * Ho + ho) * Wo + wo] = (int32_t)total;
                }
            }
        }
    }
    return ORACLE_OK;
}

/*
 * Epilogue on the accumulators (scale merge of Sec. 4.3 "Complexities", clip and
 * round of Eq. 1b-1c / Eq. 16a-16c).  Every fp32 operation is rounded on its own.
 *   y = fl(fl(acc) * S)                     S = fl(s_w * s_a), given
 *   y = fl(y * ch_scale[co])                if ch_scale
 *   y = fl(y + ch_bias[co])                 if ch_bias
 *   y = fl(y + residual[n][co][ho][wo])     if residual
 *   y = max(y, 0)                           if relu
 *   q = clamp(floor(fl(fl(y * inv_next) + 0.5)), 0, 2^next_bits - 1)   if q_out
 * Tensors are [N][Co][Ho][Wo]; y_out and q_out may each be NULL.
 */
void oracle_epilogue(const int32_t *acc, int N, int Co, int Ho, int Wo, float S, const float *ch_scale,
                     const float *ch_bias, const float *residual, int relu, float *y_out,
                     int next_bits, float inv_next, int32_t *q_out) {
    const size_t plane = (size_t)Ho * Wo;
    const int qmax = (1 << next_bits) - 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int co = 0; co < Co; ++co) {
            for (size_t p = 0; p < plane; ++p) {
                const size_t idx = ((size_t)n * Co + co) * plane + p;
                volatile float y = (float)acc[idx];
                y = y * S;
                if (ch_scale) y = y * ch_scale[co];
                if (ch_bias) y = y + ch_bias[co];
                if (residual) y = y + residual[idx];
                if (relu && !(y > 0.0f)) y = 0.0f;
                if (y_out) y_out[idx] = y;
                if (q_out) {
                    volatile float v = y * inv_next;
                    volatile float r = v + 0.5f;
                    float f = floorf(r);
                    int32_t c;
                    if (!(f >= 0.0f)) c = 0;
                    else if (f > (float)qmax) c = qmax;
                    else c = (int32_t)f;
                    q_out[idx] = c;
                }
            }
        }
    }
}

/*
 * Bit-plane words of the activations, built one bit at a time.
 *   in : qa [N][C][H][W], unsigned Ab-bit codes
 *   out: u32 [N][H][W][CW][Ab], CW = ceil(C/32); bit (c % 32) of word
 *        [n][h][w][c / 32][k] is bit k of qa[n][c][h][w]; unused bits are zero.
 */
void oracle_pack_acts(const int32_t *qa, int N, int C, int H, int W, int Ab, uint32_t *out) {
    const int CW = (C + 31) / 32;
    memset(out, 0, (size_t)N * H * W * CW * Ab * sizeof(uint32_t));
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w) {
                    const uint32_t code = (uint32_t)qa[(((size_t)n * C + c) * H + h) * W + w];
                    for (int k = 0; k < Ab; ++k)
                        if ((code >> k) & 1u)
                            out[((((size_t)n * H + h) * W + w) * CW + c / 32) * Ab + k] |= 1u << (c % 32);
                }
}

/*
 * Bit-plane words of the weights, built one bit at a time.
 *   in : qw [Co][C][kh][kw], signed Wb-bit codes (two's complement bits are taken)
 *   out: u32 [kh][kw][CW][Co][Wb]; bit (c % 32) of word [r][s][c / 32][co][m] is
 *        bit m of the two's-complement code qw[co][c][r][s]; unused bits are zero.
 */
void oracle_pack_weights(const int32_t *qw, int Co, int C, int kh, int kw, int Wb, uint32_t *out) {
    const int CW = (C + 31) / 32;
    memset(out, 0, (size_t)kh * kw * CW * Co * Wb * sizeof(uint32_t));
    for (int co = 0; co < Co; ++co)
        for (int c = 0; c < C; ++c)
            for (int r = 0; r < kh; ++r)
                for (int s = 0; s < kw; ++s) {
                    const uint32_t code = (uint32_t)qw[(((size_t)co * C + c) * kh + r) * kw + s];
                    for (int m = 0; m < Wb; ++m)
                        if ((code >> m) & 1u)
                            out[((((size_t)r * kw + s) * CW + c / 32) * Co + co) * Wb + m] |= 1u << (c % 32);
                }
}

/* Inverse of oracle_pack_acts (used by tests to read back fused packed outputs). */
void oracle_unpack_acts(const uint32_t *packed, int N, int C, int H, int W, int Ab, int32_t *qa) {
    const int CW = (C + 31) / 32;
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w) {
                    uint32_t code = 0;
                    for (int k = 0; k < Ab; ++k) {
                        const uint32_t word = packed[((((size_t)n * H + h) * W + w) * CW + c / 32) * Ab + k];
                        code |= ((word >> (c % 32)) & 1u) << k;
                    }
                    qa[(((size_t)n * C + c) * H + h) * W + w] = (int32_t)code;
                }
}
