// Implicit-GEMM bit-plane convolution on the integer pipes (AND + POPC), sm_100a.
//
// Stage 1 of the binary decomposition (Eq. 13: P = B_w B_x with AND + bitcount) and stage 2
// (Eq. 14: recombination with 2^(m+k)) are fused: a thread keeps ONE int32 accumulator per
// output and adds  +/- popc(a_k & w_m) << (m+k)  for every plane pair, so the paper's matrix P
// and its img2col matrices never exist in memory.
//
// Work split.  A CTA owns TILE_P consecutive output pixels (flattened n,ho,wo) times TILE_C
// output channels.  Lanes of a warp hold different pixels (conflict-free shared loads), all lanes
// of a warp share the same TC channels (weight words are shared-memory broadcasts).  The
// reduction runs over "k-words": one 32-channel word of one filter tap, KK = kh*kw*CW of them,
// staged KSTEP at a time into shared memory with zero fill for taps outside the image.
#pragma once

#include "ebs_internal.cuh"

namespace ebs {

template <int WB, int AB, int TP, int TC, int WARPS_P, int WARPS_C>
struct PopcTile {
    static constexpr int NT = 32 * WARPS_P * WARPS_C;
    static constexpr int TILE_P = 32 * TP * WARPS_P;
    static constexpr int TILE_C = TC * WARPS_C;
    static constexpr int KK_WORDS = AB * TILE_P + WB * TILE_C;
    static constexpr int KSTEP_RAW = (16 * 1024 / 4) / KK_WORDS;
    static constexpr int KSTEP = KSTEP_RAW < 1 ? 1 : (KSTEP_RAW > 8 ? 8 : KSTEP_RAW);
    static constexpr int STAGE_WORDS = KSTEP * KK_WORDS;
    static constexpr int OUT_WORDS = TILE_P * code_row_bytes(TILE_C) / 4;   // u8 codes of the tile for the packed output
    static constexpr int SMEM_WORDS = STAGE_WORDS > OUT_WORDS ? STAGE_WORDS : OUT_WORDS;
};

template <int WB, int AB, int TP, int TC, int WARPS_P, int WARPS_C>
__global__ void __launch_bounds__(32 * WARPS_P * WARPS_C)
conv_popc_kernel(const ConvParams p) {
    using T = PopcTile<WB, AB, TP, TC, WARPS_P, WARPS_C>;
    constexpr int NT = T::NT, TILE_P = T::TILE_P, TILE_C = T::TILE_C, KSTEP = T::KSTEP;
    static_assert((TC * WB) % 4 == 0, "weight words of a thread are read as 16-byte vectors");

    __shared__ __align__(16) uint32_t smem[T::SMEM_WORDS];
    __shared__ int pix_base[TILE_P];      // (n*H*W) of the pixel's image, or -1 past the end
    __shared__ short pix_h0[TILE_P];      // ho*sh - ph
    __shared__ short pix_w0[TILE_P];      // wo*sw - pw
    __shared__ int kinfo[2][KSTEP];       // r | s<<8 | cw<<16 for the k-words of a step, -1 past the end

    uint32_t (*A_s)[AB][TILE_P] = reinterpret_cast<uint32_t (*)[AB][TILE_P]>(smem);
    uint32_t (*W_s)[TILE_C][WB] = reinterpret_cast<uint32_t (*)[TILE_C][WB]>(smem + KSTEP * AB * TILE_P);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wp = warp % WARPS_P, wc = warp / WARPS_P;
    const int tile_p0 = blockIdx.x * TILE_P;
    const int co0 = blockIdx.y * TILE_C;

    auto decode_kk = [&](int kk) -> int {
        if (kk >= p.KK) return -1;
        const int tap = kk / p.CW, cw = kk - tap * p.CW;
        const int r = tap / p.kw, s = tap - r * p.kw;
        return r | (s << 8) | (cw << 16);
    };

    for (int i = tid; i < TILE_P; i += NT) {
        const int gp = tile_p0 + i;
        if (gp < p.P) {
            const int hw = p.Ho * p.Wo;
            const int n = gp / hw, rem = gp - n * hw;
            const int ho = rem / p.Wo, wo = rem - ho * p.Wo;
            pix_base[i] = n * p.H * p.W;
            pix_h0[i] = (short)(ho * p.sh - p.ph);
            pix_w0[i] = (short)(wo * p.sw - p.pw);
        } else {
            pix_base[i] = -1;
            pix_h0[i] = 0;
            pix_w0[i] = 0;
        }
    }
    if (tid < KSTEP) kinfo[0][tid] = decode_kk(tid);

    int acc[TP][TC];
    int wsum[TP];              // sum of the activation codes under the filter window (w_levels)
#pragma unroll
    for (int t = 0; t < TP; ++t) {
        wsum[t] = 0;
#pragma unroll
        for (int c = 0; c < TC; ++c) acc[t][c] = 0;
    }

    __syncthreads();

    int buf = 0;
    for (int kk0 = 0; kk0 < p.KK; kk0 += KSTEP, buf ^= 1) {
        // ---- stage activations: one item = (k-word q, pixel i), AB plane words each
        for (int item = tid; item < KSTEP * TILE_P; item += NT) {
            const int q = item / TILE_P, i = item - q * TILE_P;
            const int info = kinfo[buf][q];
            uint32_t words[AB];
#pragma unroll
            for (int j = 0; j < AB; ++j) words[j] = 0u;
            const int base = pix_base[i];
            if (info >= 0 && base >= 0) {
                const int hi = pix_h0[i] + (info & 0xff), wi = pix_w0[i] + ((info >> 8) & 0xff);
                if ((unsigned)hi < (unsigned)p.H && (unsigned)wi < (unsigned)p.W) {
                    const size_t off = ((size_t)(base + hi * p.W + wi) * p.CW + (info >> 16)) * AB;
                    if (EBS_IN_RANGE(p, CHK_POPC_X, off + AB - 1, p.lim_x)) load_words_global<AB>(p.x + off, words);
                }
            }
#pragma unroll
            for (int j = 0; j < AB; ++j) A_s[q][j][i] = words[j];
        }
        // ---- stage weights: KSTEP x (TILE_C*WB) words, contiguous per k-word in global memory
        for (int item = tid; item < KSTEP * TILE_C * WB; item += NT) {
            const int q = item / (TILE_C * WB), e = item - q * (TILE_C * WB);
            const int c = e / WB;
            const int kk = kk0 + q;
            uint32_t v = 0u;
            if (kk < p.KK && co0 + c < p.Co && EBS_IN_RANGE(p, CHK_POPC_W, ((long long)kk * p.Co + co0) * WB + e, p.lim_w))
                v = __ldg(p.w + ((size_t)kk * p.Co + co0) * WB + e);
            (&W_s[q][0][0])[e] = v;
        }
        __syncthreads();
        if (tid < KSTEP) kinfo[buf ^ 1][tid] = decode_kk(kk0 + KSTEP + tid);

        // ---- AND + POPC over the staged k-words
#pragma unroll
        for (int q = 0; q < KSTEP; ++q) {
            if (kk0 + q < p.KK) {
                uint32_t a[TP][AB], w[TC][WB];
#pragma unroll
                for (int t = 0; t < TP; ++t)
#pragma unroll
                    for (int j = 0; j < AB; ++j) {
                        a[t][j] = A_s[q][j][(wp * TP + t) * 32 + lane];
                        if (p.w_levels) wsum[t] += __popc(a[t][j]) << j;
                    }
                const uint4* wv = reinterpret_cast<const uint4*>(&W_s[q][wc * TC][0]);
                uint32_t* wflat = &w[0][0];
#pragma unroll
                for (int v = 0; v < TC * WB / 4; ++v) {
                    const uint4 t4 = wv[v];
                    wflat[4 * v] = t4.x; wflat[4 * v + 1] = t4.y; wflat[4 * v + 2] = t4.z; wflat[4 * v + 3] = t4.w;
                }
#pragma unroll
                for (int t = 0; t < TP; ++t)
#pragma unroll
                    for (int c = 0; c < TC; ++c)
#pragma unroll
                        for (int i = 0; i < WB; ++i)
#pragma unroll
                            for (int j = 0; j < AB; ++j) {
                                const int cnt = __popc(a[t][j] & w[c][i]) << (i + j);
                                if (i == WB - 1) acc[t][c] -= cnt;   // two's-complement top plane
                                else acc[t][c] += cnt;
                            }
            }
        }
        __syncthreads();
    }

    // ---- epilogue: accumulators, fp32 output, requantized packed planes
    const bool want_y = p.y != nullptr, want_q = p.packed_next != nullptr;
    uint8_t* out_s = reinterpret_cast<uint8_t*>(smem);      // [TILE_P][TILE_C] codes (staging is finished)
    const int qmax = (1 << p.next_bits) - 1;
#pragma unroll
    for (int t = 0; t < TP; ++t) {
        const int pl = (wp * TP + t) * 32 + lane;
        const int gp = tile_p0 + pl;
        const bool pvalid = gp < p.P;
#pragma unroll
        for (int c = 0; c < TC; ++c) {
            const int cl = wc * TC + c, co = co0 + cl;
            const bool valid = pvalid && co < p.Co;
            int code = 0;
            if (valid) {
                const size_t o = (size_t)gp * p.Co + co;
                const int av = p.w_levels ? 2 * acc[t][c] + wsum[t] : acc[t][c];
                if (p.acc && EBS_IN_RANGE(p, CHK_POPC_ACC, o, p.lim_out)) p.acc[o] = av;
                if (want_y || want_q) {
                    float yv = __fmul_rn((float)av, p.S);
                    if (p.ch_scale) yv = __fmul_rn(yv, __ldg(p.ch_scale + co));
                    if (p.ch_bias) yv = __fadd_rn(yv, __ldg(p.ch_bias + co));
                    if (p.residual) yv = __fadd_rn(yv, __ldg(p.residual + o));
                    if (p.res_packed) yv = __fadd_rn(yv, packed_residual(p, gp, co));
                    if (p.relu && !(yv > 0.0f)) yv = 0.0f;
                    if (want_y && EBS_IN_RANGE(p, CHK_POPC_Y, o, p.lim_out)) {
                        if (p.y_nchw) {
                            const int hw = p.Ho * p.Wo;
                            const int n = gp / hw, rem = gp - n * hw;
                            p.y[((size_t)n * p.Co + co) * hw + rem] = yv;
                        } else {
                            p.y[o] = yv;
                        }
                    }
                    if (want_q) code = quantize_code(yv, p.inv_next, 0, qmax);
                }
            }
            if (want_q && EBS_IN_RANGE(p, CHK_TILE_CODES, pl * code_row_bytes(TILE_C) + cl, TILE_P * code_row_bytes(TILE_C)))
                out_s[pl * code_row_bytes(TILE_C) + cl] = (uint8_t)code;
        }
    }
    if (want_q) {
        __syncthreads();
        pack_code_tile<TILE_P, TILE_C, NT>(out_s, p, tile_p0, co0);
    }
}

template <int WB, int AB, int TP, int TC, int WARPS_P, int WARPS_C>
int launch_conv_popc(const ConvParams& p, dim3 grid, cudaStream_t st) {
    conv_popc_kernel<WB, AB, TP, TC, WARPS_P, WARPS_C><<<grid, 32 * WARPS_P * WARPS_C, 0, st>>>(p);
    return EBS_OK;
}

// Variant table.  Every variant gives a thread TC = 8 output channels (except the small one) and
// TP pixels; the cap TP * 8 * WB * AB <= 512 keeps the unrolled AND+POPC block of one k-word inside
// the instruction cache.  variant = tile_c_index * 3 + tp_index, tile_c in {16, 32, 64},
// TP in {1, 2, 4}; variant 9 is the small tile (32 pixels x 16 channels, 4 warps) for problems
// that cannot fill the GPU otherwise.
template <int WB, int AB, int VARIANT>
struct VariantGeom {
    static constexpr int PAIRS = WB * AB;
    static constexpr int TP_CAP = PAIRS <= 16 ? 4 : (PAIRS <= 32 ? 2 : 1);
    static constexpr int TP_REQ = 1 << (VARIANT % 3);
    static constexpr int TP = TP_REQ > TP_CAP ? TP_CAP : TP_REQ;
    static constexpr int TC = 8;
    static constexpr int WARPS_C = 2 << (VARIANT / 3);      // 2, 4, 8 -> tile_c 16, 32, 64
    static constexpr int WARPS_P = 8 / WARPS_C;
};
template <int WB, int AB>
struct VariantGeom<WB, AB, 9> {
    static constexpr int TP = 1, TC = 4, WARPS_C = 4, WARPS_P = 1;
};

template <int WB, int AB, int VARIANT>
constexpr ConvVariant make_variant() {
    using G = VariantGeom<WB, AB, VARIANT>;
    return ConvVariant{&launch_conv_popc<WB, AB, G::TP, G::TC, G::WARPS_P, G::WARPS_C>,
                       32 * G::TP * G::WARPS_P, G::TC * G::WARPS_C, 32 * G::WARPS_P * G::WARPS_C};
}

#define EBS_VARIANT_ROW(WB, AB)                                                                       \
    {make_variant<WB, AB, 0>(), make_variant<WB, AB, 1>(), make_variant<WB, AB, 2>(),                 \
     make_variant<WB, AB, 3>(), make_variant<WB, AB, 4>(), make_variant<WB, AB, 5>(),                 \
     make_variant<WB, AB, 6>(), make_variant<WB, AB, 7>(), make_variant<WB, AB, 8>(),                 \
     make_variant<WB, AB, 9>()}

// Defines conv_popc_variant_w<WB>() for one weight bitwidth (one translation unit each, so the
// instantiations compile in parallel).
#define EBS_DEFINE_WB_TABLE(WB)                                                                       \
    const ConvVariant* conv_popc_variant_w##WB(int a_bits, int variant) {                             \
        static const ConvVariant table[8][NUM_CONV_VARIANTS] = {                                      \
            EBS_VARIANT_ROW(WB, 1), EBS_VARIANT_ROW(WB, 2), EBS_VARIANT_ROW(WB, 3),                   \
            EBS_VARIANT_ROW(WB, 4), EBS_VARIANT_ROW(WB, 5), EBS_VARIANT_ROW(WB, 6),                   \
            EBS_VARIANT_ROW(WB, 7), EBS_VARIANT_ROW(WB, 8)};                                          \
        if (a_bits < 1 || a_bits > 8 || variant < 0 || variant >= NUM_CONV_VARIANTS) return nullptr;  \
        return &table[a_bits - 1][variant];                                                           \
    }

}  // namespace ebs
