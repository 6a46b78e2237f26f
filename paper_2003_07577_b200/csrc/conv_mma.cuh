// Implicit-GEMM bit-plane convolution on the int8 tensor pipe (mma.sync m16n8k32), sm_100a.
//
// sm_100a has no native 1-bit AND+POPC matrix instruction: the toolchain expands
// mma.sync...b1.and.popc into ~110 instructions that turn bits into bytes and issue eight int8
// MMAs.  This kernel goes one step further: the planes of a 32-channel word are merged back into one
// byte per channel -- the activation code sum_k 2^k bit_k as u8, the weight code sum_m c_m 2^m bit_m
// as s8 (c_m = -1 for the top plane: two's complement) -- so that ONE int8 MMA per reduction word adds
// sum_m sum_k c_m 2^(m+k) * bitcount(AND(activation plane k, weight plane m)), stage 1 (Eq. 13) and
// stage 2 (Eq. 14) of the binary decomposition for all plane pairs at once, into one int32
// accumulator per output.  The matrix P never exists; the result is the same integer.
//
// Activation fragments are built in registers straight from the packed 32-bit words: thread (g, tq)
// of a warp owns reduction bits {8b + tq, 8b + 4 + tq : b = 0..3} of a word, so "rotate right by
// (tq - k), AND with 0x01010101 << k" puts plane k's bits at bit k of four bytes (two instructions
// per plane and register).  Weight fragments are two words of the channel's row of the byte image
// the weight packer wrote (K position 4b + i = channel 8i + b, the same assignment), so the kernel
// does not depend on the weight bit count.
//
// Layers with at most 16 input channels use only the low bits of each word; there 2, 4 or 8 staged
// taps are OR-ed into one word (shifted by 16, 8 or 4 bits) while the fragments are built, for both
// operands alike, so a 32-channel MMA step is filled with real reduction bits.
//
// Work split: a CTA owns TILE_P consecutive output pixels x TILE_C channels; a warp owns
// 16*MT pixels x 8*NT channels.  The packed activation words and the weight rows of KSTEP reduction
// words are staged with cp.async (zero fill for taps outside the image), double buffered.
#pragma once

#include "ebs_internal.cuh"

namespace ebs {

constexpr int MMA_KTAB = 256;   // reduction words (kh*kw*CW) the in-kernel tap table can hold

__device__ __forceinline__ void cp_async_bytes(void* smem_dst, const void* gsrc, int bytes, bool valid) {
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
    const int src_size = valid ? bytes : 0;        // src_size 0: nothing is read, the destination is zero filled
    if (bytes == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(gsrc), "r"(src_size));
    else if (bytes == 8)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;\n" ::"r"(dst), "l"(gsrc), "r"(src_size));
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(dst), "l"(gsrc), "r"(src_size));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

// Largest of 16/8/4 bytes that divides a run of `words` 32-bit words (and hence its alignment).
__host__ __device__ constexpr int chunk_bytes(int words) { return (words % 4 == 0) ? 16 : ((words % 2 == 0) ? 8 : 4); }

// Reads NWORDS consecutive shared-memory words whose address is aligned to chunk_bytes(NWORDS).
template <int NWORDS>
__device__ __forceinline__ void load_words_shared(const uint32_t* src, uint32_t (&dst)[NWORDS]) {
    if constexpr (NWORDS % 4 == 0) {
#pragma unroll
        for (int v = 0; v < NWORDS / 4; ++v) {
            const uint4 t = reinterpret_cast<const uint4*>(src)[v];
            dst[4 * v] = t.x; dst[4 * v + 1] = t.y; dst[4 * v + 2] = t.z; dst[4 * v + 3] = t.w;
        }
    } else if constexpr (NWORDS % 2 == 0) {
#pragma unroll
        for (int v = 0; v < NWORDS / 2; ++v) {
            const uint2 t = reinterpret_cast<const uint2*>(src)[v];
            dst[2 * v] = t.x; dst[2 * v + 1] = t.y;
        }
    } else {
#pragma unroll
        for (int v = 0; v < NWORDS; ++v) dst[v] = src[v];
    }
}

__device__ __forceinline__ void mma_u8s8(int (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int AB, int MT, int NT, int WARPS_P, int WARPS_C>
struct MmaTile {
    static constexpr int NTHREADS = 32 * WARPS_P * WARPS_C;
    static constexpr int TILE_P = 16 * MT * WARPS_P;
    static constexpr int TILE_C = 8 * NT * WARPS_C;
    static constexpr int KW_WORDS = TILE_P * AB + TILE_C * 8;           // words per staged reduction word: packed
                                                                         // activation words + 32-byte weight rows
    static constexpr int KSTEP_RAW = 4096 / KW_WORDS;                    // about 16 KB per stage
    static constexpr int KSTEP = KSTEP_RAW < 1 ? 1 : (KSTEP_RAW > 8 ? 8 : KSTEP_RAW);
    static constexpr int STAGE_WORDS = KSTEP * KW_WORDS;
    static constexpr int OUT_WORDS = TILE_P * code_row_bytes(TILE_C) / 4;
    static constexpr int SMEM_WORDS = 2 * STAGE_WORDS > OUT_WORDS ? 2 * STAGE_WORDS : OUT_WORDS;
    static constexpr int PPT = TILE_P > NTHREADS ? TILE_P / NTHREADS : 1;       // pixels staged per thread
    static constexpr int QSTRIDE = NTHREADS > TILE_P ? NTHREADS / TILE_P : 1;   // threads sharing a pixel
    static_assert(TILE_P % NTHREADS == 0 || NTHREADS % TILE_P == 0, "staging map needs a power-of-two ratio");
    static_assert(SMEM_WORDS * 4 + MMA_KTAB * 8 <= 47 * 1024, "static shared memory budget");
};

// FULL = false: the form for even c_out, NHWC, two's-complement weight codes and no per-channel or shortcut terms
// (chosen on the host), which leaves out their instructions and the general epilogue.
template <int AB, int MT, int NT, int WARPS_P, int WARPS_C, bool FULL>
__global__ void __launch_bounds__(32 * WARPS_P * WARPS_C)
conv_mma_kernel(const ConvParams p) {
    using T = MmaTile<AB, MT, NT, WARPS_P, WARPS_C>;
    constexpr int NTH = T::NTHREADS, TILE_P = T::TILE_P, TILE_C = T::TILE_C, KSTEP = T::KSTEP;
    constexpr int PPT = T::PPT, QSTRIDE = T::QSTRIDE;
    constexpr int A_CH = chunk_bytes(AB);

    __shared__ __align__(16) uint32_t smem[T::SMEM_WORDS];
    __shared__ int2 ktab[MMA_KTAB];            // per reduction word: {word offset of the tap, r | s << 8}

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, tq = lane & 3;
    const int wp = warp % WARPS_P, wc = warp / WARPS_P;
    const int tile_p0 = blockIdx.x * TILE_P;
    const int co0 = blockIdx.y * TILE_C;

    // ---- tap table (kk = tap * CW + cw)
#pragma unroll 1
    for (int kk = tid; kk < p.KK; kk += NTH) {
        const int tap = kk / p.CW, cw = kk - tap * p.CW;
        const int r = tap / p.kw, s = tap - r * p.kw;
        ktab[kk] = make_int2(((r * p.W + s) * p.CW + cw) * AB, r | (s << 8));
    }

    // ---- the pixels this thread stages: word offset of (n, h0, w0) and which taps stay inside the image
    int pix_off[PPT];
    uint32_t row_ok[PPT], col_ok[PPT];
#pragma unroll
    for (int u = 0; u < PPT; ++u) {
        const int pl = (tid % TILE_P) + u * NTH;
        const int gp = tile_p0 + pl;
        pix_off[u] = 0; row_ok[u] = 0u; col_ok[u] = 0u;
        if (gp < p.P) {
            const int hw = p.Ho * p.Wo;
            const int n = gp / hw, rem = gp - n * hw;
            const int ho = rem / p.Wo, wo = rem - ho * p.Wo;
            const int h0 = ho * p.sh - p.ph, w0 = wo * p.sw - p.pw;
            pix_off[u] = ((n * p.H + h0) * p.W + w0) * p.CW * AB;
            for (int r = 0; r < p.kh; ++r) row_ok[u] |= ((unsigned)(h0 + r) < (unsigned)p.H ? 1u : 0u) << r;
            for (int s = 0; s < p.kw; ++s) col_ok[u] |= ((unsigned)(w0 + s) < (unsigned)p.W ? 1u : 0u) << s;
        }
    }

    auto stage = [&](int kk0, int buf) {
        uint32_t* A_s = smem + buf * T::STAGE_WORDS;                       // [KSTEP][TILE_P][AB]
        uint32_t* W_s = A_s + KSTEP * TILE_P * AB;                         // [KSTEP][TILE_C][8]
#pragma unroll
        for (int qq = 0; qq < (KSTEP + QSTRIDE - 1) / QSTRIDE; ++qq) {
            const int q = qq * QSTRIDE + (QSTRIDE > 1 ? tid / TILE_P : 0);
            if (QSTRIDE > 1 && q >= KSTEP) break;
            const int kk = kk0 + q;
            const bool kvalid = kk < p.KK;
            const int2 info = kvalid ? ktab[kk] : make_int2(0, 0);
            const int r = info.y & 0xff, s = info.y >> 8;
#pragma unroll
            for (int u = 0; u < PPT; ++u) {
                const int pl = (tid % TILE_P) + u * NTH;
                const bool valid = kvalid && ((row_ok[u] >> r) & (col_ok[u] >> s) & 1u) &&
                                   EBS_IN_RANGE(p, CHK_MMA_X, (long long)pix_off[u] + info.x + AB - 1, p.lim_x) &&
                                   EBS_IN_RANGE(p, CHK_MMA_STAGE, (q * TILE_P + pl) * AB + AB - 1, KSTEP * TILE_P * AB);
                const uint32_t* src = valid ? p.x + (pix_off[u] + info.x) : p.x;
                uint32_t* dst = A_s + (q * TILE_P + pl) * AB;
#pragma unroll
                for (int c = 0; c < AB * 4 / A_CH; ++c)
                    cp_async_bytes(dst + c * (A_CH / 4), src + c * (A_CH / 4), A_CH, valid);
            }
        }
        // weights: the 32-byte rows (one s8 code per input channel) of channels co0 .. co0+TILE_C of every staged
        // reduction word, from the byte image; rows from c_out up to its multiple of 16 are zero there
#pragma unroll 1
        for (int e = tid; e < KSTEP * TILE_C * 2; e += NTH) {
            const int q = e / (TILE_C * 2), rem = e - q * (TILE_C * 2), c = rem >> 1, half = rem & 1;
            const int kk = kk0 + q;
            const bool valid = kk < p.KK && co0 + c < p.Co16 &&
                               EBS_IN_RANGE(p, CHK_MMA_W8, ((long long)kk * p.Co16 + co0 + c) * 32 + half * 16 + 15, p.lim_w8);
            const uint8_t* src = valid ? p.w8 + ((size_t)kk * p.Co16 + co0 + c) * 32 + half * 16 : p.w8;
            cp_async_bytes(W_s + (q * TILE_C + c) * 8 + half * 4, src, 16, valid);
        }
    };

    int acc[MT][NT][4];
    int wsum[MT][2];           // sum of the activation codes under the filter window, rows g and g+8 (w_levels)
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        wsum[mt][0] = 0; wsum[mt][1] = 0;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0;
    }

    __syncthreads();                                   // tap table ready
    const int nsteps = (p.KK + KSTEP - 1) / KSTEP;
    stage(0, 0);
    cp_async_commit();

    for (int st = 0; st < nsteps; ++st) {
        const int buf = st & 1;
        if (st + 1 < nsteps) {
            stage((st + 1) * KSTEP, buf ^ 1);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();

        const uint32_t* A_s = smem + buf * T::STAGE_WORDS;
        const uint32_t* W_s = A_s + KSTEP * TILE_P * AB;
#pragma unroll 1
        for (int q = 0; q < KSTEP; ++q) {
            if ((q & (p.fold - 1)) == 0 && st * KSTEP + q < p.KK) {
                if (p.w_levels) {            // window sum of the activation codes: every lane reads the whole
                                             // words of its rows g and g+8, so it can count them itself
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        const int r0 = (wp * MT + mt) * 16 + g;
                        for (int f = 0; f < p.fold && q + f < KSTEP; ++f) {
                            const uint32_t* row0 = A_s + ((q + f) * TILE_P + r0) * AB;
                            const uint32_t* row1 = row0 + 8 * AB;
#pragma unroll
                            for (int k = 0; k < AB; ++k) {
                                wsum[mt][0] += __popc(row0[k]) << k;
                                wsum[mt][1] += __popc(row1[k]) << k;
                            }
                        }
                    }
                }
                // activation fragments: the planes of a channel merged back into its code, byte = sum_k 2^k bit_k
                uint32_t af[MT][4];
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    const int r0 = (wp * MT + mt) * 16 + g;
                    const uint32_t* row0 = A_s + (q * TILE_P + r0) * AB;
                    const uint32_t* row1 = row0 + 8 * AB;
                    uint32_t wr0[AB], wr1[AB];
                    load_words_shared<AB>(row0, wr0);
                    load_words_shared<AB>(row1, wr1);
                    if (p.fold > 1) {                     // few input channels: several taps share one word
                        for (int f = 1; f < p.fold && q + f < KSTEP; ++f) {
                            uint32_t t0[AB], t1[AB];
                            load_words_shared<AB>(row0 + f * TILE_P * AB, t0);
                            load_words_shared<AB>(row1 + f * TILE_P * AB, t1);
#pragma unroll
                            for (int k = 0; k < AB; ++k) {
                                wr0[k] |= t0[k] << (f * p.fold_bits);
                                wr1[k] |= t1[k] << (f * p.fold_bits);
                            }
                        }
                    }
                    af[mt][0] = af[mt][1] = af[mt][2] = af[mt][3] = 0u;
#pragma unroll
                    for (int k = 0; k < AB; ++k) {
                        const uint32_t w0 = wr0[k], w1 = wr1[k];
                        const uint32_t mask = 0x01010101u << k;
                        af[mt][0] |= __funnelshift_r(w0, w0, tq - k) & mask;
                        af[mt][1] |= __funnelshift_r(w1, w1, tq - k) & mask;
                        af[mt][2] |= __funnelshift_r(w0, w0, tq + 4 - k) & mask;
                        af[mt][3] |= __funnelshift_r(w1, w1, tq + 4 - k) & mask;
                    }
                }
                // weight fragments: two words of the channel's byte row (the image holds the merged two's-complement
                // codes, K position 4b+i = channel 8i+b, and swaps the 16-byte halves of rows with (c_out >> 2) odd)
                uint32_t bf[NT][2];
                const int xw = (g >> 2) << 2;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const uint32_t* row = W_s + (q * TILE_C + (wc * NT + nt) * 8 + g) * 8;
                    bf[nt][0] = row[tq ^ xw];
                    bf[nt][1] = row[(4 + tq) ^ xw];
                    if (p.fold > 1) {
                        for (int f = 1; f < p.fold && q + f < KSTEP; ++f) {
                            const uint32_t* t = row + f * TILE_C * 8;
                            if (p.fold_bits >= 8) {       // channel c + f * fold_bits: same word, byte f * fold_bits / 8 up
                                bf[nt][0] |= t[tq ^ xw] << (f * p.fold_bits);
                                bf[nt][1] |= t[(4 + tq) ^ xw] << (f * p.fold_bits);
                            } else {                      // 4 channels a tap: odd taps land in the upper register
                                const uint32_t v = t[tq ^ xw] << (8 * (f >> 1));
                                if (f & 1) bf[nt][1] |= v; else bf[nt][0] |= v;
                            }
                        }
                    }
                }
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) mma_u8s8(acc[mt][nt], af[mt], bf[nt][0], bf[nt][1]);
            }
        }
        __syncthreads();
    }

    // ---- epilogue.  Fragment element e of (mt, nt): pixel row (e >> 1) * 8 + g, channel 2 * tq + (e & 1).
    const bool want_y = p.y != nullptr, want_q = p.packed_next != nullptr;
    uint8_t* out_s = reinterpret_cast<uint8_t*>(smem);      // [TILE_P][TILE_C + 4] requantized codes
    constexpr int ROWB = code_row_bytes(TILE_C);
    const int qmax = (1 << p.next_bits) - 1;
    const bool pair_ok = (p.Co & 1) == 0;                   // two adjacent channels form an aligned 8-byte pair
    // common case: even c_out, no per-channel terms, no residual, NHWC -> straight-line code
    if (p.w_levels) {                                       // accumulator = 2 * plane sum + window sum
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 2 * acc[mt][nt][e] + wsum[mt][e >> 1];
    }
    // common case: even c_out and NHWC -> two-channel vectors, per-channel terms kept in registers, the
    // shortcut codes (if the shortcut comes as packed planes) staged as bytes in the code tile
    const bool simple = !FULL || (pair_ok && !p.y_nchw);
    if (FULL && simple && p.res_packed) {
        constexpr int GROUPS = TILE_C / 8;
#pragma unroll 1
        for (int e = tid; e < TILE_P * GROUPS; e += NTH) {
            const int pl = e / GROUPS, grp = e - pl * GROUPS;
            const int gp = tile_p0 + pl, c = co0 + 8 * grp;
            uint32_t lo = 0u, hi = 0u;                          // codes of channels c .. c+3 and c+4 .. c+7, one per byte
            if (gp < p.P && c < p.Co) {
                const uint32_t* w = p.res_packed + ((size_t)gp * p.CWo + (c >> 5)) * p.res_bits;
                for (int j = 0; j < p.res_bits; ++j) {
                    const uint32_t byte = (__ldg(w + j) >> (c & 31)) & 0xFFu;         // plane j of the eight channels
                    lo |= (((byte & 0xFu) * 0x00204081u) & 0x01010101u) << j;          // bit i -> bit 8 i
                    hi |= (((byte >> 4) * 0x00204081u) & 0x01010101u) << j;
                }
            }
            uint32_t* dst = reinterpret_cast<uint32_t*>(out_s + pl * ROWB + 8 * grp);
            dst[0] = lo;
            dst[1] = hi;
        }
        __syncthreads();
    }
    if (simple) {
        // Per-channel terms and the shortcut default to exact identities (x * 1 and x + (-0) return x bit for bit), so
        // the block is straight-line code with uniform predicates on its loads and stores only; the accumulators go
        // out in a loop of their own.  (One unrolled copy instead of three keeps the kernel's code small: these
        // launches are short enough for instruction fetch to matter.)
        float cs[NT][2], cb[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int co = co0 + (wc * NT + nt) * 8 + 2 * tq;
            const bool in = co < p.Co;                          // c_out is even here: co + 1 exists with co
            cs[nt][0] = (FULL && p.ch_scale && in) ? __ldg(p.ch_scale + co) : 1.0f;
            cs[nt][1] = (FULL && p.ch_scale && in) ? __ldg(p.ch_scale + co + 1) : 1.0f;
            cb[nt][0] = (FULL && p.ch_bias && in) ? __ldg(p.ch_bias + co) : -0.0f;
            cb[nt][1] = (FULL && p.ch_bias && in) ? __ldg(p.ch_bias + co + 1) : -0.0f;
        }
        const int co_t = co0 + wc * NT * 8 + 2 * tq;            // this thread's first channel
        // plain form with further outputs: the accumulators are stored from the loop below
        const bool acc_inline = !FULL && p.acc && (want_y || want_q);
        if (p.acc && !acc_inline) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int gp = tile_p0 + (wp * MT + mt) * 16 + half * 8 + g;
                    int* row = p.acc + (size_t)gp * p.Co + co_t;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
                        if (gp < p.P && co_t + nt * 8 < p.Co && EBS_IN_RANGE(p, CHK_MMA_ACC, (long long)gp * p.Co + co_t + nt * 8 + 1, p.lim_out))
                            *reinterpret_cast<int2*>(row + nt * 8) = make_int2(acc[mt][nt][half * 2], acc[mt][nt][half * 2 + 1]);
                }
        }
        if (want_y || want_q) {
            const float relu_lo = p.relu ? 0.0f : -INFINITY;
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int pl = (wp * MT + mt) * 16 + half * 8 + g;
                    const int gp = tile_p0 + pl;
                    const size_t row_o = (size_t)gp * p.Co + co_t;
                    uint8_t* code_row = out_s + pl * ROWB + wc * NT * 8 + 2 * tq;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const bool valid = gp < p.P && co_t + nt * 8 < p.Co;
                        if constexpr (!FULL) {
                            if (acc_inline && valid && EBS_IN_RANGE(p, CHK_MMA_ACC, row_o + nt * 8 + 1, p.lim_out))
                                *reinterpret_cast<int2*>(p.acc + row_o + nt * 8) =
                                    make_int2(acc[mt][nt][half * 2], acc[mt][nt][half * 2 + 1]);
                        }
                        float y0 = __fmul_rn((float)acc[mt][nt][half * 2], p.S), y1 = __fmul_rn((float)acc[mt][nt][half * 2 + 1], p.S);
                        if constexpr (FULL) {
                            y0 = __fadd_rn(__fmul_rn(y0, cs[nt][0]), cb[nt][0]);
                            y1 = __fadd_rn(__fmul_rn(y1, cs[nt][1]), cb[nt][1]);
                        }
                        float r0 = -0.0f, r1 = -0.0f;
                        if constexpr (!FULL) {
                        } else if (p.residual) {
                            if (valid) {
                                const float2 r = __ldg(reinterpret_cast<const float2*>(p.residual + row_o + nt * 8));
                                r0 = r.x;
                                r1 = r.y;
                            }
                        } else if (p.res_packed) {
                            const uint32_t rc = *reinterpret_cast<const uint16_t*>(code_row + nt * 8);
                            r0 = __fmul_rn(p.res_scale, (float)(rc & 0xFFu));
                            r1 = __fmul_rn(p.res_scale, (float)(rc >> 8));
                        }
                        if constexpr (FULL) {
                            y0 = __fadd_rn(y0, r0);
                            y1 = __fadd_rn(y1, r1);
                        }
                        int code0, code1;
                        if constexpr (FULL) {
                            y0 = p.relu ? fmaxf(y0, 0.0f) : y0;
                            y1 = p.relu ? fmaxf(y1, 0.0f) : y1;
                            code0 = valid ? quantize_act_code(y0, p.inv_next, qmax) : 0;
                            code1 = valid ? quantize_act_code(y1, p.inv_next, qmax) : 0;
                        } else {
                            // plain form: y = acc * S is finite (the host checks S), so max(y, -inf) is y; channels past
                            // the layer have zero weight rows, hence zero codes, and pixels past it are never packed
                            y0 = fmaxf(y0, relu_lo);
                            y1 = fmaxf(y1, relu_lo);
                            code0 = quantize_act_code(y0, p.inv_next, qmax);
                            code1 = quantize_act_code(y1, p.inv_next, qmax);
                        }
                        if (want_y && valid && EBS_IN_RANGE(p, CHK_MMA_Y, row_o + nt * 8 + 1, p.lim_out))
                            *reinterpret_cast<float2*>(p.y + row_o + nt * 8) = make_float2(y0, y1);
                        if (want_q) *reinterpret_cast<uint16_t*>(code_row + nt * 8) = (uint16_t)(code0 | (code1 << 8));
                    }
                }
        }
    } else if constexpr (FULL) {
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int pl = (wp * MT + mt) * 16 + half * 8 + g;
            const int gp = tile_p0 + pl;
            const bool pvalid = gp < p.P;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int cl = (wc * NT + nt) * 8 + 2 * tq, co = co0 + cl;
                const int a0 = acc[mt][nt][half * 2], a1 = acc[mt][nt][half * 2 + 1];
                int code0 = 0, code1 = 0;
                if (pvalid && co < p.Co) {
                    const size_t o = (size_t)gp * p.Co + co;
                    const bool two = co + 1 < p.Co;
                    if (p.acc && EBS_IN_RANGE(p, CHK_MMA_ACC, o + (two ? 1 : 0), p.lim_out)) {
                        if (pair_ok) *reinterpret_cast<int2*>(p.acc + o) = make_int2(a0, a1);
                        else { p.acc[o] = a0; if (two) p.acc[o + 1] = a1; }
                    }
                    if (want_y || want_q) {
                        float y0 = __fmul_rn((float)a0, p.S), y1 = __fmul_rn((float)a1, p.S);
                        if (p.ch_scale) {
                            y0 = __fmul_rn(y0, __ldg(p.ch_scale + co));
                            if (two) y1 = __fmul_rn(y1, __ldg(p.ch_scale + co + 1));
                        }
                        if (p.ch_bias) {
                            y0 = __fadd_rn(y0, __ldg(p.ch_bias + co));
                            if (two) y1 = __fadd_rn(y1, __ldg(p.ch_bias + co + 1));
                        }
                        if (p.residual) {
                            y0 = __fadd_rn(y0, __ldg(p.residual + o));
                            if (two) y1 = __fadd_rn(y1, __ldg(p.residual + o + 1));
                        }
                        if (p.res_packed) {
                            y0 = __fadd_rn(y0, packed_residual(p, gp, co));
                            if (two) y1 = __fadd_rn(y1, packed_residual(p, gp, co + 1));
                        }
                        if (p.relu) {
                            if (!(y0 > 0.0f)) y0 = 0.0f;
                            if (!(y1 > 0.0f)) y1 = 0.0f;
                        }
                        if (want_y && EBS_IN_RANGE(p, CHK_MMA_Y, o + (two ? 1 : 0), p.lim_out)) {
                            if (p.y_nchw) {
                                const int hw = p.Ho * p.Wo;
                                const int n = gp / hw, rem = gp - n * hw;
                                p.y[((size_t)n * p.Co + co) * hw + rem] = y0;
                                if (two) p.y[((size_t)n * p.Co + co + 1) * hw + rem] = y1;
                            } else if (pair_ok) {
                                *reinterpret_cast<float2*>(p.y + o) = make_float2(y0, y1);
                            } else {
                                p.y[o] = y0;
                                if (two) p.y[o + 1] = y1;
                            }
                        }
                        if (want_q) {
                            code0 = quantize_act_code(y0, p.inv_next, qmax);
                            if (two) code1 = quantize_act_code(y1, p.inv_next, qmax);
                        }
                    }
                }
                if (want_q) *reinterpret_cast<uint16_t*>(out_s + pl * ROWB + cl) = (uint16_t)(code0 | (code1 << 8));
            }
        }
    }
    }
    if (want_q) {
        __syncthreads();
        pack_code_tile<TILE_P, TILE_C, NTH>(out_s, p, tile_p0, co0);
    }
}

template <int AB, int MT, int NT, int WARPS_P, int WARPS_C>
int launch_conv_mma(const ConvParams& p, dim3 grid, cudaStream_t st) {
    const bool full = p.ch_scale || p.ch_bias || p.residual || p.res_packed || p.y_nchw || (p.Co & 1) || p.w_levels ||
                      !isfinite(p.S);
    if (full) conv_mma_kernel<AB, MT, NT, WARPS_P, WARPS_C, true><<<grid, 32 * WARPS_P * WARPS_C, 0, st>>>(p);
    else conv_mma_kernel<AB, MT, NT, WARPS_P, WARPS_C, false><<<grid, 32 * WARPS_P * WARPS_C, 0, st>>>(p);
    return EBS_OK;
}

// Variants: variant = size_class * 3 + tile_c_index, tile_c in {16, 32, 64}.
//   class 0 (large)  the biggest warp tile the plane-pair count allows (fewest fragment rebuilds), 8 warps
//   class 1 (medium) 32 pixels x 16 channels per warp, 8 warps
//   class 2 (small)  16 pixels x 16 channels per warp, 4 warps -- for layers that otherwise leave SMs idle
// Every plane pair is one MMA per 16x8 output block per reduction word, so the large warp tile
// shrinks as the pair count grows.
template <int AB, int VARIANT>
struct MmaGeom {
    static constexpr int CLASS = VARIANT / 3;
    static constexpr int TILE_C = 16 << (VARIANT % 3);
    static constexpr int WARPS = CLASS == 2 ? TILE_C / 4 : 8;          // small: 4 pixel groups x TILE_C/16 channel groups
    static constexpr int NT_PREF = (CLASS == 0 && AB <= 4) ? 4 : 2;
    static constexpr int NT = (TILE_C / 8) < NT_PREF ? (TILE_C / 8) : NT_PREF;
    static constexpr int WARPS_C_RAW = TILE_C / (8 * NT);
    static constexpr int WARPS_C = WARPS_C_RAW > WARPS ? WARPS : WARPS_C_RAW;
    static constexpr int WARPS_P = WARPS / WARPS_C;
    static constexpr int ACC_BUDGET = AB == 1 ? 64 : (AB <= 4 ? 32 : 16);   // accumulator registers of a thread
    static constexpr int MT_RAW = ACC_BUDGET / (4 * NT);
    static constexpr int MT_AB = AB <= 2 ? 4 : (AB <= 4 ? 2 : 1);      // activation words in flight: MT*AB*2 registers
    static constexpr int MT_LARGE = MT_RAW < 1 ? 1 : (MT_RAW > MT_AB ? MT_AB : MT_RAW);
    static constexpr int MT = CLASS == 0 ? MT_LARGE : (CLASS == 1 ? (MT_AB < 2 ? MT_AB : 2) : 1);
};

constexpr int NUM_MMA_VARIANTS = 9;

template <int AB, int VARIANT>
constexpr ConvVariant make_mma_variant() {
    using G = MmaGeom<AB, VARIANT>;
    return ConvVariant{&launch_conv_mma<AB, G::MT, G::NT, G::WARPS_P, G::WARPS_C>, 16 * G::MT * G::WARPS_P,
                       8 * G::NT * G::WARPS_C, 32 * G::WARPS_P * G::WARPS_C};
}

// One translation unit per activation bit count (conv_mma_a1.cu .. conv_mma_a8.cu) defines its row of the table.
#define EBS_DEFINE_MMA_ROW(AB)                                                                           \
    const ConvVariant* conv_mma_variant_a##AB(int variant) {                                             \
        static const ConvVariant row[NUM_MMA_VARIANTS] = {                                               \
            make_mma_variant<AB, 0>(), make_mma_variant<AB, 1>(), make_mma_variant<AB, 2>(),             \
            make_mma_variant<AB, 3>(), make_mma_variant<AB, 4>(), make_mma_variant<AB, 5>(),             \
            make_mma_variant<AB, 6>(), make_mma_variant<AB, 7>(), make_mma_variant<AB, 8>()};            \
        if (variant < 0 || variant >= NUM_MMA_VARIANTS) return nullptr;                                  \
        return &row[variant];                                                                            \
    }

}  // namespace ebs
