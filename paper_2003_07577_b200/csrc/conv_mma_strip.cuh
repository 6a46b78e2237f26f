// Warp-level int8 MMA convolution for small stride-1 layers with every input pixel expanded ONCE per CTA.
//
// conv_mma_kernel rebuilds the activation fragments from the packed bits for every filter tap (two integer
// instructions per plane and register, kh*kw times per pixel) and the weight fragments in every warp.  Here a
// CTA owns TILE_P consecutive pixels of the zero-padded input frame (the numbering of conv_umma_strip_kernel:
// for stride 1 a filter tap is a constant shift), expands the strip TILE_P + (kh-1) Wp + (kw-1) of pixels into
// BYTES in shared memory once (32-byte rows per pixel and 32-channel word, byte 4b+i = channel 8i+b, the two
// 16-byte halves swapped when (pixel >> 2) & 1 so that fragment loads are bank-conflict free), copies the weight
// rows of its channel tile from the byte image that ebs_pack_weights appends (all taps and words: a few KB),
// and then only loads fragments: a0/a1 = bytes 4tq..4tq+3 of rows g and g+8, a2/a3 = bytes 16+4tq.. -- one
// 32-bit shared load per fragment register per tap.  The whole reduction of a layer fits in shared memory
// (c_in <= 128), so there is no staging pipeline.  Layers with at most 16 (8) input channels use only byte
// lanes 0-1 (0) of every register; there two (four) taps share one MMA step, the later tap's registers
// shifted left by 16 (8, 16, 24) bits, for both operands alike.
// COMPACT form (9-16 input channels, one word): 16 bytes per pixel and per weight row, so K positions 0-15 of an MMA
// step are one tap and 16-31 the next -- two taps per step without shifts and half the shared loads.
// Epilogue as in conv_mma_kernel (accumulator pairs, fp32 steps, code tile, multiply-gather pack), with the
// output pixel of a frame row looked up in a per-CTA table (rows with hp >= Ho or wp >= Wo have none).  The RES
// form carries the per-channel terms and the shortcut (fp32 or packed codes); the plain form, which the host picks
// when none of them is passed, leaves their instructions out.  These launches last a few microseconds and are
// bound by instruction issue and fetch, so the epilogue is one straight-line block and set-up loops are not unrolled.
#pragma once

#include <type_traits>

#include "conv_mma.cuh"
#include "conv_umma_strip.cuh"   // frame helpers (strip_pointwise, strip_frame_h/w)

namespace ebs {

struct MmaStripGeom {
    int strip_pix, strip_pad, smem_bytes, fold;
    bool ok;
};
inline MmaStripGeom mma_strip_geometry(const ConvParams& p, int tile_p, int tile_c) {
    MmaStripGeom g{};
    const int Wp = strip_frame_w(p), taps = p.kh * p.kw;
    g.strip_pix = tile_p + (p.kh - 1) * Wp + (p.kw - 1);
    g.strip_pad = (g.strip_pix + 7) & ~7;
    const int cin = p.CW == 1 ? p.fold_bits : 32;                 // fold_bits >= c_in for folded layers
    g.fold = (p.CW == 1 && cin <= 8) ? 4 : ((p.CW == 1 && cin <= 16) ? 2 : 1);
    const long long frame = (long long)p.N * strip_frame_h(p) * Wp;
    g.smem_bytes = p.CW * g.strip_pad * 32 + taps * p.CW * tile_c * 32 + tile_p * code_row_bytes(tile_c) + tile_p * 4 + 128;
    g.ok = ((p.sh == 1 && p.sw == 1) || strip_pointwise(p)) && p.CW <= 4 && taps * p.CW <= 64 && !p.w_levels &&
           !p.y_nchw && (p.Co & 1) == 0 && p.fold <= 4 &&
           g.smem_bytes <= 96 * 1024 && frame < (1LL << 31) - 4096 &&
           Wp < (1 << 15) && strip_frame_h(p) < (1 << 15) && g.strip_pix * p.CW < (1 << 15);   // small_div operands
    return g;
}

// floor(a / d) for 0 <= a < 2^20 and 1 <= d < 2^16 from the correctly rounded reciprocal of d: (a + 0.5) / d is at
// least 0.5 / d away from every integer and the two roundings move it by less than (a + d) 2^-23, so the floor of the
// product is the quotient (four instructions instead of a 32-bit integer division).
__device__ __forceinline__ int small_div(int a, float rcp_d) { return __float2int_rd(__fmul_rn((float)a + 0.5f, rcp_d)); }

template <int AB, int MT, int NT, int WARPS_P, int WARPS_C, bool COMPACT = false, bool RES = false>
__global__ void __launch_bounds__(32 * WARPS_P * WARPS_C)
conv_mma_strip_kernel(const ConvParams p) {
    constexpr int NTH = 32 * WARPS_P * WARPS_C, TILE_P = 16 * MT * WARPS_P, TILE_C = 8 * NT * WARPS_C;
    constexpr int ROWB = code_row_bytes(TILE_C);
    extern __shared__ __align__(16) uint8_t smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, tq = lane & 3;
    const int wp_ = warp % WARPS_P, wc = warp / WARPS_P;
    const int S = p.strip_pix, SP = (S + 7) & ~7, taps = p.kh * p.kw;
    const bool pointwise = strip_pointwise(p);
    const int Wp = strip_frame_w(p), Hp = strip_frame_h(p);
    const int frame = p.N * Hp * Wp;
    const int f0 = blockIdx.x * TILE_P, co0 = blockIdx.y * TILE_C;
    // COMPACT (one word of at most 16 channels): 16 bytes per pixel and weight row, word j = channels j, 8+j, 4+j, 12+j;
    // the weights get one more (zero) tap, the partner of the last tap when their number is odd
    uint8_t* strip = smem_raw;                                       // [CW][SP][32]   | [SP][16]
    uint8_t* wimg = strip + (COMPACT ? SP * 16 : p.CW * SP * 32);    // [taps * CW][TILE_C][32] | [taps + 1][TILE_C][16]
    uint8_t* out_s = wimg + (COMPACT ? (taps + 1) * TILE_C * 16 : taps * p.CW * TILE_C * 32);   // [TILE_P][ROWB] codes
    int* gp_s = reinterpret_cast<int*>(out_s + TILE_P * ROWB);       // output pixel of every frame row, -1: none
    // ---- weight rows of this channel tile, all taps and words (rows past c_out are zero in the image): asynchronous
    // copies issued first, so that their latency hides behind the tables and the strip expansion
    if constexpr (COMPACT) {
#pragma unroll 1
        for (int e = tid; e < (taps + 1) * TILE_C; e += NTH) {
            const int t = e / TILE_C, row = e - t * TILE_C;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (t < taps && co0 + row < p.Co16 &&
                EBS_IN_RANGE(p, CHK_MS_W8, ((long long)t * p.Co16 + co0 + row) * 32 + 31, p.lim_w8)) {
                const uint4* src = reinterpret_cast<const uint4*>(p.w8 + ((size_t)t * p.Co16 + co0 + row) * 32);
                const int sw = ((co0 + row) >> 2) & 1;                   // the image swaps the halves of these rows
                const uint4 lo = __ldg(src + sw), hi = __ldg(src + (sw ^ 1));
                v = make_uint4(__byte_perm(lo.x, hi.x, 0x5410), __byte_perm(lo.y, hi.y, 0x5410),
                               __byte_perm(lo.z, hi.z, 0x5410), __byte_perm(lo.w, hi.w, 0x5410));
            }
            reinterpret_cast<uint4*>(wimg)[e] = v;
        }
    } else {
#pragma unroll 1
        for (int e = tid; e < taps * p.CW * TILE_C * 2; e += NTH) {
            const int half = e & 1, row = (e >> 1) % TILE_C, kk = (e >> 1) / TILE_C;
            const bool valid = co0 + row < p.Co16 &&
                               EBS_IN_RANGE(p, CHK_MS_W8, ((long long)kk * p.Co16 + co0 + row) * 32 + half * 16 + 15, p.lim_w8) &&
                               EBS_IN_RANGE(p, CHK_MS_WS, (kk * TILE_C + row) * 32 + half * 16 + 15, taps * p.CW * TILE_C * 32);
            const uint8_t* src = valid ? p.w8 + ((size_t)kk * p.Co16 + co0 + row) * 32 + half * 16 : p.w8;
            cp_async_bytes(wimg + (kk * TILE_C + row) * 32 + half * 16, src, 16, valid);
        }
        cp_async_commit();
    }
    __shared__ int tap_shift_s[64];                                   // frame shift r * Wp + s of every tap
#pragma unroll 1
    for (int t = tid; t < taps; t += NTH) tap_shift_s[t] = (t / p.kw) * Wp + (t % p.kw);

    // ---- the strip: packed words -> bytes, once per pixel and word
    // frame coordinates of the tile's first pixel (two integer divisions a thread); the pixels after it are reached
    // with small quotients only
    const int n0 = f0 / (Hp * Wp), rem0 = f0 - n0 * (Hp * Wp);
    const int hp0 = rem0 / Wp, wq0 = rem0 - hp0 * Wp;
    const float rcp_w = __frcp_rn((float)Wp), rcp_h = __frcp_rn((float)Hp), rcp_cw = __frcp_rn((float)p.CW);
    // Two items per thread and round: both items' packed words are requested before either is used, so a strip of up
    // to 2 * NTH (pixel, word) items costs one round trip to memory, not two (the small layers this kernel serves are
    // a few microseconds long: a second dependent load is a tenth of that).
    constexpr int PF = 2;
    const int n_items = S * p.CW;
#pragma unroll 1
    for (int e0 = tid; e0 < n_items; e0 += PF * NTH) {
        uint32_t words[PF][AB];
        int s_[PF], cw_[PF], gp_[PF];
#pragma unroll
        for (int u = 0; u < PF; ++u) {
            const int e = e0 + u * NTH;
            s_[u] = -1;
            cw_[u] = 0;
            gp_[u] = -1;
#pragma unroll
            for (int k = 0; k < AB; ++k) words[u][k] = 0u;
            if (e >= n_items) continue;
            const int s = COMPACT ? e : small_div(e, rcp_cw), cw = COMPACT ? 0 : e - s * p.CW;
            s_[u] = s;
            cw_[u] = cw;
            const int f = f0 + s;
            if (f < frame) {
                const int cwq = small_div(wq0 + s, rcp_w), wq = wq0 + s - cwq * Wp;      // column, carry into the row
                const int chq = small_div(hp0 + cwq, rcp_h), hp = hp0 + cwq - chq * Hp;  // row, carry into the image
                const int n = n0 + chq;
                if (hp < p.Ho && wq < p.Wo) gp_[u] = (n * p.Ho + hp) * p.Wo + wq;        // the output pixel of this frame row
                const int h = pointwise ? hp * p.sh : hp - p.ph, w = pointwise ? wq * p.sw : wq - p.pw;
                if ((unsigned)h < (unsigned)p.H && (unsigned)w < (unsigned)p.W &&
                    EBS_IN_RANGE(p, CHK_MS_X, (((long long)(n * p.H + h) * p.W + w) * p.CW + cw) * AB + AB - 1, p.lim_x))
                    load_words_global<AB>(p.x + (((size_t)(n * p.H + h) * p.W + w) * p.CW + cw) * AB, words[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < PF; ++u) {
            const int s = s_[u], cw = cw_[u];
            if (s < 0) continue;
            uint32_t r[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};          // COMPACT uses r[0..3]: the four 4-channel words
            if constexpr (COMPACT) {
#pragma unroll
                for (int k = 0; k < AB; ++k) {
                    const uint32_t mask = 0x01010101u << k;
                    // bits 0-3 / 8-11 / 4-7 / 12-15 of the word to the low nibbles of bytes 0 / 1 / 2 / 3, then bit j
                    // of every byte to bit k of word j: bytes = channels j, 8+j, 4+j, 12+j
                    const uint32_t u4 = (words[u][k] & 0x0F0Fu) | ((words[u][k] & 0xF0F0u) << 12);
#pragma unroll
                    for (int j = 0; j < 4; ++j) r[j] |= __funnelshift_r(u4, u4, j - k) & mask;
                }
            } else {
                // v_k = rotl(w_k, k); byte register b = rotr(OR_k v_k & (0x01010101 << ((b + k) & 7)), b)
                uint32_t v[AB];
#pragma unroll
                for (int k = 0; k < AB; ++k) v[k] = __funnelshift_l(words[u][k], words[u][k], k);
#pragma unroll
                for (int b8 = 0; b8 < 8; ++b8) {
                    uint32_t t = v[0] & (0x01010101u << b8);
#pragma unroll
                    for (int k = 1; k < AB; ++k) t |= v[k] & (0x01010101u << ((b8 + k) & 7));
                    r[b8] = __funnelshift_r(t, t, b8);
                }
            }
            if (cw == 0 && s < TILE_P) gp_s[s] = gp_[u];
            if (!EBS_IN_RANGE(p, CHK_MS_STRIP, COMPACT ? s * 16 + 15 : (cw * SP + s) * 32 + 31, COMPACT ? SP * 16 : p.CW * SP * 32)) continue;
            if constexpr (COMPACT) {
                reinterpret_cast<uint4*>(strip)[s] = make_uint4(r[0], r[1], r[2], r[3]);
            } else {
                uint4* dst = reinterpret_cast<uint4*>(strip + (cw * SP + s) * 32);
                const int sw = (s >> 2) & 1;
                dst[sw] = make_uint4(r[0], r[1], r[2], r[3]);
                dst[sw ^ 1] = make_uint4(r[4], r[5], r[6], r[7]);
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();

    // ---- main loop: fragments are plain shared loads
    int acc[MT][NT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0;

    // taps per MMA step (1, 2 or 4, set by the launcher) as a compile-time constant of the loop body, so that the
    // fragment loads of a step are independent instructions the scheduler can overlap
    auto reduce = [&](auto fold_tag) {
        constexpr int FOLD = decltype(fold_tag)::value;
        constexpr int FSHIFT = 32 / FOLD;                              // bits a folded tap is shifted by
        const int arow0 = (wp_ * MT) * 16 + g;
        for (int cw = 0; cw < p.CW; ++cw) {
            const uint8_t* strip_w = strip + cw * SP * 32;
#pragma unroll 3           // (three taps' fragment loads in flight; nine made the ResNet-20 step 8% slower: code size)
            for (int t0 = 0; t0 < taps; t0 += FOLD) {
                uint32_t af[MT][4], bf[NT][2];
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) af[mt][0] = af[mt][1] = af[mt][2] = af[mt][3] = 0u;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) bf[nt][0] = bf[nt][1] = 0u;
#pragma unroll
                for (int ft = 0; ft < FOLD; ++ft) {
                    const int t = t0 + ft;
                    if (t < taps) {
                        const int shift = tap_shift_s[t];
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) {
                            const int pix0 = arow0 + mt * 16 + shift, pix1 = pix0 + 8;
                            const int x0 = ((pix0 >> 2) & 1) << 4, x1 = ((pix1 >> 2) & 1) << 4;
                            const uint8_t* r0 = strip_w + pix0 * 32;
                            const uint8_t* r1 = strip_w + pix1 * 32;
                            af[mt][0] |= *reinterpret_cast<const uint32_t*>(r0 + ((4 * tq) ^ x0)) << (ft * FSHIFT);
                            af[mt][1] |= *reinterpret_cast<const uint32_t*>(r1 + ((4 * tq) ^ x1)) << (ft * FSHIFT);
                            af[mt][2] |= *reinterpret_cast<const uint32_t*>(r0 + ((16 + 4 * tq) ^ x0)) << (ft * FSHIFT);
                            af[mt][3] |= *reinterpret_cast<const uint32_t*>(r1 + ((16 + 4 * tq) ^ x1)) << (ft * FSHIFT);
                        }
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            const int row = (wc * NT + nt) * 8 + g;
                            const int xb = (((co0 + row) >> 2) & 1) << 4;     // the image swaps the halves of these rows
                            const uint8_t* wr = wimg + ((t * p.CW + cw) * TILE_C + row) * 32;
                            bf[nt][0] |= *reinterpret_cast<const uint32_t*>(wr + ((4 * tq) ^ xb)) << (ft * FSHIFT);
                            bf[nt][1] |= *reinterpret_cast<const uint32_t*>(wr + ((16 + 4 * tq) ^ xb)) << (ft * FSHIFT);
                        }
                    }
                }
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) mma_u8s8(acc[mt][nt], af[mt], bf[nt][0], bf[nt][1]);
            }
        }
    };
    if constexpr (COMPACT) {
        // two taps per MMA step: K positions 0-15 are the first tap's 16 channels, 16-31 the second's
        const int arow0 = (wp_ * MT) * 16 + g;
#pragma unroll 1
        for (int t0 = 0; t0 < taps; t0 += 2) {
            const int t1 = t0 + 1;                                         // == taps: the zero weight rows
            const int sh0 = tap_shift_s[t0], sh1 = tap_shift_s[t1 < taps ? t1 : t0];
            uint32_t af[MT][4], bf[NT][2];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const uint8_t* r0 = strip + (arow0 + mt * 16 + sh0) * 16 + 4 * tq;
                const uint8_t* r1 = strip + (arow0 + mt * 16 + sh1) * 16 + 4 * tq;
                af[mt][0] = *reinterpret_cast<const uint32_t*>(r0);
                af[mt][1] = *reinterpret_cast<const uint32_t*>(r0 + 8 * 16);
                af[mt][2] = *reinterpret_cast<const uint32_t*>(r1);
                af[mt][3] = *reinterpret_cast<const uint32_t*>(r1 + 8 * 16);
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int row = (wc * NT + nt) * 8 + g;
                bf[nt][0] = *reinterpret_cast<const uint32_t*>(wimg + (t0 * TILE_C + row) * 16 + 4 * tq);
                bf[nt][1] = *reinterpret_cast<const uint32_t*>(wimg + (t1 * TILE_C + row) * 16 + 4 * tq);
            }
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) mma_u8s8(acc[mt][nt], af[mt], bf[nt][0], bf[nt][1]);
        }
    } else {
        if (p.strip_ks == 4) reduce(std::integral_constant<int, 4>{});
        else if (p.strip_ks == 2) reduce(std::integral_constant<int, 2>{});
        else reduce(std::integral_constant<int, 1>{});
    }

    // ---- epilogue.  Fragment element e of (mt, nt): tile row (e >> 1) * 8 + g, channel 2 * tq + (e & 1).
    const bool want_y = p.y != nullptr, want_q = p.packed_next != nullptr;
    const int qmax = (1 << p.next_bits) - 1;
    // Per-channel terms default to exact identities (x * 1 and x + (-0) return x bit for bit), so the block below is
    // straight-line code with uniform predicates only on its stores; accumulators go out in a loop of their own.
    float cs[NT][2], cb[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int co = co0 + (wc * NT + nt) * 8 + 2 * tq;
        const bool in = co < p.Co;                                  // c_out is even: co + 1 exists with co
        cs[nt][0] = (RES && p.ch_scale && in) ? __ldg(p.ch_scale + co) : 1.0f;
        cs[nt][1] = (RES && p.ch_scale && in) ? __ldg(p.ch_scale + co + 1) : 1.0f;
        cb[nt][0] = (RES && p.ch_bias && in) ? __ldg(p.ch_bias + co) : -0.0f;
        cb[nt][1] = (RES && p.ch_bias && in) ? __ldg(p.ch_bias + co + 1) : -0.0f;
    }
    const int co_t = co0 + wc * NT * 8 + 2 * tq;                    // this thread's first channel
    if (RES && p.res_packed) {                                      // shortcut codes of the tile, one per byte, into the code tile
        constexpr int GROUPS = TILE_C / 8;
#pragma unroll 1
        for (int e = tid; e < TILE_P * GROUPS; e += NTH) {
            const int pl = e / GROUPS, grp = e - pl * GROUPS;
            const int gp = gp_s[pl], c = co0 + 8 * grp;
            uint32_t lo = 0u, hi = 0u;                              // channels c .. c+3 and c+4 .. c+7
            if (gp >= 0 && c < p.Co) {
                const uint32_t* w = p.res_packed + ((size_t)gp * p.CWo + (c >> 5)) * p.res_bits;
#pragma unroll 1
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
    // plain form with further outputs: the accumulators are stored from the loop below (one table look-up a row)
    const bool acc_inline = !RES && p.acc && (want_y || want_q);
    if (p.acc && !acc_inline) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int gp = gp_s[(wp_ * MT + mt) * 16 + half * 8 + g];
                int* row = p.acc + (size_t)(gp < 0 ? 0 : gp) * p.Co + co_t;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
                    if (gp >= 0 && co_t + nt * 8 < p.Co && EBS_IN_RANGE(p, CHK_MS_ACC, (long long)gp * p.Co + co_t + nt * 8 + 1, p.lim_out))
                        *reinterpret_cast<int2*>(row + nt * 8) = make_int2(acc[mt][nt][half * 2], acc[mt][nt][half * 2 + 1]);
            }
    }
    if (want_y || want_q) {
        const float relu_lo = p.relu ? 0.0f : -INFINITY;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int pl = (wp_ * MT + mt) * 16 + half * 8 + g;
                const int gp = gp_s[pl];
                float* yrow = p.y + (size_t)(gp < 0 ? 0 : gp) * p.Co + co_t;
                uint8_t* code_row = out_s + pl * ROWB + wc * NT * 8 + 2 * tq;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const bool valid = gp >= 0 && co_t + nt * 8 < p.Co;
                    if constexpr (!RES) {
                        if (acc_inline && valid && EBS_IN_RANGE(p, CHK_MS_ACC, (long long)gp * p.Co + co_t + nt * 8 + 1, p.lim_out))
                            *reinterpret_cast<int2*>(p.acc + (size_t)gp * p.Co + co_t + nt * 8) =
                                make_int2(acc[mt][nt][half * 2], acc[mt][nt][half * 2 + 1]);
                    }
                    float y0 = __fmul_rn((float)acc[mt][nt][half * 2], p.S), y1 = __fmul_rn((float)acc[mt][nt][half * 2 + 1], p.S);
                    if constexpr (RES) {
                        y0 = __fadd_rn(__fmul_rn(y0, cs[nt][0]), cb[nt][0]);
                        y1 = __fadd_rn(__fmul_rn(y1, cs[nt][1]), cb[nt][1]);
                    }
                    float r0 = -0.0f, r1 = -0.0f;                    // the shortcut, if any, after the per-channel terms
                    if constexpr (!RES) {
                    } else if (p.residual) {
                        if (valid) {
                            const float2 r = __ldg(reinterpret_cast<const float2*>(p.residual + (size_t)gp * p.Co + co_t + nt * 8));
                            r0 = r.x;
                            r1 = r.y;
                        }
                    } else if (p.res_packed) {
                        const uint32_t rc = *reinterpret_cast<const uint16_t*>(code_row + nt * 8);
                        r0 = __fmul_rn(p.res_scale, (float)(rc & 0xFFu));
                        r1 = __fmul_rn(p.res_scale, (float)(rc >> 8));
                    }
                    if constexpr (RES) {
                        y0 = __fadd_rn(y0, r0);
                        y1 = __fadd_rn(y1, r1);
                    }
                    int code0, code1;
                    if constexpr (RES) {
                        y0 = p.relu ? fmaxf(y0, 0.0f) : y0;
                        y1 = p.relu ? fmaxf(y1, 0.0f) : y1;
                        code0 = valid ? quantize_act_code(y0, p.inv_next, qmax) : 0;
                        code1 = valid ? quantize_act_code(y1, p.inv_next, qmax) : 0;
                    } else {
                        // plain form: y = acc * S is finite (the host checks S), so max(y, -inf) is y; rows and channels
                        // past the layer have zero accumulators (zero weight rows), hence zero codes, without a select
                        y0 = fmaxf(y0, relu_lo);
                        y1 = fmaxf(y1, relu_lo);
                        code0 = quantize_act_code(y0, p.inv_next, qmax);
                        code1 = quantize_act_code(y1, p.inv_next, qmax);
                    }
                    if (want_y && valid && EBS_IN_RANGE(p, CHK_MS_Y, (long long)gp * p.Co + co_t + nt * 8 + 1, p.lim_out))
                        *reinterpret_cast<float2*>(yrow + nt * 8) = make_float2(y0, y1);
                    if (want_q) *reinterpret_cast<uint16_t*>(code_row + nt * 8) = (uint16_t)(code0 | (code1 << 8));
                }
            }
    }
    if (want_q) {
        __syncthreads();
        constexpr int CWL = (TILE_C + 31) / 32;
        constexpr int NW = TILE_C >= 32 ? 8 : TILE_C / 4;           // code words per 32-channel group
#pragma unroll 1
        for (int item = tid; item < TILE_P * CWL; item += NTH) {
            const int cwl = item / TILE_P, pl = item - cwl * TILE_P;
            const int gp = gp_s[pl], cwg = (co0 >> 5) + cwl;
            if (gp < 0 || cwg >= p.CWo) continue;
            const uint32_t* row = reinterpret_cast<const uint32_t*>(out_s + pl * ROWB + cwl * 32);
            uint32_t codes[NW];
#pragma unroll
            for (int k = 0; k < NW; ++k) codes[k] = row[k];
            uint32_t* dst = p.packed_next + ((size_t)gp * p.CWo + cwg) * p.next_bits;
            if (!EBS_IN_RANGE(p, CHK_MS_PN, ((long long)gp * p.CWo + cwg) * p.next_bits + p.next_bits - 1, p.lim_pn)) continue;
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
}

template <int AB, int MT, int NT, int WARPS_P, int WARPS_C>
int launch_conv_mma_strip(const ConvParams& p0, dim3 /*grid*/, cudaStream_t st) {
    constexpr int TILE_P = 16 * MT * WARPS_P, TILE_C = 8 * NT * WARPS_C;
    ConvParams p = p0;
    const MmaStripGeom g = mma_strip_geometry(p, TILE_P, TILE_C);
    if (!g.ok) return EBS_ERR_UNSUPPORTED;                    // the geometry does not apply: nothing is launched
    p.strip_pix = g.strip_pix;
    p.strip_ks = g.fold;
    // four forms of the kernel: with or without per-channel and shortcut terms (RES; layers without any do not pay
    // for them), and for the 16-channel tile the 16-byte-per-pixel form when the layer has 9-16 input channels
    const bool res = p.residual || p.res_packed || p.ch_scale || p.ch_bias || !isfinite(p.S);
    const bool compact = TILE_C == 16 && g.fold == 2;
    static bool attr_set[4][64] = {};                           // per kernel form and device
    auto go = [&](void (*kernel)(const ConvParams), int form) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (dev >= 0 && dev < 64 && !attr_set[form][dev]) {
            cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
            attr_set[form][dev] = true;
        }
        const long long frame = (long long)p.N * strip_frame_h(p) * strip_frame_w(p);
        const dim3 grid((unsigned)((frame + TILE_P - 1) / TILE_P), (unsigned)((p.Co + TILE_C - 1) / TILE_C), 1);
        kernel<<<grid, 32 * WARPS_P * WARPS_C, g.smem_bytes, st>>>(p);
    };
    if constexpr (TILE_C == 16) {
        if (compact) {
            if (res) go(conv_mma_strip_kernel<AB, MT, NT, WARPS_P, WARPS_C, true, true>, 3);
            else go(conv_mma_strip_kernel<AB, MT, NT, WARPS_P, WARPS_C, true, false>, 2);
            return EBS_OK;
        }
    }
    if (res) go(conv_mma_strip_kernel<AB, MT, NT, WARPS_P, WARPS_C, false, true>, 1);
    else go(conv_mma_strip_kernel<AB, MT, NT, WARPS_P, WARPS_C, false, false>, 0);
    return EBS_OK;
}

// Variants: channel tile 16 / 32 / 64, 256 frame pixels per CTA (8 warps).
constexpr int NUM_MMA_STRIP_VARIANTS = 3;

}  // namespace ebs
