// Persistent, warp-specialised bit-plane convolution on the tcgen05 tensor cores for every layer
// geometry the ResNet stacks contain: stride-1 k x k, strided k x k, and 1 x 1 at any stride.
//
// Arithmetic as in conv_umma_kernel (Eq. 13-14 regrouped channel by channel): the planes of a packed
// word are merged back into one byte per channel and one int8 MMA per (tap, reduction word) retires
// all Wb*Ab plane pairs of its 32 channels.  What this kernel adds:
//
//  * One addressing scheme for all strides.  Write a tap offset as r - pad_h = stride_h * qr + a with
//    0 <= a < stride_h (likewise s - pad_w = stride_w * qs + b).  The input pixels with row parity a and
//    column parity b form a "phase" image X_ab[i][j] = X[stride_h * i + a][stride_w * j + b], and tap
//    (r, s) of output (ho, wo) reads X_ab[ho + qr][wo + qs]: a stride-1 access.  Outputs are numbered in
//    a frame of Hq x Wq pixels per image (Hq = Ho + max qr - min qr, likewise Wq) and a tap becomes a
//    constant shift (qr - min qr) * Wq + (qs - min qs) inside the strip of frame pixels a CTA expands to
//    bytes.  Stride 1 has one phase (the frame is the zero-padded input); a 3x3 stride-2 layer has
//    four, a strided 1x1 layer one (only the pixels it reads).  Every input pixel is expanded once per
//    CTA and tile, whatever the stride and however many taps read it.
//  * Super-tiles: a CTA owns m_sub x 128 consecutive frame pixels x TILE_N channels with one
//    accumulator per 128 pixels in tensor memory, so a weight tile fetched into shared memory feeds
//    m_sub MMAs and the halo of the strip is shared.
//  * Weights stay resident in shared memory when all (tap, word) tiles of a channel tile fit, else they
//    stream through the stage ring by cp.async.bulk, a stage ahead of the MMAs.
//  * Roles (20 warps): warps 0-7 expand (packed words -> byte strips, global loads two chunks ahead), warps 8-9
//    issue the MMAs (two warps when a tile has an even number of accumulators: each owns the accumulators of one
//    parity; a single warp needs 140-180 clocks per MMA and was the bound of the k x k layers), warp 10 fetches weight
//    tiles (every lane one tile of a ring slot), warps 12-19 run the epilogue out of tensor memory while the next
//    tile's MMAs fill the other accumulator set.
//  * Bit <-> byte transposes by rotate and bit-select: with v_k = rotl(w_k, k) the byte register of
//    channels {b, 8+b, 16+b, 24+b} is rotr(t_b, b), byte position (b+k) & 7 of t_b taken from v_k; the
//    selects of plane pairs and quads are shared between the eight registers (planes_to_bytes), and the
//    epilogue packs requantized codes into plane words with the mirrored tree (bytes_to_planes).
//  * PAIR form (the 256-channel tile on a cluster of two CTAs): one MMA of M = 256 per (tap, word) over
//    both CTAs' shared and tensor memory (cta_group::2), each CTA fetching the weight rows of half the
//    channel tile; see the kernel.  Every copy into shared memory is a plain per-CTA copy; the MMAs' completion is
//    signalled to both CTAs by one tcgen05.commit each.
//
// Every wait on an mbarrier is bounded (ConvParams::wait_limit polls); on a timeout the CTA raises a
// shared abort flag, all its loops end, it records the event in a device counter, frees its tensor
// memory and returns.  The single-CTA forms use no clusters.
#pragma once

#include "conv_umma_strip.cuh"

namespace ebs {

constexpr int PIPE_EXPANDERS = 256;
// Warps 8 and 9 issue the MMAs, warp 10 fetches weights, warp 11 has no role (20 warps cost the same registers as 18:
// they are allotted in fours), warps 12-19 run the epilogue.
constexpr int PIPE_ISSUER_WARP = 8, PIPE_ISSUERS = 2, PIPE_PRODUCER_WARP = 10, PIPE_EPI_WARP0 = 12, PIPE_EPI_WARPS = 8;
constexpr int PIPE_THREADS = (PIPE_EPI_WARP0 + PIPE_EPI_WARPS) * 32;
constexpr int PIPE_SLOTS = 2;                      // (pixel, word) items an expander thread handles per stage
constexpr int PIPE_MAX_ITEMS = PIPE_SLOTS * PIPE_EXPANDERS;
constexpr int PIPE_MAX_TAPS = 64, PIPE_MAX_PHASES = 4, PIPE_MAX_STAGES = 4;
constexpr int PIPE_MAX_BSLOTS = 32;                // weight tiles in flight when the weights stream
constexpr int PIPE_MAX_MMAS = 512;                 // MMAs of one chunk (table of their operand offsets in shared memory)
constexpr int PIPE_SMEM_MAX = 220 * 1024;

// Exact unsigned division by a run-time constant: q = (t + ((n - t) >> s1)) >> s2, t = mulhi(m, n).
struct FastDiv {
    uint32_t m, s1, s2;
};
inline FastDiv make_fastdiv(uint32_t d) {
    FastDiv f{};
    uint32_t l = 0;
    while ((1ull << l) < d) ++l;
    f.m = (uint32_t)(((1ull << 32) * ((1ull << l) - d)) / d + 1);
    f.s1 = l < 1 ? l : 1;
    f.s2 = l > 1 ? l - 1 : 0;
    return f;
}
__device__ __forceinline__ uint32_t fastdiv(uint32_t n, const FastDiv& f) {
    const uint32_t t = __umulhi(f.m, n);
    return (t + ((n - t) >> f.s1)) >> f.s2;
}

// Launch geometry, computed on the host and passed to the kernel by value.
struct PipeGeom {
    int Wq, Hq, frame;                 // frame of one image and pixels of all images
    FastDiv div_img, div_row;          // by Hq * Wq and by Wq
    int q0r, q0s;                      // smallest tap quotients (<= 0)
    int m_sub, tile_pix;               // accumulators per super-tile; 128 * m_sub
    int n_ptiles, n_ctiles;
    int S, SP;                         // strip pixels (tile_pix + largest tap shift), rounded up to 8
    int ks, nsub, kss, nwg;            // words per expander pass; passes per stage; words per stage = ks * nsub;
                                       // word groups (stages per tile and phase) = ceil(CW / kss)
    int n_ph, nchunks;                 // phases; chunks per tile = n_ph * nwg (phase-major)
    int n_stages, a_word_bytes, a_stage_bytes, stage_bytes;
    int b_resident, b_total_bytes, taps;
    int b_slots, b_group;              // streamed weights: ring of slots of b_group (tap, word) tiles of TILE_N x 32 bytes
    int nbuf, tmem_cols, smem_bytes;
    int pair;                          // 1: two CTAs of a cluster share every MMA (256 pixels x 256 channels, half a weight tile each)
    int grid_x, grid_y;
    int ph_a[PIPE_MAX_PHASES], ph_b[PIPE_MAX_PHASES];
    int ph_tap0[PIPE_MAX_PHASES + 1];  // tap slots of phase i: [ph_tap0[i], ph_tap0[i + 1])
    short tap_shift[PIPE_MAX_TAPS];    // per tap slot: shift inside the strip, in pixels
    short tap_id[PIPE_MAX_TAPS];       // per tap slot: r * kw + s (tile index in the weight byte image)
    bool ok;
};

inline int floordiv_int(int a, int b) { return (a >= 0) ? a / b : -((-a + b - 1) / b); }

// m_sub_req / ks_req = 0: chosen here.  Returns ok = false when the kernel does not apply.
inline PipeGeom pipe_geometry(const ConvParams& p, int tile_n, int sms, int m_sub_req = 0, bool pair = false) {
    PipeGeom g{};
    if (pair && (tile_n != 256 || (p.Co % 256) != 0 || sms < 2)) return g;
    const int pw = pair ? 2 : 1;                               // CTAs that share a pixel pair-tile
    g.pair = pair ? 1 : 0;
    sms /= pw;                                                 // the unit that takes work items: a CTA, or a pair
    const int taps = p.kh * p.kw;
    if (p.w_levels || p.sh > 2 || p.sw > 2 || taps > PIPE_MAX_TAPS || p.kh > 16 || p.kw > 16) return g;
    if (tile_n != 64 && tile_n != 128 && tile_n != 256) return g;
    if ((long long)p.CW * 8 > PIPE_ZERO_WORDS) return g;      // the zero page covers a pixel's words at 8 planes (byte codes: 8 words a word)
    g.q0r = floordiv_int(-p.ph, p.sh);
    g.q0s = floordiv_int(-p.pw, p.sw);
    const int qr_max = floordiv_int(p.kh - 1 - p.ph, p.sh), qs_max = floordiv_int(p.kw - 1 - p.pw, p.sw);
    g.Hq = p.Ho + qr_max - g.q0r;
    g.Wq = p.Wo + qs_max - g.q0s;
    const long long frame = (long long)p.N * g.Hq * g.Wq;
    if (frame >= (1LL << 31) - 4096) return g;
    g.frame = (int)frame;
    g.div_img = make_fastdiv((uint32_t)(g.Hq * g.Wq));
    g.div_row = make_fastdiv((uint32_t)g.Wq);
    const int max_shift = (qr_max - g.q0r) * g.Wq + (qs_max - g.q0s);
    if (max_shift > 30000) return g;
    // phases and their taps
    g.taps = taps;
    int slot = 0;
    for (int a = 0; a < p.sh; ++a)
        for (int b = 0; b < p.sw; ++b) {
            const int first = slot;
            for (int r = 0; r < p.kh; ++r)
                for (int s = 0; s < p.kw; ++s) {
                    const int qr = floordiv_int(r - p.ph, p.sh), qs = floordiv_int(s - p.pw, p.sw);
                    if ((r - p.ph) - p.sh * qr != a || (s - p.pw) - p.sw * qs != b) continue;
                    g.tap_shift[slot] = (short)((qr - g.q0r) * g.Wq + (qs - g.q0s));
                    g.tap_id[slot] = (short)(r * p.kw + s);
                    ++slot;
                }
            if (slot > first) {
                g.ph_a[g.n_ph] = a;
                g.ph_b[g.n_ph] = b;
                g.ph_tap0[g.n_ph] = first;
                ++g.n_ph;
            }
        }
    g.ph_tap0[g.n_ph] = slot;
    int max_ph_taps = 0;
    for (int i = 0; i < g.n_ph; ++i) max_ph_taps = max_ph_taps > g.ph_tap0[i + 1] - g.ph_tap0[i] ? max_ph_taps : g.ph_tap0[i + 1] - g.ph_tap0[i];
    g.n_ctiles = (p.Co + tile_n - 1) / tile_n;
    const int b_tile = tile_n * 32 / pw;                       // a pair: each CTA holds the rows of half the channels
    g.b_total_bytes = p.CW * taps * b_tile;
    const int deep = p.CW * taps;                               // MMAs per accumulator and tile
    // candidates for the super-tile, largest first: it must leave the strip within the expanders' items and give
    // the SMs enough tiles; a deep reduction prefers the widest accumulator set even without double buffering
    const int m_cap = 512 / tile_n;                             // accumulators that fit in tensor memory at all
    int m_sub = 0;
    for (int m = m_cap; m >= 1; m >>= 1) {
        if (m_sub_req && m != m_sub_req) continue;
        const int nb = (2 * m * tile_n <= 512) ? 2 : 1;
        if (nb == 1 && deep < 64 && !m_sub_req) continue;        // shallow reductions want the epilogue overlapped
        if (m * UMMA_M + max_shift > PIPE_MAX_ITEMS) continue;
        const long long pt = (frame + (long long)m * UMMA_M * pw - 1) / ((long long)m * UMMA_M * pw);
        if (!m_sub_req && m > 1 && pt * g.n_ctiles < (deep >= 64 ? 1LL : 2LL) * sms) continue;
        m_sub = m;
        break;
    }
    if (!m_sub) return g;
    g.m_sub = m_sub;
    g.tile_pix = m_sub * UMMA_M;
    g.nbuf = (2 * m_sub * tile_n <= 512) ? 2 : 1;
    g.tmem_cols = g.nbuf * m_sub * tile_n;
    if (g.tmem_cols < 32) g.tmem_cols = 32;
    g.n_ptiles = (int)((frame + (long long)g.tile_pix * pw - 1) / ((long long)g.tile_pix * pw));   // pair-tiles for a pair
    g.S = g.tile_pix + max_shift;
    g.SP = (g.S + 7) & ~7;
    g.a_word_bytes = g.SP * 32 + 64;                           // sized with the largest skew; fixed once ks is known
    if (g.SP * 16 >= (1 << 18)) return g;
    // weights resident when they leave room for at least two activation stages
    const int budget = PIPE_SMEM_MAX - 2048 - PIPE_MAX_MMAS * 8;   // the MMA table sits behind the rings
    g.b_resident = g.b_total_bytes + 2 * ((g.a_word_bytes + 255) & ~255) <= budget && g.b_total_bytes <= 160 * 1024;
    int ks = PIPE_MAX_ITEMS / g.S;
    if (ks > 4) ks = 4;
    if (ks > p.CW) ks = p.CW;
    if (ks < 1) return g;
    while (ks > 1 && ks * taps * m_sub >= PIPE_MAX_MMAS - 2) --ks;     // (the issue loops read up to two entries ahead)
    if (ks * taps * m_sub >= PIPE_MAX_MMAS - 2) return g;
    // Streamed weights go through a ring of their own (slots of a few consecutive (tap, word) tiles), so that copies are
    // in flight all the time (a stage-sized unit would leave the copy engine idle while a stage's MMAs run).
    auto stage_bytes = [&](int k) { return (k * g.a_word_bytes + 255) & ~255; };
    const int b_ring_min = g.b_resident ? 0 : 96 * 1024 / pw;
    const int avail = budget - (g.b_resident ? g.b_total_bytes : b_ring_min);
    while (ks > 1 && 2 * stage_bytes(ks) > avail) --ks;
    if (2 * stage_bytes(ks) > avail) return g;
    // fewer words per pass when that buys a deeper ring (latency hiding matters more than stage size)
    while (ks > 1 && avail / stage_bytes(ks) < 3) --ks;
    // A stage is filled in nsub expander passes of ks words: the thread that issues the MMAs retires an instruction
    // only every ten clocks or so, so its per-stage bookkeeping has to be spread over about a dozen MMAs.
    int nsub = 1;
    while (nsub < 4 && ks * nsub * taps * m_sub < 12 && ks * nsub < p.CW &&
           ks * 2 * nsub * taps * m_sub < PIPE_MAX_MMAS - 2 && 3 * stage_bytes(ks * 2 * nsub) <= avail)
        nsub *= 2;
    // Skew between the word tiles of a pass: the 8 lanes of a quarter warp store 16 bytes each for ks words of 8 / ks
    // pixels; a skew of 128 / ks bytes (48 for three words) puts them on eight different 16-byte bank groups.
    g.a_word_bytes = g.SP * 32 + (ks == 4 ? 32 : ks == 3 ? 48 : 64);
    g.ks = ks;
    g.nsub = nsub;
    g.kss = ks * nsub;
    g.nwg = (p.CW + g.kss - 1) / g.kss;
    g.nchunks = g.n_ph * g.nwg;
    g.a_stage_bytes = stage_bytes(g.kss);
    g.stage_bytes = g.a_stage_bytes;
    g.n_stages = avail / g.stage_bytes;
    const int st_cap = g.b_resident ? PIPE_MAX_STAGES : (pair ? PIPE_MAX_STAGES : 3);
    if (g.n_stages > st_cap) g.n_stages = st_cap;
    if (!g.b_resident) {
        // a slot holds up to 32 KB of consecutive tiles of a chunk (one wait and one commit per slot, not per MMA)
        g.b_group = 32768 / b_tile;
        if (g.b_group > g.kss * max_ph_taps) g.b_group = g.kss * max_ph_taps;
        if (g.b_group < 1) g.b_group = 1;
        g.b_slots = (budget - g.n_stages * g.stage_bytes) / (g.b_group * b_tile);
        if (g.b_slots > PIPE_MAX_BSLOTS) g.b_slots = PIPE_MAX_BSLOTS;
        if (g.b_slots < 3) return g;
    }
    g.smem_bytes = (g.b_resident ? g.b_total_bytes : g.b_slots * g.b_group * b_tile) + g.n_stages * g.stage_bytes + 1024 +
                   PIPE_MAX_MMAS * 8;
    if (g.b_resident) {                                        // a CTA keeps one channel tile
        g.grid_y = g.n_ctiles;
        long long gx = sms / g.n_ctiles;
        if (gx < 1) gx = 1;
        if (gx > g.n_ptiles) gx = g.n_ptiles;
        g.grid_x = (int)gx * pw;
    } else {
        g.grid_y = 1;
        const long long items = (long long)g.n_ptiles * g.n_ctiles;
        g.grid_x = (int)(items < sms ? items : sms) * pw;
    }
    g.ok = g.n_stages >= 2 && g.smem_bytes <= PIPE_SMEM_MAX && g.grid_y <= 65535 && g.n_ctiles <= 65535;
    return g;
}

// NW plane words of one (pixel, 32-channel word) item -> eight registers of four channel bytes (row byte 4b + i = channel
// 8i + b).  With v_k = rotl(w_k, k), register b is rotr(t_b, b) where byte position (b + k) & 7 of t_b holds plane k.  The
// eight t_b pick the planes in eight cyclic orders, and orders that agree modulo 2 (modulo 4) share their pairs (quads)
// of planes: one bit-select per pair and parity, one per quad and residue, one per register - 24 selects for eight
// planes where a merge per (register, plane) takes 64.
__device__ __forceinline__ uint32_t bit_select(uint32_t a, uint32_t b, uint32_t m) { return (a & m) | (b & ~m); }

template <int NW>
__device__ __forceinline__ void planes_to_bytes(const uint32_t (&w)[NW], uint32_t (&r)[8]) {
    uint32_t v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = k < NW ? __funnelshift_l(w[k < NW ? k : 0], w[k < NW ? k : 0], k) : 0u;
    if constexpr (NW == 1) {
#pragma unroll
        for (int bb = 0; bb < 8; ++bb) {
            const uint32_t t = v[0] & (0x01010101u << bb);
            r[bb] = __funnelshift_r(t, t, bb);
        }
    } else {
        // pairs: plane 2j on the even bit positions and plane 2j + 1 on the odd ones (parity 0), or the reverse
        uint32_t pr[4][2];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            pr[j][0] = bit_select(v[2 * j], v[2 * j + 1], 0x55555555u);
            pr[j][1] = bit_select(v[2 * j + 1], v[2 * j], 0x55555555u);
        }
        if constexpr (NW == 2) {
#pragma unroll
            for (int bb = 0; bb < 8; ++bb) {
                const uint32_t t = pr[0][bb & 1] & ((0x01010101u << bb) | (0x01010101u << ((bb + 1) & 7)));
                r[bb] = __funnelshift_r(t, t, bb);
            }
        } else {
            // quads: the pair 2i on the positions = c, c + 1 (mod 4), the pair 2i + 1 on the other two
            uint32_t qd[2][4];
#pragma unroll
            for (int i = 0; i < 2; ++i)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t m2 = c == 0 ? 0x33333333u : c == 1 ? 0x66666666u : c == 2 ? 0xCCCCCCCCu : 0x99999999u;
                    qd[i][c] = bit_select(pr[2 * i][c & 1], pr[2 * i + 1][c & 1], m2);
                }
#pragma unroll
            for (int bb = 0; bb < 8; ++bb) {
                const uint32_t m3 = 0x01010101u * (uint32_t)(((0x0Fu << bb) | (0x0Fu >> (8 - bb))) & 0xFFu);
                const uint32_t t = bit_select(qd[0][bb & 3], qd[1][bb & 3], m3);   // planes 0-3 on positions bb .. bb + 3
                r[bb] = __funnelshift_r(t, t, bb);
            }
        }
    }
}

// Eight registers of four channel bytes (byte i of register b = channel 8i + b) -> plane words: the mirror image of
// planes_to_bytes.  With c_b = rotl(bytes_b, b), plane j is rotr(t_j, j) where byte position (b + j) & 7 of t_j comes from
// register b; the pair and quad selects are shared between the planes (16 + nb selects where a merge per (plane,
// register) takes 8 * nb).
__device__ __forceinline__ void bytes_to_planes(const uint32_t (&cr)[8], int nb, uint32_t (&planes)[8]) {
    uint32_t pr[4][2], qd[2][4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        pr[j][0] = bit_select(cr[2 * j], cr[2 * j + 1], 0x55555555u);
        pr[j][1] = bit_select(cr[2 * j + 1], cr[2 * j], 0x55555555u);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint32_t m2 = c == 0 ? 0x33333333u : c == 1 ? 0x66666666u : c == 2 ? 0xCCCCCCCCu : 0x99999999u;
            qd[i][c] = bit_select(pr[2 * i][c & 1], pr[2 * i + 1][c & 1], m2);
        }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        if (j >= nb) break;
        const uint32_t m3 = 0x01010101u * (uint32_t)(((0x0Fu << j) | (0x0Fu >> (8 - j))) & 0xFFu);
        const uint32_t t = bit_select(qd[0][j & 3], qd[1][j & 3], m3);
        planes[j] = __funnelshift_r(t, t, j);
    }
}

// fl(t) -> the bit pattern 0x4B000000 + clamp(floor(t), 0, qmax) without the conversion pipe and with one logic-pipe
// instruction: t + |t| is 2 * max(t, 0) exactly, the minimum with 2 * qmax + 1 bounds it (floor and clamp commute for
// integer bounds: floor(min(max(t, 0), qmax + 1/2)) = min(max(floor(t), 0), qmax)), and the halving and the 2^23 go into
// one multiply-add rounded toward -inf, whose low mantissa bits are the floor.
__device__ __forceinline__ uint32_t code_pattern(float t, float hi2) {
    const float a = __fadd_rn(t, fabsf(t));
    return __float_as_uint(__fmaf_rd(fminf(a, hi2), 0.5f, 8388608.0f));
}

// One 32-channel group of the plain epilogue: 32 accumulators of this thread's pixel -> stores, fp32 steps,
// requantized codes -> plane words.
// tcgen05.mma with both descriptors given as (low word, high word): the start-address field sits in the low word, so
// an operand is moved by a 32-bit addition.  The whole warp executes the call with the same operands and the
// instruction is predicated on `leader` (non-zero in one lane): with the issue loop free of divergent branches its
// address arithmetic stays warp-uniform, which measured faster than a loop run by one thread alone.
__device__ __forceinline__ void umma_i8_split(uint32_t leader, uint32_t tmem_d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                              uint32_t b_hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "setp.ne.b32 q, %7, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %5, p;\n\t}\n"
        :: "r"(tmem_d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate), "r"(leader)
        : "memory");
}
// The same for a CTA pair: M = 256 over the two CTAs' tensor memory, issued by the even CTA; the commit arrives on the
// barrier at this offset in both CTAs.
__device__ __forceinline__ void umma_i8_split_pair(uint32_t leader, uint32_t tmem_d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                                   uint32_t b_hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "setp.ne.b32 q, %7, 0;\n\t"
        "@q tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %5, p;\n\t}\n"
        :: "r"(tmem_d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate), "r"(leader)
        : "memory");
}
// Completion of the pair's MMAs issued so far, signalled to the barrier at this offset in both CTAs: one commit on the
// issuing (even) CTA's barrier and one on the odd CTA's, whose address in the cluster window is passed in.
__device__ __forceinline__ void umma_commit_pred_pair(uint32_t leader, uint64_t* bar, uint32_t peer_delta) {
    const uint32_t own = smem_u32(bar);
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "setp.ne.b32 q, %2, 0;\n\t"
        "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t"
        "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%1];\n\t}\n"
        ::"r"(own), "r"(own + peer_delta), "r"(leader) : "memory");
}
// Address of the same shared-memory object in the CTA of the given rank of this cluster.
__device__ __forceinline__ uint32_t cluster_addr(const void* ptr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(smem_u32(ptr)), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_address) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];\n" ::"r"(cluster_address) : "memory");
}
// Bounded wait on a barrier another CTA of the cluster arrives on.
__device__ __forceinline__ bool mbar_wait_cluster_hot(uint64_t* bar, uint32_t parity, volatile int* abort_flag, unsigned limit) {
    const uint32_t addr = smem_u32(bar);
    for (unsigned it = 0; it < limit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}\n"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void umma_commit_pred(uint32_t leader, uint64_t* bar) {
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}\n"
        ::"r"(smem_u32(bar)), "r"(leader) : "memory");
}

// Two fp32 values in one 64-bit register for the packed fp32 instructions (one issue slot for two results; each lane is
// an individually rounded IEEE operation, identical to the scalar instruction).
__device__ __forceinline__ uint64_t f32x2_pack(float lo, float hi) {
    return ((uint64_t)__float_as_uint(hi) << 32) | (uint64_t)__float_as_uint(lo);
}
__device__ __forceinline__ uint64_t f32x2_mul_rn(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t f32x2_add_rn(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t f32x2_add_rd(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rm.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

//
// The float -> int conversion issues at an eighth of the fp32 rate on this machine (16 results per clock and SM against
// 128 fp32 operations) and was what bounded the epilogue, so the floor and the clamp are done with an fp32 addition and
// integer min / max instead (see below); the fp32 steps run as packed two-lane instructions.
template <bool WANT_Q>
__device__ __forceinline__ void pipe_group32(const ConvParams& p, uint32_t (&v)[32], size_t o, bool pvalid, float S,
                                             float inv_next, int nb, int qmax, uint32_t* dst) {
    if (p.acc && pvalid && EBS_IN_RANGE(p, CHK_PIPE_ACC, o + 31, p.lim_out)) {
#pragma unroll
        for (int gq = 0; gq < 8; ++gq)
            *reinterpret_cast<int4*>(p.acc + o + 4 * gq) =
                make_int4((int)v[4 * gq], (int)v[4 * gq + 1], (int)v[4 * gq + 2], (int)v[4 * gq + 3]);
    }
    // y = fl(float(acc) * S) for the 32 channels, two to a register: pair (h, bb) = channels 16h + bb and 16h + 8 + bb
    uint64_t yy[2][8];
    const uint64_t S2 = f32x2_pack(S, S);
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int bb = 0; bb < 8; ++bb)
            yy[h][bb] = f32x2_mul_rn(f32x2_pack((float)(int)v[16 * h + bb], (float)(int)v[16 * h + 8 + bb]), S2);
    if (p.y && pvalid && EBS_IN_RANGE(p, CHK_PIPE_Y, o + 31, p.lim_out)) {
        const bool relu = p.relu != 0;
#pragma unroll
        for (int gq = 0; gq < 8; ++gq) {
            float t[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int c = 4 * gq + e;                           // channel c: pair (c / 16, c % 8), upper lane if c & 8
                const uint64_t w = yy[c >> 4][c & 7];
                t[e] = __uint_as_float((c & 8) ? (uint32_t)(w >> 32) : (uint32_t)w);
                if (relu) t[e] = t[e] > 0.f ? t[e] : 0.f;
            }
            *reinterpret_cast<float4*>(p.y + o + 4 * gq) = make_float4(t[0], t[1], t[2], t[3]);
        }
    }
    if (WANT_Q) {
        // The clamp at zero of the quantizer makes an explicit ReLU redundant here: a negative y gives
        // floor(y / step + 0.5) <= 0 and is clamped to code 0, exactly what max(y, 0) would give.
        // Floor and clamp without the conversion pipe: code_pattern above.
        // Byte register bb holds the codes of channels {bb, 8 + bb, 16 + bb, 24 + bb}, rotated left by bb.
        uint32_t cr[8];
        const float hi2 = (float)(2 * qmax + 1);
#pragma unroll
        for (int bb = 0; bb < 8; ++bb) {
            uint32_t m[4];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                // (the multiply and the addition of 0.5 are scalar instructions with explicit rounding, which the assembler
                // never contracts into a fused multiply-add; issued as a packed pair they came out fused)
                const uint64_t w = yy[h][bb];
                m[2 * h] = code_pattern(__fadd_rn(__fmul_rn(__uint_as_float((uint32_t)w), inv_next), 0.5f), hi2);
                m[2 * h + 1] = code_pattern(__fadd_rn(__fmul_rn(__uint_as_float((uint32_t)(w >> 32)), inv_next), 0.5f), hi2);
            }
            const uint32_t c4 = __byte_perm(__byte_perm(m[0], m[1], 0x0040), __byte_perm(m[2], m[3], 0x0040), 0x5410);
            cr[bb] = __funnelshift_l(c4, c4, bb);
        }
        uint32_t planes[8];
        bytes_to_planes(cr, nb, planes);
        if (pvalid && EBS_IN_RANGE(p, CHK_PIPE_PN, (dst - p.packed_next) + nb - 1, p.lim_pn)) {
            if (nb == 4) {
                *reinterpret_cast<uint4*>(dst) = make_uint4(planes[0], planes[1], planes[2], planes[3]);
            } else if (nb == 8) {
                *reinterpret_cast<uint4*>(dst) = make_uint4(planes[0], planes[1], planes[2], planes[3]);
                *reinterpret_cast<uint4*>(dst + 4) = make_uint4(planes[4], planes[5], planes[6], planes[7]);
            } else if (nb == 2) {
                *reinterpret_cast<uint2*>(dst) = make_uint2(planes[0], planes[1]);
            } else if (nb == 6) {
                *reinterpret_cast<uint2*>(dst) = make_uint2(planes[0], planes[1]);
                *reinterpret_cast<uint2*>(dst + 2) = make_uint2(planes[2], planes[3]);
                *reinterpret_cast<uint2*>(dst + 4) = make_uint2(planes[4], planes[5]);
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (j >= nb) break;
                    dst[j] = planes[j];
                }
            }
        }
    }
}

// Plane words of consecutive 32-channel groups of one pixel, held back until their run can leave in wide stores.  A
// group's nb plane words are contiguous in memory, but for an odd nb their start is only 4-byte aligned and 32 lanes
// each storing nb single words scatter 32 sectors per instruction (the wide 1x1 layers of a chain were up to 1.7 times
// slower with nb = 7 than with nb = 8).  A warp handles G consecutive groups of its pixel (G = 4 for the 256-channel tile, 2
// for the 128-channel one): their G * nb words are one contiguous run that starts on a 4 * G-byte boundary, stored as nb
// vectors of G words.  The hold is a shift register (static indices only); last = the run's last group.
template <int G>
struct PlaneHold {
    uint32_t w[G > 1 ? G : 1][8];
    int filled;
};
template <int NB, int G>
__device__ __forceinline__ void pipe_store_run(const uint32_t (&w)[G][8], uint32_t* run) {
    static_assert(G == 2 || G == 4, "two or four groups to a run");
#pragma unroll
    for (int t = 0; t < NB; ++t) {                       // vector t = words G t .. G t + G - 1 of the run; word i = group i / NB, plane i % NB
        if constexpr (G == 4)
            *reinterpret_cast<uint4*>(run + 4 * t) = make_uint4(w[(4 * t) / NB][(4 * t) % NB], w[(4 * t + 1) / NB][(4 * t + 1) % NB],
                                                                 w[(4 * t + 2) / NB][(4 * t + 2) % NB], w[(4 * t + 3) / NB][(4 * t + 3) % NB]);
        else
            *reinterpret_cast<uint2*>(run + 2 * t) = make_uint2(w[(2 * t) / NB][(2 * t) % NB], w[(2 * t + 1) / NB][(2 * t + 1) % NB]);
    }
}
template <int G>
__device__ __forceinline__ void pipe_store_planes(const uint32_t (&planes)[8], int nb, uint32_t* dst, bool pvalid, PlaneHold<G>& hold,
                                                  const ConvParams& p) {
    if constexpr (G > 1) {
        if ((nb & 1) && (p.CWo % G) == 0) {               // odd: hold the group; store the run with its last group (rows of
                                                          // CWo * nb words keep the run's alignment only if G divides CWo)
#pragma unroll
            for (int gi = 0; gi + 1 < G; ++gi)
#pragma unroll
                for (int j = 0; j < 8; ++j) hold.w[gi][j] = hold.w[gi + 1][j];
#pragma unroll
            for (int j = 0; j < 8; ++j) hold.w[G - 1][j] = planes[j];
            if (++hold.filled == G) {
                hold.filled = 0;
                uint32_t* run = dst - (G - 1) * nb;          // the first group of the run
                if (pvalid && EBS_IN_RANGE(p, CHK_PIPE_PN, (dst - p.packed_next) + nb - 1, p.lim_pn)) {
                    if (nb == 7) pipe_store_run<7, G>(hold.w, run);
                    else if (nb == 5) pipe_store_run<5, G>(hold.w, run);
                    else if (nb == 3) pipe_store_run<3, G>(hold.w, run);
                    else pipe_store_run<1, G>(hold.w, run);
                }
            }
            return;
        }
    }
    if (pvalid && EBS_IN_RANGE(p, CHK_PIPE_PN, (dst - p.packed_next) + nb - 1, p.lim_pn)) {
        if (nb == 4) {
            *reinterpret_cast<uint4*>(dst) = make_uint4(planes[0], planes[1], planes[2], planes[3]);
        } else if (nb == 8) {
            *reinterpret_cast<uint4*>(dst) = make_uint4(planes[0], planes[1], planes[2], planes[3]);
            *reinterpret_cast<uint4*>(dst + 4) = make_uint4(planes[4], planes[5], planes[6], planes[7]);
        } else if (nb == 2) {
            *reinterpret_cast<uint2*>(dst) = make_uint2(planes[0], planes[1]);
        } else if (nb == 6) {
            *reinterpret_cast<uint2*>(dst) = make_uint2(planes[0], planes[1]);
            *reinterpret_cast<uint2*>(dst + 2) = make_uint2(planes[2], planes[3]);
            *reinterpret_cast<uint2*>(dst + 4) = make_uint2(planes[4], planes[5]);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (j >= nb) break;
                dst[j] = planes[j];
            }
        }
    }
}

// The same group when only packed planes are asked for (a chained network: no accumulator and no fp32 output): the
// four channels of a byte register go from accumulator to code in one short chain, so that nothing but the 32
// accumulators and the finished code registers is alive at a time -- the general form above keeps the 32 fp32 images
// as well, which at 96 registers costs spills and the parallelism of the instruction stream.
template <int G>
__device__ __forceinline__ void pipe_group32_packed(const uint32_t (&v)[32], bool pvalid, float S, float inv_next, int nb, int qmax,
                                                    uint32_t* dst, const ConvParams& p, PlaneHold<G>& hold) {
    uint32_t cr[8];
    const uint64_t S2 = f32x2_pack(S, S);
    const float hi2 = (float)(2 * qmax + 1);
#pragma unroll
    for (int bb = 0; bb < 8; ++bb) {
        uint32_t m[4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint64_t w = f32x2_mul_rn(f32x2_pack((float)(int)v[16 * h + bb], (float)(int)v[16 * h + 8 + bb]), S2);
            m[2 * h] = code_pattern(__fadd_rn(__fmul_rn(__uint_as_float((uint32_t)w), inv_next), 0.5f), hi2);
            m[2 * h + 1] = code_pattern(__fadd_rn(__fmul_rn(__uint_as_float((uint32_t)(w >> 32)), inv_next), 0.5f), hi2);
        }
        const uint32_t c4 = __byte_perm(__byte_perm(m[0], m[1], 0x0040), __byte_perm(m[2], m[3], 0x0040), 0x5410);
        cr[bb] = __funnelshift_l(c4, c4, bb);
    }
    uint32_t planes[8];
    bytes_to_planes(cr, nb, planes);
    pipe_store_planes(planes, nb, dst, pvalid, hold, p);
}

// The packed-only group of a layer with per-channel terms and / or a shortcut (a folded batch normalisation, the
// second convolution of a residual block): the same chain per byte register with the terms applied in the library's
// order -- per-channel scale, per-channel shift, fp32 shortcut, shortcut from packed codes -- each an individually
// rounded fp32 operation.  The shortcut codes come out of their planes with the rotate-merge of the expanders, which
// leaves them in exactly the byte registers (channels bb, 8 + bb, 16 + bb, 24 + bb) this loop works on.  The ReLU is
// not applied: the quantizer's clamp at zero gives the same codes.
template <int G>
__device__ __forceinline__ void pipe_group32_affine(const uint32_t (&v)[32], const ConvParams& p, size_t o, int cbase, int gp,
                                                    bool pvalid, int nb, int qmax, uint32_t* dst, PlaneHold<G>& hold) {
    const float S = p.S, inv_next = p.inv_next;
    uint32_t rbyte[8];
    const bool has_rp = p.res_packed != nullptr;
    if (has_rp) {
        const uint32_t* rw = p.res_packed + ((size_t)gp * p.CWo + (cbase >> 5)) * p.res_bits;
        uint32_t rw8[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) rw8[j] = (pvalid && j < p.res_bits) ? __ldg(rw + j) : 0u;
        planes_to_bytes<8>(rw8, rbyte);
    }
    uint32_t cr[8];
    const float hi2 = (float)(2 * qmax + 1);
#pragma unroll
    for (int bb = 0; bb < 8; ++bb) {
        uint32_t m[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = 8 * i + bb;
            float t = __fmul_rn((float)(int)v[c], S);
            if (p.ch_scale) t = __fmul_rn(t, __ldg(p.ch_scale + cbase + c));
            if (p.ch_bias) t = __fadd_rn(t, __ldg(p.ch_bias + cbase + c));
            if (p.residual && pvalid) t = __fadd_rn(t, __ldg(p.residual + o + c));
            if (has_rp) t = __fadd_rn(t, __fmul_rn(p.res_scale, (float)((rbyte[bb] >> (8 * i)) & 0xFFu)));
            m[i] = code_pattern(__fadd_rn(__fmul_rn(t, inv_next), 0.5f), hi2);
        }
        const uint32_t c4 = __byte_perm(__byte_perm(m[0], m[1], 0x0040), __byte_perm(m[2], m[3], 0x0040), 0x5410);
        cr[bb] = __funnelshift_l(c4, c4, bb);
    }
    uint32_t planes[8];
    bytes_to_planes(cr, nb, planes);
    pipe_store_planes(planes, nb, dst, pvalid, hold, p);
}

// Packed-only epilogue with per-channel terms / shortcut of one 128-pixel accumulator (whole channel tile, NHWC).
template <int TILE_N, int G>
__device__ __forceinline__ void pipe_epilogue_affine_g(const ConvParams& p, uint32_t tmem_acc, int vwarp, int gp, bool pvalid,
                                                       int co0) {
    constexpr int COLS = TILE_N / 2;
    const uint32_t trow = tmem_acc + ((uint32_t)((vwarp & 3) * 32) << 16);
    const int cbeg = (vwarp >> 2) * COLS;
    const int nb = p.next_bits, qmax = (1 << p.next_bits) - 1;
    uint32_t v[32];
    PlaneHold<G> hold;
    hold.filled = 0;
#pragma unroll 1
    for (int c0 = cbeg; c0 < cbeg + COLS; c0 += 32) {
        uint32_t (&lo)[16] = *reinterpret_cast<uint32_t(*)[16]>(&v[0]);
        uint32_t (&hi)[16] = *reinterpret_cast<uint32_t(*)[16]>(&v[16]);
        tmem_ld16_issue(trow + (uint32_t)c0, lo);
        tmem_ld16_issue(trow + (uint32_t)(c0 + 16), hi);
        tmem_ld16_wait(lo);
        tmem_ld16_wait(hi);
        const size_t o = (size_t)gp * p.Co + co0 + c0;
        uint32_t* dst = p.packed_next + ((size_t)gp * p.CWo + ((co0 + c0) >> 5)) * nb;
        pipe_group32_affine(v, p, o, co0 + c0, gp, pvalid, nb, qmax, dst, hold);
    }
}

// Plain epilogue (no per-channel terms, no shortcut, NHWC, whole channel tile, c_out % 4 == 0) of one
// 128-pixel accumulator.  vwarp 0..7: TMEM lane quarter vwarp % 4, channel half vwarp / 4.
template <int TILE_N, int G>
__device__ __forceinline__ void pipe_epilogue_plain_g(const ConvParams& p, uint32_t tmem_acc, int vwarp, int gp, bool pvalid,
                                                      int co0) {
    constexpr int COLS = TILE_N / 2;
    const uint32_t trow = tmem_acc + ((uint32_t)((vwarp & 3) * 32) << 16);
    const int cbeg = (vwarp >> 2) * COLS;
    const bool want_q = p.packed_next != nullptr;
    const int nb = want_q ? p.next_bits : 0, qmax = (1 << p.next_bits) - 1;
    const float S = p.S, inv_next = p.inv_next;
    uint32_t v[32];
    PlaneHold<G> hold;
    hold.filled = 0;
#pragma unroll 1
    for (int c0 = cbeg; c0 < cbeg + COLS; c0 += 32) {
        uint32_t (&lo)[16] = *reinterpret_cast<uint32_t(*)[16]>(&v[0]);
        uint32_t (&hi)[16] = *reinterpret_cast<uint32_t(*)[16]>(&v[16]);
        tmem_ld16_issue(trow + (uint32_t)c0, lo);
        tmem_ld16_issue(trow + (uint32_t)(c0 + 16), hi);
        tmem_ld16_wait(lo);
        tmem_ld16_wait(hi);
        const size_t o = (size_t)gp * p.Co + co0 + c0;
        uint32_t* dst = p.packed_next + ((size_t)gp * p.CWo + ((co0 + c0) >> 5)) * nb;
        if (want_q && !p.acc && !p.y) {
            pipe_group32_packed(v, pvalid, S, inv_next, nb, qmax, dst, p, hold);
        } else if (want_q) {
            pipe_group32<true>(p, v, o, pvalid, S, inv_next, nb, qmax, dst);
        } else {
            pipe_group32<false>(p, v, o, pvalid, S, inv_next, nb, qmax, dst);
        }
    }
}

// Packed-only epilogue without per-channel terms of one 128-pixel accumulator (whole channel tile): nothing but the lean
// group, for the kernel forms that are launched only for such layers.
template <int TILE_N, int G>
__device__ __forceinline__ void pipe_epilogue_packed_g(const ConvParams& p, uint32_t tmem_acc, int vwarp, int gp, bool pvalid,
                                                       int co0) {
    constexpr int COLS = TILE_N / 2;
    const uint32_t trow = tmem_acc + ((uint32_t)((vwarp & 3) * 32) << 16);
    const int cbeg = (vwarp >> 2) * COLS;
    const int nb = p.next_bits, qmax = (1 << p.next_bits) - 1;
    const float S = p.S, inv_next = p.inv_next;
    uint32_t v[32];
    PlaneHold<G> hold;
    hold.filled = 0;
#pragma unroll 1
    for (int c0 = cbeg; c0 < cbeg + COLS; c0 += 32) {
        uint32_t (&lo)[16] = *reinterpret_cast<uint32_t(*)[16]>(&v[0]);
        uint32_t (&hi)[16] = *reinterpret_cast<uint32_t(*)[16]>(&v[16]);
        tmem_ld16_issue(trow + (uint32_t)c0, lo);
        tmem_ld16_issue(trow + (uint32_t)(c0 + 16), hi);
        tmem_ld16_wait(lo);
        tmem_ld16_wait(hi);
        uint32_t* dst = p.packed_next + ((size_t)gp * p.CWo + ((co0 + c0) >> 5)) * nb;
        pipe_group32_packed(v, pvalid, S, inv_next, nb, qmax, dst, p, hold);
    }
}

// Odd plane counts of the packed output take the form that holds the groups of a run back: a kernel instantiation of
// its own (HOLD), chosen by the launcher, because the shift register costs the other layers registers and time even
// as an untaken branch of the same kernel (even counts 15-25% slower when both forms were compiled into one kernel).
// Kernel form for a layer: 0 = every output mode and ragged channel tiles; 1 = packed planes only, whole channel tiles
// (the usual layer of a network: its epilogue holds nothing but the lean group, or the group with per-channel terms);
// 2 = form 1 with the held-back runs.
inline bool pipe_packed_only(const ConvParams& p, int tile_n) {
    return p.packed_next && !p.acc && !p.y && !p.w_levels && (p.Co % tile_n) == 0;
}
inline bool pipe_hold_applies(const ConvParams& p, int tile_n) {
    const int G = tile_n / 64;
    // (5 and 7 planes; with 1 or 3 the single-word stores are few and the held form measured slower)
    return G > 1 && p.packed_next && (p.next_bits == 5 || p.next_bits == 7) && (p.CWo % G) == 0 && !p.acc && !p.y && !p.y_nchw &&
           (p.Co & 31) == 0 && !p.w_levels;
}

template <int AB, int TILE_N, bool AFFINE, int FORM, bool PAIR = false>
__global__ void __launch_bounds__(PIPE_THREADS, 1) conv_umma_pipe_kernel(const ConvParams p, const PipeGeom g) {
    constexpr int EPI_G = FORM == 2 ? TILE_N / 64 : 1;         // groups of an output run held back (odd plane counts)
    // PAIR: the two CTAs of a cluster work as one.  Each expands its own 128 * m_sub pixels and holds the weight rows of
    // half the channel tile; the even CTA issues MMAs of M = 256 (cta_group::2) that read both CTAs' shared memory and
    // write both CTAs' tensor memory, so a weight byte is fetched from L2 once per 256 pixels instead of once per 128.
    // The odd CTA's issuing warp only reports to the even CTA when its stages, weight slots and accumulators are ready.
    constexpr int B_ROWS = PAIR ? TILE_N / 2 : TILE_N;
    constexpr int B_TILE_BYTES = B_ROWS * 32;
    static_assert(!PAIR || TILE_N == 256, "a CTA pair works on 256-channel tiles");
    __shared__ __align__(8) uint64_t st_peer[PAIR ? PIPE_MAX_STAGES : 1], bs_peer[PAIR ? PIPE_MAX_BSLOTS : 1], acc_peer[2], b_peer;
    const int crank = PAIR ? (int)(blockIdx.x & 1u) : 0;       // rank in the pair (cluster of 2 along x)
    const int bx = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, gx = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    extern __shared__ uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t st_full[PIPE_MAX_STAGES], st_empty[PIPE_MAX_STAGES], acc_full[2], acc_empty[2], b_full;
    __shared__ __align__(8) uint64_t bs_full[PIPE_MAX_BSLOTS], bs_empty[PIPE_MAX_BSLOTS];   // streamed weight tiles
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ uint32_t s_tap_shift[PIPE_MAX_TAPS];     // tap tables in shared memory: indexed at run time by single threads
    __shared__ int s_tap_id[PIPE_MAX_TAPS];

    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid < PIPE_MAX_TAPS) {
        s_tap_shift[tid] = (uint32_t)g.tap_shift[tid];
        s_tap_id[tid] = (int)g.tap_id[tid];
    }
    // Table of the MMAs of a chunk, per phase, in issue order (word, tap, accumulator): x = offset of the activation
    // operand from the stage start (16-byte units: word, tap shift, 128 pixels per accumulator) | accumulator column
    // offset << 22, y = offset of the weight tile (16-byte units) from the chunk's first tile (resident weights) or from
    // the start of its ring slot (streamed).  An issuing warp then spends a load, three additions and the MMA per step;
    // with operand addresses computed in its loop it was the slowest stage of the pipeline.
    uint2* mma_tab = reinterpret_cast<uint2*>(dyn_smem + ((1024u - (smem_u32(dyn_smem) & 1023u)) & 1023u) +
                                              (g.smem_bytes - 1024 - PIPE_MAX_MMAS * 8));
    {
        const int per_tap = g.kss * g.m_sub, total_e = per_tap * g.taps;
        const uint32_t bt16 = (uint32_t)B_TILE_BYTES >> 4;
        for (int e = tid; e < total_e; e += PIPE_THREADS) {
            int ph = 0;
            while (ph + 1 < g.n_ph && e >= per_tap * g.ph_tap0[ph + 1]) ++ph;
            const int t0 = g.ph_tap0[ph], ntp = g.ph_tap0[ph + 1] - t0;
            const int local = e - per_tap * t0;
            const int q = local / (ntp * g.m_sub), r = local - q * (ntp * g.m_sub);
            const int tl = r / g.m_sub, j = r - tl * g.m_sub;
            const uint32_t a_off = (uint32_t)(q * (g.a_word_bytes >> 4) + g.tap_shift[t0 + tl] + j * UMMA_M);
            const uint32_t b_off = g.b_resident ? (uint32_t)(q * g.taps + tl) * bt16
                                                : (uint32_t)((q * ntp + tl) % g.b_group) * bt16;
            if (EBS_IN_RANGE(p, CHK_PIPE_TAB, e, PIPE_MAX_MMAS))
                mma_tab[e] = make_uint2(a_off | ((uint32_t)(j * TILE_N) << 22), b_off);
        }
    }
    const int NST = g.n_stages, KS = g.ks, KSS = g.kss, NSUB = g.nsub, SP = g.SP, S = g.S;
    const int nchunks = g.nchunks, nwg = g.nwg;
    const bool resident = g.b_resident != 0;
    uint8_t* base = dyn_smem + ((1024u - (smem_u32(dyn_smem) & 1023u)) & 1023u);
    uint8_t* b_res = base;                                               // resident: [CW][tap slots][TILE_N][32]; else the ring of tiles
    uint8_t* stages = base + (resident ? g.b_total_bytes : g.b_slots * g.b_group * B_TILE_BYTES);   // [NST] x [KS][2][SP][16]
    const int NBS = g.b_slots, GB = g.b_group;
    // Streamed weights: every CTA of a channel tile reads the same weight tiles, and CTAs that start together would ask
    // the same few L2 slices for the same tile at the same time.  Integer accumulation is exact in any order, so each
    // CTA starts its walk over the word groups at a different one.
    const int wg_rot = resident ? 0 : bx % nwg;
    volatile int* abortp = &abort_flag;
    const unsigned wait_limit = p.wait_limit;

    // work items of this CTA: (pixel super-tile, channel tile)
    const int n_items = resident ? g.n_ptiles : g.n_ptiles * g.n_ctiles;
    const int my_items = (bx < n_items) ? (n_items - 1 - bx) / gx + 1 : 0;
    auto item_of = [&](int it, int& ptile, int& ctile) {
        const int idx = bx + it * gx;
        if (resident) { ptile = idx; ctile = (int)blockIdx.y; }
        else { ptile = idx / g.n_ctiles; ctile = idx - ptile * g.n_ctiles; }
    };

    // Issuing warps: a single warp issuing every MMA of a CTA needs 140-180 clocks per MMA (measured: its busy time, not
    // the tensor pipe, bounded the k x k layers and the GEMM), so with two or four accumulators per tile two warps share the
    // work, each owning the accumulators of one parity -- MMAs of different warps never touch the same accumulator, so
    // no order between the warps is needed.  One accumulator: one issuing warp.
    const int n_iss = (g.m_sub & 1) == 0 ? PIPE_ISSUERS : 1;
    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < PIPE_MAX_STAGES; ++s) {
            mbar_init(&st_full[s], (PIPE_EXPANDERS / 32) * g.nsub);  // every expander warp arrives once per pass
            mbar_init(&st_empty[s], n_iss);                         // every issuing warp commits its own MMAs
        }
        for (int s = 0; s < PIPE_MAX_BSLOTS; ++s) {
            mbar_init(&bs_full[s], 1);
            mbar_init(&bs_empty[s], n_iss);
        }
        mbar_init(&acc_full[0], n_iss);
        mbar_init(&acc_full[1], n_iss);
        mbar_init(&acc_empty[0], PIPE_EPI_WARPS);
        mbar_init(&acc_empty[1], PIPE_EPI_WARPS);
        mbar_init(&b_full, 1);
        if constexpr (PAIR) {
            for (int s = 0; s < PIPE_MAX_STAGES; ++s) mbar_init(&st_peer[s], 1);
            for (int s = 0; s < PIPE_MAX_BSLOTS; ++s) mbar_init(&bs_peer[s], 1);
            mbar_init(&acc_peer[0], 1);
            mbar_init(&acc_peer[1], 1);
            mbar_init(&b_peer, 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == PIPE_ISSUER_WARP) {
        if constexpr (PAIR) {                                 // the same warp of both CTAs, the same slot address
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_slot)),
                         "r"((uint32_t)g.tmem_cols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;\n" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_slot)),
                         "r"((uint32_t)g.tmem_cols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();                   // the other CTA's barriers exist before anything arrives on them
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const uint32_t tmem_base = tmem_slot;

    // Registers follow the roles (warpgroups of four warps: 0-7 expanders, 8-11 issuers / producer / no role, 12-19
    // epilogue): each role's branch opens with a setmaxnreg executed by all four warps of its warpgroups, and the
    // assembler allocates each branch for its own count.  The epilogue's 32 accumulators, their fp32 images and the code
    // registers want about 126 registers; with the 96 a CTA of 20 warps starts with it spilled and its instruction stream
    // lost its parallelism (wide 1x1 layers 15-20% slower, and no better with twelve epilogue warps).  The other roles
    // need fewer than 96.  The increase waits in hardware until the CTA's pool has the registers, so the counts must fit
    // into what the launch allots: checked at compile time.  (80 / 56 / 128 measured best of three splits.)
    constexpr int REG_LAUNCH = 96, REG_EXP = 80, REG_MID = 56, REG_EPI = 128;
    static_assert(8 * REG_EXP + 4 * REG_MID + 8 * REG_EPI <= 20 * REG_LAUNCH, "setmaxnreg: the roles' registers exceed the CTA's pool");
    static_assert(PIPE_EPI_WARP0 == 12 && PIPE_EPI_WARPS == 8 && PIPE_THREADS == 640, "role layout changed: revisit the register split");
    if (warp < 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(REG_EXP));
        // =========================== expanders ===========================
        int slot_q[PIPE_SLOTS], slot_pix[PIPE_SLOTS], slot_dst[PIPE_SLOTS];
#pragma unroll
        // An even number of words per pass: a thread takes two adjacent words of one pixel, so that for an odd plane count
        // its 2 * AB packed words still start on an 8-byte boundary and load as pairs.  Otherwise items tid and tid + 256.
        constexpr int NW = AB == 0 ? 8 : AB;                  // words of one (pixel, 32-channel word) item; AB = 0: byte codes
        const bool paired = (NW & 1) != 0 && (KS & 1) == 0 && (p.CW & 1) == 0;
        for (int j = 0; j < PIPE_SLOTS; ++j) {
            const int e = paired ? 2 * tid + j : tid + j * PIPE_EXPANDERS;
            const int s = e / KS, q = e - s * KS;            // consecutive lanes: consecutive words of one pixel
            slot_q[j] = s < S ? q : -1;                       // -1: no item
            slot_pix[j] = s;
            slot_dst[j] = q * g.a_word_bytes + s * 16;
        }
        // Loader state: runs several passes ahead of the expansion, also across tile boundaries.  Per (tile, phase) a
        // thread keeps one pointer per slot -- its pixel's words at its word position, or a page of zero words for
        // padding, pixels past the batch and threads without an item -- so that a pass adds one warp-uniform word offset,
        // bounded per thread so that the ragged last word group stays inside the pixel (those words feed no MMA).
        int ld_it = 0, ld_c = 0, ld_sub = 0, ld_lim[PIPE_SLOTS];
        const uint32_t* ld_src[PIPE_SLOTS];
#ifdef EBS_CHECKED
        bool ld_real[PIPE_SLOTS];
#endif
#pragma unroll
        for (int j = 0; j < PIPE_SLOTS; ++j) ld_lim[j] = p.CW - ((paired && j == 0) ? 2 : 1) - max(slot_q[j], 0);
        auto chunk_offsets = [&](int it, int ph) {
            int ptile, ctile;
            item_of(it, ptile, ctile);
            const int f0 = (PAIR ? 2 * ptile + crank : ptile) * g.tile_pix;
            const int pa = g.ph_a[ph], pb = g.ph_b[ph];
#pragma unroll
            for (int j = 0; j < PIPE_SLOTS; ++j) {
                const int qn = max(slot_q[j], 0) * NW;
                ld_src[j] = p.zero_words + qn;                  // padding or past the batch -> zero bytes
#ifdef EBS_CHECKED
                ld_real[j] = false;
#endif
                const int f = f0 + slot_pix[j];
                if (slot_q[j] >= 0 && f < g.frame) {
                    const uint32_t n = fastdiv((uint32_t)f, g.div_img);
                    const uint32_t rem = (uint32_t)f - n * (uint32_t)(g.Hq * g.Wq);
                    const uint32_t hq = fastdiv(rem, g.div_row), wq = rem - hq * (uint32_t)g.Wq;
                    const int h = p.sh * ((int)hq + g.q0r) + pa, w = p.sw * ((int)wq + g.q0s) + pb;
                    if ((unsigned)h < (unsigned)p.H && (unsigned)w < (unsigned)p.W) {
                        ld_src[j] = p.x + ((size_t)((((int)n * p.H + h) * p.W + w) * p.CW) * NW + qn);
#ifdef EBS_CHECKED
                        ld_real[j] = true;
#endif
                    }
                }
            }
        };
        // register ring of packed words: SETS - 1 chunks of global loads in flight per thread (about 48 registers whatever
        // the plane count: the latency of these loads, not their bandwidth, is what a deep reduction waits for)
        constexpr int SETS = NW <= 4 ? 4 : 3;
        uint32_t a_set[SETS][PIPE_SLOTS][NW];
        int ld_ph = 0, ld_wg = 0;
        auto load_next = [&](int set) {
            int wg = ld_wg + wg_rot;
            if (wg >= nwg) wg -= nwg;
            if (ld_wg == 0 && ld_sub == 0) chunk_offsets(ld_it, ld_ph);
            const int base = wg * KSS + ld_sub * KS;            // first word of the pass (warp-uniform)
#ifdef EBS_CHECKED
            auto load_ok = [&](int j, const uint32_t* a, int n) {
                return ld_real[j] ? EBS_IN_RANGE(p, CHK_PIPE_X, (a - p.x) + n - 1, p.lim_x)
                                  : EBS_IN_RANGE(p, CHK_PIPE_X, (a - p.zero_words) + n - 1, PIPE_ZERO_WORDS);
            };
#else
            auto load_ok = [](int, const uint32_t*, int) { return true; };
#endif
            if (paired) {                                       // both words of the pixel in one run of 2 * AB words
                const uint32_t* a = ld_src[0] + min(base, ld_lim[0]) * NW;
                if (load_ok(0, a, 2 * NW)) load_words_global<2 * NW>(a, *reinterpret_cast<uint32_t(*)[2 * NW]>(&a_set[set][0][0]));
            } else {
#pragma unroll
                for (int j = 0; j < PIPE_SLOTS; ++j) {
                    const uint32_t* a = ld_src[j] + min(base, ld_lim[j]) * NW;
                    if (load_ok(j, a, NW)) load_words_global<NW>(a, a_set[set][j]);
                }
            }
            if (++ld_sub == NSUB) {
                ld_sub = 0;
                if (++ld_wg == nwg) { ld_wg = 0; ++ld_ph; }
                if (++ld_c == nchunks) { ld_c = 0; ld_ph = 0; ++ld_it; }
            }
        };
        const int total = my_items * nchunks * NSUB;           // expander passes
#pragma unroll
        for (int u = 0; u < SETS - 1; ++u)
            if (u < total) load_next(u);
        bool ok = true;
        int st = 0, sub = 0;
        uint32_t st_round = 0;                                  // how many times the ring has wrapped
        for (int g0 = 0; g0 < total && ok; g0 += SETS) {
#pragma unroll
            for (int u = 0; u < SETS; ++u) {
                const int gi = g0 + u;
                if (gi >= total) break;
                uint8_t* A_st = stages + st * g.stage_bytes + sub * KS * g.a_word_bytes;
                if (gi + SETS - 1 < total) load_next((u + SETS - 1) % SETS);
                if (st_round > 0 && sub == 0) {                 // the MMAs that read this stage one round ago must be done
                    if (!mbar_wait_bounded(&st_empty[st], (st_round - 1) & 1u, abortp, wait_limit)) { ok = false; break; }
                }
#pragma unroll
                for (int j = 0; j < PIPE_SLOTS; ++j) {
                    if (slot_q[j] < 0) continue;
                    // v_k = rotl(w_k, k); byte register bb = rotr(OR_k v_k & (0x01010101 << ((bb + k) & 7)), bb)
                    uint32_t r[8];
                    if constexpr (AB == 0) {
                        // byte codes, channel c in byte c of the item: only the order changes (row byte 4b + i = channel
                        // 8i + b, the order of the weight image): register b takes byte b % 4 of words b / 4, 2 + b / 4, ...
                        const uint32_t (&w)[8] = a_set[u][j];
#pragma unroll
                        for (int bb = 0; bb < 8; ++bb) {
                            const uint32_t sel = 0x0040u + 0x11u * (uint32_t)(bb & 3);          // byte (bb & 3) of both operands
                            const uint32_t lo = __byte_perm(w[bb >> 2], w[2 + (bb >> 2)], sel);
                            const uint32_t hi = __byte_perm(w[4 + (bb >> 2)], w[6 + (bb >> 2)], sel);
                            r[bb] = __byte_perm(lo, hi, 0x5410);
                        }
                    } else {
                        planes_to_bytes<NW>(a_set[u][j], r);
                    }
                    uint8_t* dst = A_st + slot_dst[j];
                    if (!EBS_IN_RANGE(p, CHK_PIPE_STAGE, (dst + SP * 16 + 15) - stages, NST * g.stage_bytes) ||
                        !EBS_IN_RANGE(p, CHK_PIPE_STAGE, dst - stages, NST * g.stage_bytes))
                        continue;
                    *reinterpret_cast<uint4*>(dst) = make_uint4(r[0], r[1], r[2], r[3]);
                    *reinterpret_cast<uint4*>(dst + SP * 16) = make_uint4(r[4], r[5], r[6], r[7]);
                }
                // every lane makes its bytes visible to the tensor core's proxy, then one lane arrives for the warp (32
                // arrivals on one barrier word would be served one after the other)
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                __syncwarp();
                if ((tid & 31) == 0) mbar_arrive(&st_full[st]);
                if (++sub == NSUB) {
                    sub = 0;
                    if (++st == NST) { st = 0; ++st_round; }
                }
            }
        }
    } else if (warp < PIPE_EPI_WARP0) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(REG_MID));
      if (PAIR && crank == 1 && warp < PIPE_PRODUCER_WARP) {
        // =========================== the odd CTA of a pair: reports ===========================
        // One warp follows this CTA's own barriers in the order the even CTA's issuing warps wait for them and passes
        // each completion on with one arrival on the even CTA's barrier of the same name.
        if (warp == PIPE_ISSUER_WARP) {
            const bool lane0 = (tid & 31) == 0;
            const uint32_t r_st = cluster_addr(&st_peer[0], 0), r_bs = cluster_addr(&bs_peer[0], 0);
            const uint32_t r_acc = cluster_addr(&acc_peer[0], 0), r_b = cluster_addr(&b_peer, 0);
            bool ok = true;
            if (my_items > 0 && resident) {
                ok = mbar_wait_bounded_hot(&b_full, 0u, abortp, wait_limit);
                if (ok && lane0) mbar_arrive_cluster(r_b);
            }
            int st = 0, bs = 0;
            uint32_t st_round = 0, bs_round = 0;
            for (int it = 0; it < my_items && ok; ++it) {
                const int buf = g.nbuf == 2 ? (it & 1) : 0;
                const int use = g.nbuf == 2 ? (it >> 1) : it;
                if (use > 0) {
                    if (!mbar_wait_bounded_hot(&acc_empty[buf], (uint32_t)((use - 1) & 1), abortp, wait_limit)) break;
                    if (lane0) mbar_arrive_cluster(r_acc + 8u * (uint32_t)buf);
                }
                int ph = 0, wg = 0;
                for (int c = 0; c < nchunks && ok; ++c) {
                    if (!mbar_wait_bounded_hot(&st_full[st], st_round & 1u, abortp, wait_limit)) { ok = false; break; }
                    if (lane0) mbar_arrive_cluster(r_st + 8u * (uint32_t)st);
                    if (!resident) {
                        const int wgr = wg + wg_rot >= nwg ? wg + wg_rot - nwg : wg + wg_rot;
                        const int words = min(KSS, p.CW - wgr * KSS);
                        const int ntiles = words * (g.ph_tap0[ph + 1] - g.ph_tap0[ph]);
                        for (int i0 = 0; i0 < ntiles; i0 += GB) {
                            if (!mbar_wait_bounded_hot(&bs_full[bs], bs_round & 1u, abortp, wait_limit)) { ok = false; break; }
                            if (lane0) mbar_arrive_cluster(r_bs + 8u * (uint32_t)bs);
                            if (++bs == NBS) { bs = 0; ++bs_round; }
                        }
                    }
                    __syncwarp();
                    if (++st == NST) { st = 0; ++st_round; }
                    if (++wg == nwg) { wg = 0; ++ph; }
                }
            }
        }
      } else if (warp >= PIPE_ISSUER_WARP && warp < PIPE_ISSUER_WARP + n_iss) {
        // =========================== issuers ===========================
        const int k_iss = warp - PIPE_ISSUER_WARP;                // this warp takes the MMAs k_iss, k_iss + n_iss, ... of a chunk
        // The issuing thread is a pipeline stage of its own: every address is advanced by additions (descriptor start
        // addresses are in 16-byte units), a handful of instructions per MMA.
        constexpr uint32_t IDESC = PAIR ? (umma_idesc_i8(TILE_N) & ~(0x1Fu << 24)) | ((256u >> 4) << 24) : umma_idesc_i8(TILE_N);
        constexpr uint32_t BT16 = B_TILE_BYTES >> 4;
        const bool skip_mma = (p.test_flags & 1) != 0;            // test hook: issue nothing, so that waits run out
        bool ok = my_items == 0 || !resident || mbar_wait_bounded_hot(&b_full, 0u, abortp, wait_limit);
        if (PAIR && ok && my_items > 0 && resident) ok = mbar_wait_cluster_hot(&b_peer, 0u, abortp, wait_limit);
        const uint64_t da_ring = umma_desc_interleaved(smem_u32(stages), (uint32_t)(SP * 16));
        const uint64_t db_res = umma_desc_sw32(smem_u32(b_res));   // resident tiles, or slot 0 of the ring
        const uint32_t da_lo = (uint32_t)da_ring, da_hi = (uint32_t)(da_ring >> 32);
        const uint32_t db_lo = (uint32_t)db_res, db_hi = (uint32_t)(db_res >> 32);
        const uint32_t stage16 = (uint32_t)(g.stage_bytes >> 4);
        const int m_sub = g.m_sub;
        const uint32_t leader = (tid & 31) == 0 ? 1u : 0u;
        auto mma_issue = [](uint32_t ld, uint32_t d, uint32_t al, uint32_t ah, uint32_t bl, uint32_t bh, uint32_t idesc, uint32_t accu) {
            if constexpr (PAIR) umma_i8_split_pair(ld, d, al, ah, bl, bh, idesc, accu);
            else umma_i8_split(ld, d, al, ah, bl, bh, idesc, accu);
        };
        // (a pair: the odd CTA's shared window lies at a fixed distance from this one's in the cluster window)
        const uint32_t peer_delta = PAIR ? cluster_addr(&abort_flag, 1) - smem_u32(&abort_flag) : 0u;
        auto mma_commit = [peer_delta](uint32_t ld, uint64_t* bar) {
            if constexpr (PAIR) umma_commit_pred_pair(ld, bar, peer_delta);
            else umma_commit_pred(ld, bar);
        };
        int st = 0, bs = 0;
        uint32_t st_round = 0, bs_round = 0;
        for (int it = 0; it < my_items && ok; ++it) {
            const int buf = g.nbuf == 2 ? (it & 1) : 0;
            const int use = g.nbuf == 2 ? (it >> 1) : it;          // how often this accumulator set was used before
            if (use > 0) {                                          // its epilogue must have drained it
                if (!mbar_wait_bounded_hot(&acc_empty[buf], (uint32_t)((use - 1) & 1), abortp, wait_limit)) break;
                if (PAIR && !mbar_wait_cluster_hot(&acc_peer[buf], (uint32_t)((use - 1) & 1), abortp, wait_limit)) break;
            }
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            const uint32_t tmem_d = tmem_base + (uint32_t)(buf * m_sub * TILE_N);
            int ph = 0, wg = 0;
            for (int c = 0; c < nchunks; ++c) {
                if (!mbar_wait_bounded_hot(&st_full[st], st_round & 1u, abortp, wait_limit)) { ok = false; break; }
                if (PAIR && !mbar_wait_cluster_hot(&st_peer[st], st_round & 1u, abortp, wait_limit)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                if (!skip_mma) {
                    const int wgr = wg + wg_rot >= nwg ? wg + wg_rot - nwg : wg + wg_rot;
                    const int words = min(KSS, p.CW - wgr * KSS);
                    const int t0 = g.ph_tap0[ph], ntp = g.ph_tap0[ph + 1] - t0;
                    const uint2* tab = mma_tab + KSS * m_sub * t0;
                    const int zero_n = c == 0 ? m_sub : 0;         // the first MMA into each accumulator of a tile overwrites it
                    const uint32_t a_lo = da_lo + (uint32_t)st * stage16;
                    if (resident) {
                        const uint32_t b_lo = db_lo + (uint32_t)((wgr * KSS) * g.taps + t0) * BT16;
                        const int n = words * ntp * m_sub;
                        uint2 e = tab[k_iss];
                        for (int i = k_iss; i < n; i += n_iss) {
                            const uint2 nxt = tab[i + n_iss];             // (past the end: inside the table's allocation)
                            mma_issue(leader, tmem_d + (e.x >> 22), a_lo + (e.x & 0x3FFFFFu), da_hi, b_lo + e.y, db_hi, IDESC,
                                          i >= zero_n ? 1u : 0u);
                            e = nxt;
                        }
                    } else {
                        // streamed weights: the chunk's (word, tap) tiles in order, GB consecutive tiles per ring slot
                        const int ntiles = words * ntp;
                        int i = k_iss;
                        for (int i0 = 0; i0 < ntiles; i0 += GB) {
                            if (!mbar_wait_bounded_hot(&bs_full[bs], bs_round & 1u, abortp, wait_limit)) { ok = false; break; }
                            if (PAIR && !mbar_wait_cluster_hot(&bs_peer[bs], bs_round & 1u, abortp, wait_limit)) { ok = false; break; }
                            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                            const uint32_t b_lo = db_lo + (uint32_t)(bs * GB) * BT16;
                            const int n = (i0 + min(GB, ntiles - i0)) * m_sub;
                            uint2 e = tab[i];
                            for (; i < n; i += n_iss) {
                                const uint2 nxt = tab[i + n_iss];
                                mma_issue(leader, tmem_d + (e.x >> 22), a_lo + (e.x & 0x3FFFFFu), da_hi, b_lo + e.y, db_hi, IDESC,
                                              i >= zero_n ? 1u : 0u);
                                e = nxt;
                            }
                            mma_commit(leader, &bs_empty[bs]);
                            if (++bs == NBS) { bs = 0; ++bs_round; }
                        }
                        if (!ok) break;
                    }
                    mma_commit(leader, &st_empty[st]);
                    if (c == nchunks - 1) mma_commit(leader, &acc_full[buf]);
                }
                __syncwarp();
                if (++st == NST) { st = 0; ++st_round; }
                if (++wg == nwg) { wg = 0; ++ph; }
            }
        }
    } else if (warp == PIPE_PRODUCER_WARP) {
        // =========================== weight tiles ===========================
        // The whole warp runs the loops with uniform control flow and every lane issues the copy of one tile of a slot
        // (its own address arithmetic, side by side with the other lanes'): a single lane working through the tiles one
        // after the other retired an instruction every dozen clocks and needed about 360 clocks per tile -- more than
        // the two MMAs that consume a 256-channel tile -- which bounded every layer whose weights stream.
        const int lane = tid & 31;
        if (my_items > 0) {
            if (resident) {                                      // all tiles of this CTA's channel tile, once
                const int co0 = (int)blockIdx.y * TILE_N + crank * B_ROWS;   // a pair: this CTA's half of the channel tile
                const uint32_t rows = (uint32_t)min(B_ROWS, p.Co16 - co0);
                const int total_tiles = p.CW * g.taps;
                if (lane == 0) mbar_arrive_expect_tx(&b_full, rows * 32u * (uint32_t)total_tiles);
                __syncwarp();
                for (int t = lane; t < total_tiles; t += 32) {
                    const int cw = t / g.taps, ts = t - cw * g.taps;
                    if (EBS_IN_RANGE(p, CHK_PIPE_W8, ((long long)(s_tap_id[ts] * p.CW + cw) * p.Co16 + co0) * 32 + rows * 32 - 1, p.lim_w8))
                        bulk_copy_g2s(b_res + t * B_TILE_BYTES,
                                      p.w8 + ((size_t)(s_tap_id[ts] * p.CW + cw) * p.Co16 + co0) * 32, rows * 32u, &b_full);
                }
            } else {
                int bs = 0;
                uint32_t bs_round = 0;
                bool ok = true;
                for (int it = 0; it < my_items && ok; ++it) {
                    int ptile, ctile;
                    item_of(it, ptile, ctile);
                    const int co0 = ctile * TILE_N + crank * B_ROWS;
                    const uint32_t bytes = (uint32_t)min(B_ROWS, p.Co16 - co0) * 32u;
                    int ph = 0, wg = -1;
                    for (int c = 0; c < nchunks && ok; ++c) {
                        if (++wg == nwg) { wg = 0; ++ph; }
                        const int wgr = wg + wg_rot >= nwg ? wg + wg_rot - nwg : wg + wg_rot;
                        const int words = min(KSS, p.CW - wgr * KSS);
                        const int t0 = g.ph_tap0[ph], ntaps = g.ph_tap0[ph + 1] - t0, ntiles = words * ntaps;
                        for (int i0 = 0; i0 < ntiles; i0 += GB) {
                            if (bs_round > 0) {                     // the MMAs that read this slot one round ago must be done
                                const bool free = mbar_wait_bounded_hot(&bs_empty[bs], (bs_round - 1) & 1u, abortp, wait_limit);
                                if (!__all_sync(0xffffffffu, free)) { ok = false; break; }
                            }
                            const int n = min(GB, ntiles - i0);
                            if (lane == 0) mbar_arrive_expect_tx(&bs_full[bs], bytes * (uint32_t)n);
                            __syncwarp();
                            if (lane < n) {
                                const int t = i0 + lane;                          // tile of the chunk: word-major, taps inside
                                const int q = t / ntaps, ts = t0 + (t - q * ntaps);
                                const size_t src = ((size_t)(s_tap_id[ts] * p.CW + wgr * KSS + q) * p.Co16 + co0) * 32;
                                // (a copy skipped by the range-checked build leaves its barrier incomplete: the CTA then gives
                                // up at its bounded wait, which is reported as well)
                                if (EBS_IN_RANGE(p, CHK_PIPE_W8, src + bytes - 1, p.lim_w8))
                                    bulk_copy_g2s(b_res + (bs * GB + lane) * B_TILE_BYTES, p.w8 + src, bytes, &bs_full[bs]);
                            }
                            if (++bs == NBS) { bs = 0; ++bs_round; }
                        }
                    }
                }
            }
        }
      }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(REG_EPI));
        // =========================== epilogue ===========================
        const int half = (warp - PIPE_EPI_WARP0) >> 2;           // which half of the channels
        const int vwarp = (warp & 3) + 4 * half;                 // TMEM lane quarter = warp % 4 (hardware rule)
        const int row = (warp & 3) * 32 + (tid & 31);
        const bool plain_ok = !AFFINE && !p.ch_scale && !p.ch_bias && !p.residual && !p.res_packed && !p.y_nchw &&
                              (p.Co & 3) == 0;
        // layers with per-channel terms or a shortcut that only hand packed planes on (the usual layer of a network)
        const bool affine_ok = AFFINE && p.packed_next && !p.y && !p.acc && !p.w_levels && (p.Co & 31) == 0;
        for (int it = 0; it < my_items; ++it) {
            const int buf = g.nbuf == 2 ? (it & 1) : 0;
            const int use = g.nbuf == 2 ? (it >> 1) : it;
            if (!mbar_wait_bounded(&acc_full[buf], (uint32_t)(use & 1), abortp, wait_limit)) break;
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            int ptile, ctile;
            item_of(it, ptile, ctile);
            const int co0 = ctile * TILE_N;
            for (int j = 0; j < g.m_sub; ++j) {
                const int f = (PAIR ? 2 * ptile + crank : ptile) * g.tile_pix + j * UMMA_M + row;
                bool pvalid = false;
                int gp = 0;
                if (f < g.frame) {
                    const uint32_t n = fastdiv((uint32_t)f, g.div_img);
                    const uint32_t rem = (uint32_t)f - n * (uint32_t)(g.Hq * g.Wq);
                    const uint32_t hq = fastdiv(rem, g.div_row), wq = rem - hq * (uint32_t)g.Wq;
                    pvalid = (int)hq < p.Ho && (int)wq < p.Wo;
                    gp = ((int)n * p.Ho + (int)hq) * p.Wo + (int)wq;
                }
                if (!__any_sync(0xffffffffu, pvalid)) continue;   // 32 frame pixels without an output
                const uint32_t tmem_acc = tmem_base + (uint32_t)((buf * g.m_sub + j) * TILE_N);
                if constexpr (FORM != 0) {
                    if constexpr (AFFINE) pipe_epilogue_affine_g<TILE_N, EPI_G>(p, tmem_acc, vwarp, gp, pvalid, co0);
                    else pipe_epilogue_packed_g<TILE_N, EPI_G>(p, tmem_acc, vwarp, gp, pvalid, co0);
                } else {
                    if (plain_ok && co0 + TILE_N <= p.Co) pipe_epilogue_plain_g<TILE_N, 1>(p, tmem_acc, vwarp, gp, pvalid, co0);
                    else if (affine_ok && co0 + TILE_N <= p.Co) pipe_epilogue_affine_g<TILE_N, 1>(p, tmem_acc, vwarp, gp, pvalid, co0);
                    else umma_epilogue<TILE_N, AFFINE>(p, tmem_acc, vwarp, gp, pvalid, 0, co0);
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
            __syncwarp();
            if ((tid & 31) == 0) mbar_arrive(&acc_empty[buf]);
        }
    }

    // a CTA that gave up may still have weight copies in flight towards its shared memory: give them time to land
    // (bounded) before the block ends and the memory is handed to another block
    if (warp == PIPE_PRODUCER_WARP && *abortp) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();                   // neither CTA leaves while the other may still arrive on its barriers
    if (abort_flag != 0 && tid == 0) atomicAdd(&g_umma_timeouts, 1ull);
    if (warp == PIPE_ISSUER_WARP) {
        if constexpr (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols)
                         : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols)
                         : "memory");
    }
}

int pipe_sm_count();

template <int AB, int TILE_N, int HOLD>
int launch_conv_umma_pipe_form(const ConvParams& p, const PipeGeom& g, cudaStream_t st) {
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaFuncSetAttribute(conv_umma_pipe_kernel<AB, TILE_N, false, HOLD>, cudaFuncAttributeMaxDynamicSharedMemorySize, PIPE_SMEM_MAX);
        cudaFuncSetAttribute(conv_umma_pipe_kernel<AB, TILE_N, true, HOLD>, cudaFuncAttributeMaxDynamicSharedMemorySize, PIPE_SMEM_MAX);
        attr_set[dev] = true;
    }
    const dim3 grid((unsigned)g.grid_x, (unsigned)g.grid_y, 1);
    if (p.ch_scale || p.ch_bias || p.residual || p.res_packed)
        conv_umma_pipe_kernel<AB, TILE_N, true, HOLD><<<grid, PIPE_THREADS, g.smem_bytes, st>>>(p, g);
    else
        conv_umma_pipe_kernel<AB, TILE_N, false, HOLD><<<grid, PIPE_THREADS, g.smem_bytes, st>>>(p, g);
    return EBS_OK;
}

// The CTA-pair form: clusters of two CTAs along x; packed-only whole tiles (form 1) or every output mode (form 0),
// no per-channel terms.
template <int AB, int FORM>
int launch_conv_umma_pipe_pair_form(const ConvParams& p, const PipeGeom& g, cudaStream_t st) {
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    auto kern = conv_umma_pipe_kernel<AB, 256, false, FORM, true>;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, PIPE_SMEM_MAX);
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)g.grid_x, (unsigned)g.grid_y, 1);
    cfg.blockDim = dim3(PIPE_THREADS, 1, 1);
    cfg.dynamicSmemBytes = (size_t)g.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, p, g) == cudaSuccess ? EBS_OK : EBS_ERR_CUDA;
}

inline bool pipe_pair_request_ok(const ConvParams& p) {
    return !p.ch_scale && !p.ch_bias && !p.residual && !p.res_packed && !p.w_levels && (p.Co % 256) == 0;
}

template <int AB>
int launch_conv_umma_pipe_pair(const ConvParams& p, dim3 /*grid*/, cudaStream_t st) {
    if (!pipe_pair_request_ok(p)) return EBS_ERR_UNSUPPORTED;
    const PipeGeom g = pipe_geometry(p, 256, pipe_sm_count(), p.pipe_m_sub, true);
    if (!g.ok) return EBS_ERR_UNSUPPORTED;
    if (!p.zero_words) return EBS_ERR_CUDA;                   // the device's zero page could not be found
    if (pipe_packed_only(p, 256)) return launch_conv_umma_pipe_pair_form<AB, 1>(p, g, st);
    return launch_conv_umma_pipe_pair_form<AB, 0>(p, g, st);
}

template <int AB, int TILE_N>
int launch_conv_umma_pipe(const ConvParams& p, dim3 /*grid*/, cudaStream_t st) {
    const PipeGeom g = pipe_geometry(p, TILE_N, pipe_sm_count(), p.pipe_m_sub);
    if (!g.ok) return EBS_ERR_UNSUPPORTED;                    // the geometry does not apply: nothing is launched
    if (!p.zero_words) return EBS_ERR_CUDA;                   // the device's zero page could not be found
    if (pipe_packed_only(p, TILE_N)) {
        if constexpr (TILE_N >= 128) {
            if (pipe_hold_applies(p, TILE_N)) return launch_conv_umma_pipe_form<AB, TILE_N, 2>(p, g, st);
        }
        return launch_conv_umma_pipe_form<AB, TILE_N, 1>(p, g, st);
    }
    return launch_conv_umma_pipe_form<AB, TILE_N, 0>(p, g, st);
}

constexpr int NUM_UMMA_PIPE_VARIANTS = 4;          // TILE_N = 64, 128, 256; 256 on a CTA pair

// One translation unit per activation bit count (conv_umma_pipe_a1.cu .. a8.cu): its three channel tiles and
// its share of the give-up counter.
#define EBS_DEFINE_PIPE_ROW(AB)                                                                             \
    const ConvVariant* conv_umma_pipe_variant_a##AB(int variant) {                                          \
        static const ConvVariant row[NUM_UMMA_PIPE_VARIANTS] = {                                            \
            ConvVariant{&launch_conv_umma_pipe<AB, 64>, UMMA_M, 64, PIPE_THREADS},                          \
            ConvVariant{&launch_conv_umma_pipe<AB, 128>, UMMA_M, 128, PIPE_THREADS},                        \
            ConvVariant{&launch_conv_umma_pipe<AB, 256>, UMMA_M, 256, PIPE_THREADS},                        \
            ConvVariant{&launch_conv_umma_pipe_pair<AB>, UMMA_M, 256, PIPE_THREADS}};                       \
        if (variant < 0 || variant >= NUM_UMMA_PIPE_VARIANTS) return nullptr;                               \
        return &row[variant];                                                                               \
    }                                                                                                       \
    unsigned long long conv_umma_pipe_timeouts_a##AB() {                                                    \
        unsigned long long v = 0;                                                                           \
        cudaMemcpyFromSymbol(&v, g_umma_timeouts, sizeof(v));                                               \
        return v;                                                                                           \
    }

}  // namespace ebs
