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
//  * Roles: warps 0-7 expand (packed words -> byte strips, global loads two chunks ahead), warp 8
//    issues the MMAs, warp 9 fetches weight tiles, warps 10-17 run the epilogue out of tensor memory
//    while the next tile's MMAs fill the other accumulator set.
//  * Bit <-> byte transposes with one masked merge per plane and register: with v_k = rotl(w_k, k) the
//    byte register of channels {b, 8+b, 16+b, 24+b} is rotr(OR_k v_k & (0x01010101 << ((b+k) & 7)), b);
//    the epilogue packs requantized codes into plane words with the mirrored identity.
//
// Every wait on an mbarrier is bounded (ConvParams::wait_limit polls); on a timeout the CTA raises a
// shared abort flag, all its loops end, it records the event in a device counter, frees its tensor
// memory and returns.  No clusters, no multicast.
#pragma once

#include "conv_umma_strip.cuh"

namespace ebs {

constexpr int PIPE_EXPANDERS = 256;
constexpr int PIPE_ISSUER_WARP = 8, PIPE_PRODUCER_WARP = 9, PIPE_EPI_WARP0 = 10, PIPE_EPI_WARPS = 8;
constexpr int PIPE_THREADS = (PIPE_EPI_WARP0 + PIPE_EPI_WARPS) * 32;
constexpr int PIPE_SLOTS = 2;                      // (pixel, word) items an expander thread handles per stage
constexpr int PIPE_MAX_ITEMS = PIPE_SLOTS * PIPE_EXPANDERS;
constexpr int PIPE_MAX_TAPS = 64, PIPE_MAX_PHASES = 4, PIPE_MAX_STAGES = 4;
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
    int ks, nwg;                       // reduction words per stage; word groups = ceil(CW / ks)
    int n_ph, nchunks;                 // phases; chunks per tile = n_ph * nwg (phase-major)
    int n_stages, a_word_bytes, a_stage_bytes, stage_bytes;
    int b_resident, b_total_bytes, taps;
    int nbuf, tmem_cols, smem_bytes;
    int grid_x, grid_y;
    int ph_a[PIPE_MAX_PHASES], ph_b[PIPE_MAX_PHASES];
    int ph_tap0[PIPE_MAX_PHASES + 1];  // tap slots of phase i: [ph_tap0[i], ph_tap0[i + 1])
    short tap_shift[PIPE_MAX_TAPS];    // per tap slot: shift inside the strip, in pixels
    short tap_id[PIPE_MAX_TAPS];       // per tap slot: r * kw + s (tile index in the weight byte image)
    bool ok;
};

inline int floordiv_int(int a, int b) { return (a >= 0) ? a / b : -((-a + b - 1) / b); }

// m_sub_req / ks_req = 0: chosen here.  Returns ok = false when the kernel does not apply.
inline PipeGeom pipe_geometry(const ConvParams& p, int tile_n, int sms, int m_sub_req = 0) {
    PipeGeom g{};
    const int taps = p.kh * p.kw;
    if (p.w_levels || p.sh > 2 || p.sw > 2 || taps > PIPE_MAX_TAPS || p.kh > 16 || p.kw > 16) return g;
    if (tile_n != 64 && tile_n != 128 && tile_n != 256) return g;
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
    const int b_tile = tile_n * 32;
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
        const long long pt = (frame + (long long)m * UMMA_M - 1) / ((long long)m * UMMA_M);
        if (!m_sub_req && m > 1 && pt * g.n_ctiles < 2LL * sms) continue;
        m_sub = m;
        break;
    }
    if (!m_sub) return g;
    g.m_sub = m_sub;
    g.tile_pix = m_sub * UMMA_M;
    g.nbuf = (2 * m_sub * tile_n <= 512) ? 2 : 1;
    g.tmem_cols = g.nbuf * m_sub * tile_n;
    if (g.tmem_cols < 32) g.tmem_cols = 32;
    g.n_ptiles = (int)((frame + g.tile_pix - 1) / g.tile_pix);
    g.S = g.tile_pix + max_shift;
    g.SP = (g.S + 7) & ~7;
    g.a_word_bytes = g.SP * 32 + 32;
    if (g.SP * 16 >= (1 << 18)) return g;
    // weights resident when they leave room for at least two activation stages
    const int budget = PIPE_SMEM_MAX - 2048;
    g.b_resident = g.b_total_bytes + 2 * ((g.a_word_bytes + 255) & ~255) <= budget && g.b_total_bytes <= 160 * 1024;
    int ks = PIPE_MAX_ITEMS / g.S;
    if (ks > 4) ks = 4;
    if (ks > p.CW) ks = p.CW;
    if (ks < 1) return g;
    auto stage_bytes = [&](int k) {
        const int a = (k * g.a_word_bytes + 255) & ~255;
        return a + (g.b_resident ? 0 : k * max_ph_taps * b_tile);
    };
    const int avail = budget - (g.b_resident ? g.b_total_bytes : 0);
    while (ks > 1 && 2 * stage_bytes(ks) > avail) --ks;
    if (2 * stage_bytes(ks) > avail) return g;
    // fewer words per stage when that buys a deeper ring (latency hiding matters more than stage size)
    while (ks > 1 && avail / stage_bytes(ks) < 3) --ks;
    g.ks = ks;
    g.nwg = (p.CW + ks - 1) / ks;
    g.nchunks = g.n_ph * g.nwg;
    g.a_stage_bytes = (ks * g.a_word_bytes + 255) & ~255;
    g.stage_bytes = stage_bytes(ks);
    g.n_stages = avail / g.stage_bytes;
    if (g.n_stages > PIPE_MAX_STAGES) g.n_stages = PIPE_MAX_STAGES;
    g.smem_bytes = (g.b_resident ? g.b_total_bytes : 0) + g.n_stages * g.stage_bytes + 1024;
    if (g.b_resident) {                                        // a CTA keeps one channel tile
        g.grid_y = g.n_ctiles;
        long long gx = sms / g.n_ctiles;
        if (gx < 1) gx = 1;
        if (gx > g.n_ptiles) gx = g.n_ptiles;
        g.grid_x = (int)gx;
    } else {
        g.grid_y = 1;
        const long long items = (long long)g.n_ptiles * g.n_ctiles;
        g.grid_x = (int)(items < sms ? items : sms);
    }
    g.ok = g.n_stages >= 2 && g.smem_bytes <= PIPE_SMEM_MAX && g.grid_y <= 65535 && g.n_ctiles <= 65535;
    return g;
}

// One 32-channel group of the plain epilogue: 32 accumulators of this thread's pixel -> stores, fp32 steps,
// requantized codes -> plane words.
template <bool WANT_Q>
__device__ __forceinline__ void pipe_group32(const ConvParams& p, uint32_t (&v)[32], size_t o, bool pvalid, float S,
                                             float inv_next, int nb, int qmax, uint32_t* dst) {
    if (p.acc && pvalid) {
#pragma unroll
        for (int gq = 0; gq < 8; ++gq)
            *reinterpret_cast<int4*>(p.acc + o + 4 * gq) =
                make_int4((int)v[4 * gq], (int)v[4 * gq + 1], (int)v[4 * gq + 2], (int)v[4 * gq + 3]);
    }
    float y[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) y[e] = __fmul_rn((float)(int)v[e], S);
    if (p.y && pvalid) {
        const bool relu = p.relu != 0;
#pragma unroll
        for (int gq = 0; gq < 8; ++gq) {
            float4 t = make_float4(y[4 * gq], y[4 * gq + 1], y[4 * gq + 2], y[4 * gq + 3]);
            if (relu) { t.x = t.x > 0.f ? t.x : 0.f; t.y = t.y > 0.f ? t.y : 0.f; t.z = t.z > 0.f ? t.z : 0.f; t.w = t.w > 0.f ? t.w : 0.f; }
            *reinterpret_cast<float4*>(p.y + o + 4 * gq) = t;
        }
    }
    if (WANT_Q) {
        // The clamp at zero of the quantizer makes an explicit ReLU redundant here: a negative y gives
        // floor(y / step + 0.5) <= 0 and is clamped to code 0, exactly what max(y, 0) would give.
        // Byte register bb holds the codes of channels {bb, 8 + bb, 16 + bb, 24 + bb}, rotated left by bb.
        uint32_t cr[8];
#pragma unroll
        for (int bb = 0; bb < 8; ++bb) {
            int q[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                q[i] = min(__float2int_rd(__fadd_rn(__fmul_rn(y[8 * i + bb], inv_next), 0.5f)), qmax);
            const uint32_t c4 = pack_sat_u8x4(q[0], q[1], q[2], q[3]);      // saturates at 0 (negative values)
            cr[bb] = __funnelshift_l(c4, c4, bb);
        }
        uint32_t planes[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (j >= nb) break;
            uint32_t t = cr[0] & (0x01010101u << (j & 7));
#pragma unroll
            for (int bb = 1; bb < 8; ++bb) t |= cr[bb] & (0x01010101u << ((bb + j) & 7));
            planes[j] = __funnelshift_r(t, t, j);
        }
        if (pvalid) {
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

// Plain epilogue (no per-channel terms, no shortcut, NHWC, whole channel tile, c_out % 4 == 0) of one
// 128-pixel accumulator.  vwarp 0..7: TMEM lane quarter vwarp % 4, channel half vwarp / 4.
template <int TILE_N>
__device__ __forceinline__ void pipe_epilogue_plain(const ConvParams& p, uint32_t tmem_acc, int vwarp, int gp, bool pvalid,
                                                    int co0) {
    constexpr int COLS = TILE_N / 2;
    const uint32_t trow = tmem_acc + ((uint32_t)((vwarp & 3) * 32) << 16);
    const int cbeg = (vwarp >> 2) * COLS;
    const bool want_q = p.packed_next != nullptr;
    const int nb = want_q ? p.next_bits : 0, qmax = (1 << p.next_bits) - 1;
    const float S = p.S, inv_next = p.inv_next;
    uint32_t v[32];
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
        if (want_q) pipe_group32<true>(p, v, o, pvalid, S, inv_next, nb, qmax, dst);
        else pipe_group32<false>(p, v, o, pvalid, S, inv_next, nb, qmax, dst);
    }
}

template <int AB, int TILE_N, bool AFFINE>
__global__ void __launch_bounds__(PIPE_THREADS, 1) conv_umma_pipe_kernel(const ConvParams p, const PipeGeom g) {
    constexpr int B_TILE_BYTES = TILE_N * 32;
    extern __shared__ uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t st_full[PIPE_MAX_STAGES], st_empty[PIPE_MAX_STAGES], acc_full[2], acc_empty[2], b_full;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int NST = g.n_stages, KS = g.ks, SP = g.SP, S = g.S;
    const int nchunks = g.nchunks, nwg = g.nwg;
    const bool resident = g.b_resident != 0;
    uint8_t* base = dyn_smem + ((1024u - (smem_u32(dyn_smem) & 1023u)) & 1023u);
    uint8_t* b_res = base;                                               // [CW][tap slots][TILE_N][32] when resident
    uint8_t* stages = base + (resident ? g.b_total_bytes : 0);           // [NST] x ([KS][2][SP][16] A, then B tiles)
    volatile int* abortp = &abort_flag;
    const unsigned wait_limit = p.wait_limit;

    // work items of this CTA: (pixel super-tile, channel tile)
    const int n_items = resident ? g.n_ptiles : g.n_ptiles * g.n_ctiles;
    const int my_items = ((int)blockIdx.x < n_items) ? (n_items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    auto item_of = [&](int it, int& ptile, int& ctile) {
        const int idx = (int)blockIdx.x + it * (int)gridDim.x;
        if (resident) { ptile = idx; ctile = (int)blockIdx.y; }
        else { ptile = idx / g.n_ctiles; ctile = idx - ptile * g.n_ctiles; }
    };

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < PIPE_MAX_STAGES; ++s) {
            mbar_init(&st_full[s], PIPE_EXPANDERS + (resident ? 0 : 1));   // expanders (+ the thread that announces the weight copies)
            mbar_init(&st_empty[s], 1);
        }
        mbar_init(&acc_full[0], 1);
        mbar_init(&acc_full[1], 1);
        mbar_init(&acc_empty[0], PIPE_EPI_WARPS * 32);
        mbar_init(&acc_empty[1], PIPE_EPI_WARPS * 32);
        mbar_init(&b_full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == PIPE_ISSUER_WARP) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_slot)),
                     "r"((uint32_t)g.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const uint32_t tmem_base = tmem_slot;

    if (warp < 8) {
        // =========================== expanders ===========================
        int slot_q[PIPE_SLOTS], slot_pix[PIPE_SLOTS], slot_dst[PIPE_SLOTS];
#pragma unroll
        for (int j = 0; j < PIPE_SLOTS; ++j) {
            const int e = tid + j * PIPE_EXPANDERS;
            const int s = e / KS, q = e - s * KS;            // consecutive lanes: consecutive words of one pixel
            slot_q[j] = s < S ? q : -1;                       // -1: no item
            slot_pix[j] = s;
            slot_dst[j] = q * g.a_word_bytes + s * 16;
        }
        // loader state: runs two chunks ahead of the expansion, also across tile boundaries
        int ld_it = 0, ld_c = 0, ld_off[PIPE_SLOTS];
        auto chunk_offsets = [&](int it, int ph) {
            int ptile, ctile;
            item_of(it, ptile, ctile);
            const int f0 = ptile * g.tile_pix;
            const int pa = g.ph_a[ph], pb = g.ph_b[ph];
#pragma unroll
            for (int j = 0; j < PIPE_SLOTS; ++j) {
                ld_off[j] = -1;                                 // -1: padding or past the batch -> zero bytes
                const int f = f0 + slot_pix[j];
                if (slot_q[j] >= 0 && f < g.frame) {
                    const uint32_t n = fastdiv((uint32_t)f, g.div_img);
                    const uint32_t rem = (uint32_t)f - n * (uint32_t)(g.Hq * g.Wq);
                    const uint32_t hq = fastdiv(rem, g.div_row), wq = rem - hq * (uint32_t)g.Wq;
                    const int h = p.sh * ((int)hq + g.q0r) + pa, w = p.sw * ((int)wq + g.q0s) + pb;
                    if ((unsigned)h < (unsigned)p.H && (unsigned)w < (unsigned)p.W)
                        ld_off[j] = (((int)n * p.H + h) * p.W + w) * p.CW * AB;
                }
            }
        };
        uint32_t a_set[3][PIPE_SLOTS][AB];
        auto load_next = [&](int set) {
            const int ph = ld_c / nwg, wg = ld_c - ph * nwg;
            if (wg == 0) chunk_offsets(ld_it, ph);
#pragma unroll
            for (int j = 0; j < PIPE_SLOTS; ++j) {
#pragma unroll
                for (int k = 0; k < AB; ++k) a_set[set][j][k] = 0u;
                const int cw = wg * KS + slot_q[j];
                if (slot_q[j] >= 0 && ld_off[j] >= 0 && cw < p.CW)
                    load_words_global<AB>(p.x + (ld_off[j] + cw * AB), a_set[set][j]);
            }
            if (++ld_c == nchunks) { ld_c = 0; ++ld_it; }
        };
        const int total = my_items * nchunks;
        if (total > 0) load_next(0);
        if (total > 1) load_next(1);
        bool ok = true;
        int st = 0;
        uint32_t st_round = 0;                                  // how many times the ring has wrapped
        for (int g0 = 0; g0 < total && ok; g0 += 3) {
#pragma unroll
            for (int u = 0; u < 3; ++u) {
                const int gi = g0 + u;
                if (gi >= total) break;
                uint8_t* A_st = stages + st * g.stage_bytes;
                if (gi + 2 < total) load_next((u + 2) % 3);
                if (st_round > 0) {                             // the MMAs that read this stage one round ago must be done
                    if (!mbar_wait_bounded(&st_empty[st], (st_round - 1) & 1u, abortp, wait_limit)) { ok = false; break; }
                }
#pragma unroll
                for (int j = 0; j < PIPE_SLOTS; ++j) {
                    if (slot_q[j] < 0) continue;
                    // v_k = rotl(w_k, k); byte register bb = rotr(OR_k v_k & (0x01010101 << ((bb + k) & 7)), bb)
                    uint32_t v[AB];
#pragma unroll
                    for (int k = 0; k < AB; ++k) v[k] = __funnelshift_l(a_set[u][j][k], a_set[u][j][k], k);
                    uint32_t r[8];
#pragma unroll
                    for (int bb = 0; bb < 8; ++bb) {
                        uint32_t t = v[0] & (0x01010101u << bb);
#pragma unroll
                        for (int k = 1; k < AB; ++k) t |= v[k] & (0x01010101u << ((bb + k) & 7));
                        r[bb] = __funnelshift_r(t, t, bb);
                    }
                    uint8_t* dst = A_st + slot_dst[j];
                    *reinterpret_cast<uint4*>(dst) = make_uint4(r[0], r[1], r[2], r[3]);
                    *reinterpret_cast<uint4*>(dst + SP * 16) = make_uint4(r[4], r[5], r[6], r[7]);
                }
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                mbar_arrive(&st_full[st]);
                if (++st == NST) { st = 0; ++st_round; }
            }
        }
    } else if (warp == PIPE_ISSUER_WARP) {
        // =========================== issuer ===========================
        constexpr uint32_t IDESC = umma_idesc_i8(TILE_N);
        const bool skip_mma = (p.test_flags & 1) != 0;            // test hook: issue nothing, so that waits run out
        bool ok = my_items == 0 || !resident || mbar_wait_bounded(&b_full, 0u, abortp, wait_limit);
        int st = 0;
        uint32_t st_round = 0;
        for (int it = 0; it < my_items && ok; ++it) {
            const int buf = g.nbuf == 2 ? (it & 1) : 0;
            const int use = g.nbuf == 2 ? (it >> 1) : it;          // how often this accumulator set was used before
            if (use > 0) {                                          // its epilogue must have drained it
                if (!mbar_wait_bounded(&acc_empty[buf], (uint32_t)((use - 1) & 1), abortp, wait_limit)) break;
            }
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            const uint32_t tmem_d = tmem_base + (uint32_t)(buf * g.m_sub * TILE_N);
            for (int c = 0; c < nchunks; ++c) {
                if (!mbar_wait_bounded(&st_full[st], st_round & 1u, abortp, wait_limit)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                if ((tid & 31) == 0 && !skip_mma) {
                    const int ph = c / nwg, wg = c - ph * nwg;
                    const int words = min(KS, p.CW - wg * KS);
                    const int t0 = g.ph_tap0[ph], t1 = g.ph_tap0[ph + 1];
                    uint8_t* stage = stages + st * g.stage_bytes;
                    const uint64_t da0 = umma_desc_interleaved(smem_u32(stage), (uint32_t)(SP * 16));
                    const uint32_t b_stage = smem_u32(stage + g.a_stage_bytes);
                    for (int q = 0; q < words; ++q) {
                        const uint64_t da_q = da0 + (uint64_t)(q * (g.a_word_bytes >> 4));
                        for (int ts = t0; ts < t1; ++ts) {
                            const uint32_t b_addr = resident
                                ? smem_u32(b_res) + (uint32_t)(((wg * KS + q) * g.taps + ts) * B_TILE_BYTES)
                                : b_stage + (uint32_t)((q * (t1 - t0) + (ts - t0)) * B_TILE_BYTES);
                            const uint64_t db = umma_desc_sw32(b_addr);
                            const uint64_t da_t = da_q + (uint64_t)g.tap_shift[ts];
                            const uint32_t acc_flag = (c | q | (ts - t0)) != 0 ? 1u : 0u;
                            for (int j = 0; j < g.m_sub; ++j)
                                umma_i8(tmem_d + (uint32_t)(j * TILE_N), da_t + (uint64_t)(j * (UMMA_M * 16 >> 4)), db, IDESC, acc_flag);
                        }
                    }
                    umma_commit(&st_empty[st]);
                    if (c == nchunks - 1) umma_commit(&acc_full[buf]);
                }
                __syncwarp();
                if (++st == NST) { st = 0; ++st_round; }
            }
        }
    } else if (warp == PIPE_PRODUCER_WARP) {
        // =========================== weight tiles ===========================
        if ((tid & 31) == 0 && my_items > 0) {
            if (resident) {                                      // all tiles of this CTA's channel tile, once
                const int co0 = (int)blockIdx.y * TILE_N;
                const uint32_t rows = (uint32_t)min(TILE_N, p.Co16 - co0);
                mbar_arrive_expect_tx(&b_full, rows * 32u * (uint32_t)(p.CW * g.taps));
                for (int cw = 0; cw < p.CW; ++cw)
                    for (int ts = 0; ts < g.taps; ++ts)
                        bulk_copy_g2s(b_res + (cw * g.taps + ts) * B_TILE_BYTES,
                                      p.w8 + ((size_t)(g.tap_id[ts] * p.CW + cw) * p.Co16 + co0) * 32, rows * 32u, &b_full);
            } else {
                int st = 0;
                uint32_t st_round = 0;
                bool ok = true;
                for (int it = 0; it < my_items && ok; ++it) {
                    int ptile, ctile;
                    item_of(it, ptile, ctile);
                    const int co0 = ctile * TILE_N;
                    const uint32_t rows = (uint32_t)min(TILE_N, p.Co16 - co0);
                    for (int c = 0; c < nchunks; ++c) {
                        if (st_round > 0) {
                            if (!mbar_wait_bounded(&st_empty[st], (st_round - 1) & 1u, abortp, wait_limit)) { ok = false; break; }
                        }
                        const int ph = c / nwg, wg = c - ph * nwg;
                        const int words = min(KS, p.CW - wg * KS);
                        const int t0 = g.ph_tap0[ph], t1 = g.ph_tap0[ph + 1];
                        uint8_t* b_stage = stages + st * g.stage_bytes + g.a_stage_bytes;
                        mbar_arrive_expect_tx(&st_full[st], rows * 32u * (uint32_t)(words * (t1 - t0)));
                        for (int q = 0; q < words; ++q)
                            for (int ts = t0; ts < t1; ++ts)
                                bulk_copy_g2s(b_stage + (q * (t1 - t0) + (ts - t0)) * B_TILE_BYTES,
                                              p.w8 + ((size_t)(g.tap_id[ts] * p.CW + wg * KS + q) * p.Co16 + co0) * 32,
                                              rows * 32u, &st_full[st]);
                        if (++st == NST) { st = 0; ++st_round; }
                    }
                }
            }
        }
    } else {
        // =========================== epilogue ===========================
        const int half = (warp - PIPE_EPI_WARP0) >> 2;           // which half of the channels
        const int vwarp = (warp & 3) + 4 * half;                 // TMEM lane quarter = warp % 4 (hardware rule)
        const int row = (warp & 3) * 32 + (tid & 31);
        const bool plain_ok = !AFFINE && !p.ch_scale && !p.ch_bias && !p.residual && !p.res_packed && !p.y_nchw &&
                              (p.Co & 3) == 0;
        for (int it = 0; it < my_items; ++it) {
            const int buf = g.nbuf == 2 ? (it & 1) : 0;
            const int use = g.nbuf == 2 ? (it >> 1) : it;
            if (!mbar_wait_bounded(&acc_full[buf], (uint32_t)(use & 1), abortp, wait_limit)) break;
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            int ptile, ctile;
            item_of(it, ptile, ctile);
            const int co0 = ctile * TILE_N;
            for (int j = 0; j < g.m_sub; ++j) {
                const int f = ptile * g.tile_pix + j * UMMA_M + row;
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
                if (plain_ok && co0 + TILE_N <= p.Co) pipe_epilogue_plain<TILE_N>(p, tmem_acc, vwarp, gp, pvalid, co0);
                else umma_epilogue<TILE_N, AFFINE>(p, tmem_acc, vwarp, gp, pvalid, 0, co0);
            }
            asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
            mbar_arrive(&acc_empty[buf]);
        }
    }

    // a CTA that gave up may still have weight copies in flight towards its shared memory: give them time to land
    // (bounded) before the block ends and the memory is handed to another block
    if (warp == PIPE_PRODUCER_WARP && *abortp) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (abort_flag != 0 && tid == 0) atomicAdd(&g_umma_timeouts, 1ull);
    if (warp == PIPE_ISSUER_WARP) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols)
                     : "memory");
    }
}

int pipe_sm_count();

template <int AB, int TILE_N>
int launch_conv_umma_pipe(const ConvParams& p, dim3 /*grid*/, cudaStream_t st) {
    const PipeGeom g = pipe_geometry(p, TILE_N, pipe_sm_count(), p.pipe_m_sub);
    if (!g.ok) return EBS_ERR_UNSUPPORTED;                    // the geometry does not apply: nothing is launched
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaFuncSetAttribute(conv_umma_pipe_kernel<AB, TILE_N, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PIPE_SMEM_MAX);
        cudaFuncSetAttribute(conv_umma_pipe_kernel<AB, TILE_N, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PIPE_SMEM_MAX);
        attr_set[dev] = true;
    }
    const dim3 grid((unsigned)g.grid_x, (unsigned)g.grid_y, 1);
    if (p.ch_scale || p.ch_bias || p.residual || p.res_packed)
        conv_umma_pipe_kernel<AB, TILE_N, true><<<grid, PIPE_THREADS, g.smem_bytes, st>>>(p, g);
    else
        conv_umma_pipe_kernel<AB, TILE_N, false><<<grid, PIPE_THREADS, g.smem_bytes, st>>>(p, g);
    return EBS_OK;
}

constexpr int NUM_UMMA_PIPE_VARIANTS = 3;          // TILE_N = 64, 128, 256

// One translation unit per activation bit count (conv_umma_pipe_a1.cu .. a8.cu): its three channel tiles and
// its share of the give-up counter.
#define EBS_DEFINE_PIPE_ROW(AB)                                                                             \
    const ConvVariant* conv_umma_pipe_variant_a##AB(int variant) {                                          \
        static const ConvVariant row[NUM_UMMA_PIPE_VARIANTS] = {                                            \
            ConvVariant{&launch_conv_umma_pipe<AB, 64>, UMMA_M, 64, PIPE_THREADS},                          \
            ConvVariant{&launch_conv_umma_pipe<AB, 128>, UMMA_M, 128, PIPE_THREADS},                        \
            ConvVariant{&launch_conv_umma_pipe<AB, 256>, UMMA_M, 256, PIPE_THREADS}};                       \
        if (variant < 0 || variant >= NUM_UMMA_PIPE_VARIANTS) return nullptr;                               \
        return &row[variant];                                                                               \
    }                                                                                                       \
    unsigned long long conv_umma_pipe_timeouts_a##AB() {                                                    \
        unsigned long long v = 0;                                                                           \
        cudaMemcpyFromSymbol(&v, g_umma_timeouts, sizeof(v));                                               \
        return v;                                                                                           \
    }

}  // namespace ebs
