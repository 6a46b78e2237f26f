// Persistent form of the strip kernel: the weight bytes of a channel tile stay in shared memory and a
// CTA walks over many pixel tiles, with the three phases of a tile in different warps.
//
// Same arithmetic and addressing as conv_umma_strip_kernel (outputs numbered in the padded input
// frame, a filter tap = a shifted operand descriptor, weights from the byte image).  The non-persistent
// kernel fetches the kh*kw*CW weight tiles of its channel tile again in every CTA -- 147 KB per 128
// output pixels for a 3x3 128->128 layer, 250 MB of L2 traffic per layer -- and runs set-up, loads,
// expansion, MMAs and epilogue of a tile one after the other.  Here a CTA
//   * fetches all weight tiles of its channel tile ONCE (cp.async.bulk onto one mbarrier),
//   * owns pixel tiles t = blockIdx.x, blockIdx.x + gridDim.x, ... and runs 17 warps:
//       warps 0-7   expanders: packed words -> byte strips in a two-stage ring (loads run two chunks
//                   ahead, across tile boundaries),
//       warp  8     issuer: one tcgen05.mma per (tap, word) into one of TWO accumulators in tensor
//                   memory, tcgen05.commit onto the stage's "empty" barrier and, after a tile's last
//                   MMA, onto the accumulator's "full" barrier,
//       warps 9-16  epilogue: wait for "full", read the accumulator (tcgen05.ld), store / requantize /
//                   pack, arrive on the accumulator's "empty" barrier;
//     so the expansion of tile i+1, the MMAs of tile i and the epilogue of tile i-1 overlap.
// Applies when the strip kernel does, the weight tiles fit (<= 150 KB) and the layer has no window-sum
// term (w_levels = 0).  Bounded waits and the abort path as in conv_umma_kernel.
#pragma once

#include "conv_umma_strip.cuh"

namespace ebs {

constexpr int RES_THREADS = 17 * 32;
constexpr int RES_EPI_WARP0 = 9;
constexpr int RES_B_BYTES_MAX = 150 * 1024;

struct ResidentGeom {
    StripGeom strip;
    int b_bytes;        // all weight tiles of one channel tile
    int smem_bytes;
    int grid_x;         // CTAs along the pixel tiles
    bool ok;
};
inline ResidentGeom resident_geometry(const ConvParams& p, int tile_n, int sms) {
    ResidentGeom g{};
    g.strip = strip_geometry(p, tile_n);
    const int taps = p.kh * p.kw;
    g.b_bytes = p.CW * taps * tile_n * 32;
    int ks = g.strip.ks;
    while (ks > 1 && ks * strip_word_bytes(g.strip.strip_pad) > 24 * 1024) --ks;
    g.strip.ks = ks;
    g.smem_bytes = g.b_bytes + 2 * (ks * strip_word_bytes(g.strip.strip_pad) + 256) + 1024;
    const long long frame = (long long)p.N * strip_frame_h(p) * strip_frame_w(p);
    const long long ftiles = (frame + UMMA_M - 1) / UMMA_M;
    const int cotiles = (p.Co + tile_n - 1) / tile_n;
    long long gx = sms / cotiles;
    if (gx < 1) gx = 1;
    if (gx > ftiles) gx = ftiles;
    g.grid_x = (int)gx;
    g.ok = g.strip.ok && !p.w_levels && g.b_bytes <= RES_B_BYTES_MAX && g.b_bytes < (1 << 20) &&
           g.smem_bytes <= 210 * 1024 && cotiles <= 65535;
    return g;
}

template <int AB, int TILE_N, bool AFFINE>
__global__ void __launch_bounds__(RES_THREADS, 1) conv_umma_resident_kernel(const ConvParams p) {
    constexpr int TMEM_COLS = 2 * TILE_N < 32 ? 32 : 2 * TILE_N;     // two accumulators
    constexpr int B_TILE_BYTES = TILE_N * 32;
    extern __shared__ uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t a_full[2], a_empty[2], acc_full[2], acc_empty[2], b_full;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int S = p.strip_pix, SP = (S + 7) & ~7, KS = p.strip_ks;
    const int taps = p.kh * p.kw;
    const bool pointwise = strip_pointwise(p);
    const int Wp = strip_frame_w(p), Hp = strip_frame_h(p);
    const int frame = p.N * Hp * Wp;
    const int ftiles = (frame + UMMA_M - 1) / UMMA_M;
    const int my_tiles = ((int)blockIdx.x < ftiles) ? (ftiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int co0 = blockIdx.y * TILE_N;
    const int a_word_bytes = strip_word_bytes(SP);
    const int a_stage_bytes = (KS * a_word_bytes + 255) & ~255;
    uint8_t* base = dyn_smem + ((1024u - (smem_u32(dyn_smem) & 1023u)) & 1023u);
    uint8_t* b_tiles = base;                                             // [CW][taps][TILE_N][32]
    uint8_t* a_stages = base + p.CW * taps * B_TILE_BYTES;               // [2][KS][2][SP][16]
    volatile int* abortp = &abort_flag;
    const int nchunks = (p.CW + KS - 1) / KS;

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(&a_full[0], UMMA_EXPANDERS);
        mbar_init(&a_full[1], UMMA_EXPANDERS);
        mbar_init(&a_empty[0], 1);
        mbar_init(&a_empty[1], 1);
        mbar_init(&acc_full[0], 1);
        mbar_init(&acc_full[1], 1);
        mbar_init(&acc_empty[0], 256);
        mbar_init(&acc_empty[1], 256);
        mbar_init(&b_full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_slot)),
                     "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const uint32_t tmem_base = tmem_slot;

    if (warp < 8) {
        // =========================== expanders ===========================
        if (tid == 0 && my_tiles > 0) {                        // all weight tiles of this channel tile, once
            const uint32_t rows = (uint32_t)min(TILE_N, p.Co16 - co0);
            mbar_arrive_expect_tx(&b_full, rows * 32u * (uint32_t)(p.CW * taps));
            for (int cw = 0; cw < p.CW; ++cw)
                for (int t = 0; t < taps; ++t)
                    bulk_copy_g2s(b_tiles + (cw * taps + t) * B_TILE_BYTES,
                                  p.w8 + ((size_t)(t * p.CW + cw) * p.Co16 + co0) * 32, rows * 32u, &b_full);
        }
        int slot_q[STRIP_SLOTS], slot_pix[STRIP_SLOTS], slot_dst[STRIP_SLOTS];
#pragma unroll
        for (int j = 0; j < STRIP_SLOTS; ++j) {
            const int e = tid + j * UMMA_EXPANDERS;
            const int s = e / KS, q = e - s * KS;            // consecutive lanes: consecutive words of one pixel
            slot_q[j] = s < S ? q : -1;
            slot_pix[j] = s;
            slot_dst[j] = q * a_word_bytes + s * 16;
        }
        // loader state: runs two chunks ahead of the expansion, also across tile boundaries
        int ld_tile = 0, ld_ch = 0, ld_off[STRIP_SLOTS];
        auto tile_offsets = [&](int it) {
            const int f0 = ((int)blockIdx.x + it * (int)gridDim.x) * UMMA_M;
#pragma unroll
            for (int j = 0; j < STRIP_SLOTS; ++j) {
                ld_off[j] = -1;                                 // -1: padding or past the batch -> zero bytes
                const int f = f0 + slot_pix[j];
                if (slot_q[j] >= 0 && f < frame) {
                    const int n = f / (Hp * Wp), rem = f - n * (Hp * Wp);
                    const int hp = rem / Wp, wp = rem - hp * Wp;
                    const int h = pointwise ? hp * p.sh : hp - p.ph, w = pointwise ? wp * p.sw : wp - p.pw;
                    if ((unsigned)h < (unsigned)p.H && (unsigned)w < (unsigned)p.W)
                        ld_off[j] = ((n * p.H + h) * p.W + w) * p.CW * AB;
                }
            }
        };
        uint32_t a_set[3][STRIP_SLOTS][AB];
        auto load_next = [&](int set) {
#pragma unroll
            for (int j = 0; j < STRIP_SLOTS; ++j) {
#pragma unroll
                for (int k = 0; k < AB; ++k) a_set[set][j][k] = 0u;
                const int cw = ld_ch * KS + slot_q[j];
                if (slot_q[j] >= 0 && ld_off[j] >= 0 && cw < p.CW)
                    load_words_global<AB>(p.x + (ld_off[j] + cw * AB), a_set[set][j]);
            }
            if (++ld_ch == nchunks) {
                ld_ch = 0;
                if (++ld_tile < my_tiles) tile_offsets(ld_tile);
            }
        };
        const int total = my_tiles * nchunks;
        if (total > 0) { tile_offsets(0); load_next(0); }
        if (total > 1) load_next(1);
        bool ok = true;
        for (int g0 = 0; g0 < total && ok; g0 += 6) {
#pragma unroll
            for (int u6 = 0; u6 < 6; ++u6) {                    // 6 = lcm of the 3 register sets and the 2 stages
                const int g = g0 + u6;
                if (g >= total) break;
                const int u = u6 % 3, st = u6 & 1;
                uint8_t* A_st = a_stages + st * a_stage_bytes;
                if (g + 2 < total) load_next((u + 2) % 3);
                if (g >= 2) {                                   // the MMAs of chunk g-2 must have read the stage
                    if (!mbar_wait_bounded(&a_empty[st], (uint32_t)(((g >> 1) - 1) & 1), abortp)) { ok = false; break; }
                }
#pragma unroll
                for (int j = 0; j < STRIP_SLOTS; ++j) {
                    if (slot_q[j] < 0) continue;
                    uint32_t r[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
                    for (int k = 0; k < AB; ++k) {
                        const uint32_t w = a_set[u][j][k];
                        const uint32_t mask = 0x01010101u << k;
#pragma unroll
                        for (int bb = 0; bb < 8; ++bb) r[bb] |= __funnelshift_r(w, w, bb - k) & mask;
                    }
                    uint8_t* dst = A_st + slot_dst[j];
                    *reinterpret_cast<uint4*>(dst) = make_uint4(r[0], r[1], r[2], r[3]);
                    *reinterpret_cast<uint4*>(dst + SP * 16) = make_uint4(r[4], r[5], r[6], r[7]);
                }
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                mbar_arrive(&a_full[st]);
            }
        }
    } else if (warp == 8) {
        // =========================== issuer ===========================
        constexpr uint32_t IDESC = umma_idesc_i8(TILE_N);
        bool ok = my_tiles == 0 || mbar_wait_bounded(&b_full, 0u, abortp);
        const uint32_t b_base = smem_u32(b_tiles);
        int g = 0;
        for (int it = 0; it < my_tiles && ok; ++it) {
            const int buf = it & 1;
            if (it >= 2) {                                      // the epilogue of tile it-2 must have drained this accumulator
                if (!mbar_wait_bounded(&acc_empty[buf], (uint32_t)(((it >> 1) - 1) & 1), abortp)) break;
            }
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            const uint32_t tmem_d = tmem_base + (uint32_t)(buf * TILE_N);
            for (int ch = 0; ch < nchunks; ++ch, ++g) {
                const int st = g & 1;
                if (!mbar_wait_bounded(&a_full[st], (uint32_t)((g >> 1) & 1), abortp)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                if ((tid & 31) == 0) {
                    // descriptors built once per chunk and advanced by additions: a few instructions per MMA
                    const uint32_t a_base = smem_u32(a_stages + st * a_stage_bytes);
                    const int words = min(KS, p.CW - ch * KS);
                    const uint64_t da0 = umma_desc_interleaved(a_base, (uint32_t)(SP * 16));
                    uint64_t db = umma_desc_sw32(b_base + (uint32_t)(ch * KS * taps * B_TILE_BYTES));
                    uint32_t acc_flag = ch != 0 ? 1u : 0u;
                    for (int q = 0; q < words; ++q) {
                        uint64_t da_r = da0 + (uint64_t)(q * (a_word_bytes >> 4));
                        for (int r = 0; r < p.kh; ++r, da_r += (uint64_t)Wp) {
                            for (int s = 0; s < p.kw; ++s) {
                                umma_i8(tmem_d, da_r + (uint64_t)s, db, IDESC, acc_flag);
                                db += (uint64_t)(B_TILE_BYTES >> 4);
                                acc_flag = 1u;
                            }
                        }
                    }
                    umma_commit(&a_empty[st]);
                    if (ch == nchunks - 1) umma_commit(&acc_full[buf]);
                }
                __syncwarp();
            }
        }
    } else {
        // =========================== epilogue ===========================
        const int half = (warp - RES_EPI_WARP0) >> 2;            // which half of the channels (tiles of >= 64)
        const int vwarp = (warp & 3) + 4 * half;                 // TMEM lane quarter = warp % 4 (hardware rule)
        const int row = (warp & 3) * 32 + (tid & 31);
        for (int it = 0; it < my_tiles; ++it) {
            const int buf = it & 1;
            if (!mbar_wait_bounded(&acc_full[buf], (uint32_t)((it >> 1) & 1), abortp)) break;
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            const int f = ((int)blockIdx.x + it * (int)gridDim.x) * UMMA_M + row;
            bool pvalid = false;
            int gp = 0;
            if (f < frame) {
                const int n = f / (Hp * Wp), rem = f - n * (Hp * Wp);
                const int hp = rem / Wp, wp = rem - hp * Wp;
                pvalid = hp < p.Ho && wp < p.Wo;
                gp = (n * p.Ho + hp) * p.Wo + wp;
            }
            umma_epilogue<TILE_N, AFFINE>(p, tmem_base + (uint32_t)(buf * TILE_N), vwarp, gp, pvalid, 0, co0);
            asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
            mbar_arrive(&acc_empty[buf]);
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (abort_flag != 0 && tid == 0) atomicAdd(&g_umma_timeouts, 1ull);
    if (warp == 8) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS)
                     : "memory");
    }
}

int resident_sm_count();

template <int AB, int TILE_N>
int launch_conv_umma_resident(const ConvParams& p0, dim3 /*grid*/, cudaStream_t st) {
    ConvParams p = p0;
    const ResidentGeom g = resident_geometry(p, TILE_N, resident_sm_count());
    if (!g.ok) return EBS_ERR_UNSUPPORTED;                    // the geometry does not apply: nothing is launched
    p.strip_pix = g.strip.strip_pix;
    p.strip_ks = g.strip.ks;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaFuncSetAttribute(conv_umma_resident_kernel<AB, TILE_N, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 210 * 1024);
        cudaFuncSetAttribute(conv_umma_resident_kernel<AB, TILE_N, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 210 * 1024);
        attr_set[dev] = true;
    }
    const dim3 grid((unsigned)g.grid_x, (unsigned)((p.Co + TILE_N - 1) / TILE_N), 1);
    if (p.ch_scale || p.ch_bias || p.residual || p.res_packed)
        conv_umma_resident_kernel<AB, TILE_N, true><<<grid, RES_THREADS, g.smem_bytes, st>>>(p);
    else
        conv_umma_resident_kernel<AB, TILE_N, false><<<grid, RES_THREADS, g.smem_bytes, st>>>(p);
    return EBS_OK;
}

constexpr int NUM_UMMA_RESIDENT_VARIANTS = 5;      // TILE_N = 16, 32, 64, 128, 256

}  // namespace ebs
