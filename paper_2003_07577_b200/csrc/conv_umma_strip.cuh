// Stride-1 (and strided 1x1) bit-plane convolution on the tcgen05 tensor cores with every input pixel
// expanded ONCE per thread block, however many filter taps read it.
//
// Arithmetic as in conv_umma_kernel: the planes of a packed word are merged back into one byte per
// channel and one int8 MMA per (tap, reduction word) retires all Wb*Ab plane pairs of its 32 channels.
// What differs is the addressing.  Output pixels are numbered in the zero-padded input frame,
//     f = (n * Hp + hp) * Wp + wp,   Hp = H + 2 pad_h,  Wp = W + 2 pad_w,
// so that for stride 1 the input under tap (r, s) of output f is simply f + r * Wp + s: a filter tap is
// a constant shift.  A CTA owns 128 consecutive f and TILE_N channels.  Per reduction word its
// expanders write the bytes of the strip f0 .. f0 + 127 + (kh-1) * Wp + (kw-1) into shared memory once
// (zero where f falls in the padding or past the batch), in the un-swizzled K-major layout
// [16-byte half][pixel][16 bytes], in which 8 consecutive pixels form one 128-byte core matrix.  The
// MMA of tap (r, s) then reads the same strip through a descriptor whose start address is moved by
// (r * Wp + s) * 16 bytes.  Outputs whose f has hp >= Ho or wp >= Wo do not exist and are dropped in
// the epilogue; this costs (Hp * Wp) / (Ho * Wo) - 1 extra MMA rows and saves a factor kh * kw in
// bit-to-byte expansion, which is what bounds the per-tap kernel.
//
// The weight operand comes from the byte image that ebs_pack_weights appends to the plane words: a
// (tap, word) tile of TILE_N rows x 32 bytes is contiguous there in exactly the swizzled layout the MMA
// reads, so one thread fetches it with cp.async.bulk straight into shared memory, completing on the
// stage's "full" mbarrier; no thread touches weight bits.
//
// Roles, barriers, bounded waits and the epilogue are those of conv_umma_kernel (warps 0-7 expand,
// warp 8 issues; two stages).
#pragma once

#include "conv_umma.cuh"

namespace ebs {

constexpr int STRIP_SLOTS = 2;                 // (pixel, word) items an expander thread handles per stage
constexpr int STRIP_MAX_ITEMS = STRIP_SLOTS * UMMA_EXPANDERS;

// Shared-memory matrix descriptor: K-major operand without swizzle.  Rows (pixels) are 16 bytes apart
// inside a core matrix of 8 rows, core matrices of consecutive row groups 128 bytes apart, the two
// 16-byte halves of the 32-byte reduction step `lbo` bytes apart.
__device__ __forceinline__ uint64_t umma_desc_interleaved(uint32_t smem_addr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);      // start address, 16-byte units
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16; // leading byte offset: between the two K halves
    d |= (uint64_t)(128u >> 4) << 32;                 // stride byte offset: between 8-row groups
    d |= (uint64_t)1u << 46;                          // descriptor version of this architecture
    return d;                                         // layout type 0: no swizzle
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Contiguous global -> shared copy by the copy engine; both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                 ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// A 1x1 convolution without padding reads exactly one input pixel per output whatever its stride, so
// it runs in the same kernel with the frame taken over the OUTPUT pixels: Hp = Ho, Wp = Wo and input
// pixel (hp * stride_h, wp * stride_w).
__host__ __device__ inline bool strip_pointwise(const ConvParams& p) {
    return p.kh == 1 && p.kw == 1 && p.ph == 0 && p.pw == 0;
}
__host__ __device__ inline int strip_frame_h(const ConvParams& p) { return strip_pointwise(p) ? p.Ho : p.H + 2 * p.ph; }
__host__ __device__ inline int strip_frame_w(const ConvParams& p) { return strip_pointwise(p) ? p.Wo : p.W + 2 * p.pw; }

// Bytes from one reduction word of a strip to the next: two halves of strip_pad x 16 bytes plus 32 bytes, so
// that the 16-byte stores of lanes that hold consecutive words of one pixel fall into different banks.
__host__ __device__ inline int strip_word_bytes(int strip_pad) { return strip_pad * 32 + 32; }

// Host-side geometry of a launch (also used by the library to decide whether the kernel applies).
struct StripGeom {
    int strip_pix;      // pixels of a strip: 128 + (kh-1) * Wp + (kw-1)
    int strip_pad;      // rounded up to 8 (core matrices)
    int ks;             // reduction words per stage
    int smem_bytes;     // dynamic shared memory
    bool ok;
};
inline StripGeom strip_geometry(const ConvParams& p, int tile_n) {
    StripGeom g{};
    const int Wp = strip_frame_w(p), taps = p.kh * p.kw;
    g.strip_pix = UMMA_M + (p.kh - 1) * Wp + (p.kw - 1);
    g.strip_pad = (g.strip_pix + 7) & ~7;
    const long long frame = (long long)p.N * strip_frame_h(p) * Wp;
    const int word_bytes = strip_word_bytes(g.strip_pad) + taps * tile_n * 32;
    int ks = STRIP_MAX_ITEMS / g.strip_pix;
    if (ks > 4) ks = 4;
    if (ks > p.CW) ks = p.CW;
    while (ks > 1 && ks * word_bytes > 48 * 1024) --ks;
    g.ks = ks;
    g.smem_bytes = 2 * (ks * word_bytes + 256) + 1024 + g.strip_pad * 4;
    g.ok = ((p.sh == 1 && p.sw == 1) || strip_pointwise(p)) && ks >= 1 && g.strip_pix <= STRIP_MAX_ITEMS && taps <= 64 &&
           g.smem_bytes <= 200 * 1024 && frame < (1LL << 31) - 256 && g.strip_pad * 16 < (1 << 18);
    return g;
}

template <int AB, int TILE_N, bool AFFINE>
__global__ void __launch_bounds__(UMMA_THREADS) conv_umma_strip_kernel(const ConvParams p) {
    constexpr int TMEM_COLS = TILE_N < 32 ? 32 : TILE_N;
    constexpr int B_TILE_BYTES = TILE_N * 32;
    extern __shared__ uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t full_bar[2];
    __shared__ __align__(8) uint64_t empty_bar[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int S = p.strip_pix, SP = (S + 7) & ~7, KS = p.strip_ks;
    const int taps = p.kh * p.kw;
    const bool pointwise = strip_pointwise(p);
    const int Wp = strip_frame_w(p), Hp = strip_frame_h(p);
    const int frame = p.N * Hp * Wp;                          // outputs are numbered in the padded input frame
    const int f0 = blockIdx.x * UMMA_M;
    const int co0 = blockIdx.y * TILE_N;
    const int a_word_bytes = strip_word_bytes(SP);            // one reduction word of the strip: two halves of SP x 16 B (+ skew)
    const int a_stage_bytes = (KS * a_word_bytes + 255) & ~255;   // the weight tiles behind it keep their 256-byte alignment
    const int stage_bytes = a_stage_bytes + KS * taps * B_TILE_BYTES;
    uint8_t* tiles = dyn_smem + ((1024u - (smem_u32(dyn_smem) & 1023u)) & 1023u);
    int* csum_s = reinterpret_cast<int*>(tiles + 2 * stage_bytes);      // per strip pixel: sum of its codes (w_levels)
    volatile int* abortp = &abort_flag;

    for (int i = tid; i < SP; i += UMMA_THREADS) csum_s[i] = 0;
    if (tid == 0) {
        abort_flag = 0;
        mbar_init(&full_bar[0], UMMA_EXPANDERS + 1);          // 256 expanders + the thread that announces the copies
        mbar_init(&full_bar[1], UMMA_EXPANDERS + 1);
        mbar_init(&empty_bar[0], 1);
        mbar_init(&empty_bar[1], 1);
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

    const int nchunks = (p.CW + KS - 1) / KS;

    if (warp < 8) {
        // =========================== expanders ===========================
        // slot j of this thread: strip pixel s_j of reduction word q_j of the stage
        int slot_q[STRIP_SLOTS], slot_off[STRIP_SLOTS], slot_dst[STRIP_SLOTS], slot_pix[STRIP_SLOTS];
#pragma unroll
        for (int j = 0; j < STRIP_SLOTS; ++j) {
            const int e = tid + j * UMMA_EXPANDERS;
            const int s = e / KS, q = e - s * KS;            // consecutive lanes: consecutive words of one pixel (contiguous in memory)
            slot_q[j] = s < S ? q : -1;                       // -1: no item
            slot_pix[j] = s;
            slot_dst[j] = q * a_word_bytes + s * 16;
            slot_off[j] = -1;                                 // -1: padding or past the batch -> zero bytes
            const int f = f0 + s;
            if (s < S && f < frame) {
                const int n = f / (Hp * Wp), rem = f - n * (Hp * Wp);
                const int hp = rem / Wp, wp = rem - hp * Wp;
                const int h = pointwise ? hp * p.sh : hp - p.ph, w = pointwise ? wp * p.sw : wp - p.pw;
                if ((unsigned)h < (unsigned)p.H && (unsigned)w < (unsigned)p.W)
                    slot_off[j] = ((n * p.H + h) * p.W + w) * p.CW * AB;
            }
        }
        const uint32_t b_rows = (uint32_t)min(TILE_N, p.Co16 - co0);
        uint32_t a_set[3][STRIP_SLOTS][AB];                   // packed words of three consecutive chunks (ring)

        auto load_chunk = [&](int ch, int set) {
#pragma unroll
            for (int j = 0; j < STRIP_SLOTS; ++j) {
#pragma unroll
                for (int k = 0; k < AB; ++k) a_set[set][j][k] = 0u;
                const int cw = ch * KS + slot_q[j];
                if (slot_q[j] >= 0 && slot_off[j] >= 0 && cw < p.CW)
                    load_words_global<AB>(p.x + (slot_off[j] + cw * AB), a_set[set][j]);
            }
        };
        load_chunk(0, 0);
        if (nchunks > 1) load_chunk(1, 1);
        bool expanders_ok = true;
        int csum[STRIP_SLOTS] = {};
        for (int ch0 = 0; ch0 < nchunks && expanders_ok; ch0 += 3) {
#pragma unroll
            for (int u = 0; u < 3; ++u) {
                const int ch = ch0 + u;
                if (ch >= nchunks) break;
                const int st = ch & 1;
                uint8_t* A_st = tiles + st * stage_bytes;
                if (ch + 2 < nchunks) load_chunk(ch + 2, (u + 2) % 3);
                if (ch >= 2) {                                 // the MMAs of chunk ch-2 must have read the stage
                    if (!mbar_wait_bounded(&empty_bar[st], (uint32_t)(((ch >> 1) - 1) & 1), abortp)) {
                        expanders_ok = false;
                        break;
                    }
                }
                if (tid == 0) {                                // weight tiles of this stage: one bulk copy per (word, tap)
                    const int words = min(KS, p.CW - ch * KS);
                    const uint32_t bytes = b_rows * 32u;
                    mbar_arrive_expect_tx(&full_bar[st], bytes * (uint32_t)(words * taps));
                    for (int q = 0; q < words; ++q)
                        for (int t = 0; t < taps; ++t)
                            bulk_copy_g2s(A_st + a_stage_bytes + (q * taps + t) * B_TILE_BYTES,
                                          p.w8 + ((size_t)(t * p.CW + ch * KS + q) * p.Co16 + co0) * 32, bytes,
                                          &full_bar[st]);
                }
#pragma unroll
                for (int j = 0; j < STRIP_SLOTS; ++j) {
                    if (slot_q[j] < 0) continue;
                    // activation codes: register b of the pixel holds channels {b, 8+b, 16+b, 24+b}
                    uint32_t r[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
                    for (int k = 0; k < AB; ++k) {
                        const uint32_t w = a_set[u][j][k];
                        if (p.w_levels) csum[j] += __popc(w) << k;
                        const uint32_t mask = 0x01010101u << k;
#pragma unroll
                        for (int bb = 0; bb < 8; ++bb) r[bb] |= __funnelshift_r(w, w, bb - k) & mask;
                    }
                    uint8_t* dst = A_st + slot_dst[j];
                    *reinterpret_cast<uint4*>(dst) = make_uint4(r[0], r[1], r[2], r[3]);
                    *reinterpret_cast<uint4*>(dst + SP * 16) = make_uint4(r[4], r[5], r[6], r[7]);
                }
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");  // generic writes -> tensor-core reads
                mbar_arrive(&full_bar[st]);
            }
        }
        if (p.w_levels) {
#pragma unroll
            for (int j = 0; j < STRIP_SLOTS; ++j)
                if (slot_q[j] >= 0 && csum[j]) atomicAdd(&csum_s[slot_pix[j]], csum[j]);
        }
    } else {
        // =========================== issuer ===========================
        constexpr uint32_t IDESC = umma_idesc_i8(TILE_N);
        for (int ch = 0; ch < nchunks; ++ch) {
            const int st = ch & 1;
            if (!mbar_wait_bounded(&full_bar[st], (uint32_t)((ch >> 1) & 1), abortp)) break;
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            if ((tid & 31) == 0) {
                // the issuing thread is the pipeline stage that feeds the tensor core: descriptors are built once
                // and advanced by additions (start addresses are in 16-byte units), a few instructions per MMA
                const uint32_t a_base = smem_u32(tiles + st * stage_bytes);
                const int words = min(KS, p.CW - ch * KS);
                const uint64_t da0 = umma_desc_interleaved(a_base, (uint32_t)(SP * 16));
                uint64_t db = umma_desc_sw32(a_base + a_stage_bytes);
                uint32_t acc_flag = ch != 0 ? 1u : 0u;
                for (int q = 0; q < words; ++q) {
                    uint64_t da_r = da0 + (uint64_t)(q * (a_word_bytes >> 4));
                    for (int r = 0; r < p.kh; ++r, da_r += (uint64_t)Wp) {
                        for (int s = 0; s < p.kw; ++s) {
                            umma_i8(tmem_base, da_r + (uint64_t)s, db, IDESC, acc_flag);
                            db += (uint64_t)(B_TILE_BYTES >> 4);
                            acc_flag = 1u;
                        }
                    }
                }
                umma_commit(&empty_bar[st]);
            }
            __syncwarp();
        }
        // all MMAs done (the last commit covers every earlier one); only this warp polls, the expanders
        // sleep in the block barrier below
        if (!*abortp) mbar_wait_bounded(&empty_bar[(nchunks - 1) & 1], (uint32_t)(((nchunks - 1) >> 1) & 1), abortp);
    }

    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const bool aborted = abort_flag != 0;

    // ---- epilogue: expander threads read the accumulators of their own row f0 + (tid % 128)
    if (!aborted && warp < 8) {
        const int row = tid & (UMMA_M - 1);
        const int f = f0 + row;
        bool pvalid = false;
        int gp = 0;
        if (f < frame) {
            const int n = f / (Hp * Wp), rem = f - n * (Hp * Wp);
            const int hp = rem / Wp, wp = rem - hp * Wp;
            pvalid = hp < p.Ho && wp < p.Wo;
            gp = (n * p.Ho + hp) * p.Wo + wp;
        }
        int wsum_row = 0;
        if (p.w_levels)
            for (int r = 0; r < p.kh; ++r)
                for (int s = 0; s < p.kw; ++s) wsum_row += csum_s[row + r * Wp + s];
        umma_epilogue<TILE_N, AFFINE>(p, tmem_base, warp, gp, pvalid, wsum_row, co0);
    }
    if (aborted && tid == 0) atomicAdd(&g_umma_timeouts, 1ull);

    // ---- release tensor memory (every path reaches this)
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 8) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS)
                     : "memory");
    }
}

template <int AB, int TILE_N>
int launch_conv_umma_strip(const ConvParams& p0, dim3 /*grid*/, cudaStream_t st) {
    ConvParams p = p0;
    const StripGeom g = strip_geometry(p, TILE_N);
    if (!g.ok) return EBS_ERR_UNSUPPORTED;                    // the geometry does not apply: nothing is launched
    p.strip_pix = g.strip_pix;
    p.strip_ks = g.ks;
    const bool affine = p.ch_scale || p.ch_bias || p.residual || p.res_packed;
    static bool attr_set[64] = {};                            // dynamic shared memory limit raised, per device
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaFuncSetAttribute(conv_umma_strip_kernel<AB, TILE_N, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        cudaFuncSetAttribute(conv_umma_strip_kernel<AB, TILE_N, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        attr_set[dev] = true;
    }
    const long long frame = (long long)p.N * strip_frame_h(p) * strip_frame_w(p);
    const dim3 grid((unsigned)((frame + UMMA_M - 1) / UMMA_M), (unsigned)((p.Co + TILE_N - 1) / TILE_N), 1);
    if (affine) conv_umma_strip_kernel<AB, TILE_N, true><<<grid, UMMA_THREADS, g.smem_bytes, st>>>(p);
    else conv_umma_strip_kernel<AB, TILE_N, false><<<grid, UMMA_THREADS, g.smem_bytes, st>>>(p);
    return EBS_OK;
}

constexpr int NUM_UMMA_STRIP_VARIANTS = 5;      // TILE_N = 16, 32, 64, 128, 256

}  // namespace ebs
