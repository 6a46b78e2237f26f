// Whole-network kernel for basic-block CIFAR ResNets: one CTA carries one image through every layer
// with its activations resident in shared memory.
//
// The per-layer kernels spend most of a ResNet-20 layer's 5-18 us on launch, prologue and moving 4-37 KB
// of activations per image through L2.  Here the activation codes of an image live in shared memory as
// BYTES, already in the un-swizzled K-major strip layout the tcgen05 operand descriptors read
// ([16-byte half][frame pixel][16 bytes] per 32-channel word, frame = zero-padded image), so between
// layers there is no bit-to-byte expansion, no global traffic and no launch.  Per layer the CTA
//   1. has the layer's weight byte image (the second part of an ebs_pack_weights buffer) fetched into one
//      of two shared buffers by cp.async.bulk while the previous layer runs,
//   2. lets one thread issue all MMAs of the layer -- every 128-row tile of the frame x every tap x every
//      32-channel word, a tap being a shifted descriptor -- into tensor-memory accumulators (tile t at
//      columns 32 t or 64 t), then tcgen05.commit onto an mbarrier,
//   3. runs the fp32 steps of the epilogue out of tensor memory (scale, per-channel scale/shift, shortcut,
//      ReLU, requantize: the same individually rounded operations as the per-layer kernels) and writes the
//      codes as bytes at frame position f + Wp + 1 of the destination strip: outputs that do not exist
//      (frame columns >= Wo, rows >= Ho) land exactly on padding positions and are written as zero.
// Stride-2 3x3 layers are computed at stride 1 and subsampled in the epilogue (4x the MMAs of two or three
// layers, no phase logic); a 1x1 stride-2 projection runs on a subsampled copy of its input laid out in the
// output frame, keeps its accumulators in tensor memory, and the next layer's epilogue adds them as the
// shortcut.  The identity shortcut is read from the destination strip (the block input) just before it is
// overwritten in place.  After the last block: average pooling (pixels added in order), 8-bit
// quantization, and the classifier as a plain integer dot product.
// Every wait is bounded; on a timeout the CTA sets its abort flag, skips the rest, frees tensor memory.
#include "conv_umma_strip.cuh"

namespace ebs {

constexpr int FUSED_THREADS = 768;
constexpr int FUSED_ACT_PIX = 1360;                    // pixels an activation strip holds (34 x 34 frame + halo, 128-row tiles)
constexpr int FUSED_ACT_BYTES = FUSED_ACT_PIX * 32;    // one 32-channel word
constexpr int FUSED_W_BYTES = 37 * 1024;               // largest weight image (3x3 64->64)
constexpr int FUSED_SMEM = 3 * FUSED_ACT_BYTES + 2 * FUSED_W_BYTES + 1024;
constexpr int FUSED_HOLD_COL = 320;                    // accumulator columns of a held projection

using FusedLayer = ebs_fused_layer;
using FusedHead = ebs_fused_head;

__device__ __forceinline__ uint8_t* strip_ptr(uint8_t* acts, int buf) { return acts + buf * FUSED_ACT_BYTES; }
// A strip holds one 32-channel word of up to 1360 frame pixels or two words of up to 680: pixels per word.
__host__ __device__ inline int strip_cap(int channels) { return channels > 32 ? FUSED_ACT_PIX / 2 : FUSED_ACT_PIX; }

__global__ void __launch_bounds__(FUSED_THREADS, 1)
fused_resnet_kernel(const uint8_t* __restrict__ images, int img_h, int img_w, const FusedLayer* __restrict__ layers,
                    int n_layers, const FusedHead head, float* __restrict__ logits, uint8_t* __restrict__ trace,
                    long long trace_stride) {
    extern __shared__ uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t w_bar[2], mma_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int fc_codes[64];
    __shared__ float s_cs[64], s_cb[64], s_pcs[64], s_pcb[64];    // per-channel terms of the layer / of the held projection
    __shared__ float s_proj_S;
    __shared__ int s_proj_flags;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int img = blockIdx.x;
    uint8_t* base = dyn_smem + ((1024u - (smem_u32(dyn_smem) & 1023u)) & 1023u);
    uint8_t* acts = base;                                        // three strips
    uint8_t* wbuf = base + 3 * FUSED_ACT_BYTES;                  // two weight images
    volatile int* abortp = &abort_flag;

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(&w_bar[0], 1);
        mbar_init(&w_bar[1], 1);
        mbar_init(&mma_bar, 4);                                   // the four issuing threads
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_slot)),
                     "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    // all strips start as zeros (padding positions are never written with anything else)
    for (int i = tid; i < 3 * FUSED_ACT_BYTES / 16; i += FUSED_THREADS) reinterpret_cast<uint4*>(acts)[i] = make_uint4(0, 0, 0, 0);
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const uint32_t tmem_base = tmem_slot;

    auto fetch_weights = [&](int li) {                           // one thread: the whole byte image of layer li
        const FusedLayer& L = layers[li];
        const int cw = (L.c_in + 31) >> 5, co16 = (L.c_out + 15) & ~15;
        const uint32_t bytes = (uint32_t)(L.k * L.k * cw * co16 * 32);
        mbar_arrive_expect_tx(&w_bar[li & 1], bytes);
        bulk_copy_g2s(wbuf + (li & 1) * FUSED_W_BYTES, L.w8, bytes, &w_bar[li & 1]);
    };
    if (tid == 0 && n_layers > 0) fetch_weights(0);

    // ---- the image: u8 NHWC, 3 channels -> bytes of strip 0 in the padded frame (channel c is byte 4c of word 0)
    {
        const int Wp = img_w + 2;
        const uint8_t* src = images + (size_t)img * img_h * img_w * 3;
        for (int pix = tid; pix < img_h * img_w; pix += FUSED_THREADS) {
            const int h = pix / img_w, w = pix - h * img_w;
            const uint32_t r = src[pix * 3], g = src[pix * 3 + 1], b = src[pix * 3 + 2];
            uint32_t* dst = reinterpret_cast<uint32_t*>(strip_ptr(acts, 0) + ((h + 1) * Wp + (w + 1)) * 16);
            dst[0] = r; dst[1] = g; dst[2] = b;                   // words 0..2 of the first 16-byte half: channels 0, 1, 2
        }
    }
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    __syncthreads();

    bool ok = true;
    int mma_phase = 0;
    float* pool_scratch = reinterpret_cast<float*>(strip_ptr(acts, 0));      // [pixels][c_out] of the last layer

    for (int li = 0; li < n_layers && ok; ++li) {
        const FusedLayer L = layers[li];
        const int cw = (L.c_in + 31) >> 5, co16 = (L.c_out + 15) & ~15;
        const int Ho = L.stride == 2 ? L.h_in / 2 : L.h_in, Wo = L.stride == 2 ? L.w_in / 2 : L.w_in;
        // frame in which the MMAs run: the padded input for a 3x3 layer, the padded OUTPUT frame for the projection
        const int Hf = L.k == 3 ? L.h_in + 2 : Ho + 2, Wf = L.k == 3 ? L.w_in + 2 : Wo + 2;
        const int frame = Hf * Wf;
        const int tiles = (frame + UMMA_M - 1) / UMMA_M;
        const int acc_stride = co16 > 32 ? co16 : 32;
        const int col0 = L.hold ? FUSED_HOLD_COL : 0;

        const int Wp_out = Wo + 2;                                 // frame of the destination strip
        const int cap_in = strip_cap(L.c_in), cap_out = strip_cap(L.c_out);   // pixels per word of the strips read / written
        uint8_t* src_strip = strip_ptr(acts, L.src);
        uint8_t* dst_strip = L.dst >= 0 ? strip_ptr(acts, L.dst) : nullptr;

        if (tid == 0 && li + 1 < n_layers) fetch_weights(li + 1);  // its buffer was last read by layer li-1, finished
        if (tid < 64) {                                            // per-channel terms -> shared memory (read by every row)
            const bool in = tid < L.c_out;
            s_cs[tid] = (L.ch_scale && in) ? __ldg(L.ch_scale + tid) : 1.0f;
            s_cb[tid] = (L.ch_bias && in) ? __ldg(L.ch_bias + tid) : 0.0f;
            if (L.res == 2) {
                const FusedLayer& P = layers[li - 1];              // the projection whose accumulators are held
                s_pcs[tid] = (P.ch_scale && in) ? __ldg(P.ch_scale + tid) : 1.0f;
                s_pcb[tid] = (P.ch_bias && in) ? __ldg(P.ch_bias + tid) : 0.0f;
                if (tid == 0) { s_proj_S = P.S; s_proj_flags = (P.ch_scale ? 1 : 0) | (P.ch_bias ? 2 : 0); }
            }
        }

        if (L.k == 1) {
            // projection: its input is the stride-2 subsample of strip src, copied into strip dst in the output frame
            for (int i = tid; i < FUSED_ACT_BYTES / 16; i += FUSED_THREADS)
                reinterpret_cast<uint4*>(dst_strip)[i] = make_uint4(0, 0, 0, 0);
            __syncthreads();
            const int Wp_in = L.w_in + 2;
            for (int e = tid; e < Ho * Wo * cw * 2; e += FUSED_THREADS) {
                const int half = e & 1, rest = e >> 1, wd = rest % cw, pix = rest / cw;
                const int ho = pix / Wo, wo = pix - ho * Wo;
                const uint8_t* s = src_strip + wd * cap_in * 32 + half * cap_in * 16 + ((2 * ho + 1) * Wp_in + 2 * wo + 1) * 16;
                uint8_t* d = dst_strip + wd * cap_in * 32 + half * cap_in * 16 + ((ho + 1) * Wf + wo + 1) * 16;
                *reinterpret_cast<uint4*>(d) = *reinterpret_cast<const uint4*>(s);
            }
        } else if (L.zero_dst && dst_strip) {
            for (int i = tid; i < FUSED_ACT_BYTES / 16; i += FUSED_THREADS)
                reinterpret_cast<uint4*>(dst_strip)[i] = make_uint4(0, 0, 0, 0);
        }
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
        __syncthreads();

        // ---- MMAs of the whole layer
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        if (lane == 0 && warp < 4 && mbar_wait_bounded(&w_bar[li & 1], (uint32_t)((li >> 1) & 1), abortp)) {
            // Four threads issue (lane 0 of warps 0-3, tiles dealt round-robin): the issue loop of one thread,
            // not the tensor core, bounds a layer of many small MMAs.  Descriptors are built once and advanced
            // by additions (start addresses are in 16-byte units).  Each thread's commit arrives once.
            if (warp < tiles) {
                const uint32_t idesc = umma_idesc_i8(co16);
                const uint8_t* a_src = L.k == 1 ? dst_strip : src_strip;   // the projection reads its subsampled copy
                const uint64_t da0 = umma_desc_interleaved(smem_u32(a_src), (uint32_t)(cap_in * 16));
                uint64_t db = umma_desc_sw32(smem_u32(wbuf + (li & 1) * FUSED_W_BYTES));
                const uint64_t db_step = (uint64_t)((co16 * 32) >> 4), db_word = db_step * (uint64_t)cw;
                for (int wd = 0; wd < cw; ++wd) {
                    const uint64_t da_w = da0 + (uint64_t)(wd * cap_in * 2);   // one word = cap_in * 32 bytes
                    uint64_t db_t = db + db_step * (uint64_t)wd;                // weight tiles are ordered [tap][word]
                    for (int r = 0; r < L.k; ++r) {
                        for (int s = 0; s < L.k; ++s, db_t += db_word) {
                            const int shift = L.k == 3 ? r * Wf + s : Wf + 1;    // 1x1: the centre of the output frame
                            const uint32_t acc_flag = (wd | r | s) != 0 ? 1u : 0u;
                            uint64_t da = da_w + (uint64_t)(warp * UMMA_M + shift);
                            uint32_t tm = tmem_base + (uint32_t)(col0 + warp * acc_stride);
                            for (int t = warp; t < tiles; t += 4, da += 4 * UMMA_M, tm += 4 * acc_stride)
                                umma_i8(tm, da, db_t, idesc, acc_flag);
                        }
                    }
                }
                umma_commit(&mma_bar);
            } else {
                mbar_arrive(&mma_bar);
            }
        }
        // one warp polls for the MMAs' completion; the others sleep in the block barrier instead of spinning
        if (warp == 4) mbar_wait_bounded(&mma_bar, (uint32_t)(mma_phase & 1), abortp);
        __syncthreads();
        if (abort_flag != 0) { ok = false; break; }
        ++mma_phase;
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");

        // ---- epilogue (a held projection has none: the next layer reads its accumulators)
        if (!L.hold) {
            const int qmax = (1 << L.out_bits) - 1;
            const int quarter = warp & 3;
            const bool has_cs = L.ch_scale != nullptr, has_cb = L.ch_bias != nullptr;
            const bool p_cs = s_proj_flags & 1, p_cb = s_proj_flags & 2;
            const float S = L.S, inv_step = L.out_inv_step, res_step = L.res_step, PS = s_proj_S;
            // a unit of work is (tile, 16 channels); the four warps of a TMEM lane quarter take units in turn
            const int nb16 = co16 >> 4, units = tiles * nb16;
            for (int u = warp >> 2; u < units; u += FUSED_THREADS / 128) {
                const int t = u / nb16, c0 = (u - t * nb16) << 4;
                const int f = t * UMMA_M + quarter * 32 + lane;
                const int hp = f / Wf, wp = f - hp * Wf;
                // does this frame row have an output, and where does it go in the destination frame
                bool valid = f < frame;
                int ho = hp, wo = wp;
                if (L.stride == 2) { valid = valid && !(hp & 1) && !(wp & 1); ho = hp >> 1; wo = wp >> 1; }
                valid = valid && ho < Ho && wo < Wo;
                const int target = L.stride == 2 ? (ho + 1) * Wp_out + wo + 1 : f + Wf + 1;
                const bool in_frame = f < frame && (L.stride == 1 || valid);   // stride 1 also writes the zeros of the padding
                const uint32_t trow = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(col0 + t * acc_stride);
                const uint32_t prow = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(FUSED_HOLD_COL + t * acc_stride);
                const int lane0 = (c0 & 16) >> 3;                        // byte lane of channels c0 .. c0+7 in words 0..7
                uint32_t resw[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};      // the identity shortcut's word at the same pixel
                if (L.res == 1 && valid) {
                    const uint8_t* rp = strip_ptr(acts, L.res_buf) + (c0 >> 5) * cap_out * 32 + target * 16;
                    const uint4 a = *reinterpret_cast<const uint4*>(rp), b = *reinterpret_cast<const uint4*>(rp + cap_out * 16);
                    resw[0] = a.x; resw[1] = a.y; resw[2] = a.z; resw[3] = a.w;
                    resw[4] = b.x; resw[5] = b.y; resw[6] = b.z; resw[7] = b.w;
                }
                uint32_t v[16], pv[16];
                tmem_ld16(trow + (uint32_t)c0, v);                      // whole warp, also for rows without an output
                if (L.res == 2) tmem_ld16(prow + (uint32_t)c0, pv);
                int q[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const int c = c0 + e;
                    float y = __fmul_rn((float)(int)v[e], S);
                    if (has_cs) y = __fmul_rn(y, s_cs[c]);
                    if (has_cb) y = __fadd_rn(y, s_cb[c]);
                    if (L.res == 2) {                               // projection shortcut: its own scale and per-channel terms
                        float r = __fmul_rn((float)(int)pv[e], PS);
                        if (p_cs) r = __fmul_rn(r, s_pcs[c]);
                        if (p_cb) r = __fadd_rn(r, s_pcb[c]);
                        y = __fadd_rn(y, r);
                    }
                    if (L.res == 1)                                 // identity shortcut: channel 8 i + k is byte i of word k
                        y = __fadd_rn(y, __fmul_rn(res_step, (float)((resw[e & 7] >> (8 * (lane0 + (e >> 3)))) & 0xFFu)));
                    if (L.relu && !(y > 0.0f)) y = 0.0f;
                    int code = 0;
                    if (valid && c < L.c_out) {
                        if (L.dst < 0) pool_scratch[(ho * Wo + wo) * L.c_out + c] = y;
                        else code = min(__float2int_rd(__fadd_rn(__fmul_rn(y, inv_step), 0.5f)), qmax);
                    }
                    q[e] = code;
                }
                if (L.dst >= 0 && in_frame) {
                    // word k of the pixel holds channels k, 8+k, 16+k, 24+k as bytes: these 16 channels are two
                    // adjacent bytes of each of the eight words (negative codes saturate to 0)
                    uint8_t* wp_ = dst_strip + (c0 >> 5) * cap_out * 32 + target * 16 + lane0;
#pragma unroll
                    for (int k8 = 0; k8 < 8; ++k8) {
                        uint32_t two;
                        asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;\n" : "=r"(two) : "r"(q[8 + k8]), "r"(q[k8]), "r"(0));
                        *reinterpret_cast<uint16_t*>(wp_ + (k8 >> 2) * cap_out * 16 + (k8 & 3) * 4) = (uint16_t)two;
                    }
                    if (trace && L.trace_off >= 0 && valid) {
                        uint8_t* tp = trace + (size_t)img * trace_stride + L.trace_off + (size_t)(ho * Wo + wo) * L.c_out + c0;
#pragma unroll
                        for (int e = 0; e < 16; ++e)
                            if (c0 + e < L.c_out) tp[e] = (uint8_t)max(q[e], 0);
                    }
                }
            }
        }
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
        __syncthreads();
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    }
    // ---- pooling, 8-bit quantization, classifier
    if (ok && !abort_flag && n_layers > 0) {
        const FusedLayer L = layers[n_layers - 1];
        const int Ho = L.stride == 2 ? L.h_in / 2 : L.h_in, Wo = L.stride == 2 ? L.w_in / 2 : L.w_in;
        const int hw = Ho * Wo, C = L.c_out;
        if (tid < C && tid < 64) {
            float acc = 0.0f;
            for (int p = 0; p < hw; ++p) acc = __fadd_rn(acc, pool_scratch[p * C + tid]);
            const float m = __fmul_rn(acc, 1.0f / (float)hw);
            fc_codes[tid] = quantize_act_code(m, head.a_inv_step, 255);
        }
        __syncthreads();
        if (tid < head.c_out) {
            const int co16 = (head.c_out + 15) & ~15, cwf = (head.c_in + 31) >> 5;
            int acc = 0;
            for (int c = 0; c < head.c_in; ++c) {
                const int wd = c >> 5, cc = c & 31, j = 4 * (cc & 7) + (cc >> 3);      // byte 4b + i of the row
                const int jj = j ^ (((tid >> 2) & 1) << 4);                               // halves swapped for these rows
                const int8_t wv = (int8_t)head.w8[((size_t)wd * co16 + tid) * 32 + jj];
                acc += (int)wv * fc_codes[c];
            }
            (void)cwf;
            float y = __fmul_rn((float)acc, head.S);
            if (head.ch_scale) y = __fmul_rn(y, __ldg(head.ch_scale + tid));
            if (head.ch_bias) y = __fadd_rn(y, __ldg(head.ch_bias + tid));
            logits[(size_t)img * head.c_out + tid] = y;
        }
    }
    if (abort_flag != 0 && tid == 0) atomicAdd(&g_umma_timeouts, 1ull);

    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// Limits of the kernel for one layer; returns EBS_OK or the reason it cannot run.
static int check_layer(const FusedLayer& L, const FusedLayer* prev) {
    if (!L.w8 || (L.k != 1 && L.k != 3) || (L.stride != 1 && L.stride != 2)) return EBS_ERR_INVALID_ARG;
    if (L.c_in < 1 || L.c_in > 64 || L.c_out < 1 || L.c_out > 64 || L.h_in < 1 || L.w_in < 1) return EBS_ERR_UNSUPPORTED;
    if (L.k == 1 && (L.stride != 2 || !L.hold)) return EBS_ERR_UNSUPPORTED;        // 1x1 only as the strided projection
    if (L.stride == 2 && ((L.h_in | L.w_in) & 1)) return EBS_ERR_UNSUPPORTED;
    if (L.src < 0 || L.src > 2 || L.dst < -1 || L.dst > 2 || (L.hold && L.dst < 0)) return EBS_ERR_INVALID_ARG;
    if (L.res < 0 || L.res > 2 || (L.res == 1 && (L.res_buf < 0 || L.res_buf > 2))) return EBS_ERR_INVALID_ARG;
    if (L.res == 2 && (!prev || !prev->hold || prev->c_out != L.c_out)) return EBS_ERR_INVALID_ARG;
    if (L.dst >= 0 && !L.hold && (L.out_bits < 1 || L.out_bits > 8 || !(L.out_inv_step > 0.0f))) return EBS_ERR_INVALID_ARG;
    const int Ho = L.stride == 2 ? L.h_in / 2 : L.h_in, Wo = L.stride == 2 ? L.w_in / 2 : L.w_in;
    const int Hf = L.k == 3 ? L.h_in + 2 : Ho + 2, Wf = L.k == 3 ? L.w_in + 2 : Wo + 2;
    const int tiles = (Hf * Wf + UMMA_M - 1) / UMMA_M, co16 = (L.c_out + 15) & ~15, cw = (L.c_in + 31) >> 5;
    if (tiles * UMMA_M + 2 * Wf + 2 > strip_cap(L.c_in)) return EBS_ERR_UNSUPPORTED;          // rows the MMAs read
    if (L.dst >= 0 && !L.hold && (Ho + 2) * (Wo + 2) + Wo + 3 > strip_cap(L.c_out)) return EBS_ERR_UNSUPPORTED;   // rows written
    if ((L.hold ? FUSED_HOLD_COL : 0) + tiles * (co16 > 32 ? co16 : 32) > (L.hold ? 512 : FUSED_HOLD_COL)) return EBS_ERR_UNSUPPORTED;
    if (L.k * L.k * cw * co16 * 32 > FUSED_W_BYTES) return EBS_ERR_UNSUPPORTED;
    if (L.dst < 0 && Ho * Wo * L.c_out * 4 > FUSED_ACT_BYTES) return EBS_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(L.w8) & 15u) != 0) return EBS_ERR_INVALID_ARG;
    return EBS_OK;
}

int fused_plan_upload(const void* layers_host, int n_layers, void* layers_dev, cudaStream_t st) {
    const FusedLayer* L = static_cast<const FusedLayer*>(layers_host);
    for (int i = 0; i < n_layers; ++i) {
        const int rc = check_layer(L[i], i > 0 ? &L[i - 1] : nullptr);
        if (rc) return rc;
    }
    if (L[0].c_in > 4 || L[0].src != 0) return EBS_ERR_UNSUPPORTED;                   // the image goes to strip 0, <= 4 channels
    if (L[n_layers - 1].dst != -1 || L[n_layers - 1].c_out > 64) return EBS_ERR_INVALID_ARG;
    return check_cuda(cudaMemcpyAsync(layers_dev, layers_host, (size_t)n_layers * sizeof(FusedLayer), cudaMemcpyHostToDevice, st));
}

int launch_fused_resnet(const uint8_t* images, int n, int img_h, int img_w, const void* layers_dev, int n_layers,
                        const void* head_host, float* logits, uint8_t* trace, long long trace_stride, cudaStream_t st) {
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (check_cuda(cudaFuncSetAttribute(fused_resnet_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FUSED_SMEM)))
            return EBS_ERR_CUDA;
        attr_set[dev] = true;
    }
    FusedHead head;
    memcpy(&head, head_host, sizeof(head));
    fused_resnet_kernel<<<n, FUSED_THREADS, FUSED_SMEM, st>>>(images, img_h, img_w, static_cast<const FusedLayer*>(layers_dev),
                                                               n_layers, head, logits, trace, trace_stride);
    return check_cuda(cudaGetLastError());
}

unsigned long long fused_net_timeouts() {
    unsigned long long v = 0;
    cudaMemcpyFromSymbol(&v, g_umma_timeouts, sizeof(v));
    return v;
}

int fused_layer_bytes() { return (int)sizeof(FusedLayer); }
int fused_head_bytes() { return (int)sizeof(FusedHead); }

}  // namespace ebs

