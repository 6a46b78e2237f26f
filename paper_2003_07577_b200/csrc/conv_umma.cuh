// Implicit-GEMM bit-plane convolution on the 5th-generation tensor cores (tcgen05.mma kind::i8,
// accumulator in tensor memory), sm_100a.
//
// Same arithmetic as conv_mma_kernel.  The plane-pair sum of the binary decomposition,
//     sum_m sum_k c_m 2^(m+k) * bitcount(AND(activation plane k, weight plane m)),
// regroups channel by channel into (sum_k 2^k a_k) * (sum_m c_m 2^m w_m): the expanders merge the
// planes of a packed word back into one byte per channel (the activation code as u8, the weight code
// as two's-complement s8, the top plane supplying the sign extension), and ONE int8 MMA per reduction
// word then retires all Wb*Ab plane pairs of its 32 channels into one int32 accumulator per output.
// An MMA covers 128 output pixels x TILE_N channels x 32 channels of one tap, reads both operands
// from shared memory and accumulates in tensor memory (TMEM).  Operands stay bit planes in global
// memory; bytes exist only in shared memory.
//
// A CTA owns 128 consecutive output pixels x TILE_N channels and has 9 warps:
//   warps 0-7 (expanders)  load packed words ahead into registers and expand them into 32-byte rows of
//      K-major, 32-byte-swizzled shared tiles (one tile per reduction word; byte 4b+i of a row <- bit
//      8i+b of the words, the same map for both operands): threads t and t+128 build the two 16-byte
//      halves of pixel row t, and the weight rows are dealt out over all 256 threads; then
//      fence.proxy.async and arrive on the stage's "full" mbarrier;
//   warp 8 (issuer)        waits for "full", issues one tcgen05.mma per reduction word and a
//      tcgen05.commit that arrives on the stage's "empty" mbarrier once the tensor core has read the
//      stage.
// Two stages, so expansion of the next reduction words overlaps the MMAs of the current ones.
// Epilogue: tcgen05.ld gives every expander thread accumulators of its pixel (warps w and w+4 split
// the channels); it stores them, applies the fp32 steps and packs the requantized codes of its pixel
// into plane words in registers.
//
// Every wait on an mbarrier is bounded; on a timeout the CTA raises a shared abort flag, all its
// loops end, it records the event in a device counter, frees its tensor memory and returns.
#pragma once

#include "ebs_internal.cuh"

namespace ebs {

constexpr int UMMA_KTAB = 256;          // reduction words the in-kernel tap table can hold
constexpr int UMMA_M = 128;             // pixels per CTA = TMEM lanes
constexpr unsigned UMMA_WAIT_LIMIT = 1u << 20;

static __device__ unsigned long long g_umma_timeouts = 0ull;   // CTAs that gave up waiting (0 in a healthy run)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait for the phase with the given parity; false = gave up (or another thread already had).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                  unsigned limit = UMMA_WAIT_LIMIT) {
    const uint32_t addr = smem_u32(bar);
    for (unsigned it = 0; it < limit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}\n"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if (*abort_flag) return false;
        __nanosleep(it < 8 ? 40 : 200);   // leave the issue slots to the warps that have work
    }
    *abort_flag = 1;
    return false;
}
// The same wait for the single warps that feed the tensor core (issuer, weight producer): no sleep between polls (the
// try_wait itself suspends the thread for a while), so that they react as soon as the barrier flips.
__device__ __forceinline__ bool mbar_wait_bounded_hot(uint64_t* bar, uint32_t parity, volatile int* abort_flag, unsigned limit) {
    const uint32_t addr = smem_u32(bar);
    for (unsigned it = 0; it < limit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}\n"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

// Shared-memory matrix descriptor: K-major operand, 32-byte swizzle, rows of 32 bytes (K = 32 int8),
// 8-row groups 256 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw32(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);     // start address, 16-byte units
    d |= (uint64_t)1u << 16;                         // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(256u >> 4) << 32;                // stride byte offset between 8-row groups
    d |= (uint64_t)1u << 46;                         // descriptor version of this architecture
    d |= (uint64_t)6u << 61;                         // layout type: 32-byte swizzle
    return d;
}

// Instruction descriptor: D = s32, A = u8 (activations), B = s8 (weights), both K-major, M = 128.
__host__ __device__ constexpr uint32_t umma_idesc_i8(int n) {
    return (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(UMMA_M >> 4) << 24);
}

__device__ __forceinline__ void umma_i8(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                        uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}\n"
        :: "r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}

// Address of 16-byte chunk c (0/1) of row `row` in a 32-byte-swizzled tile (tile base 256-byte aligned).
__device__ __forceinline__ uint8_t* sw32_chunk(uint8_t* tile, int row, int c) {
    return tile + row * 32 + ((c ^ ((row >> 2) & 1)) << 4);
}

// The two halves of a tensor-memory load: issue, and later wait.  The wait names the destination registers
// as read-write operands so that no use of them is scheduled before it.
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld16_wait(uint32_t (&v)[16]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;\n"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
                 :: "memory");
}

// Four integers -> four bytes a | b << 8 | c << 16 | d << 24, each saturated to 0 .. 255.
__device__ __forceinline__ uint32_t pack_sat_u8x4(int a, int b, int c, int d) {
    uint32_t hi, out;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;\n" : "=r"(hi) : "r"(d), "r"(c), "r"(0));
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;\n" : "=r"(out) : "r"(b), "r"(a), "r"(hi));
    return out;
}

// Epilogue straight out of tensor memory.  Warp w reads TMEM lanes 32 * (w % 4) .. + 31: thread `lane`
// of it owns the accumulators of one pixel row (global output pixel gp; pvalid false = row without an
// output).  Warps w and w + 4 split the channels when the tile is wide enough.  The thread stores the
// accumulators, applies the fp32 steps and packs the requantized codes of its pixel into plane words.
// AFFINE = false compiles the straight-line path without per-channel terms and shortcuts (layers that have
// them then take the general path); kernels that are built in both forms pick the form on the host, so the
// extra registers of the terms do not lower the occupancy of layers without them.
template <int TILE_N, bool AFFINE = false>
__device__ __forceinline__ void umma_epilogue(const ConvParams& p, uint32_t tmem_base, int warp, int gp, bool pvalid,
                                              int wsum_row, int co0) {
    constexpr int EPI_WARPS = TILE_N >= 64 ? 8 : 4;
    constexpr int COLS_PER_WARP = TILE_N >= 64 ? TILE_N / 2 : TILE_N;
    if (warp < EPI_WARPS) {
        const bool want_y = p.y != nullptr, want_q = p.packed_next != nullptr;
        const int qmax = (1 << p.next_bits) - 1;
        const bool vec_ok = (p.Co & 3) == 0;                        // 16-byte aligned groups of four channels
        const uint32_t trow = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const int hw = p.Ho * p.Wo;
        const int img = pvalid ? gp / hw : 0, rem = pvalid ? gp - img * hw : 0;
        const int cbeg = (warp >> 2) * COLS_PER_WARP;
        // Common case -- the whole channel tile exists, channels in aligned groups of four, no per-channel
        // terms, no shortcut, NHWC: straight-line code, 32 channels (one packed output word) per round.
        const bool terms_aligned = (((uintptr_t)p.ch_scale | (uintptr_t)p.ch_bias) & 15u) == 0;
        const bool no_terms = !p.ch_scale && !p.ch_bias && !p.residual && !p.res_packed;
        if (COLS_PER_WARP % 32 == 0 && co0 + TILE_N <= p.Co && vec_ok && !p.y_nchw &&
            (AFFINE ? terms_aligned : no_terms)) {
            const int nb = want_q ? p.next_bits : 0;
            const float S = p.S, inv_next = p.inv_next;
            const bool relu = p.relu != 0, w_levels = p.w_levels != 0;
            // 16 channels of this thread's pixel: store, fp32 steps, requantize, shift their plane bits into `planes`
            uint32_t resw[8];                                   // shortcut planes of the current 32-channel word
            auto process16 = [&](uint32_t (&v)[16], int cbase, uint32_t (&planes)[8]) {
                if (w_levels) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) v[e] = (uint32_t)(2 * (int)v[e] + wsum_row);
                }
                const size_t o = (size_t)gp * p.Co + co0 + cbase;
                if (p.acc && pvalid) {
#pragma unroll
                    for (int gq = 0; gq < 4; ++gq)
                        *reinterpret_cast<int4*>(p.acc + o + 4 * gq) =
                            make_int4((int)v[4 * gq], (int)v[4 * gq + 1], (int)v[4 * gq + 2], (int)v[4 * gq + 3]);
                }
                if (want_y || want_q) {
                    float y[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) y[e] = __fmul_rn((float)(int)v[e], S);
                    if (AFFINE && p.ch_scale) {                 // the same 16 values for every lane: broadcast vector loads
#pragma unroll
                        for (int gq = 0; gq < 4; ++gq) {
                            const float4 t = __ldg(reinterpret_cast<const float4*>(p.ch_scale + co0 + cbase) + gq);
                            y[4 * gq] = __fmul_rn(y[4 * gq], t.x); y[4 * gq + 1] = __fmul_rn(y[4 * gq + 1], t.y);
                            y[4 * gq + 2] = __fmul_rn(y[4 * gq + 2], t.z); y[4 * gq + 3] = __fmul_rn(y[4 * gq + 3], t.w);
                        }
                    }
                    if (AFFINE && p.ch_bias) {
#pragma unroll
                        for (int gq = 0; gq < 4; ++gq) {
                            const float4 t = __ldg(reinterpret_cast<const float4*>(p.ch_bias + co0 + cbase) + gq);
                            y[4 * gq] = __fadd_rn(y[4 * gq], t.x); y[4 * gq + 1] = __fadd_rn(y[4 * gq + 1], t.y);
                            y[4 * gq + 2] = __fadd_rn(y[4 * gq + 2], t.z); y[4 * gq + 3] = __fadd_rn(y[4 * gq + 3], t.w);
                        }
                    }
                    if (AFFINE && p.residual && pvalid) {
#pragma unroll
                        for (int gq = 0; gq < 4; ++gq) {
                            const float4 t = __ldg(reinterpret_cast<const float4*>(p.residual + o) + gq);
                            y[4 * gq] = __fadd_rn(y[4 * gq], t.x); y[4 * gq + 1] = __fadd_rn(y[4 * gq + 1], t.y);
                            y[4 * gq + 2] = __fadd_rn(y[4 * gq + 2], t.z); y[4 * gq + 3] = __fadd_rn(y[4 * gq + 3], t.w);
                        }
                    }
                    if (AFFINE && p.res_packed) {               // shortcut codes from packed planes: bit i of a nibble -> byte i
                        const int sh = cbase & 16;
#pragma unroll
                        for (int gq = 0; gq < 4; ++gq) {
                            uint32_t c4r = 0u;
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                if (j >= p.res_bits) break;
                                c4r |= ((((resw[j] >> (sh + 4 * gq)) & 0xFu) * 0x00204081u) & 0x01010101u) << j;
                            }
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                y[4 * gq + e] = __fadd_rn(y[4 * gq + e],
                                                          __fmul_rn(p.res_scale, (float)((c4r >> (8 * e)) & 0xFFu)));
                        }
                    }
                    if (relu) {
#pragma unroll
                        for (int e = 0; e < 16; ++e) y[e] = y[e] > 0.0f ? y[e] : 0.0f;
                    }
                    if (want_y && pvalid) {
#pragma unroll
                        for (int gq = 0; gq < 4; ++gq)
                            *reinterpret_cast<float4*>(p.y + o + 4 * gq) =
                                make_float4(y[4 * gq], y[4 * gq + 1], y[4 * gq + 2], y[4 * gq + 3]);
                    }
                    if (want_q) {
#pragma unroll
                        for (int gq = 3; gq >= 0; --gq) {
                            // codes of four channels as bytes: floor(y / step + 0.5), at most qmax; the pack
                            // instruction saturates at 0 (negative values, and NaN converts to 0)
                            int q[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                q[e] = min(__float2int_rd(__fadd_rn(__fmul_rn(y[4 * gq + e], inv_next), 0.5f)), qmax);
                            const uint32_t c4 = pack_sat_u8x4(q[0], q[1], q[2], q[3]);
                            // plane j of the four codes -> the top nibble of a product, shifted into the plane word
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                if (j >= nb) break;
                                const uint32_t bits = j <= 4 ? (c4 & (0x01010101u << j)) * (0x10204080u >> j)
                                                             : ((c4 >> j) & 0x01010101u) * 0x10204080u;
                                planes[j] = __funnelshift_l(bits, planes[j], 4);
                            }
                        }
                    }
                }
            };
            // the load of the next 16 channels is in flight while the current ones are processed; the upper
            // half of a 32-channel word comes first because the plane words grow by shifting left
            uint32_t va[16], vb[16];
            tmem_ld16_issue(trow + (uint32_t)(cbeg + 16), va);     // whole warp, also for rows past the end
#pragma unroll 1
            for (int c0 = cbeg; c0 < cbeg + COLS_PER_WARP; c0 += 32) {
                uint32_t planes[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
                if (AFFINE && p.res_packed) {
                    const uint32_t* rw = p.res_packed + ((size_t)gp * p.CWo + ((co0 + c0) >> 5)) * p.res_bits;
#pragma unroll
                    for (int j = 0; j < 8; ++j) resw[j] = (pvalid && j < p.res_bits) ? __ldg(rw + j) : 0u;
                }
                tmem_ld16_wait(va);
                tmem_ld16_issue(trow + (uint32_t)c0, vb);
                process16(va, c0 + 16, planes);
                tmem_ld16_wait(vb);
                if (c0 + 32 < cbeg + COLS_PER_WARP) tmem_ld16_issue(trow + (uint32_t)(c0 + 48), va);
                process16(vb, c0, planes);
                if (want_q && pvalid) {
                    uint32_t* dst = p.packed_next + ((size_t)gp * p.CWo + ((co0 + c0) >> 5)) * nb;
                    if (nb == 4) {
                        *reinterpret_cast<uint4*>(dst) = make_uint4(planes[0], planes[1], planes[2], planes[3]);
                    } else if (nb == 8) {
                        *reinterpret_cast<uint4*>(dst) = make_uint4(planes[0], planes[1], planes[2], planes[3]);
                        *reinterpret_cast<uint4*>(dst + 4) = make_uint4(planes[4], planes[5], planes[6], planes[7]);
                    } else if (nb == 2) {
                        *reinterpret_cast<uint2*>(dst) = make_uint2(planes[0], planes[1]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            if (j >= nb) break;
                            dst[j] = planes[j];
                        }
                    }
                }
            }
            return;
        }
        uint32_t planes[8];
#pragma unroll 1
        for (int c0 = cbeg; c0 < cbeg + COLS_PER_WARP; c0 += 16) {
            uint32_t v[16];
            tmem_ld16(trow + (uint32_t)c0, v);                       // whole warp, also for rows past the end
            if (p.w_levels) {
#pragma unroll
                for (int e = 0; e < 16; ++e) v[e] = (uint32_t)(2 * (int)v[e] + wsum_row);
            }
            if ((c0 & 31) == 0) {
#pragma unroll
                for (int j = 0; j < 8; ++j) planes[j] = 0u;
            }
#pragma unroll
            for (int gq = 0; gq < 4; ++gq) {                          // four channels at a time
                const int co = co0 + c0 + 4 * gq;
                uint32_t code4 = 0u;
                float yv[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int a = (int)v[4 * gq + e];
                    float y = __fmul_rn((float)a, p.S);
                    if (co + e < p.Co) {
                        if (p.ch_scale) y = __fmul_rn(y, __ldg(p.ch_scale + co + e));
                        if (p.ch_bias) y = __fadd_rn(y, __ldg(p.ch_bias + co + e));
                        if (p.residual && pvalid) y = __fadd_rn(y, __ldg(p.residual + (size_t)gp * p.Co + co + e));
                        if (p.res_packed && pvalid) y = __fadd_rn(y, packed_residual(p, gp, co + e));
                    }
                    if (p.relu && !(y > 0.0f)) y = 0.0f;
                    yv[e] = y;
                    if (want_q && co + e < p.Co) code4 |= (uint32_t)quantize_act_code(y, p.inv_next, qmax) << (8 * e);
                }
                if (pvalid && co < p.Co) {
                    const size_t o = (size_t)gp * p.Co + co;
                    if (p.acc) {
                        if (vec_ok) *reinterpret_cast<int4*>(p.acc + o) =
                            make_int4((int)v[4 * gq], (int)v[4 * gq + 1], (int)v[4 * gq + 2], (int)v[4 * gq + 3]);
                        else
                            for (int e = 0; e < 4 && co + e < p.Co; ++e) p.acc[o + e] = (int)v[4 * gq + e];
                    }
                    if (want_y) {
                        if (p.y_nchw) {
                            for (int e = 0; e < 4 && co + e < p.Co; ++e)
                                p.y[((size_t)img * p.Co + co + e) * hw + rem] = yv[e];
                        } else if (vec_ok) {
                            *reinterpret_cast<float4*>(p.y + o) = make_float4(yv[0], yv[1], yv[2], yv[3]);
                        } else {
                            for (int e = 0; e < 4 && co + e < p.Co; ++e) p.y[o + e] = yv[e];
                        }
                    }
                }
                if (want_q) {
                    const int nib_pos = ((c0 & 16) >> 2) + gq;          // which nibble of the 32-channel word
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j < p.next_bits)
                            planes[j] |= ((((code4 >> j) & 0x01010101u) * 0x01020408u) >> 24) << (4 * nib_pos);
                }
            }
            const bool word_done = ((c0 & 16) != 0) || (c0 + 16 >= TILE_N);
            if (want_q && word_done && pvalid) {
                const int cwg = (co0 + c0) >> 5;
                if (cwg < p.CWo) {
                    uint32_t* dst = p.packed_next + ((size_t)gp * p.CWo + cwg) * p.next_bits;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j < p.next_bits) dst[j] = planes[j];
                }
            }
        }
    }
}

constexpr int UMMA_EXPANDERS = 256;     // threads of warps 0-7
constexpr int UMMA_THREADS = UMMA_EXPANDERS + 32;

constexpr int umma_min(int a, int b) { return a < b ? a : b; }

template <int WB, int AB, int TILE_N>
struct UmmaTile {
    static constexpr int A_TILE_BYTES = UMMA_M * 32;                    // activation codes of one reduction word
    static constexpr int B_TILE_BYTES = TILE_N * 32;                    // weight codes of one reduction word
    static constexpr int KW_BYTES = A_TILE_BYTES + B_TILE_BYTES;
    // reduction words per stage: bounded by shared memory (32 KB a stage) and by the registers that hold
    // the packed words of three chunks in flight (about 16 activation and 16 weight words per chunk)
    static constexpr int KS_SMEM = (32 * 1024) / KW_BYTES;
    static constexpr int KS_A = 16 / AB;
    static constexpr int KS_B = (16 * UMMA_EXPANDERS) / (WB * TILE_N);
    static constexpr int KS_MIN = umma_min(umma_min(KS_SMEM, KS_A), umma_min(KS_B, 4));
    static constexpr int KS = KS_MIN < 1 ? 1 : KS_MIN;
    static constexpr int STAGE_BYTES = KS * KW_BYTES;
    static constexpr int SMEM_BYTES = 2 * STAGE_BYTES + 1024;           // + slack to align the tiles to 1 KB
    static constexpr int TMEM_COLS = TILE_N < 32 ? 32 : TILE_N;
    static constexpr int B_ITEMS = (KS * TILE_N + UMMA_EXPANDERS - 1) / UMMA_EXPANDERS;   // weight rows per thread
    static_assert(TILE_N % 16 == 0 && TILE_N >= 16 && TILE_N <= 256, "tcgen05.mma N for M = 128");
    static_assert((STAGE_BYTES % 256) == 0, "tiles keep the swizzle alignment");
    static_assert(SMEM_BYTES <= 220 * 1024, "shared memory per CTA");
};

template <int WB, int AB, int TILE_N>
__global__ void __launch_bounds__(UMMA_THREADS) conv_umma_kernel(const ConvParams p) {
    using T = UmmaTile<WB, AB, TILE_N>;
    constexpr int KS = T::KS;
    extern __shared__ uint8_t dyn_smem[];
    __shared__ int2 ktab[UMMA_KTAB];
    __shared__ __align__(8) uint64_t full_bar[2];
    __shared__ __align__(8) uint64_t empty_bar[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int wsum_s[2][UMMA_M];          // per pixel row: window sum of the activation codes, one part per half

    const int tid = threadIdx.x, warp = tid >> 5;
    const int tile_p0 = blockIdx.x * UMMA_M;
    const int co0 = blockIdx.y * TILE_N;
    uint8_t* tiles = dyn_smem + ((1024u - (smem_u32(dyn_smem) & 1023u)) & 1023u);
    volatile int* abortp = &abort_flag;

    // ---- set-up: tap table, barriers, tensor memory
    for (int kk = tid; kk < p.KK; kk += UMMA_THREADS) {
        const int tap = kk / p.CW, cw = kk - tap * p.CW;
        const int r = tap / p.kw, s = tap - r * p.kw;
        ktab[kk] = make_int2(((r * p.W + s) * p.CW + cw) * AB, r | (s << 8));
    }
    if (tid == 0) {
        abort_flag = 0;
        mbar_init(&full_bar[0], UMMA_EXPANDERS);
        mbar_init(&full_bar[1], UMMA_EXPANDERS);
        mbar_init(&empty_bar[0], 1);
        mbar_init(&empty_bar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_slot)),
                     "r"((uint32_t)T::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const uint32_t tmem_base = tmem_slot;

    const int kwords = (p.KK + p.fold - 1) / p.fold;          // reduction words after tap folding
    const int nchunks = (kwords + KS - 1) / KS;
    const int row = tid & (UMMA_M - 1);                        // pixel row of an expander thread
    const int gp = tile_p0 + row;

    if (warp < 8) {
        // =========================== expanders ===========================
        const int half = tid >> 7;                             // which 16-byte half of its pixel row it builds
        int pix_off = 0;
        uint32_t row_ok = 0u, col_ok = 0u;
        if (gp < p.P) {
            const int hw = p.Ho * p.Wo;
            const int n = gp / hw, rem = gp - n * hw;
            const int ho = rem / p.Wo, wo = rem - ho * p.Wo;
            const int h0 = ho * p.sh - p.ph, w0 = wo * p.sw - p.pw;
            pix_off = ((n * p.H + h0) * p.W + w0) * p.CW * AB;
            for (int r = 0; r < p.kh; ++r) row_ok |= ((unsigned)(h0 + r) < (unsigned)p.H ? 1u : 0u) << r;
            for (int s = 0; s < p.kw; ++s) col_ok |= ((unsigned)(w0 + s) < (unsigned)p.W ? 1u : 0u) << s;
        }
        uint32_t a_set[3][KS][AB], b_set[3][T::B_ITEMS][WB];   // packed words of three consecutive chunks (ring)

        // per-thread constants of the weight rows it expands: which (reduction word, channel row), where
        // that row starts in global memory (for reduction word 0) and in the stage
        int b_q[T::B_ITEMS], b_goff[T::B_ITEMS], b_soff[T::B_ITEMS];
#pragma unroll
        for (int i = 0; i < T::B_ITEMS; ++i) {
            const int item = tid + i * UMMA_EXPANDERS;
            const int q = item / TILE_N, nrow = item - q * TILE_N;
            const bool live = q < KS && co0 + nrow < p.Co;
            b_q[i] = q < KS ? q : -1;                            // -1: no row (more threads than rows)
            b_goff[i] = live ? (co0 + nrow) * WB : -1;            // -1: channel past c_out -> zero row
            b_soff[i] = KS * T::A_TILE_BYTES + q * T::B_TILE_BYTES + nrow * 32;
        }
        const int a_soff = row * 32 + ((half ^ ((row >> 2) & 1)) << 4);   // this thread's chunk, 32-byte swizzle
        const int co_wb = p.Co * WB;                              // weight words per reduction word

        // packed words of chunk `ch` -> registers (zero past the end, outside the image, past c_out)
        auto load_chunk = [&](int ch, int set) {
            uint32_t (&a_nxt)[KS][AB] = a_set[set];
            uint32_t (&b_nxt)[T::B_ITEMS][WB] = b_set[set];
#pragma unroll
            for (int q = 0; q < KS; ++q) {
                const int kw = ch * KS + q;
#pragma unroll
                for (int k = 0; k < AB; ++k) a_nxt[q][k] = 0u;
                if (kw < kwords) {
                    if (p.fold == 1) {
                        const int2 info = ktab[kw];
                        if ((row_ok >> (info.y & 0xff)) & (col_ok >> (info.y >> 8)) & 1u)
                            load_words_global<AB>(p.x + (pix_off + info.x), a_nxt[q]);
                    } else {
                        for (int f = 0; f < p.fold; ++f) {
                            const int kk = kw * p.fold + f;
                            if (kk >= p.KK) break;
                            const int2 info = ktab[kk];
                            if ((row_ok >> (info.y & 0xff)) & (col_ok >> (info.y >> 8)) & 1u) {
                                uint32_t t[AB];
                                load_words_global<AB>(p.x + (pix_off + info.x), t);
#pragma unroll
                                for (int k = 0; k < AB; ++k) a_nxt[q][k] |= t[k] << (f * p.fold_bits);
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < T::B_ITEMS; ++i) {
#pragma unroll
                for (int m = 0; m < WB; ++m) b_nxt[i][m] = 0u;
                const int kw = ch * KS + b_q[i];
                if (b_q[i] >= 0 && b_goff[i] >= 0 && kw < kwords) {
                    if (p.fold == 1) {
                        load_words_global<WB>(p.w + ((size_t)kw * co_wb + b_goff[i]), b_nxt[i]);
                    } else {
                        for (int f = 0; f < p.fold; ++f) {
                            const int kk = kw * p.fold + f;
                            if (kk >= p.KK) break;
                            uint32_t t[WB];
                            load_words_global<WB>(p.w + ((size_t)kk * co_wb + b_goff[i]), t);
#pragma unroll
                            for (int m = 0; m < WB; ++m) b_nxt[i][m] |= t[m] << (f * p.fold_bits);
                        }
                    }
                }
            }
        };

        // the words of chunks ch+1 and ch+2 are in flight while chunk ch is expanded; the ring index is a
        // compile-time constant after unrolling, so the three sets stay in registers and no pending load is moved
        load_chunk(0, 0);
        if (nchunks > 1) load_chunk(1, 1);
        bool expanders_ok = true;
        int wsum = 0;                                              // this thread's share of its row's window sum
        for (int ch0 = 0; ch0 < nchunks && expanders_ok; ch0 += 3) {
#pragma unroll
            for (int u = 0; u < 3; ++u) {
                const int ch = ch0 + u;
                if (ch >= nchunks) break;
                const int st = ch & 1;
                uint8_t* A_st = tiles + st * T::STAGE_BYTES;           // [KS] tiles of 128 rows x 32 B, then
                                                                       // [KS] tiles of TILE_N rows x 32 B
                if (ch + 2 < nchunks) load_chunk(ch + 2, (u + 2) % 3);
                if (ch >= 2) {                                         // the MMAs of chunk ch-2 must have read the stage
                    if (!mbar_wait_bounded(&empty_bar[st], (uint32_t)(((ch >> 1) - 1) & 1), abortp)) {
                        expanders_ok = false;
                        break;
                    }
                }
                const uint32_t (&a_cur)[KS][AB] = a_set[u];
                const uint32_t (&b_cur)[T::B_ITEMS][WB] = b_set[u];
#pragma unroll
                for (int q = 0; q < KS; ++q) {
                    // activation codes: register b of the row holds channels {b, 8+b, 16+b, 24+b}
                    uint32_t r[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                    for (int k = 0; k < AB; ++k) {
                        const uint32_t w = a_cur[q][k];
                        if (p.w_levels && (k & 1) == half) wsum += __popc(w) << k;
                        const uint32_t mask = 0x01010101u << k;
#pragma unroll
                        for (int bb = 0; bb < 4; ++bb) r[bb] |= __funnelshift_r(w, w, 4 * half + bb - k) & mask;
                    }
                    *reinterpret_cast<uint4*>(A_st + q * T::A_TILE_BYTES + a_soff) = make_uint4(r[0], r[1], r[2], r[3]);
                }
#pragma unroll
                for (int i = 0; i < T::B_ITEMS; ++i) {
                    if (b_q[i] >= 0) {
                        // weight codes: planes below the top one give the low bits, the top plane the byte
                        // 256 - 2^(WB-1) (bits WB-1 .. 7 set): two's-complement sign extension
                        uint32_t r[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
                        for (int m = 0; m < WB; ++m) {
                            const uint32_t w = b_cur[i][m];
                            const uint32_t mask = 0x01010101u << m;
                            const uint32_t scale = (m == WB - 1 && WB < 8) ? ((1u << (9 - WB)) - 1u) : 1u;
#pragma unroll
                            for (int bb = 0; bb < 8; ++bb) r[bb] |= (__funnelshift_r(w, w, bb - m) & mask) * scale;
                        }
                        uint8_t* dst = A_st + b_soff[i];
                        const int bsw = (b_soff[i] >> 3) & 16;           // ((row >> 2) & 1) << 4 with row = offset / 32
                        *reinterpret_cast<uint4*>(dst + bsw) = make_uint4(r[0], r[1], r[2], r[3]);
                        *reinterpret_cast<uint4*>(dst + (bsw ^ 16)) = make_uint4(r[4], r[5], r[6], r[7]);
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");  // generic writes -> tensor-core reads
                mbar_arrive(&full_bar[st]);
            }
        }
        wsum_s[half][row] = wsum;
        // all MMAs done (the last commit covers every earlier one)
        if (!*abortp) mbar_wait_bounded(&empty_bar[(nchunks - 1) & 1], (uint32_t)(((nchunks - 1) >> 1) & 1), abortp);
    } else {
        // =========================== issuer ===========================
        constexpr uint32_t IDESC = umma_idesc_i8(TILE_N);
        for (int ch = 0; ch < nchunks; ++ch) {
            const int st = ch & 1;
            if (!mbar_wait_bounded(&full_bar[st], (uint32_t)((ch >> 1) & 1), abortp)) break;
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            if ((tid & 31) == 0) {
                const uint32_t a_base = smem_u32(tiles + st * T::STAGE_BYTES);
                const uint32_t b_base = a_base + KS * T::A_TILE_BYTES;
                const uint64_t da0 = umma_desc_sw32(a_base), db0 = umma_desc_sw32(b_base);
#pragma unroll
                for (int q = 0; q < KS; ++q) {
                    if (ch * KS + q >= kwords) break;
                    umma_i8(tmem_base, da0 + (uint64_t)((q * T::A_TILE_BYTES) >> 4),
                            db0 + (uint64_t)((q * T::B_TILE_BYTES) >> 4), IDESC, (ch | q) != 0 ? 1u : 0u);
                }
                umma_commit(&empty_bar[st]);
            }
            __syncwarp();
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const bool aborted = abort_flag != 0;

    // ---- epilogue: expander threads read the accumulators of their own pixel row
    if (!aborted) {
        const int wsum_row = (p.w_levels && warp < 8) ? wsum_s[0][row] + wsum_s[1][row] : 0;
        umma_epilogue<TILE_N>(p, tmem_base, warp, gp, gp < p.P, wsum_row, co0);
    }
    if (aborted && tid == 0) atomicAdd(&g_umma_timeouts, 1ull);

    // ---- release tensor memory (every path reaches this)
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 8) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"((uint32_t)T::TMEM_COLS)
                     : "memory");
    }
}

template <int WB, int AB, int TILE_N>
int launch_conv_umma(const ConvParams& p, dim3 grid, cudaStream_t st) {
    using T = UmmaTile<WB, AB, TILE_N>;
    // raising the dynamic shared-memory limit is a per-device attribute of the kernel: set it once per device
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaFuncSetAttribute(conv_umma_kernel<WB, AB, TILE_N>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             T::SMEM_BYTES);
        attr_set[dev] = true;
    }
    conv_umma_kernel<WB, AB, TILE_N><<<grid, UMMA_THREADS, T::SMEM_BYTES, st>>>(p);
    return EBS_OK;
}

constexpr int NUM_UMMA_VARIANTS = 5;           // TILE_N = 16, 32, 64, 128, 256

template <int WB, int AB, int VARIANT>
constexpr ConvVariant make_umma_variant() {
    constexpr int TILE_N = 16 << VARIANT;
    return ConvVariant{&launch_conv_umma<WB, AB, TILE_N>, UMMA_M, TILE_N, UMMA_THREADS};
}

#define EBS_UMMA_ROW(WB, AB)                                                                              \
    {make_umma_variant<WB, AB, 0>(), make_umma_variant<WB, AB, 1>(), make_umma_variant<WB, AB, 2>(),      \
     make_umma_variant<WB, AB, 3>(), make_umma_variant<WB, AB, 4>()}

#define EBS_DEFINE_UMMA_TABLE(WB)                                                                         \
    const ConvVariant* conv_umma_variant_w##WB(int a_bits, int variant) {                                 \
        static const ConvVariant table[8][NUM_UMMA_VARIANTS] = {                                          \
            EBS_UMMA_ROW(WB, 1), EBS_UMMA_ROW(WB, 2), EBS_UMMA_ROW(WB, 3), EBS_UMMA_ROW(WB, 4),           \
            EBS_UMMA_ROW(WB, 5), EBS_UMMA_ROW(WB, 6), EBS_UMMA_ROW(WB, 7), EBS_UMMA_ROW(WB, 8)};          \
        if (a_bits < 1 || a_bits > 8 || variant < 0 || variant >= NUM_UMMA_VARIANTS) return nullptr;      \
        return &table[a_bits - 1][variant];                                                               \
    }                                                                                                     \
    unsigned long long conv_umma_timeouts_w##WB() {                                                       \
        unsigned long long v = 0;                                                                         \
        cudaMemcpyFromSymbol(&v, g_umma_timeouts, sizeof(v));                                             \
        return v;                                                                                         \
    }

}  // namespace ebs
