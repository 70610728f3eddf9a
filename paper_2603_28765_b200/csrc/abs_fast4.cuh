// Fast path of the group-quantize kernel for the 4-bit formats (IF4, NVFP4), round-to-nearest,
// no Hadamard / stochastic options.  Same arithmetic as the generic kernel, bit for bit, written
// for the sm_100a issue budget: packed f32x2 multiply / FMA for the per-element work, the integer
// candidate rounded by one fused add of 1.5*2^23 + 8 (the low mantissa nibble of the sum is the
// offset-binary code), three-input max for the group maximum, integer Horner packing of the codes.
#pragma once
#include "abs_device.cuh"

namespace absq {


// 1.5 * 2^23 + 8: adding it to an integer-valued-after-rounding k in [-8, 7] leaves k + 8 in the
// low mantissa nibble, so eight such sums combine into eight offset-binary nibbles without borrows.
constexpr float kMagic8 = 12582920.0f;
constexpr uint32_t kMagic8Bits = 0x4B400008u;

// Bytes b0..b3 (each < 256) -> b0 | b1<<8 | b2<<16 | b3<<24 with multiply-adds (FMA pipe, not the ALU).
__device__ __forceinline__ uint32_t merge_bytes(uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3) {
    return ((b3 * 256u + b2) * 256u + b1) * 256u + b0;
}


// Step 4 for eight scaled values at once: four e2m1x2 converts whose bytes are packed into one word
// inside the asm block (no byte masks), plus the half2 values of each byte for the error terms.
__device__ __forceinline__ uint32_t e2m1x8_encode_decode(const float (&y)[8], uint32_t (&h)[4]) {
    uint32_t w;
    asm("{ .reg .b8 a, b, c, d;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 a, %6, %5;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b, %8, %7;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 c, %10, %9;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 d, %12, %11;\n"
        "  cvt.rn.f16x2.e2m1x2 %1, a;\n"
        "  cvt.rn.f16x2.e2m1x2 %2, b;\n"
        "  cvt.rn.f16x2.e2m1x2 %3, c;\n"
        "  cvt.rn.f16x2.e2m1x2 %4, d;\n"
        "  mov.b32 %0, {a, b, c, d}; }"
        : "=&r"(w), "=&r"(h[0]), "=&r"(h[1]), "=&r"(h[2]), "=&r"(h[3])
        : "f"(y[0]), "f"(y[1]), "f"(y[2]), "f"(y[3]), "f"(y[4]), "f"(y[5]), "f"(y[6]), "f"(y[7]));
    return w;
}
__device__ __forceinline__ uint32_t e2m1x8_encode(const float (&y)[8]) {
    uint32_t w;
    asm("{ .reg .b8 a, b, c, d;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 a, %2, %1;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 b, %4, %3;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 c, %6, %5;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 d, %8, %7;\n"
        "  mov.b32 %0, {a, b, c, d}; }"
        : "=r"(w)
        : "f"(y[0]), "f"(y[1]), "f"(y[2]), "f"(y[3]), "f"(y[4]), "f"(y[5]), "f"(y[6]), "f"(y[7]));
    return w;
}

// Per-element work of one group (steps 3-10 of Fig. 3a) once the scale is known.
// CLAMP is the rare variant for scale bytes that are subnormal (1..7) or saturated (0x7E): there
// |y * 7/6| can exceed 7.5, so the integer candidate must be clamped to +-7; for every other scale
// byte |y| <= 6 * 17/16 and the rounded integer is within +-7 by construction.
// D_INT_GIVEN: the caller also passes d * fp32(6/7) (from the block's table) instead of having it computed here.
template <bool HAS_INT, bool CLAMP, bool D_INT_GIVEN = false>
__device__ __forceinline__ void encode_body4(const float (&x)[16], uint32_t sb, float d, float r, uint32_t& sbyte,
                                             uint32_t& c_lo, uint32_t& c_hi, float d_int_given = 0.0f) {
    const uint64_t R2 = pack2(r, r);
    if constexpr (!HAS_INT) {
#pragma unroll
        for (int hgrp = 0; hgrp < 2; ++hgrp) {
            float y[8];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                unpack2(mul2(pack2(x[8 * hgrp + 2 * i], x[8 * hgrp + 2 * i + 1]), R2), y[2 * i], y[2 * i + 1]);   // E1
            (hgrp ? c_hi : c_lo) = e2m1x8_encode(y);                                                           // E2
        }
        sbyte = sb;
    } else {
        const float c_pre = __uint_as_float(0x3F955555u);    // fp32(7/6)
        const float c_post = __uint_as_float(0x3F5B6DB7u);   // fp32(6/7)
        const float d_int = D_INT_GIVEN ? d_int_given : __fmul_rn(d, c_post);
        const uint64_t ND2 = pack2(-d, -d), NDI2 = pack2(-d_int, -d_int), CP2 = pack2(c_pre, c_pre);
        const uint64_t MG2 = pack2(kMagic8, kMagic8);
        uint64_t accF[2], accI[2];                                           // (S0,S1) and (S2,S3) chains
        uint32_t fw[2], kb[16];
#pragma unroll
        for (int hgrp = 0; hgrp < 2; ++hgrp) {
            uint64_t X[4], Y[4];
            float y[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                X[i] = pack2(x[8 * hgrp + 2 * i], x[8 * hgrp + 2 * i + 1]);
                Y[i] = mul2(X[i], R2);                                       // E1 (step 3)
                unpack2(Y[i], y[2 * i], y[2 * i + 1]);
            }
            uint32_t h[4];
            fw[hgrp] = e2m1x8_encode_decode(y, h);                           // E2 (step 4) and the code values
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&h[i]));
                const uint64_t E = fma2(pack2(v.x, v.y), ND2, X[i]);         // E3: -(v*d - x); squared below
                accF[hgrp] = (i == 0) ? mul2(E, E) : fma2(E, E, accF[hgrp]);   // fma(e, e, 0) == e * e
                uint64_t KZ = fma2(Y[i], CP2, MG2);                          // E4 (step 7): exact product, one rounding
                if constexpr (CLAMP) {
                    float k0, k1;
                    unpack2(KZ, k0, k1);
                    k0 = fminf(fmaxf(k0, kMagic8 - 7.0f), kMagic8 + 7.0f);
                    k1 = fminf(fmaxf(k1, kMagic8 - 7.0f), kMagic8 + 7.0f);
                    KZ = pack2(k0, k1);
                }
                const uint64_t KF = sub2(KZ, MG2);                           // k as a float
                const uint64_t FI = fma2(KF, NDI2, X[i]);                    // E5 (steps 8-9)
                accI[hgrp] = (i == 0) ? mul2(FI, FI) : fma2(FI, FI, accI[hgrp]);
                float kz0, kz1;
                unpack2(KZ, kz0, kz1);
                kb[8 * hgrp + 2 * i] = __float_as_uint(kz0);
                kb[8 * hgrp + 2 * i + 1] = __float_as_uint(kz1);
            }
        }
        // S1-S2 (step 10).
        float f0, f1, f2, f3, i0, i1, i2, i3;
        unpack2(accF[0], f0, f1); unpack2(accF[1], f2, f3);
        unpack2(accI[0], i0, i1); unpack2(accI[1], i2, i3);
        const float E_fp = __fadd_rn(__fadd_rn(f0, f1), __fadd_rn(f2, f3));
        const float E_int = __fadd_rn(__fadd_rn(i0, i1), __fadd_rn(i2, i3));
        const bool flag = E_int < E_fp;
        // S3-S4: integer codes by Horner on the raw sums (each holds kMagic8Bits + k), then remove the
        // constant part and turn offset-binary nibbles (k + 8) into two's complement (xor 8).
        constexpr uint32_t kConst = kMagic8Bits * 0x11111111u - 0x88888888u;   // sum of (bits - (k+8)) * 16^j
        uint32_t il = kb[7], ih = kb[15];
#pragma unroll
        for (int j = 6; j >= 0; --j) {
            il = il * 16u + kb[j];
            ih = ih * 16u + kb[8 + j];
        }
        il = (il - kConst) ^ 0x88888888u;
        ih = (ih - kConst) ^ 0x88888888u;
        c_lo = flag ? il : fw[0];
        c_hi = flag ? ih : fw[1];
        sbyte = sb | (flag ? 0x80u : 0u);
    }
}

constexpr int kFastMinBlocks = 4;   // resident blocks of 256 threads per SM the IF4 instance is compiled for

// Grid-stride kernel: every thread encodes groups g, g + stride, ... (a handful of them: the host sizes the
// grid as a few waves of resident blocks) and fetches the next group's 32 bytes before it works on the
// current one, so loads stay in flight under the math.
// IdxT is int32_t whenever the group count allows it (shorter address arithmetic).
template <bool HAS_INT, typename IdxT, bool ALIGNED32, bool FROM_SLOT, bool SCALE_MUL, bool SWZ>
__global__ void __launch_bounds__(256, HAS_INT ? kFastMinBlocks : 5)
quantize4_fast_kernel(const uint4* __restrict__ in, uint2* __restrict__ codes, uint8_t* __restrict__ scales,
                      const AlphaSrc alpha_src, IdxT ngroups, uint32_t gpr, uint32_t ktiles, bool l2_prefetch) {
    pdl_launch_dependents();
    const IdxT stride = (IdxT)(gridDim.x * blockDim.x);
    IdxT g = (IdxT)(blockIdx.x * blockDim.x + threadIdx.x);
    if (l2_prefetch && g < ngroups)          // before the wait: see prefetch_l2
        prefetch_l2(in + 2 * (size_t)((FROM_SLOT && !HAS_INT) ? (IdxT)(ngroups - 1 - g) : g));
    pdl_wait();
    // The first group's load goes out before alpha is resolved: its latency hides the alpha read.
    uint32_t w[8], wn[8];
    const bool active = g < ngroups;
    // The memory-bound NVFP4 instance walks the tensor backwards when it follows the amax pass of the same call:
    // the end of the tensor is what the L2 still holds (abs_quantize 44.1 -> 41.7 us at 4096x14336).  The IF4
    // instance is bound by arithmetic and measured 1 % slower that way, so it walks forwards.
    auto at = [&](IdxT gg) -> IdxT { return (FROM_SLOT && !HAS_INT) ? (IdxT)(ngroups - 1 - gg) : gg; };
    if (active) load32B<ALIGNED32>(in + 2 * (size_t)at(g), w);
    const float alpha = resolve_alpha_per_thread<FROM_SLOT>(alpha_src);      // T2
    // G5 once per block for every scale byte 0x00..0x7E: d = Delta * alpha, 1 / d, d * 6/7 (8192x4096: 16.68 -> 16.56 us)
    __shared__ float4 scale_lut[128];
    if (threadIdx.x < 127) {
        const float dd = __fmul_rn(e4m3_value(threadIdx.x), alpha);
        scale_lut[threadIdx.x] = make_float4(dd, __frcp_rn(dd), __fmul_rn(dd, __uint_as_float(0x3F5B6DB7u)), 0.0f);
    }
    __syncthreads();
    if (!active) return;
    const float inv_a6 = __frcp_rn(__fmul_rn(alpha, 6.0f));                  // T3
    // one group: G1-G5, steps 3-10, stores
    auto process = [&](const uint32_t (&ww)[8], IdxT gg) {
        float x[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            x[2 * i] = __uint_as_float(ww[i] << 16);
            x[2 * i + 1] = __uint_as_float(ww[i] & 0xFFFF0000u);
        }
        const float m0 = max3abs(x[0], x[1], x[2]), m1 = max3abs(x[3], x[4], x[5]);
        const float m2 = max3abs(x[6], x[7], x[8]), m3 = max3abs(x[9], x[10], x[11]);
        const float m4 = max3abs(x[12], x[13], x[14]);
        const float gmax = fmaxf(max3abs(m0, m1, m2), max3abs(m3, m4, x[15]));   // G1: three-input max
        float t = __fmul_rn(gmax, inv_a6);                                   // G2-G3 (Eq. 2)
        if constexpr (SCALE_MUL) t = __fmul_rn(t, 1.0625f);                  // the 17/16 option
        const uint32_t sb = e4m3_encode(t);
        uint32_t sbyte = 0u, c_lo = 0u, c_hi = 0u;
        // G5 from the block's table (d = Delta * alpha, 1 / d, d * 6/7: the same three roundings, done once per scale
        // byte and block instead of once per group)
        const float4 e = scale_lut[sb];
        const float d = e.x, r = e.y;
        if ((sb - 8u) >= 118u) {
            // rare path: zero scale (G4: all codes 0), subnormal scale bytes 1..7 and the saturated 0x7E
            if (sb != 0u) encode_body4<HAS_INT, HAS_INT, true>(x, sb, d, r, sbyte, c_lo, c_hi, e.z);
        } else {
            encode_body4<HAS_INT, false, true>(x, sb, d, r, sbyte, c_lo, c_hi, e.z);
        }
        scales[scale_offset<SWZ>((size_t)gg, gpr, ktiles)] = (uint8_t)sbyte;
        codes[gg] = make_uint2(c_lo, c_hi);
    };
    // two groups per trip, the two register buffers swapping roles: the next group's load is always in flight
    // under the current group's arithmetic and nothing is copied between the buffers
    // Besides the register prefetch of the next group, every group is requested into the L2 one group further
    // ahead (no register cost): the register load then finds it there, which shortens the waits on memory of
    // blocks that have just started (8192x4096, input not in the L2: 17.7 -> 17.3 us; two groups further ahead
    // measured slower).  The host switches it off when the amax pass of the same call has just left the input
    // in the L2, where the three extra instructions per group only cost (0.3 us at that size).
    const IdxT pf_end = l2_prefetch ? ngroups : (IdxT)0;
    auto request_ahead = [&](IdxT gp) {
        if (gp < pf_end) prefetch_l2(in + 2 * (size_t)at(gp));
    };
    request_ahead(g + stride);
    while (true) {
        const IdxT gn = g + stride;
        const bool more = gn < ngroups;
        if (more) load32B<ALIGNED32>(in + 2 * (size_t)at(gn), wn);
        request_ahead(gn + stride);
        process(w, at(g));
        if (!more) break;
        const IdxT g2 = gn + stride;
        const bool more2 = g2 < ngroups;
        if (more2) load32B<ALIGNED32>(in + 2 * (size_t)at(g2), w);
        request_ahead(g2 + stride);
        process(wn, at(gn));
        if (!more2) break;
        g = g2;
    }
}


// ----------------------------------------------------------------------------- 4-bit dequantize

// FP32 -> packed bf16 pair, round to nearest even (Sec. 4.1).
__device__ __forceinline__ uint32_t bf16x2_rn(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
// FP32 = (one f16 half of h2) + addend, one mixed-precision add (exact for the small values used here).
__device__ __forceinline__ float half_plus_f32(uint32_t h2, bool upper, float addend) {
    const uint16_t h = upper ? (uint16_t)(h2 >> 16) : (uint16_t)(h2 & 0xFFFFu);
    float d;
    asm("add.rn.f32.f16 %0, %1, %2;" : "=f"(d) : "h"(h), "f"(addend));
    return d;
}

// Eight 4-bit codes of one word -> eight products value * d, as four packed bf16 pairs.  Branch-free:
// both decodes are formed as f16 pairs (elements 2j, 2j+1 in register j) and selected per lane.
//   FP decode: e2m1x2 -> f16x2 per byte; value = half + (-0).
//   Integer decode: nibble n goes into the mantissa of the f16 constant 1024 as n ^ 8 = k + 8, so the
//   half is 1032 + k and value = half + (-1032) = k exactly.
template <bool HAS_INT>
__device__ __forceinline__ void dequant_word4(uint32_t w, bool is_int, float addend, uint64_t D2, uint32_t (&out)[4]) {
    uint32_t h[4];
    asm("{ .reg .b8 a, b, c, d;\n"
        "  mov.b32 {a, b, c, d}, %4;\n"
        "  cvt.rn.f16x2.e2m1x2 %0, a;\n"
        "  cvt.rn.f16x2.e2m1x2 %1, b;\n"
        "  cvt.rn.f16x2.e2m1x2 %2, c;\n"
        "  cvt.rn.f16x2.e2m1x2 %3, d; }"
        : "=r"(h[0]), "=r"(h[1]), "=r"(h[2]), "=r"(h[3]) : "r"(w));
    if constexpr (HAS_INT) {
        const uint32_t L = w & 0x0F0F0F0Fu, H = (w >> 4) & 0x0F0F0F0Fu;   // even / odd nibbles, one per byte
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            // bytes [L_j, L_j, H_j, H_j] -> keep one nibble per half, set the f16 exponent of 1024, flip bit 3
            const uint32_t r = (__byte_perm(L, H, 0x4400u + 0x1111u * j) & 0x000F000Fu) ^ 0x64086408u;
            h[j] = is_int ? r : h[j];
        }
    }
    float f[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        f[2 * j] = half_plus_f32(h[j], false, addend);
        f[2 * j + 1] = half_plus_f32(h[j], true, addend);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float p0, p1;
        unpack2(mul2(pack2(f[2 * j], f[2 * j + 1]), D2), p0, p1);
        out[j] = bf16x2_rn(p0, p1);
    }
}

// SEL 0: ordinary dequantize.  SEL 1: FP groups only (integer groups -> +0).  SEL 2: integer groups only and
// without the 6/7 de-scale (FP groups -> +0): the two exact halves used for the MAC arithmetic of Sec. 5.2.
template <bool HAS_INT, typename IdxT, bool ALIGNED32, bool SWZ, int SEL>
__global__ void __launch_bounds__(256) dequantize4_fast_kernel(const uint2* __restrict__ codes,
                                                               const uint8_t* __restrict__ scales,
                                                               const float* __restrict__ alpha_p, IdxT ngroups,
                                                               uint4* __restrict__ out, uint32_t gpr, uint32_t ktiles) {
    pdl_launch_dependents();
    const float c_post = __uint_as_float(0x3F5B6DB7u);   // fp32(6/7)
    const IdxT stride = (IdxT)(gridDim.x * blockDim.x);
    if ((IdxT)(blockIdx.x * blockDim.x + threadIdx.x) < ngroups)              // before the wait: see prefetch_l2
        prefetch_l2(codes + (size_t)(blockIdx.x * blockDim.x + threadIdx.x));
    pdl_wait();
    const float alpha = __ldg(alpha_p);
    for (IdxT g = (IdxT)(blockIdx.x * blockDim.x + threadIdx.x); g < ngroups; g += stride) {
        const uint2 c = __ldg(codes + (size_t)g);
        const uint32_t sbyte = __ldg(scales + scale_offset<SWZ>((size_t)g, gpr, ktiles));
        const uint32_t mag = sbyte & 0x7Fu;
        const bool is_int = HAS_INT && (sbyte & 0x80u);
        float Delta = e4m3_value(mag);
        if (mag == 0x7Fu) Delta = __uint_as_float(0x7FC00000u);        // E4M3 NaN propagates
        float d = __fmul_rn(Delta, alpha);
        if (is_int && SEL != 2) d = __fmul_rn(d, c_post);              // de-scale integer groups (Sec. 3)
        const float addend = is_int ? -1032.0f : -0.0f;
        const uint64_t D2 = pack2(d, d);
        uint32_t lo[4], hi[4];
        dequant_word4<HAS_INT>(c.x, is_int, addend, D2, lo);
        dequant_word4<HAS_INT>(c.y, is_int, addend, D2, hi);
        uint32_t o[8] = {lo[0], lo[1], lo[2], lo[3], hi[0], hi[1], hi[2], hi[3]};
        if ((SEL == 1 && is_int) || (SEL == 2 && !is_int)) {
#pragma unroll
            for (int j = 0; j < 8; ++j) o[j] = 0u;                      // the other half of the split: +0
        }
        store32B<ALIGNED32>(out + 2 * (size_t)g, o);
    }
}

}  // namespace absq
