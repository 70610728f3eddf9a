// Packed round-to-nearest group-quantize kernels for the formats beside IF4 / NVFP4: the block-size-8
// variants of the 4-bit formats (Sec. 5.1, Table 5), the 6-bit formats IF6-E2M3 / IF6-E3M2 and IF3 (Sec. 5.1).  Same
// arithmetic as the generic kernel, bit for bit, in the style of abs_fast4.cuh: persistent grid-stride
// threads that prefetch the next 32 bytes, f32x2 arithmetic, magic-number integer rounding, Horner packing.
#pragma once
#include "abs_fast4.cuh"

namespace absq {

// ----------------------------------------------------------------------------- decode helpers

// Eight 3-bit fields of a 24-bit chunk (field j at bit 3j) spread to the low three bits of eight nibbles:
// 12-bit halves to 16-bit halves, 6-bit pairs to bytes, 3-bit fields to nibbles, each step one mask and
// one multiply-add (moving a part left by s bits adds (2^s - 1) times that part).
__device__ __forceinline__ uint32_t spread3to4(uint32_t x) {
    const uint32_t y = x + (x >> 12) * 0xF000u;
    const uint32_t z = y + (y & 0x0FC00FC0u) * 3u;
    return z + (z & 0x38383838u);
}

// Eight 3-bit codes (a 24-bit chunk) -> eight products value * d as four packed bf16 pairs, through the 4-bit
// decoder: an E2M0 code s|ee is the E2M1 code s|ee|0 (values 0, 1, 2, 4 are the E2M1 codes with a zero mantissa
// bit), and a 3-bit two's-complement integer sign-extends to a nibble.  d already holds the 4/3 factor of
// integer groups.
__device__ __forceinline__ void decode3x8(uint32_t chunk, bool is_int, float d, uint32_t (&r)[4]) {
    const uint32_t u = spread3to4(chunk);
    const uint32_t w = is_int ? (u + (u & 0x44444444u) * 2u) : (u << 1);
    dequant_word4<true>(w, is_int, is_int ? -1032.0f : -0.0f, pack2(d, d), r);
}

// Four 6-bit fields of a 24-bit chunk (field j at bit 6j) spread to one field per byte: the inverse of
// squeeze6x4 (below), again one mask and one multiply-add per step.
__device__ __forceinline__ uint32_t spread6to8(uint32_t c) {
    const uint32_t t = c + (c >> 12) * 0xF000u;
    return t + (t & 0x0FC00FC0u) * 3u;
}

// Sixteen 6-bit codes (three words) -> sixteen products value * d as eight packed bf16 pairs.  Branch-free like
// the 4-bit decoder: the FP decode is the hardware convert to f16 pairs, the integer decode places the field
// k + 32 (field xor 32) in the mantissa of the f16 constant 1024, so the half is 1056 + k; one shared tail adds
// -0 or -1056 in FP32, multiplies by the group scale (which already holds the de-scale factor of integer
// groups) and rounds to bf16 pairs.
template <ElemKind EK>
__device__ __forceinline__ void decode6x16(uint32_t w0, uint32_t w1, uint32_t w2, bool is_int, float d, uint32_t (&o)[8]) {
    const float addend = is_int ? -1056.0f : -0.0f;
    const uint64_t D2 = pack2(d, d);
    const uint32_t chunk[4] = {w0 & 0xFFFFFFu, (w0 >> 24) | ((w1 & 0xFFFFu) << 8), (w1 >> 16) | ((w2 & 0xFFu) << 16), w2 >> 8};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const uint32_t bytes = spread6to8(chunk[q]);                       // codes 4q .. 4q+3, one per byte
        uint32_t h0, h1;
        if constexpr (EK == EK_E2M3) {
            asm("{ .reg .b16 lo, hi;\n"
                "  mov.b32 {lo, hi}, %2;\n"
                "  cvt.rn.f16x2.e2m3x2 %0, lo;\n"
                "  cvt.rn.f16x2.e2m3x2 %1, hi; }" : "=&r"(h0), "=&r"(h1) : "r"(bytes));
        } else {
            asm("{ .reg .b16 lo, hi;\n"
                "  mov.b32 {lo, hi}, %2;\n"
                "  cvt.rn.f16x2.e3m2x2 %0, lo;\n"
                "  cvt.rn.f16x2.e3m2x2 %1, hi; }" : "=&r"(h0), "=&r"(h1) : "r"(bytes));
        }
        const uint32_t r0 = __byte_perm(bytes, 0u, 0x4140) ^ 0x64206420u;  // halves 1056 + k of codes 4q, 4q+1
        const uint32_t r1 = __byte_perm(bytes, 0u, 0x4342) ^ 0x64206420u;  // ... of codes 4q+2, 4q+3
        const uint32_t s0 = is_int ? r0 : h0, s1 = is_int ? r1 : h1;
        float p0, p1, p2, p3;
        unpack2(mul2(pack2(half_plus_f32(s0, false, addend), half_plus_f32(s0, true, addend)), D2), p0, p1);
        unpack2(mul2(pack2(half_plus_f32(s1, false, addend), half_plus_f32(s1, true, addend)), D2), p2, p3);
        o[2 * q] = bf16x2_rn(p0, p1);
        o[2 * q + 1] = bf16x2_rn(p2, p3);
    }
}

// ----------------------------------------------------------------------------- 4-bit, one scale per 8 values

// Steps 3-10 of Fig. 3a for one group of EIGHT values (one 32-bit word of codes).  The error sums of a
// group of 8 are S0 + S1 (the other two chains of the 16-value order are +0).
template <bool HAS_INT, bool CLAMP>
__device__ __forceinline__ void encode_half4(const float* x, uint32_t sb, float d, float r, uint32_t& sbyte,
                                             uint32_t& cword) {
    const uint64_t R2 = pack2(r, r);
    float y[8];
    uint64_t X[4], Y[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        X[i] = pack2(x[2 * i], x[2 * i + 1]);
        Y[i] = mul2(X[i], R2);                                               // E1 (step 3)
        unpack2(Y[i], y[2 * i], y[2 * i + 1]);
    }
    if constexpr (!HAS_INT) {
        cword = e2m1x8_encode(y);                                            // E2
        sbyte = sb;
    } else {
        const float c_pre = __uint_as_float(0x3F955555u);    // fp32(7/6)
        const float c_post = __uint_as_float(0x3F5B6DB7u);   // fp32(6/7)
        const float d_int = __fmul_rn(d, c_post);
        const uint64_t ND2 = pack2(-d, -d), NDI2 = pack2(-d_int, -d_int), CP2 = pack2(c_pre, c_pre);
        const uint64_t MG2 = pack2(kMagic8, kMagic8), NMG2 = pack2(-kMagic8, -kMagic8);
        uint64_t accF = 0, accI = 0;
        uint32_t h[4], kb[8];
        const uint32_t fw = e2m1x8_encode_decode(y, h);                      // E2 (step 4) and the code values
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&h[i]));
            const uint64_t E = fma2(pack2(v.x, v.y), ND2, X[i]);             // E3, negated; squared below
            accF = (i == 0) ? mul2(E, E) : fma2(E, E, accF);
            uint64_t KZ = fma2(Y[i], CP2, MG2);                              // E4 (step 7)
            if constexpr (CLAMP) {
                float k0, k1;
                unpack2(KZ, k0, k1);
                k0 = fminf(fmaxf(k0, kMagic8 - 7.0f), kMagic8 + 7.0f);
                k1 = fminf(fmaxf(k1, kMagic8 - 7.0f), kMagic8 + 7.0f);
                KZ = pack2(k0, k1);
            }
            const uint64_t FI = fma2(add2(KZ, NMG2), NDI2, X[i]);            // E5 (steps 8-9)
            accI = (i == 0) ? mul2(FI, FI) : fma2(FI, FI, accI);
            float kz0, kz1;
            unpack2(KZ, kz0, kz1);
            kb[2 * i] = __float_as_uint(kz0);
            kb[2 * i + 1] = __float_as_uint(kz1);
        }
        float f0, f1, i0, i1;
        unpack2(accF, f0, f1);
        unpack2(accI, i0, i1);
        const bool flag = __fadd_rn(i0, i1) < __fadd_rn(f0, f1);             // S1-S2 (step 10)
        constexpr uint32_t kConst = kMagic8Bits * 0x11111111u - 0x88888888u;
        uint32_t il = kb[7];
#pragma unroll
        for (int j = 6; j >= 0; --j) il = il * 16u + kb[j];
        il = (il - kConst) ^ 0x88888888u;
        cword = flag ? il : fw;
        sbyte = sb | (flag ? 0x80u : 0u);
    }
}

// One thread per aligned block of 16 values = two groups of 8: two scales, one 64-bit store of codes and
// one 16-bit store of scale bytes.  scale_mul is 17/16 with that option and 1 otherwise.
// EMUL (all kernels of this file): the emulation pass of Sec. 4.1, as in quantize4_opt_kernel: the group is decoded
// from the registers that hold its codes and scale and written to `out` as bf16; codes and scale bytes are
// stored only when `store_codes` is set.
template <bool HAS_INT, bool FROM_SLOT, bool EMUL = false>
__global__ void __launch_bounds__(256, HAS_INT ? 4 : 5)
quantize4_bs8_kernel(const uint4* __restrict__ in, uint2* __restrict__ codes, uint16_t* __restrict__ scales,
                     const AlphaSrc alpha_src, int32_t nblocks16, float scale_mul, bool aligned32,
                     uint4* __restrict__ out = nullptr, bool out_aligned32 = false, bool store_codes = true) {
    pdl_launch_dependents();
    const int32_t stride = (int32_t)(gridDim.x * blockDim.x);
    int32_t g = (int32_t)(blockIdx.x * blockDim.x + threadIdx.x);
    if (g < nblocks16) prefetch_l2(in + 2 * (size_t)g);                  // before the wait: see prefetch_l2
    pdl_wait();
    uint32_t w[8], wn[8];
    const bool active = g < nblocks16;
    if (active) {
        if (aligned32) load32B<true>(in + 2 * (size_t)g, w);
        else load32B<false>(in + 2 * (size_t)g, w);
    }
    const float alpha = resolve_alpha_per_thread<FROM_SLOT>(alpha_src);      // T2
    __shared__ float2 scale_table[128];
    fill_scale_table(scale_table, alpha);                                    // G5 for every scale byte, once per block
    if (!active) return;
    const float inv_a6 = __frcp_rn(__fmul_rn(alpha, 6.0f));                  // T3
    // one block of 16 values held in `w`, index `g`
    auto process = [&](const uint32_t (&w)[8], const int32_t g) {
        float x[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
        uint32_t cw[2], sbytes = 0u, o[8];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const float* xs = x + 8 * h;
            const float gmax = max3abs(max3abs(xs[0], xs[1], xs[2]), max3abs(xs[3], xs[4], xs[5]), fmaxf(fabsf(xs[6]), fabsf(xs[7])));   // G1
            const float t = __fmul_rn(__fmul_rn(gmax, inv_a6), scale_mul);   // G2
            const uint32_t sb = e4m3_encode(t);                              // G3
            const float2 dr = scale_table[sb];                                 // G5: d = Delta * alpha and 1 / d
            const float d = dr.x, r = dr.y;
            uint32_t sbyte = 0u, c = 0u;
            if ((sb - 8u) >= 118u) {
                if (sb != 0u) encode_half4<HAS_INT, HAS_INT>(xs, sb, d, r, sbyte, c);      // G4: zero scale -> zeros
            } else {
                encode_half4<HAS_INT, false>(xs, sb, d, r, sbyte, c);
            }
            cw[h] = c;
            sbytes |= sbyte << (8 * h);
            if constexpr (EMUL) {
                const bool is_int = HAS_INT && (sbyte & 0x80u);
                const float dd = is_int ? __fmul_rn(d, __uint_as_float(0x3F5B6DB7u)) : d;
                uint32_t rr[4];
                dequant_word4<HAS_INT>(c, is_int, is_int ? -1032.0f : -0.0f, pack2(dd, dd), rr);
                o[4 * h] = rr[0]; o[4 * h + 1] = rr[1]; o[4 * h + 2] = rr[2]; o[4 * h + 3] = rr[3];
            }
        }
        if (!EMUL || store_codes) {
            scales[g] = (uint16_t)sbytes;
            codes[g] = make_uint2(cw[0], cw[1]);
        }
        if constexpr (EMUL) {
            if (out_aligned32) store32B<true>(out + 2 * (size_t)g, o);
            else store32B<false>(out + 2 * (size_t)g, o);
        }
    };
    auto fetch = [&](uint32_t (&buf)[8], int32_t gg) {
        if (aligned32) load32B<true>(in + 2 * (size_t)gg, buf);
        else load32B<false>(in + 2 * (size_t)gg, buf);
    };
    // two blocks per trip, the two register buffers swapping roles: the next load is always in flight under
    // the current arithmetic and nothing is copied between the buffers
    while (true) {
        const int32_t gn = g + stride;
        const bool more = gn < nblocks16;
        if (more) fetch(wn, gn);
        process(w, g);
        if (!more) break;
        const int32_t g2 = gn + stride;
        const bool more2 = g2 < nblocks16;
        if (more2) fetch(w, g2);
        process(wn, gn);
        if (!more2) break;
        g = g2;
    }
}

// ----------------------------------------------------------------------------- 6-bit formats (IF6)

constexpr float kMagic32 = 12582944.0f;               // 1.5 * 2^23 + 32: the low six mantissa bits of k + kMagic32 are k + 32
constexpr uint32_t kMagic32Bits = 0x4B400020u;

// Step 4 for eight scaled values: four 6-bit x2 converts (one code per byte) give the eight code bytes
// as two words; the half2 values of the codes are then decoded from the 16-bit halves of those words.
template <ElemKind EK>
__device__ __forceinline__ void fp6x8_encode_decode(const float (&y)[8], uint32_t (&h)[4], uint32_t& w0, uint32_t& w1) {
    if constexpr (EK == EK_E2M3) {
        w0 = e2m3x2_encode(y[0], y[1]) | (e2m3x2_encode(y[2], y[3]) << 16);
        w1 = e2m3x2_encode(y[4], y[5]) | (e2m3x2_encode(y[6], y[7]) << 16);
        asm("{ .reg .b16 lo, hi;\n"
            "  mov.b32 {lo, hi}, %2;\n"
            "  cvt.rn.f16x2.e2m3x2 %0, lo;\n"
            "  cvt.rn.f16x2.e2m3x2 %1, hi; }" : "=&r"(h[0]), "=&r"(h[1]) : "r"(w0));
        asm("{ .reg .b16 lo, hi;\n"
            "  mov.b32 {lo, hi}, %2;\n"
            "  cvt.rn.f16x2.e2m3x2 %0, lo;\n"
            "  cvt.rn.f16x2.e2m3x2 %1, hi; }" : "=&r"(h[2]), "=&r"(h[3]) : "r"(w1));
    } else {
        w0 = e3m2x2_encode(y[0], y[1]) | (e3m2x2_encode(y[2], y[3]) << 16);
        w1 = e3m2x2_encode(y[4], y[5]) | (e3m2x2_encode(y[6], y[7]) << 16);
        asm("{ .reg .b16 lo, hi;\n"
            "  mov.b32 {lo, hi}, %2;\n"
            "  cvt.rn.f16x2.e3m2x2 %0, lo;\n"
            "  cvt.rn.f16x2.e3m2x2 %1, hi; }" : "=&r"(h[0]), "=&r"(h[1]) : "r"(w0));
        asm("{ .reg .b16 lo, hi;\n"
            "  mov.b32 {lo, hi}, %2;\n"
            "  cvt.rn.f16x2.e3m2x2 %0, lo;\n"
            "  cvt.rn.f16x2.e3m2x2 %1, hi; }" : "=&r"(h[2]), "=&r"(h[3]) : "r"(w1));
    }
}

// Four 6-bit codes, one per byte of w, squeezed into 24 bits (code j at bit 6j) with multiply-adds:
// b0 + b1*2^8 + b2*2^16 + b3*2^24  ->  pairs (b0 + b1*2^6) at bits 0 and 16  ->  b0 + b1*2^6 + b2*2^12 + b3*2^18.
__device__ __forceinline__ uint32_t squeeze6x4(uint32_t w) {
    const uint32_t t = w - 192u * ((w >> 8) & 0x00FF00FFu);
    return t - 0xF000u * (t >> 16);
}

// Steps 3-10 of Fig. 3a for one group of 16 values of a 6-bit format; the 96 bits of codes leave as
// three words.  The integer candidate is always clamped: |y| reaches M_FP * 17/16, and 31 * 17/16 > 31.5.
template <ElemKind EK>
__device__ __forceinline__ void encode_body6(const float (&x)[16], uint32_t sb, float d, float r, float c_pre,
                                             float c_post, uint32_t& sbyte, uint32_t (&cw)[3]) {
    const uint64_t R2 = pack2(r, r);
    const float d_int = __fmul_rn(d, c_post);
    const uint64_t ND2 = pack2(-d, -d), NDI2 = pack2(-d_int, -d_int), CP2 = pack2(c_pre, c_pre);
    const uint64_t MG2 = pack2(kMagic32, kMagic32), NMG2 = pack2(-kMagic32, -kMagic32);
    uint64_t accF[2], accI[2];
    uint32_t fchunk[4], ichunk[4];
#pragma unroll
    for (int hgrp = 0; hgrp < 2; ++hgrp) {
        uint64_t X[4], Y[4];
        float y[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            X[i] = pack2(x[8 * hgrp + 2 * i], x[8 * hgrp + 2 * i + 1]);
            Y[i] = mul2(X[i], R2);                                           // E1 (step 3)
            unpack2(Y[i], y[2 * i], y[2 * i + 1]);
        }
        uint32_t h[4], w0, w1, kb[8];
        fp6x8_encode_decode<EK>(y, h, w0, w1);                               // E2 (step 4) and the code values
        fchunk[2 * hgrp] = squeeze6x4(w0);
        fchunk[2 * hgrp + 1] = squeeze6x4(w1);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&h[i]));
            const uint64_t E = fma2(pack2(v.x, v.y), ND2, X[i]);             // E3, negated; squared below
            accF[hgrp] = (i == 0) ? mul2(E, E) : fma2(E, E, accF[hgrp]);
            float k0, k1;
            unpack2(fma2(Y[i], CP2, MG2), k0, k1);                           // E4 (step 7): exact product, one rounding
            k0 = fminf(fmaxf(k0, kMagic32 - 31.0f), kMagic32 + 31.0f);
            k1 = fminf(fmaxf(k1, kMagic32 - 31.0f), kMagic32 + 31.0f);
            const uint64_t FI = fma2(add2(pack2(k0, k1), NMG2), NDI2, X[i]); // E5 (steps 8-9)
            accI[hgrp] = (i == 0) ? mul2(FI, FI) : fma2(FI, FI, accI[hgrp]);
            kb[2 * i] = __float_as_uint(k0);
            kb[2 * i + 1] = __float_as_uint(k1);
        }
        // integer codes: Horner over four raw sums (each kMagic32Bits + k + 32), constant part removed,
        // offset-binary fields (k + 32) turned into two's complement (flip bit 5 of every field)
        constexpr uint32_t kConst = (kMagic32Bits - 32u) * (1u + 64u + 4096u + 262144u);   // leaves the fields k + 32
        ichunk[2 * hgrp] = ((((kb[3] * 64u + kb[2]) * 64u + kb[1]) * 64u + kb[0]) - kConst) ^ 0x820820u;
        ichunk[2 * hgrp + 1] = ((((kb[7] * 64u + kb[6]) * 64u + kb[5]) * 64u + kb[4]) - kConst) ^ 0x820820u;
    }
    float f0, f1, f2, f3, i0, i1, i2, i3;
    unpack2(accF[0], f0, f1); unpack2(accF[1], f2, f3);
    unpack2(accI[0], i0, i1); unpack2(accI[1], i2, i3);
    const float E_fp = __fadd_rn(__fadd_rn(f0, f1), __fadd_rn(f2, f3));         // S1-S2 (step 10)
    const float E_int = __fadd_rn(__fadd_rn(i0, i1), __fadd_rn(i2, i3));
    const bool flag = E_int < E_fp;
    const uint32_t c0 = flag ? ichunk[0] : fchunk[0], c1 = flag ? ichunk[1] : fchunk[1];
    const uint32_t c2 = flag ? ichunk[2] : fchunk[2], c3 = flag ? ichunk[3] : fchunk[3];
    cw[0] = c0 | (c1 << 24);                                                    // S4: 4 x 24 bits -> 3 words
    cw[1] = (c1 >> 8) | (c2 << 16);
    cw[2] = (c2 >> 16) | (c3 << 8);
    sbyte = sb | (flag ? 0x80u : 0u);                                           // S3
}

template <int FMT, bool FROM_SLOT, bool EMUL = false>
__global__ void __launch_bounds__(256, 3)
quantize6_fast_kernel(const uint4* __restrict__ in, uint32_t* __restrict__ codes, uint8_t* __restrict__ scales,
                      const AlphaSrc alpha_src, int32_t ngroups, float scale_mul, bool aligned32,
                      uint4* __restrict__ out = nullptr, bool out_aligned32 = false, bool store_codes = true) {
    using F = Fmt<FMT>;
    pdl_launch_dependents();
    const int32_t stride = (int32_t)(gridDim.x * blockDim.x);
    int32_t g = (int32_t)(blockIdx.x * blockDim.x + threadIdx.x);
    if (g < ngroups) prefetch_l2(in + 2 * (size_t)g);                  // before the wait: see prefetch_l2
    pdl_wait();
    uint32_t w[8], wn[8];
    const bool active = g < ngroups;
    if (active) {
        if (aligned32) load32B<true>(in + 2 * (size_t)g, w);
        else load32B<false>(in + 2 * (size_t)g, w);
    }
    const float alpha = resolve_alpha_per_thread<FROM_SLOT>(alpha_src);      // T2
    if (!active) return;
    const float inv_a6 = __frcp_rn(__fmul_rn(alpha, F::M_FP));               // T3
    const float c_pre = __fdiv_rn(F::M_INT, F::M_FP), c_post = __fdiv_rn(F::M_FP, F::M_INT);
    // one block of 16 values held in `w`, index `g`
    auto process = [&](const uint32_t (&w)[8], const int32_t g) {
        float x[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
        const float m0 = max3abs(x[0], x[1], x[2]), m1 = max3abs(x[3], x[4], x[5]);                        // G1
        const float m2 = max3abs(x[6], x[7], x[8]), m3 = max3abs(x[9], x[10], x[11]);
        const float m4 = max3abs(x[12], x[13], x[14]);
        const float gmax = fmaxf(max3abs(m0, m1, m2), max3abs(m3, m4, x[15]));
        const float t = __fmul_rn(__fmul_rn(gmax, inv_a6), scale_mul);       // G2
        const uint32_t sb = e4m3_encode(t);                                  // G3
        const float d = __fmul_rn(e4m3_value(sb), alpha);                    // G5
        const float r = __frcp_rn(d);
        uint32_t sbyte = 0u, cw[3] = {0u, 0u, 0u};
        if (sb != 0u) encode_body6<F::EK>(x, sb, d, r, c_pre, c_post, sbyte, cw);   // G4: zero scale -> zeros
        if (!EMUL || store_codes) {
            scales[g] = (uint8_t)sbyte;
            uint32_t* cp = codes + 3 * (size_t)g;
            cp[0] = cw[0]; cp[1] = cw[1]; cp[2] = cw[2];
        }
        if constexpr (EMUL) {
            const bool is_int = sbyte & 0x80u;
            uint32_t o[8];
            decode6x16<F::EK>(cw[0], cw[1], cw[2], is_int, is_int ? __fmul_rn(d, c_post) : d, o);
            if (out_aligned32) store32B<true>(out + 2 * (size_t)g, o);
            else store32B<false>(out + 2 * (size_t)g, o);
        }
    };
    auto fetch = [&](uint32_t (&buf)[8], int32_t gg) {
        if (aligned32) load32B<true>(in + 2 * (size_t)gg, buf);
        else load32B<false>(in + 2 * (size_t)gg, buf);
    };
    // two blocks per trip, the two register buffers swapping roles: the next load is always in flight under
    // the current arithmetic and nothing is copied between the buffers
    while (true) {
        const int32_t gn = g + stride;
        const bool more = gn < ngroups;
        if (more) fetch(wn, gn);
        process(w, g);
        if (!more) break;
        const int32_t g2 = gn + stride;
        const bool more2 = g2 < ngroups;
        if (more2) fetch(w, g2);
        process(wn, gn);
        if (!more2) break;
        g = g2;
    }
}

// ----------------------------------------------------------------------------- 3-bit format (IF3)

constexpr float kMagic4 = 12582916.0f;                // 1.5 * 2^23 + 4: the low three mantissa bits of k + kMagic4 are k + 4
constexpr uint32_t kMagic4Bits = 0x4B400004u;
constexpr float kMagic0 = 12582912.0f;                // 1.5 * 2^23
constexpr uint32_t kMagic0Bits = 0x4B400000u;

// Sign bits of eight bf16 values (four bf16x2 words) moved to bits 3j+2, the sign position of 3-bit code j.
// PRMT collects the four high bytes of two words (signs at bits 7, 15, 23, 31); the high half of a product
// with 2^27 + 2^22 + 2^17 + 2^12 drops them at bits 2, 5, 8, 11 (all sixteen partial products fall on
// different bits, so nothing carries; the mask removes the strays).
__device__ __forceinline__ uint32_t sign_bits3x8(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3) {
    const uint32_t a = __umulhi(__byte_perm(w0, w1, 0x7531) & 0x80808080u, 0x08421000u) & 0x924u;
    const uint32_t b = __umulhi(__byte_perm(w2, w3, 0x7531) & 0x80808080u, 0x08421000u) & 0x924u;
    return a | (b << 12);
}

// Candidates of EIGHT values of IF3 (E2M0 magnitudes {0, 1, 2, 4} or INT3), steps 3-9 of Fig. 3a: the
// 24-bit chunks of FP and integer codes and the two error chains (even / odd elements) of each candidate.
// E2M0 has no hardware convert.  Round-to-nearest-even onto {0, 1, 2, 4} of a = min(|y|, 4) is the sum of
// two exact integer roundings, RNE(min(a, 2)) + 2 * RNE((max(a, 2) - 2) / 2): the first covers 0..2 (ties
// 0.5 -> 0, 1.5 -> 2), the second the step from 2 to 4 (tie 3 -> 2); the code index is the sum of the two
// rounded integers.  FP errors are taken on magnitudes (|x| and |v| carry the same sign, so the squares
// agree).  CLAMP as in the 4-bit kernel: only subnormal or saturated scale bytes let |y * 3/4| pass 3.5.
// w holds the four bf16x2 words of the eight values (for their sign bits).
template <bool CLAMP>
__device__ __forceinline__ void candidates3x8(const float* x, const uint32_t* w, float d, float r, uint32_t& fchunk,
                                              uint32_t& ichunk, float& f0, float& f1, float& i0, float& i1) {
    const float c_pre = 0.75f, c_post = __fdiv_rn(4.0f, 3.0f);
    const float d_int = __fmul_rn(d, c_post);
    const uint64_t R2 = pack2(r, r), NDI2 = pack2(-d_int, -d_int), CP2 = pack2(c_pre, c_pre);
    const uint64_t MG = pack2(kMagic0, kMagic0);
    const uint64_t MG4 = pack2(kMagic4, kMagic4), NMG4 = pack2(-kMagic4, -kMagic4);
    // 1.5 * 2^24 has ulp 2: adding it rounds to even integers, i.e. 2 * RNE(. / 2), with the rounded integer in the
    // low mantissa bits.  kStep - 2 folds the "- 2" of max(a, 2) - 2 into the same add; kBoth removes both magics.
    constexpr float kStep = 25165824.0f;                                     // 1.5 * 2^24
    const uint64_t STEP = pack2(kStep - 2.0f, kStep - 2.0f), NBOTH = pack2(-(kStep + kMagic0), -(kStep + kMagic0));
    uint64_t accI = 0, accF = 0;
    uint32_t ib[8], kb[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint64_t X = pack2(x[2 * i], x[2 * i + 1]);
        const uint64_t Y = mul2(X, R2);                                      // E1 (step 3)
        float y0, y1;
        unpack2(Y, y0, y1);
        // E2 (step 4): E2M0 index and value of the magnitude.  Without CLAMP |y| <= 4 * 17/16, which rounds like 4
        // (max(a, 2) / 2 - 1 <= 1.13), so the saturation at 4 is only needed for the rare scale bytes.
        float a0 = fabsf(y0), a1 = fabsf(y1);
        if constexpr (CLAMP) {
            a0 = fminf(a0, 4.0f);
            a1 = fminf(a1, 4.0f);
        }
        const uint64_t M1 = add2(pack2(fminf(a0, 2.0f), fminf(a1, 2.0f)), MG);                // RNE(min(a, 2)) + magic
        const uint64_t M2 = add2(pack2(fmaxf(a0, 2.0f), fmaxf(a1, 2.0f)), STEP);              // 2 * RNE((max(a, 2) - 2) / 2) + kStep
        float m10, m11, m20, m21;
        unpack2(M1, m10, m11);
        unpack2(M2, m20, m21);
        ib[2 * i] = __float_as_uint(m10) + __float_as_uint(m20);             // kMagic0Bits + kStepBits + index
        ib[2 * i + 1] = __float_as_uint(m11) + __float_as_uint(m21);
        float v0, v1;
        unpack2(add2(add2(M2, NBOTH), M1), v0, v1);                          // the E2M0 magnitude r1 + 2 * r2 (both adds exact)
        // E3 (steps 5-6) on magnitudes
        const uint64_t E = pack2(__fmaf_rn(v0, -d, fabsf(x[2 * i])), __fmaf_rn(v1, -d, fabsf(x[2 * i + 1])));
        accF = (i == 0) ? mul2(E, E) : fma2(E, E, accF);
        // E4-E5 (steps 7-9): integer candidate, signed
        uint64_t KZ = fma2(Y, CP2, MG4);
        if constexpr (CLAMP) {
            float k0, k1;
            unpack2(KZ, k0, k1);
            k0 = fminf(fmaxf(k0, kMagic4 - 3.0f), kMagic4 + 3.0f);
            k1 = fminf(fmaxf(k1, kMagic4 - 3.0f), kMagic4 + 3.0f);
            KZ = pack2(k0, k1);
        }
        const uint64_t FI = fma2(add2(KZ, NMG4), NDI2, X);
        accI = (i == 0) ? mul2(FI, FI) : fma2(FI, FI, accI);
        float kz0, kz1;
        unpack2(KZ, kz0, kz1);
        kb[2 * i] = __float_as_uint(kz0);
        kb[2 * i + 1] = __float_as_uint(kz1);
    }
    unpack2(accI, i0, i1);
    unpack2(accF, f0, f1);
    // eight 3-bit fields by Horner on the raw sums; the constant parts are removed afterwards
    constexpr uint32_t kS8 = 0x249249u;                                      // 1 + 8 + ... + 8^7
    constexpr uint32_t kConstF = (kMagic0Bits + 0x4BC00000u) * kS8;          // bits of 1.5 * 2^23 and 1.5 * 2^24: leaves the indices 0..3
    constexpr uint32_t kConstI = (kMagic4Bits - 4u) * kS8;                   // leaves the fields k + 4
    uint32_t fc = ib[7], ic = kb[7];
#pragma unroll
    for (int j = 6; j >= 0; --j) {
        fc = fc * 8u + ib[j];
        ic = ic * 8u + kb[j];
    }
    fchunk = (fc - kConstF) | sign_bits3x8(w[0], w[1], w[2], w[3]);
    ichunk = (ic - kConstI) ^ 0x924924u;                                     // offset-binary -> two's complement
}

// Steps 3-10 for one group of 16 values: both halves under one scale, selection on (S0 + S1) + (S2 + S3).
template <bool CLAMP>
__device__ __forceinline__ void encode_body3(const float (&x)[16], const uint32_t (&w)[8], uint32_t sb, float d, float r,
                                             uint32_t& sbyte, uint32_t& c_lo, uint32_t& c_hi) {
    uint32_t fchunk[2], ichunk[2];
    float f[4], in[4];
    candidates3x8<CLAMP>(x, w, d, r, fchunk[0], ichunk[0], f[0], f[1], in[0], in[1]);
    candidates3x8<CLAMP>(x + 8, w + 4, d, r, fchunk[1], ichunk[1], f[2], f[3], in[2], in[3]);
    const float E_fp = __fadd_rn(__fadd_rn(f[0], f[1]), __fadd_rn(f[2], f[3]));       // S1-S2 (step 10)
    const float E_int = __fadd_rn(__fadd_rn(in[0], in[1]), __fadd_rn(in[2], in[3]));
    const bool flag = E_int < E_fp;
    const uint32_t c0 = flag ? ichunk[0] : fchunk[0], c1 = flag ? ichunk[1] : fchunk[1];
    c_lo = c0 | (c1 << 24);                                                  // S4: 2 x 24 bits -> 48 bits
    c_hi = c1 >> 8;
    sbyte = sb | (flag ? 0x80u : 0u);                                        // S3
}

constexpr int kIf3MinBlocks = 3;   // resident blocks of 256 threads per SM the IF3 kernel is compiled for

// G = 16: one scale per thread's 16 values.  G = 8 (IF3-BS8): each half has its own scale and selection.
template <int G, bool FROM_SLOT, bool EMUL = false>
__global__ void __launch_bounds__(256, kIf3MinBlocks)
quantize3_fast_kernel(const uint4* __restrict__ in, uint16_t* __restrict__ codes, uint8_t* __restrict__ scales,
                      const AlphaSrc alpha_src, int32_t ngroups, float scale_mul, bool aligned32,
                      uint4* __restrict__ out = nullptr, bool out_aligned32 = false, bool store_codes = true) {
    pdl_launch_dependents();
    const int32_t stride = (int32_t)(gridDim.x * blockDim.x);
    int32_t g = (int32_t)(blockIdx.x * blockDim.x + threadIdx.x);
    if (g < ngroups) prefetch_l2(in + 2 * (size_t)g);                  // before the wait: see prefetch_l2
    pdl_wait();
    uint32_t w[8], wn[8];
    const bool active = g < ngroups;
    if (active) {
        if (aligned32) load32B<true>(in + 2 * (size_t)g, w);
        else load32B<false>(in + 2 * (size_t)g, w);
    }
    const float alpha = resolve_alpha_per_thread<FROM_SLOT>(alpha_src);      // T2
    if (!active) return;
    const float inv_a6 = __frcp_rn(__fmul_rn(alpha, 4.0f));                  // T3
    // one block of 16 values held in `w`, index `g`
    auto process = [&](const uint32_t (&w)[8], const int32_t g) {
        float x[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
        uint32_t c_lo = 0u, c_hi = 0u, o[8];
        const float c_post3 = __fdiv_rn(4.0f, 3.0f);
        if constexpr (G == 16) {
            const float m0 = max3abs(x[0], x[1], x[2]), m1 = max3abs(x[3], x[4], x[5]);                    // G1
            const float m2 = max3abs(x[6], x[7], x[8]), m3 = max3abs(x[9], x[10], x[11]);
            const float m4 = max3abs(x[12], x[13], x[14]);
            const float gmax = fmaxf(max3abs(m0, m1, m2), max3abs(m3, m4, x[15]));
            const float t = __fmul_rn(__fmul_rn(gmax, inv_a6), scale_mul);   // G2
            const uint32_t sb = e4m3_encode(t);                              // G3
            const float d = __fmul_rn(e4m3_value(sb), alpha);                    // G5
            const float r = __frcp_rn(d);
            uint32_t sbyte = 0u;
            if ((sb - 8u) >= 118u) {
                if (sb != 0u) encode_body3<true>(x, w, sb, d, r, sbyte, c_lo, c_hi);         // G4: zero scale -> zeros
            } else {
                encode_body3<false>(x, w, sb, d, r, sbyte, c_lo, c_hi);
            }
            if (!EMUL || store_codes) scales[g] = (uint8_t)sbyte;
            if constexpr (EMUL) {
                const bool is_int = sbyte & 0x80u;
                const float dd = is_int ? __fmul_rn(d, c_post3) : d;
                uint32_t r0[4], r1[4];
                decode3x8(c_lo & 0xFFFFFFu, is_int, dd, r0);
                decode3x8((c_lo >> 24) | (c_hi << 8), is_int, dd, r1);
#pragma unroll
                for (int j = 0; j < 4; ++j) { o[j] = r0[j]; o[4 + j] = r1[j]; }
            }
        } else {
            uint32_t chunk[2] = {0u, 0u}, sbytes = 0u;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float* xs = x + 8 * h;
                const float gmax = max3abs(max3abs(xs[0], xs[1], xs[2]), max3abs(xs[3], xs[4], xs[5]),
                                           fmaxf(fabsf(xs[6]), fabsf(xs[7])));              // G1
                const float t = __fmul_rn(__fmul_rn(gmax, inv_a6), scale_mul);
                const uint32_t sb = e4m3_encode(t);
                const float d = __fmul_rn(e4m3_value(sb), alpha);                    // G5
                const float r = __frcp_rn(d);
                if (sb != 0u) {
                    uint32_t fc, ic;
                    float f0, f1, i0, i1;
                    if ((sb - 8u) >= 118u) candidates3x8<true>(xs, w + 4 * h, d, r, fc, ic, f0, f1, i0, i1);
                    else candidates3x8<false>(xs, w + 4 * h, d, r, fc, ic, f0, f1, i0, i1);
                    const bool flag = __fadd_rn(i0, i1) < __fadd_rn(f0, f1);  // a group of 8: S0 + S1
                    chunk[h] = flag ? ic : fc;
                    sbytes |= (sb | (flag ? 0x80u : 0u)) << (8 * h);
                    if constexpr (EMUL) {
                        uint32_t rr[4];
                        decode3x8(chunk[h], flag, flag ? __fmul_rn(d, c_post3) : d, rr);
#pragma unroll
                        for (int j = 0; j < 4; ++j) o[4 * h + j] = rr[j];
                    }
                } else if constexpr (EMUL) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) o[4 * h + j] = 0u;           // zero scale: the group decodes to +0
                }
            }
            c_lo = chunk[0] | (chunk[1] << 24);
            c_hi = chunk[1] >> 8;
            if (!EMUL || store_codes) reinterpret_cast<uint16_t*>(scales)[g] = (uint16_t)sbytes;
        }
        if (!EMUL || store_codes) {
            uint16_t* cp = codes + 3 * (size_t)g;                            // 6 bytes per block of 16
            cp[0] = (uint16_t)c_lo; cp[1] = (uint16_t)(c_lo >> 16); cp[2] = (uint16_t)c_hi;
        }
        if constexpr (EMUL) {
            if (out_aligned32) store32B<true>(out + 2 * (size_t)g, o);
            else store32B<false>(out + 2 * (size_t)g, o);
        }
    };
    auto fetch = [&](uint32_t (&buf)[8], int32_t gg) {
        if (aligned32) load32B<true>(in + 2 * (size_t)gg, buf);
        else load32B<false>(in + 2 * (size_t)gg, buf);
    };
    // two blocks per trip, the two register buffers swapping roles: the next load is always in flight under
    // the current arithmetic and nothing is copied between the buffers
    while (true) {
        const int32_t gn = g + stride;
        const bool more = gn < ngroups;
        if (more) fetch(wn, gn);
        process(w, g);
        if (!more) break;
        const int32_t g2 = gn + stride;
        const bool more2 = g2 < ngroups;
        if (more2) fetch(w, g2);
        process(wn, gn);
        if (!more2) break;
        g = g2;
    }
}

// ----------------------------------------------------------------------------- 3-bit dequantize

// IF3 / IF3-BS8 dequantize (decode3x8).  One thread per aligned block of 16 values; G = 8 gives each word of
// eight codes its own scale.
template <int G, bool ALIGNED32>
__global__ void __launch_bounds__(256) dequantize3_fast_kernel(const uint16_t* __restrict__ codes,
                                                               const uint8_t* __restrict__ scales,
                                                               const float* __restrict__ alpha_p, int32_t nblocks16,
                                                               uint4* __restrict__ out) {
    constexpr int NSUB = 16 / G;
    pdl_launch_dependents();
    const float c_post = __fdiv_rn(4.0f, 3.0f);
    const int32_t stride = (int32_t)(gridDim.x * blockDim.x);
    if ((int32_t)(blockIdx.x * blockDim.x + threadIdx.x) < nblocks16)        // before the wait: see prefetch_l2
        prefetch_l2(codes + 3 * (size_t)(blockIdx.x * blockDim.x + threadIdx.x));
    pdl_wait();
    const float alpha = __ldg(alpha_p);
    for (int32_t g = (int32_t)(blockIdx.x * blockDim.x + threadIdx.x); g < nblocks16; g += stride) {
        const uint16_t* cp = codes + 3 * (size_t)g;
        const uint32_t c0 = __ldg(cp), c1 = __ldg(cp + 1), c2 = __ldg(cp + 2);
        const uint32_t chunk[2] = {c0 | ((c1 & 0xFFu) << 16), (c1 >> 8) | (c2 << 8)};
        uint32_t sb[2];
        if constexpr (NSUB == 2) {
            const uint32_t two = __ldg(reinterpret_cast<const uint16_t*>(scales) + g);
            sb[0] = two & 0xFFu; sb[1] = two >> 8;
        } else {
            sb[0] = sb[1] = __ldg(scales + g);
        }
        uint32_t o[8];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t mag = sb[h] & 0x7Fu;
            const bool is_int = sb[h] & 0x80u;
            float Delta = e4m3_value(mag);
            if (mag == 0x7Fu) Delta = __uint_as_float(0x7FC00000u);        // E4M3 NaN propagates
            float d = __fmul_rn(Delta, alpha);
            if (is_int) d = __fmul_rn(d, c_post);                          // de-scale integer groups (Sec. 3)
            uint32_t r[4];
            decode3x8(chunk[h], is_int, d, r);
            o[4 * h] = r[0]; o[4 * h + 1] = r[1]; o[4 * h + 2] = r[2]; o[4 * h + 3] = r[3];
        }
        store32B<ALIGNED32>(out + 2 * (size_t)g, o);
    }
}

// ----------------------------------------------------------------------------- 4-bit dequantize, one scale per 8 values

// One thread per aligned block of 16 values: each word of eight codes has its own scale byte.
template <bool HAS_INT, bool ALIGNED32>
__global__ void __launch_bounds__(256) dequantize4_bs8_kernel(const uint2* __restrict__ codes,
                                                              const uint16_t* __restrict__ scales,
                                                              const float* __restrict__ alpha_p, int32_t nblocks16,
                                                              uint4* __restrict__ out) {
    pdl_launch_dependents();
    const float c_post = __uint_as_float(0x3F5B6DB7u);   // fp32(6/7)
    const int32_t stride = (int32_t)(gridDim.x * blockDim.x);
    if ((int32_t)(blockIdx.x * blockDim.x + threadIdx.x) < nblocks16)        // before the wait: see prefetch_l2
        prefetch_l2(codes + (size_t)(blockIdx.x * blockDim.x + threadIdx.x));
    pdl_wait();
    const float alpha = __ldg(alpha_p);
    for (int32_t g = (int32_t)(blockIdx.x * blockDim.x + threadIdx.x); g < nblocks16; g += stride) {
        const uint2 c = __ldg(codes + (size_t)g);
        const uint32_t two = __ldg(scales + g);
        const uint32_t cw[2] = {c.x, c.y};
        uint32_t o[8];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t sbyte = (two >> (8 * h)) & 0xFFu;
            const uint32_t mag = sbyte & 0x7Fu;
            const bool is_int = HAS_INT && (sbyte & 0x80u);
            float Delta = e4m3_value(mag);
            if (mag == 0x7Fu) Delta = __uint_as_float(0x7FC00000u);        // E4M3 NaN propagates
            float d = __fmul_rn(Delta, alpha);
            if (is_int) d = __fmul_rn(d, c_post);                          // de-scale integer groups (Sec. 3)
            uint32_t r[4];
            dequant_word4<HAS_INT>(cw[h], is_int, is_int ? -1032.0f : -0.0f, pack2(d, d), r);
            o[4 * h] = r[0]; o[4 * h + 1] = r[1]; o[4 * h + 2] = r[2]; o[4 * h + 3] = r[3];
        }
        store32B<ALIGNED32>(out + 2 * (size_t)g, o);
    }
}

// ----------------------------------------------------------------------------- 6-bit dequantize

// IF6 dequantize (decode6x16): one thread per group of 16 (three words of codes in, 32 bytes of bf16 out).
template <ElemKind EK, bool ALIGNED32>
__global__ void __launch_bounds__(256) dequantize6_fast_kernel(const uint32_t* __restrict__ codes,
                                                               const uint8_t* __restrict__ scales,
                                                               const float* __restrict__ alpha_p, int32_t ngroups,
                                                               uint4* __restrict__ out, float c_post) {
    pdl_launch_dependents();
    const int32_t stride = (int32_t)(gridDim.x * blockDim.x);
    if ((int32_t)(blockIdx.x * blockDim.x + threadIdx.x) < ngroups)          // before the wait: see prefetch_l2
        prefetch_l2(codes + 3 * (size_t)(blockIdx.x * blockDim.x + threadIdx.x));
    pdl_wait();
    const float alpha = __ldg(alpha_p);
    for (int32_t g = (int32_t)(blockIdx.x * blockDim.x + threadIdx.x); g < ngroups; g += stride) {
        const uint32_t* cp = codes + 3 * (size_t)g;
        const uint32_t w0 = __ldg(cp), w1 = __ldg(cp + 1), w2 = __ldg(cp + 2);
        const uint32_t sbyte = __ldg(scales + g);
        const uint32_t mag = sbyte & 0x7Fu;
        const bool is_int = sbyte & 0x80u;
        float Delta = e4m3_value(mag);
        if (mag == 0x7Fu) Delta = __uint_as_float(0x7FC00000u);            // E4M3 NaN propagates
        float d = __fmul_rn(Delta, alpha);
        if (is_int) d = __fmul_rn(d, c_post);                              // de-scale integer groups (Sec. 3)
        uint32_t o[8];
        decode6x16<EK>(w0, w1, w2, is_int, d, o);
        store32B<ALIGNED32>(out + 2 * (size_t)g, o);
    }
}

}  // namespace absq
