// Group-quantize kernel for the 4-bit formats (IF4, NVFP4) with the training options of Sec. 4.1:
// the 16-point random Hadamard transform and / or stochastic rounding (App. B).  Same arithmetic as the
// generic kernel, bit for bit, in the packed style of the round-to-nearest fast path: f32x2 butterflies
// for the transform stages that pair whole registers, f32x2 index-domain rounding, integer Horner packing.
#pragma once
#include "abs_fast4.cuh"

namespace absq {

constexpr float kMagic = 12582912.0f;                 // 1.5 * 2^23: x + kMagic leaves RNE(x) in the low mantissa bits
constexpr uint32_t kMagicBits = 0x4B400000u;

__device__ __forceinline__ float min3f(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float max3f(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint32_t sign_of(float y) { return __float_as_uint(y) & 0x80000000u; }

__device__ __forceinline__ uint64_t add2_rp(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rp.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t fma2_rp(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rp.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// Per-element work of one group under stochastic rounding (steps 3-10 of Fig. 3a with both candidates
// rounded stochastically, App. B).  rnd[i] holds the two 16-bit random fields h of elements 2i (low half)
// and 2i+1; u = (h + 1/2) * 2^-16.
//
// The rule "lo if a == lo, else hi iff u < (a - lo) / (hi - lo)" is evaluated as a ceiling.  With phi the
// grid's fractional-index map (grid point g_i -> i, linear in between), the rounded index is ceil(phi(a) - u):
// for phi = n + f it is n when u >= f and n + 1 when u < f.  For E2M1 phi(a) = min(2a, a + 2, a/2 + 4); the
// pieces, the subtraction of u and the final add of 1.5 * 2^23 (which leaves the ceiling in the low mantissa
// bits) all round toward +infinity, and that changes nothing: u is an odd multiple of 2^-17, every rounding
// here is to a grid at least as fine as 2^-21, so a sum rounded up crosses neither u nor an integer that the
// exact sum does not reach.  The value of an index is max(i/2, i - 2, 2i - 8).  The integer candidate is the
// same ceiling on |z|, z = y * 7/6 rounded to FP32 as in the round-to-nearest path, clamped to 7.
template <bool HAS_INT>
__device__ __forceinline__ void encode_body4_sr(const float (&x)[16], const uint32_t (&rnd)[8], uint32_t sb, float d,
                                                float r, uint32_t& sbyte, uint32_t& c_lo, uint32_t& c_hi) {
    const uint64_t R2 = pack2(r, r);
    const uint64_t TWO = pack2(2.0f, 2.0f), HALF = pack2(0.5f, 0.5f), FOUR = pack2(4.0f, 4.0f);
    const uint64_t MG = pack2(kMagic, kMagic), NMG = pack2(-kMagic, -kMagic);
    const uint64_t NSC16 = pack2(-1.0f / 65536.0f, -1.0f / 65536.0f);
    const uint64_t P128MH = pack2(128.0f - 1.0f / 131072.0f, 128.0f - 1.0f / 131072.0f);   // 128 - 2^-17, 24 bits

    const float c_pre = __uint_as_float(0x3F955555u);    // fp32(7/6)
    const float c_post = __uint_as_float(0x3F5B6DB7u);   // fp32(6/7)
    const float d_int = __fmul_rn(d, c_post);
    const uint64_t ND2 = pack2(-d, -d), NDI2 = pack2(-d_int, -d_int), CP2 = pack2(c_pre, c_pre);
    const uint64_t MG8 = pack2(kMagic8, kMagic8);
    const uint64_t NMGH = pack2(-0.5f * kMagic, -0.5f * kMagic), NMG2 = pack2(-(kMagic + 2.0f), -(kMagic + 2.0f));
    const uint64_t NMG8 = pack2(-(2.0f * kMagic + 8.0f), -(2.0f * kMagic + 8.0f));

    uint64_t accF[2], accI[2];
    uint32_t fw[2], kb[16], ib[16];
#pragma unroll
    for (int hgrp = 0; hgrp < 2; ++hgrp) {
        float vs[8], ys[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = 8 * hgrp + 2 * i;
            const uint64_t X = pack2(x[e], x[e + 1]);
            const uint64_t Y = mul2(X, R2);                                    // E1 (step 3)
            float y0, y1;
            unpack2(Y, y0, y1);
            ys[2 * i] = y0; ys[2 * i + 1] = y1;
            // -u = -(h + 1/2) * 2^-16 from the 16-bit fields: 2^23 + h as a float, then one multiply-add whose exact
            // result -(2^23 + h) * 2^-16 + 128 - 2^-17 has 17 significant bits, so nothing is rounded
            const uint32_t rw = rnd[e >> 1];
            const float m0 = __uint_as_float((rw & 0xFFFFu) | 0x4B000000u);
            const float m1 = __uint_as_float(__byte_perm(rw, 0x4B00u, 0x5432));
            const uint64_t NU = fma2(pack2(m0, m1), NSC16, P128MH);
            // E2 under stochastic rounding: index = ceil(phi(a) - u)
            const float a0 = fminf(fabsf(y0), 6.0f), a1 = fminf(fabsf(y1), 6.0f);
            const uint64_t A = pack2(a0, a1);
            float p00, p01, p10, p11, p20, p21;
            unpack2(add2(A, A), p00, p01);                                     // exact
            unpack2(add2_rp(A, TWO), p10, p11);
            unpack2(fma2_rp(A, HALF, FOUR), p20, p21);
            const uint64_t PHI = pack2(min3f(p00, p10, p20), min3f(p01, p11, p21));
            const uint64_t IM = add2_rp(add2_rp(PHI, NU), MG);                 // low mantissa bits = index 0..7
            float im0, im1;
            unpack2(IM, im0, im1);
            ib[e] = __float_as_uint(im0);
            ib[e + 1] = __float_as_uint(im1);
            if constexpr (HAS_INT) {
                // value of the index i = IM - kMagic: max(i/2, i - 2, 2i - 8), each piece formed from IM in one
                // exact operation (kMagic / 2, kMagic + 2 and 2 * kMagic + 8 are all FP32 numbers)
                float q00, q01, q10, q11, q20, q21;
                unpack2(fma2(IM, HALF, NMGH), q00, q01);
                unpack2(add2(IM, NMG2), q10, q11);
                unpack2(fma2(IM, TWO, NMG8), q20, q21);
                const float v0 = max3f(q00, q10, q20), v1 = max3f(q01, q11, q21);          // value of the index
                const float vs0 = __uint_as_float((__float_as_uint(v0) & 0x7FFFFFFFu) | sign_of(y0));
                const float vs1 = __uint_as_float((__float_as_uint(v1) & 0x7FFFFFFFu) | sign_of(y1));
                vs[2 * i] = vs0; vs[2 * i + 1] = vs1;
                const uint64_t E = fma2(pack2(vs0, vs1), ND2, X);              // E3 (steps 5-6), negated; squared below
                accF[hgrp] = (i == 0) ? mul2(E, E) : fma2(E, E, accF[hgrp]);
                // E4 (step 7) under stochastic rounding: |k| = ceil(min(|z|, 7) - u), sign of z put back
                float z0, z1;
                unpack2(mul2(Y, CP2), z0, z1);
                const uint64_t AZ = pack2(fminf(fabsf(z0), 7.0f), fminf(fabsf(z1), 7.0f));
                float k0, k1;
                unpack2(add2(add2_rp(add2_rp(AZ, NU), MG), NMG), k0, k1);
                const float ks0 = __uint_as_float((__float_as_uint(k0) & 0x7FFFFFFFu) | sign_of(z0));
                const float ks1 = __uint_as_float((__float_as_uint(k1) & 0x7FFFFFFFu) | sign_of(z1));
                const uint64_t KS = pack2(ks0, ks1);
                const uint64_t FI = fma2(KS, NDI2, X);                         // E5 (steps 8-9)
                accI[hgrp] = (i == 0) ? mul2(FI, FI) : fma2(FI, FI, accI[hgrp]);
                float km0, km1;
                unpack2(add2(KS, MG8), km0, km1);                              // low nibble = k + 8
                kb[e] = __float_as_uint(km0);
                kb[e + 1] = __float_as_uint(km1);
            }
        }
        if constexpr (HAS_INT) fw[hgrp] = e2m1x8_encode(vs);                   // exact: the values are on the grid
        else fw[hgrp] = e2m1x8_encode(ys) & 0x88888888u;                       // only the signs of y
    }
    if constexpr (!HAS_INT) {
        // codes = index nibbles by Horner on the raw sums (each holds kMagicBits + index) | sign bits
        constexpr uint32_t kConstI = kMagicBits * 0x11111111u;
        uint32_t il = ib[7], ih = ib[15];
#pragma unroll
        for (int j = 6; j >= 0; --j) {
            il = il * 16u + ib[j];
            ih = ih * 16u + ib[8 + j];
        }
        c_lo = (il - kConstI) | fw[0];
        c_hi = (ih - kConstI) | fw[1];
        sbyte = sb;
    } else {
        float f0, f1, f2, f3, i0, i1, i2, i3;
        unpack2(accF[0], f0, f1); unpack2(accF[1], f2, f3);
        unpack2(accI[0], i0, i1); unpack2(accI[1], i2, i3);
        const float E_fp = __fadd_rn(__fadd_rn(f0, f1), __fadd_rn(f2, f3));     // S1-S2 (step 10)
        const float E_int = __fadd_rn(__fadd_rn(i0, i1), __fadd_rn(i2, i3));
        const bool flag = E_int < E_fp;
        constexpr uint32_t kConst = kMagic8Bits * 0x11111111u - 0x88888888u;
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

// Resident blocks of 256 threads per SM the kernel is compiled and launched for: the stochastic-rounding
// instances need about 120 registers, the Hadamard-only ones run best with three blocks, the plain
// round-to-nearest instance (used by the emulation pass only) with four.
constexpr int opt_blocks_per_sm(bool sr, bool rht = true) { return sr ? 2 : (rht ? 3 : 4); }

// Persistent grid-stride kernel, one group of 16 per thread and iteration, next group's 32 bytes fetched
// before the current one is encoded.  scale_mul is 17/16 with that option and 1 otherwise (times 1 is exact).
// EMUL = true is the emulation pass of Sec. 4.1 (every format was emulated by dequantizing right after
// quantizing): the group is decoded from the registers that hold its codes and scale, with the arithmetic of
// the dequantize kernel, and written to `out` as bf16; codes and scale bytes are stored only when
// `store_codes` is set.
template <bool HAS_INT, bool RHT, bool SR, bool FROM_SLOT, bool EMUL>
__global__ void __launch_bounds__(256, opt_blocks_per_sm(SR, RHT))
quantize4_opt_kernel(const uint4* __restrict__ in, uint2* __restrict__ codes, uint8_t* __restrict__ scales,
                     const AlphaSrc alpha_src, int32_t ngroups, float scale_mul, uint32_t sign_mask,
                     const PhiloxKeys keys, uint64_t ctr_base, bool aligned32, uint4* __restrict__ out, bool out_aligned32,
                     bool store_codes) {
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
    __shared__ float2 scale_table[128];
    fill_scale_table(scale_table, alpha);                                    // G5 for every scale byte, once per block
    if (!active) return;
    const float inv_a6 = __frcp_rn(__fmul_rn(alpha, 6.0f));                  // T3
    uint32_t smask[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
        smask[i] = (((sign_mask >> (2 * i)) & 1u) << 15) | (((sign_mask >> (2 * i + 1)) & 1u) << 31);
    while (true) {
        const int32_t gn = g + stride;
        const bool more = gn < ngroups;
        if (more) {
            if (aligned32) load32B<true>(in + 2 * (size_t)gn, wn);
            else load32B<false>(in + 2 * (size_t)gn, wn);
        }
        float x[16];
        if constexpr (RHT) {
            hadamard16_packed(w, smask, x);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                x[2 * i] = __uint_as_float(w[i] << 16);
                x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
            }
        }
        uint32_t rnd[8];
        if constexpr (SR) {
            // Philox blocks 2g and 2g+1 hold the sixteen 16-bit fields of elements 16g .. 16g+15; ctr_base (even)
            // is the block index of the call's first element in the whole tensor (sr_index_offset / 8)
            const uint64_t i8 = ctr_base + (uint64_t)(uint32_t)g * 2u;
            const uint4 p0 = philox4x32_10((uint32_t)i8, (uint32_t)(i8 >> 32), keys);
            const uint4 p1 = philox4x32_10((uint32_t)i8 + 1u, (uint32_t)(i8 >> 32), keys);
            rnd[0] = p0.x; rnd[1] = p0.y; rnd[2] = p0.z; rnd[3] = p0.w;
            rnd[4] = p1.x; rnd[5] = p1.y; rnd[6] = p1.z; rnd[7] = p1.w;
        }
        // G1: group maximum with three-input max.
        const float m0 = max3abs(x[0], x[1], x[2]), m1 = max3abs(x[3], x[4], x[5]);
        const float m2 = max3abs(x[6], x[7], x[8]), m3 = max3abs(x[9], x[10], x[11]);
        const float m4 = max3abs(x[12], x[13], x[14]);
        const float gmax = fmaxf(max3abs(m0, m1, m2), max3abs(m3, m4, x[15]));
        // G2-G3 (Eq. 2), with the 17/16 option folded into scale_mul.
        const float t = __fmul_rn(__fmul_rn(gmax, inv_a6), scale_mul);
        const uint32_t sb = e4m3_encode(t);
        const float2 dr = scale_table[sb];                                 // G5: d = Delta * alpha and 1 / d
        const float d = dr.x, r = dr.y;
        uint32_t sbyte = 0u, c_lo = 0u, c_hi = 0u;
        if constexpr (SR) {
            if (sb != 0u) encode_body4_sr<HAS_INT>(x, rnd, sb, d, r, sbyte, c_lo, c_hi);      // G4: zero scale -> zeros
        } else {
            if ((sb - 8u) >= 118u) {
                if (sb != 0u) encode_body4<HAS_INT, HAS_INT>(x, sb, d, r, sbyte, c_lo, c_hi);
            } else {
                encode_body4<HAS_INT, false>(x, sb, d, r, sbyte, c_lo, c_hi);
            }
        }
        if (!EMUL || store_codes) {
            scales[g] = (uint8_t)sbyte;
            codes[g] = make_uint2(c_lo, c_hi);
        }
        if constexpr (EMUL) {
            const bool is_int = HAS_INT && (sbyte & 0x80u);
            const float dd = is_int ? __fmul_rn(d, __uint_as_float(0x3F5B6DB7u)) : d;        // d * fp32(6/7) for integer groups
            const float addend = is_int ? -1032.0f : -0.0f;
            const uint64_t D2 = pack2(dd, dd);
            uint32_t lo[4], hi[4];
            dequant_word4<HAS_INT>(c_lo, is_int, addend, D2, lo);
            dequant_word4<HAS_INT>(c_hi, is_int, addend, D2, hi);
            const uint32_t o[8] = {lo[0], lo[1], lo[2], lo[3], hi[0], hi[1], hi[2], hi[3]};
            if (out_aligned32) store32B<true>(out + 2 * (size_t)g, o);
            else store32B<false>(out + 2 * (size_t)g, o);
        }
        if (!more) break;
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = wn[i];
        g = gn;
    }
}

}  // namespace absq
