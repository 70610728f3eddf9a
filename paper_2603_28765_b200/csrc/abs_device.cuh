// Device-side building blocks of the IF quantize / dequantize kernels (sm_100a only).
//
// Every floating-point operation that decides a stored bit is written with an explicit
// rounding intrinsic (__fmul_rn, __fmaf_rn, ...), so the compiler never contracts or
// reorders it; the file is compiled with -fmad=false as a second line of defence.
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <nvtx3/nvToolsExt.h>

namespace absq {

// Host-side NVTX range around the enqueue work of one library call, so that a timeline tool shows which call
// launched which kernels.  Header-only NVTX: without a tool attached a push / pop is one load and a branch.
struct CallRange {
    explicit CallRange(const char* name) { nvtxRangePushA(name); }
    ~CallRange() { nvtxRangePop(); }
    CallRange(const CallRange&) = delete;
    CallRange& operator=(const CallRange&) = delete;
};

enum ElemKind { EK_E2M1 = 0, EK_E2M0 = 1, EK_E2M3 = 2, EK_E3M2 = 3 };

// Format traits: (M_FP, M_INT, bits) per Sec. 3 (IF4) and the Sec. 5.1 footnote (IF3, IF6).
template <int FMT> struct Fmt;
template <> struct Fmt<0> {  // NVFP4: Fig. 3a stops after step 4
    static constexpr int BITS = 4; static constexpr int GROUP = 16; static constexpr bool HAS_INT = false; static constexpr ElemKind EK = EK_E2M1;
    static constexpr float M_FP = 6.0f, M_INT = 0.0f; static constexpr int EMIN = 0, MBITS = 1;
};
template <> struct Fmt<1> {  // IF4
    static constexpr int BITS = 4; static constexpr int GROUP = 16; static constexpr bool HAS_INT = true; static constexpr ElemKind EK = EK_E2M1;
    static constexpr float M_FP = 6.0f, M_INT = 7.0f; static constexpr int EMIN = 0, MBITS = 1;
};
template <> struct Fmt<2> {  // IF3: E2M0 or INT3
    static constexpr int BITS = 3; static constexpr int GROUP = 16; static constexpr bool HAS_INT = true; static constexpr ElemKind EK = EK_E2M0;
    static constexpr float M_FP = 4.0f, M_INT = 3.0f; static constexpr int EMIN = 0, MBITS = 0;
};
template <> struct Fmt<3> {  // IF6-E2M3
    static constexpr int BITS = 6; static constexpr int GROUP = 16; static constexpr bool HAS_INT = true; static constexpr ElemKind EK = EK_E2M3;
    static constexpr float M_FP = 7.5f, M_INT = 31.0f; static constexpr int EMIN = 0, MBITS = 3;
};
template <> struct Fmt<4> {  // IF6-E3M2
    static constexpr int BITS = 6; static constexpr int GROUP = 16; static constexpr bool HAS_INT = true; static constexpr ElemKind EK = EK_E3M2;
    static constexpr float M_FP = 28.0f, M_INT = 31.0f; static constexpr int EMIN = -2, MBITS = 2;
};

// Block-size-8 variants (Sec. 5.1, Table 5): the same element formats with one scale per 8 values.
template <> struct Fmt<5> : Fmt<0> { static constexpr int GROUP = 8; };   // NVFP4-BS8
template <> struct Fmt<6> : Fmt<1> { static constexpr int GROUP = 8; };   // IF4-BS8
template <> struct Fmt<7> : Fmt<2> { static constexpr int GROUP = 8; };   // IF3-BS8

// ----------------------------------------------------------------------------- conversions

// Fig. 3a step 2: FP32 -> E4M3 byte, nearest-even, saturating at 448 (hardware convert).
__device__ __forceinline__ uint32_t e4m3_encode(float t) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.0f), "f"(t));
    return (uint32_t)r;                      // the upper byte is the code of the first source, +0.0, i.e. 0x00
}

// Value of an E4M3 magnitude byte 0x00..0x7E: the byte placed in FP32's exponent/mantissa top
// bits is (1+m/8)*2^(e-127) (or m*2^-129 for e = 0, an FP32 subnormal); times 2^120 it is exact.
__device__ __forceinline__ float e4m3_value(uint32_t mag7) {
    return __fmul_rn(__uint_as_float(mag7 << 20), 1.329227995784916e36f /* 2^120 */);
}

// Step 4 for E2M1, two values at once: returns (code(y1) << 4) | code(y0).
__device__ __forceinline__ uint32_t e2m1x2_encode(float y0, float y1) {
    uint16_t r;
    asm("{ .reg .b8 t; cvt.rn.satfinite.e2m1x2.f32 t, %1, %2; cvt.u16.u8 %0, t; }" : "=h"(r) : "f"(y1), "f"(y0));
    return (uint32_t)r;
}
// Values of the two E2M1 codes of a byte as a half2 (low nibble in the low half).
__device__ __forceinline__ __half2 e2m1x2_decode(uint32_t byte) {
    uint32_t h2;
    asm("{ .reg .b8 t; cvt.u8.u16 t, %1; cvt.rn.f16x2.e2m1x2 %0, t; }" : "=r"(h2) : "h"((uint16_t)byte));
    return *reinterpret_cast<__half2*>(&h2);
}
// E2M3 / E3M2: two 6-bit codes in the two bytes of a 16-bit container (y0 in the low byte).
__device__ __forceinline__ uint32_t e2m3x2_encode(float y0, float y1) {
    uint16_t r;
    asm("cvt.rn.satfinite.e2m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(y1), "f"(y0));
    return (uint32_t)r;
}
__device__ __forceinline__ uint32_t e3m2x2_encode(float y0, float y1) {
    uint16_t r;
    asm("cvt.rn.satfinite.e3m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(y1), "f"(y0));
    return (uint32_t)r;
}
__device__ __forceinline__ __half2 e2m3x2_decode(uint32_t two_bytes) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e2m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)two_bytes));
    return *reinterpret_cast<__half2*>(&h2);
}
__device__ __forceinline__ __half2 e3m2x2_decode(uint32_t two_bytes) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e3m2x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)two_bytes));
    return *reinterpret_cast<__half2*>(&h2);
}

// E2M0 has no hardware convert: magnitudes {0,1,2,4}, ties to the even code
// (0.5 -> 0, 1.5 -> 2, 3 -> 2), saturating at 4.  Returns the 3-bit code s|ee.
__device__ __forceinline__ uint32_t e2m0_encode(float y) {
    float a = fabsf(y);
    uint32_t idx = (a > 0.5f ? 1u : 0u) + (a >= 1.5f ? 1u : 0u) + (a > 3.0f ? 1u : 0u);
    return idx | ((__float_as_uint(y) >> 31) << 2);
}
__device__ __forceinline__ float e2m0_value(uint32_t code) {
    uint32_t idx = code & 3u;
    float v = (idx == 3u) ? 4.0f : (float)idx;
    return (code & 4u) ? -v : v;
}

// FP element codes and their values for a pair of scaled inputs (steps 4-5).
template <ElemKind EK>
__device__ __forceinline__ void fp_encode_pair(float y0, float y1, uint32_t& c0, uint32_t& c1, float& v0, float& v1) {
    if constexpr (EK == EK_E2M1) {
        uint32_t byte = e2m1x2_encode(y0, y1);
        c0 = byte & 0xFu; c1 = byte >> 4;
        float2 v = __half22float2(e2m1x2_decode(byte));
        v0 = v.x; v1 = v.y;
    } else if constexpr (EK == EK_E2M3) {
        uint32_t w = e2m3x2_encode(y0, y1);
        c0 = w & 0x3Fu; c1 = (w >> 8) & 0x3Fu;
        float2 v = __half22float2(e2m3x2_decode(w));
        v0 = v.x; v1 = v.y;
    } else if constexpr (EK == EK_E3M2) {
        uint32_t w = e3m2x2_encode(y0, y1);
        c0 = w & 0x3Fu; c1 = (w >> 8) & 0x3Fu;
        float2 v = __half22float2(e3m2x2_decode(w));
        v0 = v.x; v1 = v.y;
    } else {
        c0 = e2m0_encode(y0); c1 = e2m0_encode(y1);
        v0 = e2m0_value(c0); v1 = e2m0_value(c1);
    }
}

// Value of one FP element code (dequantize path).
template <ElemKind EK>
__device__ __forceinline__ float2 fp_decode_pair(uint32_t c0, uint32_t c1) {
    if constexpr (EK == EK_E2M1) return __half22float2(e2m1x2_decode((c0 & 0xFu) | ((c1 & 0xFu) << 4)));
    else if constexpr (EK == EK_E2M3) return __half22float2(e2m3x2_decode((c0 & 0x3Fu) | ((c1 & 0x3Fu) << 8)));
    else if constexpr (EK == EK_E3M2) return __half22float2(e3m2x2_decode((c0 & 0x3Fu) | ((c1 & 0x3Fu) << 8)));
    else return make_float2(e2m0_value(c0), e2m0_value(c1));
}

// ----------------------------------------------------------------------------- stochastic rounding

// Philox4x32-10 (Salmon et al.): counter (c0,c1,0,0), key (k0,k1).
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t k0, uint32_t k1) {
    uint32_t c2 = 0u, c3 = 0u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

// The same generator with its ten round keys (key + r * Weyl constant) computed once on the host and passed as a
// kernel parameter: every key is then a constant-bank operand of the XOR that consumes it, and the two additions
// per round disappear from the kernel (40 instructions per group of 16 values).
struct PhiloxKeys { uint32_t k0[10], k1[10]; };
inline PhiloxKeys philox_keys(uint64_t seed) {
    PhiloxKeys K;
    uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) { K.k0[r] = a; K.k1[r] = b; a += 0x9E3779B9u; b += 0xBB67AE85u; }
    return K;
}
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, const PhiloxKeys& K) {
    uint32_t c2 = 0u, c3 = 0u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ K.k0[r]; c1 = lo1; c2 = hi0 ^ c3 ^ K.k1[r]; c3 = lo0;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Stochastic rounding of a magnitude onto a minifloat grid with MBITS mantissa bits and smallest
// normal exponent EMIN: clamp to the top; step s = 2^(max(exponent, EMIN) - MBITS); lo = floor to
// the step; round up iff u < (a - lo) / s.  All operations are exact in FP32.
template <int EMIN, int MBITS>
__device__ __forceinline__ float sr_round_fp(float a, float top, float u) {
    a = fminf(a, top);
    int e = (int)(__float_as_uint(a) >> 23) - 127;
    e = max(e, EMIN);
    float s = __uint_as_float((uint32_t)(e - MBITS + 127) << 23);
    float inv_s = __uint_as_float((uint32_t)(MBITS - e + 127) << 23);
    float lo = __fmul_rn(floorf(__fmul_rn(a, inv_s)), s);
    float p = __fmul_rn(__fsub_rn(a, lo), inv_s);
    return (u < p) ? __fadd_rn(lo, s) : lo;
}
__device__ __forceinline__ float sr_round_int(float a, float top, float u) {
    a = fminf(a, top);
    float lo = floorf(a);
    float p = __fsub_rn(a, lo);
    return (u < p) ? __fadd_rn(lo, 1.0f) : lo;
}

// ----------------------------------------------------------------------------- packed f32x2 arithmetic

__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float max3abs(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(fabsf(a)), "f"(fabsf(b)), "f"(fabsf(c)));
    return d;
}

// ----------------------------------------------------------------------------- Hadamard option

// 16-point transform of one group held in registers: sign flips from the mask, natural-order
// Sylvester butterflies h = 1,2,4,8 with every add/sub rounded to FP32, then times 1/4.
__device__ __forceinline__ void hadamard16(float (&a)[16], uint32_t sign_mask) {
#pragma unroll
    for (int i = 0; i < 16; ++i) a[i] = __uint_as_float(__float_as_uint(a[i]) ^ (((sign_mask >> i) & 1u) << 31));
#pragma unroll
    for (int h = 1; h < 16; h <<= 1) {
#pragma unroll
        for (int base = 0; base < 16; base += 2 * h) {
#pragma unroll
            for (int j = base; j < base + h; ++j) {
                float p = a[j], q = a[j + h];
                a[j] = __fadd_rn(p, q);
                a[j + h] = __fsub_rn(p, q);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 16; ++i) a[i] = __fmul_rn(a[i], 0.25f);
}

// 16-point transform of one group given as eight bf16x2 words: sign flips on the packed words (smask has
// bit 15 / 31 of word i set where elements 2i / 2i+1 are negated), the h = 1 stage inside each pair with
// scalar adds, the h = 2, 4, 8 stages on whole pairs with packed add and fused (p - q = fma(q, -1, p), one
// rounding), then times 1/4.  Natural-order Sylvester butterflies, every result rounded to FP32.
// SCALE = false leaves out the final factor 1/4 (for a maximum it can be applied once at the end:
// rounding is monotone, so max_i fl(x_i / 4) = fl(max_i x_i / 4)).
template <bool SCALE = true>
__device__ __forceinline__ void hadamard16_packed(const uint32_t (&w)[8], const uint32_t (&smask)[8], float (&x)[16]) {
    uint64_t P[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t v = w[i] ^ smask[i];
        const float p = __uint_as_float(v << 16), q = __uint_as_float(v & 0xFFFF0000u);
        P[i] = pack2(__fadd_rn(p, q), __fsub_rn(p, q));
    }
    const uint64_t NEG1 = pack2(-1.0f, -1.0f), QUARTER = pack2(0.25f, 0.25f);
#pragma unroll
    for (int h = 1; h < 8; h <<= 1) {
#pragma unroll
        for (int base = 0; base < 8; base += 2 * h) {
#pragma unroll
            for (int j = base; j < base + h; ++j) {
                const uint64_t p = P[j], q = P[j + h];
                P[j] = add2(p, q);
                P[j + h] = fma2(q, NEG1, p);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) unpack2(SCALE ? mul2(P[i], QUARTER) : P[i], x[2 * i], x[2 * i + 1]);
}


// ----------------------------------------------------------------------------- loads / stores / launch order

// 32 contiguous bytes per thread.  With a 32-byte aligned base one 256-bit access covers a group's
// bf16 values, so a warp touches 1 KiB of whole sectors per instruction; otherwise two 128-bit ones.
template <bool ALIGNED32>
__device__ __forceinline__ void load32B(const void* p, uint32_t (&w)[8]) {
    if constexpr (ALIGNED32) {
        asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                     : "l"(p));
    } else {
        const uint4 a = __ldg(reinterpret_cast<const uint4*>(p)), b = __ldg(reinterpret_cast<const uint4*>(p) + 1);
        w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w; w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
    }
}
template <bool ALIGNED32>
__device__ __forceinline__ void store32B(void* p, const uint32_t (&w)[8]) {
    if constexpr (ALIGNED32) {
        asm volatile("st.global.L1::no_allocate.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                     :: "l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                     : "memory");
    } else {
        reinterpret_cast<uint4*>(p)[0] = make_uint4(w[0], w[1], w[2], w[3]);
        reinterpret_cast<uint4*>(p)[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
}

// Programmatic dependent launch: every kernel lets the next kernel of the stream be scheduled
// early and itself waits for the previous kernel's completion (and memory) before it touches
// global memory, so only block scheduling and register set-up overlap.  Both are no-ops for a
// kernel launched without the attribute.
// Requests the line at p into the L2.  A prefetch consumes nothing and the L2 is where writes of other SMs land,
// so it may be issued BEFORE griddepcontrol.wait: a block that is resident but still waiting for the previous
// kernel of the stream has its first data on the way when the wait ends (group-quantize kernel at 8192x4096,
// launched back to back: 17.3 -> 16.7 us).
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" :: "l"(p)); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// How a quantize kernel learns alpha (Eq. 1): either a float the caller supplied, or the running
// maximum that the amax pass of the same call left in a scratch slot.  The slot holds
// (generation << 32) | bits(max |x|): every call uses a larger generation, so a 64-bit atomicMax never
// needs the slot cleared and the amax pass needs no "last block" epilogue.
struct AlphaSrc {
    const float* alpha_p;                 // used when slot == nullptr
    const unsigned long long* slot;       // tagged maximum written by amax_kernel
    uint32_t gen;                         // generation of this call
    float denom;                          // M_FP * 448
    float* alpha_out;                     // where alpha is published for the caller
    uint32_t* overrun;                    // host-mapped word set when the slot carries another call's generation
};
// After the amax pass of the same call the slot holds this call's generation.  Any other generation means
// that a later call reused the slot while this one was still in flight (more than ABS_MAX_INFLIGHT calls
// between the two): the maximum is lost.  The kernel then reports it through the host-mapped word, which
// the next library call on the device turns into ABS_ERR_SIZE, and continues with alpha = 1.
__device__ __forceinline__ float slot_amax(const AlphaSrc& a, unsigned long long v, bool reporter) {
    if ((uint32_t)(v >> 32) == a.gen) return __uint_as_float((uint32_t)v);
    if (reporter && a.overrun) *reinterpret_cast<volatile uint32_t*>(a.overrun) = 1u;
    return 0.0f;
}
// Must be called by every thread of the block (it synchronises): thread 0 reads the slot, divides once
// (Eq. 1) and shares alpha through shared memory, so one-group-per-thread launches do not pay a division
// per thread.  Block 0 also publishes alpha for the caller.
template <bool FROM_SLOT>
__device__ __forceinline__ float resolve_alpha(const AlphaSrc& a) {
    if constexpr (!FROM_SLOT) return __ldg(a.alpha_p);
    __shared__ float alpha_shared;
    if (threadIdx.x == 0) {
        const unsigned long long v = *reinterpret_cast<const volatile unsigned long long*>(a.slot);
        const float A = slot_amax(a, v, blockIdx.x == 0);
        const float alpha = (A == 0.0f) ? 1.0f : __fdiv_rn(A, a.denom);                   // Eq. 1
        alpha_shared = alpha;
        if (blockIdx.x == 0) *a.alpha_out = alpha;
    }
    __syncthreads();
    return alpha_shared;
}

// The same without a barrier: every thread reads the slot (one L2 line, broadcast) and divides for itself.
// For the grid-stride kernels whose threads handle several groups each: the dozen instructions of the IEEE
// division are spread over those groups, and no block waits at a barrier before its first group
// (measured 1 % faster for abs_quantize at 256 MiB than the shared-memory version).
template <bool FROM_SLOT>
__device__ __forceinline__ float resolve_alpha_per_thread(const AlphaSrc& a) {
    if constexpr (!FROM_SLOT) return __ldg(a.alpha_p);
    const unsigned long long v = __ldcg(a.slot);
    const float A = slot_amax(a, v, blockIdx.x == 0 && threadIdx.x == 0);
    const float alpha = (A == 0.0f) ? 1.0f : __fdiv_rn(A, a.denom);                           // Eq. 1
    if (blockIdx.x == 0 && threadIdx.x == 0) *a.alpha_out = alpha;
    return alpha;
}

// Per-block table of G5 for every scale byte 0x00..0x7E: d = Delta * alpha and its IEEE reciprocal depend only on
// the byte, so a block computes the 127 pairs once and a group reads its pair with one 8-byte load instead of a
// multiply, a multiply and a reciprocal (same operations, same bits).  Every thread of the block must call this
// (it ends with a barrier); entry 0 (d = 0) is never read.
__device__ __forceinline__ void fill_scale_table(float2* table, float alpha) {
    if (threadIdx.x < 127) {
        const float d = __fmul_rn(e4m3_value(threadIdx.x), alpha);
        table[threadIdx.x] = make_float2(d, __frcp_rn(d));
    }
    __syncthreads();
}

// Byte offset of the scale of (row, k-th group of the row) in the 128x4-tile layout read by Blackwell
// block-scaled MMAs; ktiles = ceil(groups_per_row / 4).
__device__ __forceinline__ size_t swizzled_scale_offset(uint32_t row, uint32_t k, uint32_t ktiles) {
    return ((size_t)(row >> 7) * ktiles + (k >> 2)) * 512u + (row & 31u) * 16u + ((row >> 5) & 3u) * 4u + (k & 3u);
}
// Where group g's scale byte goes: row-major, or the tiled layout when `gpr` (groups per row) is non-zero.
template <bool SWZ>
__device__ __forceinline__ size_t scale_offset(size_t g, uint32_t gpr, uint32_t ktiles) {
    if constexpr (!SWZ) return g;
    const uint32_t row = (uint32_t)(g / gpr);
    return swizzled_scale_offset(row, (uint32_t)(g - (size_t)row * gpr), ktiles);
}

// ----------------------------------------------------------------------------- unpack

__device__ __forceinline__ void unpack_bf16x8(const uint4& v, float* x) {
    x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xFFFF0000u);
    x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xFFFF0000u);
    x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xFFFF0000u);
    x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xFFFF0000u);
}

// Pack 16 b-bit codes into the little-endian bitstream (code j at bits [b*j, b*j+b)).
template <int BITS>
__device__ __forceinline__ void pack_codes(const uint32_t (&c)[16], uint32_t (&w)[3]) {
    w[0] = w[1] = w[2] = 0u;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const int pos = BITS * j, word = pos >> 5, sh = pos & 31;
        w[word] |= c[j] << sh;
        if (sh + BITS > 32) w[word + 1] |= c[j] >> (32 - sh);
    }
}
template <int BITS>
__device__ __forceinline__ uint32_t extract_code(const uint32_t (&w)[3], int j) {
    const int pos = BITS * j, word = pos >> 5, sh = pos & 31;
    uint32_t v = w[word] >> sh;
    if (sh + BITS > 32) v |= w[word + 1] << (32 - sh);
    return v & ((1u << BITS) - 1u);
}

}  // namespace absq
