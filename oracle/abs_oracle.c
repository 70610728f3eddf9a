/*
 * abs_oracle.c -- CPU oracle for Adaptive Block-Scaled (IF) quantize / dequantize.
 *
 * TEST INFRASTRUCTURE, NOT PRODUCT.  This file is the slow, plain, scalar statement of
 * what the method computes.  It shares no code, header, table or constant with the CUDA
 * path; only tests, the smoke check and the bench's cpu_baseline / reference arm may call it.
 *
 * What it follows (all section / equation / figure numbers are the paper's):
 *   - Eq. 1 (tensor scale alpha) and Eq. 2 (E4M3 block scale Delta_i), Sec. 3.
 *   - Fig. 3a pseudocode, steps 1-10: NVFP4 is steps 1-4; IF4 evaluates an FP4 and a scaled
 *     INT4 candidate, measures each one's squared error against the input and keeps the
 *     integer candidate iff its error is strictly smaller.
 *   - Sec. 3, "6/7 method": integer groups are pre-scaled by M_INT/M_FP (7/6) and de-scaled by
 *     M_FP/M_INT (6/7); the choice is stored in the sign bit of the group's E4M3 scale.
 *   - Sec. 5.1 footnote: the factor is 4/3 for IF3, 7.5/31 for IF6-E2M3, 28/31 for IF6-E3M2.
 *   - Sec. 4.1: dequantize to FP32, then convert to BF16; random Hadamard transform and
 *     stochastic rounding as options; the 16/17 factor in the gradient scale calculation.
 *   - Appendix B: with stochastic rounding both candidates are rounded stochastically and the
 *     selection then runs on those candidates.
 *
 * The paper states the procedure in real arithmetic.  For a bit-exact comparison the
 * arithmetic is fixed here as IEEE-754 binary32, round-to-nearest-even, subnormals kept,
 * no contraction except where fmaf() is written.  Each step below carries the label used
 * in the design notes (T = per tensor, G = per group, E = per element, S = selection).
 *
 * Parity pins (see tests, "-m 'not gpu'"): worked example of Fig. 3a; FP4 / INT4 grids;
 * Table 1 MSE over N(0,1) for NVFP4 and IF4; flag-0 groups equal NVFP4 byte for byte;
 * exact round trips; chosen error <= other error; brute force per element and per group.
 * Parity unpinned by the paper (pinned only by algebraic identities / statistics of our own
 * reading): the Hadamard option's size, signs and normalisation; the bit pattern of the
 * stochastic-rounding stream; the 17/16 scale option; IF3 / IF6 beyond the printed factors.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fPIC -shared (x86-64, SSE2 math).
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define ORACLE_API __attribute__((visibility("default")))

enum { FMT_NVFP4 = 0, FMT_IF4 = 1, FMT_IF3 = 2, FMT_IF6_E2M3 = 3, FMT_IF6_E3M2 = 4,
       FMT_NVFP4_BS8 = 5, FMT_IF4_BS8 = 6, FMT_IF3_BS8 = 7, FMT_COUNT = 8 };   /* BS8: one scale per 8 values (Sec. 5.1, Table 5) */

enum {
    F_HADAMARD16 = 1u << 0,
    F_STOCHASTIC = 1u << 1,
    F_SR_SCALE_17_16 = 1u << 2,
    F_ALPHA_GIVEN = 1u << 3,
    F_OUT_FP32 = 1u << 4,
    F_FP_GROUPS_ONLY = 1u << 7,   /* dequantize: groups stored as integers come out as +0          */
    F_INT_GROUPS_RAW = 1u << 8    /* dequantize: FP groups come out as +0; integer groups as k * Delta * alpha,
                                     without the M_FP/M_INT de-scale (the MAC applies it on the scale path) */
};

/* Element format of the floating-point candidate plus the integer alternative. */
typedef struct {
    int ebits, mbits, bias; /* minifloat layout s|e..|m.. of the FP candidate           */
    int bits;               /* b: stored bits per element, sign included                 */
    int has_int;            /* 0 for plain NVFP4 (procedure stops after step 4)          */
    float m_fp;             /* largest FP magnitude: 6, 4, 7.5, 28                       */
    float m_int;            /* largest integer magnitude: 7, 3, 31, 31                   */
    int group;              /* values per scale: 16, or 8 for the block-size-8 variants  */
} fmt_desc;

static const fmt_desc FMTS[FMT_COUNT] = {
    /* NVFP4     */ {2, 1, 1, 4, 0, 6.0f, 0.0f, 16},
    /* IF4       */ {2, 1, 1, 4, 1, 6.0f, 7.0f, 16},
    /* IF3       */ {2, 0, 1, 3, 1, 4.0f, 3.0f, 16},
    /* IF6-E2M3  */ {2, 3, 1, 6, 1, 7.5f, 31.0f, 16},
    /* IF6-E3M2  */ {3, 2, 3, 6, 1, 28.0f, 31.0f, 16},
    /* NVFP4-BS8 */ {2, 1, 1, 4, 0, 6.0f, 0.0f, 8},
    /* IF4-BS8   */ {2, 1, 1, 4, 1, 6.0f, 7.0f, 8},
    /* IF3-BS8   */ {2, 0, 1, 3, 1, 4.0f, 3.0f, 8},
};

/* ------------------------------------------------------------------ small helpers */

static float bits_to_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }
static uint32_t f32_to_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }

static float bf16_to_f32(uint16_t h) { return bits_to_f32((uint32_t)h << 16); }

/* FP32 -> BF16, round to nearest, ties to even (Sec. 4.1: FP32 result converted to BF16). */
static uint16_t f32_to_bf16_rne(float f) {
    uint32_t u = f32_to_bits(f);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return (uint16_t)((u >> 16) | 0x0040u); /* NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* Magnitude of minifloat magnitude-code c (sign stripped) for layout (ebits, mbits, bias). */
static double minifloat_value(int mbits, int bias, int c) {
    int e = c >> mbits, m = c & ((1 << mbits) - 1);
    if (e == 0) return ldexp((double)m, 1 - bias - mbits);          /* subnormal / zero */
    return ldexp((double)((1 << mbits) + m), e - bias - mbits);       /* normal           */
}

/* Sorted magnitude grid of a minifloat; returns the number of entries. */
static int build_fp_grid(const fmt_desc* F, double* g) {
    int n = 1 << (F->bits - 1);
    for (int c = 0; c < n; ++c) g[c] = minifloat_value(F->mbits, F->bias, c);
    return n;
}

/* E4M3 magnitudes 0x00..0x7E (0x7F is NaN): 0, k*2^-9 (k=1..7), (8+m)*2^(e-10), max 448. */
static int build_e4m3_grid(double* g) {
    for (int c = 0; c < 127; ++c) g[c] = minifloat_value(3, 7, c);
    return 127;
}

/* Nearest grid index to a >= 0; exact ties go to the even index; above the top saturates. */
static int grid_round_rne(const double* g, int n, float a) {
    if (!(a < g[n - 1])) return n - 1;
    int lo = 0;
    while (lo + 1 < n && g[lo + 1] <= (double)a) ++lo;   /* g[lo] <= a < g[lo+1] */
    double dl = (double)a - g[lo], dh = g[lo + 1] - (double)a;  /* exact in double */
    if (dl < dh) return lo;
    if (dh < dl) return lo + 1;
    return (lo & 1) ? lo + 1 : lo;
}

/* Stochastic rounding on a sorted magnitude grid (Sec. 4.1, App. B): a is clamped to the
 * top; an exact grid value stays; otherwise round up with probability (a-lo)/(hi-lo),
 * realised as "u < p" with u in (0,1). */
static int grid_round_sr(const double* g, int n, float a, float u) {
    if (!(a < g[n - 1])) return n - 1;
    int lo = 0;
    while (lo + 1 < n && g[lo + 1] <= (double)a) ++lo;
    float flo = (float)g[lo], fhi = (float)g[lo + 1];
    if (a == flo) return lo;
    float p = (a - flo) / (fhi - flo);
    return (u < p) ? lo + 1 : lo;
}

/* ------------------------------------------------------------------ Philox4x32-10 */

static void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The uniform in (0,1) that element idx draws: 16-bit field (idx & 7) of the Philox block
 * whose counter is idx / 8; u = (h + 0.5) * 2^-16. */
static float sr_uniform(uint64_t seed, uint64_t idx) {
    uint64_t i8 = idx >> 3;
    uint32_t ctr[4] = {(uint32_t)i8, (uint32_t)(i8 >> 32), 0u, 0u};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t w[4];
    philox4x32_10(ctr, key, w);
    uint32_t h = (w[(idx & 7) >> 1] >> (16 * (idx & 1))) & 0xFFFFu;
    return ((float)h + 0.5f) * (1.0f / 65536.0f);
}

/* ------------------------------------------------------------------ Hadamard option */

/* 16-point blockwise random Hadamard transform (Sec. 4.1 names the transform only):
 * u_i = s_i * x_i with s_i = -1 where bit i of sign_mask is set, natural-order Sylvester
 * butterflies h = 1, 2, 4, 8, every add / subtract rounded to FP32, result times 1/4. */
static void hadamard16(const float in[16], uint16_t sign_mask, float out[16]) {
    float a[16];
    for (int i = 0; i < 16; ++i) a[i] = ((sign_mask >> i) & 1) ? -in[i] : in[i];
    for (int h = 1; h < 16; h <<= 1)
        for (int base = 0; base < 16; base += 2 * h)
            for (int j = base; j < base + h; ++j) {
                float p = a[j], q = a[j + h];
                a[j] = p + q;
                a[j + h] = p - q;
            }
    for (int i = 0; i < 16; ++i) out[i] = a[i] * 0.25f;
}

/* Load one group of 16 inputs as FP32, applying the Hadamard option if asked. */
static void load_group(const uint16_t* in_bf16, uint32_t flags, uint16_t sign_mask, float x[16]) {
    float raw[16];
    for (int i = 0; i < 16; ++i) raw[i] = bf16_to_f32(in_bf16[i]);
    if (flags & F_HADAMARD16) hadamard16(raw, sign_mask, x);
    else memcpy(x, raw, sizeof raw);
}

/* ------------------------------------------------------------------ error sum */

/* Sum of squares of 16 errors in the fixed order: four fused chains over the element sets
 * {0,2,4,6}, {1,3,5,7}, {8,10,12,14}, {9,11,13,15}, then (S0+S1)+(S2+S3); a group of 8 values
 * has the first two chains and the sum S0+S1.  (Fig. 3a steps
 * 6 and 9 print a mean, but the printed value 46.0 is the sum; n = 16 is constant, so the
 * comparison of step 10 is the same either way.) */
static float sum16_sq(const float* e, int n) {
    float s[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    for (int c = 0; c < n / 4; ++c) {
        int first = (c & 1) + 8 * (c >> 1);
        float acc = 0.0f;
        for (int k = 0; k < 4; ++k) { float v = e[first + 2 * k]; acc = fmaf(v, v, acc); }
        s[c] = acc;
    }
    if (n == 8) return s[0] + s[1];          /* a group of 8 has the first two chains only */
    return (s[0] + s[1]) + (s[2] + s[3]);
}

/* ------------------------------------------------------------------ packing */

/* Code j of a group occupies bits [b*j, b*j+b) of a 16*b-bit little-endian integer. */
static void pack_codes(const uint32_t code[16], int b, uint8_t* out) {
    int nbytes = 2 * b;
    memset(out, 0, (size_t)nbytes);
    for (int j = 0; j < 16; ++j)
        for (int k = 0; k < b; ++k)
            if ((code[j] >> k) & 1u) { int pos = b * j + k; out[pos >> 3] |= (uint8_t)(1u << (pos & 7)); }
}

static void unpack_codes(const uint8_t* in, int b, uint32_t code[16]) {
    for (int j = 0; j < 16; ++j) {
        uint32_t c = 0;
        for (int k = 0; k < b; ++k) { int pos = b * j + k; c |= (uint32_t)((in[pos >> 3] >> (pos & 7)) & 1u) << k; }
        code[j] = c;
    }
}

/* E4 (step 7), round-to-nearest path: integer candidate of y.  int(.) rounds the real product
 * y * M_INT/M_FP once: the product of two floats is exact in double, then nearest integer with
 * ties to even, clamped to +-M_INT. */
static float int_candidate_rne(float y, float c_pre, float m_int) {
    float kf = (float)nearbyint((double)y * (double)c_pre);
    if (kf > m_int) kf = m_int;
    if (kf < -m_int) kf = -m_int;
    return kf;
}

/* ------------------------------------------------------------------ exported element-level pieces */

ORACLE_API int abs_oracle_fmt_bits(int fmt) { return (fmt >= 0 && fmt < FMT_COUNT) ? FMTS[fmt].bits : -1; }
ORACLE_API int abs_oracle_fmt_group(int fmt) { return (fmt >= 0 && fmt < FMT_COUNT) ? FMTS[fmt].group : -1; }
ORACLE_API float abs_oracle_fmt_mfp(int fmt) { return FMTS[fmt].m_fp; }
ORACLE_API float abs_oracle_fmt_mint(int fmt) { return FMTS[fmt].m_int; }
/* c_pre = fp32(M_INT / M_FP), c_post = fp32(M_FP / M_INT) (the "6/7 method" constants). */
ORACLE_API float abs_oracle_c_pre(int fmt) { return FMTS[fmt].m_int / FMTS[fmt].m_fp; }
ORACLE_API float abs_oracle_c_post(int fmt) { return FMTS[fmt].m_fp / FMTS[fmt].m_int; }

/* Signed value of FP element code (sign in bit b-1). */
ORACLE_API float abs_oracle_fp_value(int fmt, uint32_t code) {
    const fmt_desc* F = &FMTS[fmt];
    uint32_t sign = (code >> (F->bits - 1)) & 1u;
    float v = (float)minifloat_value(F->mbits, F->bias, (int)(code & ((1u << (F->bits - 1)) - 1u)));
    return sign ? -v : v;
}

/* Step 4: FP element code of y, nearest-even, saturating, sign of y kept (also for -0). */
ORACLE_API uint32_t abs_oracle_fp_encode(int fmt, float y) {
    const fmt_desc* F = &FMTS[fmt];
    double g[64];
    int n = build_fp_grid(F, g);
    uint32_t sign = f32_to_bits(y) >> 31;
    return (sign << (F->bits - 1)) | (uint32_t)grid_round_rne(g, n, fabsf(y));
}

/* Step 7: integer candidate k of a scaled value y (round-to-nearest path). */
ORACLE_API int abs_oracle_int_encode(int fmt, float y) {
    const fmt_desc* F = &FMTS[fmt];
    return (int)int_candidate_rne(y, F->m_int / F->m_fp, F->m_int);
}

/* Step 2: E4M3 byte (0x00..0x7E) nearest to t >= 0, ties to even, saturating at 448. */
ORACLE_API uint32_t abs_oracle_e4m3_encode(float t) {
    double g[127];
    int n = build_e4m3_grid(g);
    return (uint32_t)grid_round_rne(g, n, t);
}

ORACLE_API float abs_oracle_e4m3_value(uint32_t byte) {
    uint32_t c = byte & 0x7Fu;
    if (c == 0x7Fu) return NAN;
    return (float)minifloat_value(3, 7, (int)c);
}

ORACLE_API void abs_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    philox4x32_10(ctr, key, out);
}
ORACLE_API float abs_oracle_sr_uniform(uint64_t seed, uint64_t idx) { return sr_uniform(seed, idx); }
/* Stochastically rounded index of a magnitude on a format's FP grid for a given u (element-level piece for the pins). */
ORACLE_API int abs_oracle_fp_sr(int fmt, float a, float u) {
    double g[64];
    const int n = build_fp_grid(&FMTS[fmt], g);
    return grid_round_sr(g, n, a, u);
}
ORACLE_API void abs_oracle_hadamard16(const float in[16], uint16_t sign_mask, float out[16]) {
    hadamard16(in, sign_mask, out);
}
ORACLE_API uint16_t abs_oracle_f32_to_bf16(float f) { return f32_to_bf16_rne(f); }

/* ------------------------------------------------------------------ T1: amax */

/* T1: A = max |x| over rows [row0,row1) (after the Hadamard option when asked). Exact. */
ORACLE_API float abs_oracle_amax(const uint16_t* in_bf16, int64_t cols, int64_t row0, int64_t row1,
                                 uint32_t flags, uint16_t sign_mask) {
    float A = 0.0f;
    for (int64_t r = row0; r < row1; ++r)
        for (int64_t c = 0; c < cols; c += 16) {
            float x[16];
            load_group(in_bf16 + r * cols + c, flags, sign_mask, x);
            for (int i = 0; i < 16; ++i) { float a = fabsf(x[i]); if (a > A) A = a; }
        }
    return A;
}

/* T2 (Eq. 1): alpha = A / (M_FP * 448); an all-zero tensor gets alpha = 1. */
ORACLE_API float abs_oracle_alpha(int fmt, float amax) {
    float den = FMTS[fmt].m_fp * 448.0f;
    return (amax == 0.0f) ? 1.0f : amax / den;
}

/* ------------------------------------------------------------------ quantize */

/* Quantize rows [row0,row1) of a row-major bf16 matrix with tensor scale alpha.
 * Outputs: codes (rows x cols*b/8 bytes), scales (rows x cols/G bytes, G = values per scale); optional
 * per-group E_FP / E_INT (rows x cols/G floats each, may be NULL) for the selection invariants.
 * sr_index_offset: App. B draws one random stream over the whole tensor; when this matrix is a row shard
 * of a larger one, the offset is the index of its element (0, 0) in that tensor, so that element (r, c)
 * draws field sr_index_offset + r*cols + c. */
ORACLE_API int abs_oracle_quantize_rows(int fmt, const uint16_t* in_bf16, int64_t rows, int64_t cols,
                                        int64_t row0, int64_t row1, float alpha, uint32_t flags,
                                        uint16_t sign_mask, uint64_t sr_seed, uint64_t sr_index_offset,
                                        uint8_t* codes, uint8_t* scales, float* dbg_e_fp, float* dbg_e_int) {
    if (fmt < 0 || fmt >= FMT_COUNT || cols % 16 != 0 || row0 < 0 || row1 > rows) return 1;
    const fmt_desc* F = &FMTS[fmt];
    const int b = F->bits;
    const int m_int = (int)F->m_int;
    double fpg[64], e4g[127], intg[64];
    const int nfp = build_fp_grid(F, fpg);
    const int ne4 = build_e4m3_grid(e4g);
    for (int i = 0; i <= m_int; ++i) intg[i] = (double)i;

    /* T3: per-tensor constants. */
    const float a6 = alpha * F->m_fp;
    const float inv_a6 = 1.0f / a6;
    const float c_pre = F->has_int ? F->m_int / F->m_fp : 0.0f;
    const float c_post = F->has_int ? F->m_fp / F->m_int : 0.0f;
    const int64_t gpr = cols / 16;

    const int G = F->group;                 /* values per scale */
    const int nsub = 16 / G;                /* groups per aligned block of 16 (the Hadamard block) */

    for (int64_t r = row0; r < row1; ++r)
        for (int64_t gi = 0; gi < gpr; ++gi) {
            float x[16];
            load_group(in_bf16 + r * cols + gi * 16, flags, sign_mask, x);
            uint8_t* code_out = codes + (r * gpr + gi) * (2 * b);
            uint32_t chosen[16];
            for (int sub = 0; sub < nsub; ++sub) {
                const float* xs = x + sub * G;
                const int64_t sidx = (r * gpr + gi) * nsub + sub;
                uint32_t q_fp[16], q_int[16];
                float e_fp[16], e_int[16];

                /* G1: group maximum (exact). */
                float gmax = 0.0f;
                for (int i = 0; i < G; ++i) { float a = fabsf(xs[i]); if (a > gmax) gmax = a; }
                /* G2 (Eq. 2; steps 1-2): t = gmax / (alpha * M_FP), as a multiply by the reciprocal. */
                float t = gmax * inv_a6;
                if (flags & F_SR_SCALE_17_16) t = t * 1.0625f;
                /* G3: E4M3 round-to-nearest-even, saturating. */
                uint32_t sb = (uint32_t)grid_round_rne(e4g, ne4, t);
                /* G4: a scale that rounds to zero encodes an all-zero group. */
                if (sb == 0) {
                    for (int i = 0; i < G; ++i) chosen[sub * G + i] = 0u;
                    scales[sidx] = 0x00;
                    if (dbg_e_fp) dbg_e_fp[sidx] = 0.0f;
                    if (dbg_e_int) dbg_e_int[sidx] = 0.0f;
                    continue;
                }
                /* G5: decoded block scale, combined scale and its reciprocal. */
                const float Delta = (float)e4g[sb];
                const float d = Delta * alpha;
                const float rcp = 1.0f / d;
                const float d_int = d * c_post;

                for (int i = 0; i < G; ++i) {
                    const float xi = xs[i];
                    float u = 0.0f;
                    if (flags & F_STOCHASTIC)
                        u = sr_uniform(sr_seed, sr_index_offset + (uint64_t)(r * cols + gi * 16 + sub * G + i));
                    /* E1 (step 3). */
                    const float y = xi * rcp;
                    const uint32_t ysign = f32_to_bits(y) >> 31;
                    /* E2 (step 4): FP candidate code. */
                    int mi = (flags & F_STOCHASTIC) ? grid_round_sr(fpg, nfp, fabsf(y), u)
                                                    : grid_round_rne(fpg, nfp, fabsf(y));
                    q_fp[i] = (ysign << (b - 1)) | (uint32_t)mi;
                    /* E3 (steps 5-6): error of the dequantized FP candidate, one fused rounding. */
                    float vfp = (float)fpg[mi];
                    if (ysign) vfp = -vfp;
                    e_fp[i] = fmaf(vfp, d, -xi);
                    if (!F->has_int) continue;
                    /* E4 (step 7): integer candidate of y * M_INT / M_FP, clamped to +-M_INT. */
                    float kf;
                    if (flags & F_STOCHASTIC) {
                        const float z = y * c_pre;   /* the stochastic draw needs the FP32 value itself */
                        kf = (float)grid_round_sr(intg, m_int + 1, fabsf(z), u);
                        if (f32_to_bits(z) >> 31) kf = -kf;
                    } else {
                        kf = int_candidate_rne(y, c_pre, F->m_int);
                    }
                    const int k = (int)kf;
                    q_int[i] = (uint32_t)k & ((1u << b) - 1u);   /* two's complement in b bits */
                    /* E5 (steps 8-9): error of the dequantized integer candidate. */
                    e_int[i] = fmaf((float)k, d_int, -xi);
                }

                /* S1-S3 (step 10): keep the integer candidate iff its error is strictly smaller. */
                int flag = 0;
                float E_fp = sum16_sq(e_fp, G), E_int = 0.0f;
                if (F->has_int) {
                    E_int = sum16_sq(e_int, G);
                    flag = (E_int < E_fp) ? 1 : 0;
                }
                if (dbg_e_fp) dbg_e_fp[sidx] = E_fp;
                if (dbg_e_int) dbg_e_int[sidx] = E_int;
                scales[sidx] = (uint8_t)(sb | ((uint32_t)flag << 7));
                for (int i = 0; i < G; ++i) chosen[sub * G + i] = flag ? q_int[i] : q_fp[i];
            }
            /* S4: the 16 codes of the block form one little-endian bitstream, whatever the group size. */
            pack_codes(chosen, b, code_out);
        }
    return 0;
}

/* ------------------------------------------------------------------ dequantize */

/* Dequantize rows [row0,row1): value(code) * (Delta * alpha [* M_FP/M_INT for integer groups]),
 * product in FP32, then BF16 round-to-nearest-even (or FP32 when out_fp32 != 0).  `select` splits the
 * tensor for the MAC arithmetic of Sec. 5.2: FP groups only, or integer groups only and without de-scale. */
ORACLE_API int abs_oracle_dequantize_rows(int fmt, const uint8_t* codes, const uint8_t* scales, float alpha,
                                          int64_t rows, int64_t cols, int64_t row0, int64_t row1,
                                          int out_fp32, void* out, uint32_t select) {
    if (fmt < 0 || fmt >= FMT_COUNT || cols % 16 != 0 || row0 < 0 || row1 > rows) return 1;
    const fmt_desc* F = &FMTS[fmt];
    const int b = F->bits;
    const float c_post = F->has_int ? F->m_fp / F->m_int : 0.0f;
    const int64_t gpr = cols / 16;
    const int G = F->group, nsub = 16 / G;
    for (int64_t r = row0; r < row1; ++r)
        for (int64_t gi = 0; gi < gpr; ++gi) {
            uint32_t code[16];
            unpack_codes(codes + (r * gpr + gi) * (2 * b), b, code);
            for (int i = 0; i < 16; ++i) {
                const uint8_t sbyte = scales[(r * gpr + gi) * nsub + i / G];
                /* Sec. 3: the flag lives in the sign bit that an NVFP4 scale leaves unused; a plain NVFP4
                 * tensor has no integer groups, so there the bit is ignored and the byte is its magnitude. */
                const int flag = F->has_int ? (sbyte >> 7) : 0;
                const float Delta = abs_oracle_e4m3_value(sbyte);
                float d = Delta * alpha;
                if (flag && !(select & F_INT_GROUPS_RAW)) d = d * c_post;
                const int masked = (flag && (select & F_FP_GROUPS_ONLY)) || (!flag && (select & F_INT_GROUPS_RAW));
                float v;
                if (flag) {
                    int k = (int)code[i];
                    if (k & (1 << (b - 1))) k -= (1 << b);   /* sign-extend b bits */
                    v = (float)k;
                } else {
                    v = abs_oracle_fp_value(fmt, code[i]);
                }
                const float o = masked ? 0.0f : v * d;
                const int64_t at = r * cols + gi * 16 + i;
                if (out_fp32) ((float*)out)[at] = o;
                else ((uint16_t*)out)[at] = f32_to_bf16_rne(o);
            }
        }
    return 0;
}
