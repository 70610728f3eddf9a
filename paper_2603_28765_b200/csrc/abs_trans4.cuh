// Transposed group-quantize kernel for the 4-bit formats (IF4, NVFP4): groups run down the columns of the
// row-major input (Sec. 4.1: both operands of the weight-gradient product are quantized along the token
// dimension), with the Hadamard and stochastic-rounding options of the gradient path.
#pragma once
#include "abs_opt4.cuh"
#include <type_traits>

namespace absq {

// ----------------------------------------------------------------------------- transposed quantize

// Quantizes the TRANSPOSE of a row-major [rows, cols] matrix without materialising it: groups are 16
// consecutive ROWS of one column (Sec. 4.1: both operands of the weight-gradient product are quantized
// along the token dimension).  Output = what the plain kernel would give for the [cols, rows] matrix:
// codes_t [cols, rows/2 bytes], scales_t [cols, rows/16].
// Persistent blocks walk over tiles of 64 rows x 256 columns.  A tile is brought into shared memory with
// 16-byte asynchronous copies (cp.async), double buffered: the copies of the block's next tile are in
// flight while it encodes the current one.  Thread c reads its column's values down the tile and encodes
// the four groups of 16 rows; those are neighbours in the transposed output, so their codes leave as one
// 256-bit store and their scale bytes as one 32-bit store whenever the tile is complete and the output
// addresses allow it.
constexpr int kTransUnroll = 4;
constexpr int kTransTileCols = 256;
constexpr int kTransTileRowBlocks = 4;
constexpr int kTransStageElems = 16 * kTransTileRowBlocks * kTransTileCols;        // bf16 elements per stage
constexpr int kTransSmemBytes = 2 * kTransStageElems * 2;                           // two stages

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

// 16-point transform of one group held as sixteen floats: sign flips, the h = 1 stage with scalar adds,
// the h = 2, 4, 8 stages on register pairs with packed add / fused subtract, times 1/4 (same arithmetic as
// hadamard16, every result rounded to FP32 once).
__device__ __forceinline__ void hadamard16_pairs(float (&x)[16], uint32_t sign_mask) {
    uint64_t P[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float p = __uint_as_float(__float_as_uint(x[2 * i]) ^ (((sign_mask >> (2 * i)) & 1u) << 31));
        const float q = __uint_as_float(__float_as_uint(x[2 * i + 1]) ^ (((sign_mask >> (2 * i + 1)) & 1u) << 31));
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
    for (int i = 0; i < 8; ++i) unpack2(mul2(P[i], QUARTER), x[2 * i], x[2 * i + 1]);
}

// MODE 0: quantize.  MODE 1: only the maximum of the Hadamard-transformed column groups (the amax pass of
// the transposed path with the Hadamard option; publishes a tagged maximum like amax_kernel).
// SR: stochastic rounding of both candidates (App. B); element indices, and so the Philox counters, are
// those of the transposed matrix.  scale_mul is 17/16 with that option and 1 otherwise.
// EMUL (MODE 0 only): the emulation pass of Sec. 4.1 along the columns.  Every group is decoded from the
// registers that hold its codes and written back over its own input values in the shared-memory tile; the
// finished tile then leaves with coalesced 16-byte stores to `out`, a [rows, cols] matrix in the ORIGINAL
// orientation.  Codes and scales (transposed layout) are stored only when `store_codes` is set.
template <bool HAS_INT, bool FROM_SLOT, bool RHT, bool SR, int MODE, bool EMUL>
__device__ __forceinline__ void quantize4_transposed_body(const uint16_t* __restrict__ in, uint2* __restrict__ codes_t,
                                                          uint8_t* __restrict__ scales_t, const AlphaSrc alpha_src,
                                                          int64_t rows, int64_t cols, uint32_t sign_mask,
                                                          unsigned long long* amax_slot, uint32_t amax_gen,
                                                          float scale_mul, const PhiloxKeys& keys,
                                                          uint64_t ctr_base, uint16_t* __restrict__ out,
                                                          bool store_codes) {
    extern __shared__ __align__(16) uint16_t trans_smem[];
    pdl_launch_dependents();
    pdl_wait();
    float alpha = 1.0f, inv_a6 = 1.0f;
    if constexpr (MODE == 0) {
        alpha = resolve_alpha<FROM_SLOT>(alpha_src);                         // T2
        inv_a6 = __frcp_rn(__fmul_rn(alpha, 6.0f));                          // T3
    }
    uint32_t local_max = 0u;
    const int64_t rblocks = rows / 16;
    const int64_t ntx = (cols + kTransTileCols - 1) / kTransTileCols;
    const int64_t nty = (rblocks + kTransTileRowBlocks - 1) / kTransTileRowBlocks;
    const int64_t ntiles = ntx * nty;
    // vector stores need 32-byte aligned code addresses and 4-byte aligned scale addresses for every column
    const bool vec_ok = (rblocks % kTransTileRowBlocks) == 0 &&
                        ((reinterpret_cast<uintptr_t>(codes_t) & 31u) == 0) && ((reinterpret_cast<uintptr_t>(scales_t) & 3u) == 0);

    // issue the asynchronous copies of tile t = (ty, tx) into stage s (one commit group per call, possibly empty).
    auto issue = [&](int64_t t, uint32_t ty, uint32_t tx, int s) {
        if (t < ntiles) {
            const int64_t rb0 = (int64_t)ty * kTransTileRowBlocks, c0 = (int64_t)tx * kTransTileCols;
            const int nrb = (int)min((int64_t)kTransTileRowBlocks, rblocks - rb0);
            const int ncols = (int)min((int64_t)kTransTileCols, cols - c0);
            uint16_t* stage = trans_smem + s * kTransStageElems;
            const uint16_t* src = in + rb0 * 16 * cols + c0;
            if (ncols == kTransTileCols && nrb == kTransTileRowBlocks) {
                // complete tile: 2048 chunks of 16 bytes, chunk ch = thread + 256 j lands at stage + 8 ch and comes
                // from row (thread / 32) + 8 j, columns 8 (thread % 32) ...
                uint16_t* dst = stage + 8 * threadIdx.x;
                const uint16_t* from = src + (int64_t)(threadIdx.x >> 5) * cols + 8 * (threadIdx.x & 31);
                const int64_t step = 8 * cols;
#pragma unroll
                for (int j = 0; j < 16 * kTransTileRowBlocks * (kTransTileCols / 8) / 256; ++j)
                    cp_async16(dst + j * 8 * 256, from + j * step);
            } else if (ncols == kTransTileCols) {        // full-width tile: 32 chunks of 16 bytes per row
                for (int ch = threadIdx.x; ch < 16 * nrb * (kTransTileCols / 8); ch += blockDim.x) {
                    const int r = ch >> 5, q = ch & 31;
                    cp_async16(stage + r * kTransTileCols + q * 8, src + (int64_t)r * cols + q * 8);
                }
            } else {                                     // ragged last column tile
                const int chunks_per_row = ncols / 8;
                for (int ch = threadIdx.x; ch < 16 * nrb * chunks_per_row; ch += blockDim.x) {
                    const int r = ch / chunks_per_row, q = ch - r * chunks_per_row;
                    cp_async16(stage + r * kTransTileCols + q * 8, src + (int64_t)r * cols + q * 8);
                }
            }
        }
        cp_async_commit();
    };

    int s = 0;
    // Tile counts fit 32 bits (a tile is 16384 elements).  The block's tiles are t, t + grid, ...: their
    // coordinates advance by (grid / ntx, grid % ntx) with one carry, so only the first needs a division.
    int64_t t = blockIdx.x;
    const uint32_t ntx32 = (uint32_t)ntx, step_y = gridDim.x / ntx32, step_x = gridDim.x - step_y * ntx32;
    uint32_t ty = blockIdx.x / ntx32, tx = blockIdx.x - ty * ntx32;
    issue(t, ty, tx, 0);
    for (; t < ntiles; t += gridDim.x, s ^= 1) {
        uint32_t ty_next = ty + step_y, tx_next = tx + step_x;
        if (tx_next >= ntx32) { tx_next -= ntx32; ++ty_next; }
        issue(t + gridDim.x, ty_next, tx_next, s ^ 1);   // prefetch the block's next tile into the other stage
        cp_async_wait_all_but_one();                 // this thread's copies of tile t have landed
        __syncthreads();                             // ... and everybody else's
        const int64_t rb0 = (int64_t)ty * kTransTileRowBlocks, c0 = (int64_t)tx * kTransTileCols;
        const int nrb = (int)min((int64_t)kTransTileRowBlocks, rblocks - rb0);
        const int ncols = (int)min((int64_t)kTransTileCols, cols - c0);
        uint16_t* stage = trans_smem + s * kTransStageElems;
        const int c = threadIdx.x;
        // FULL: a complete 64 x 256 tile whose outputs may leave as vector stores (the usual case): no per-group
        // bounds checks.  Otherwise the ragged-tile path with the same arithmetic.
        auto encode_column = [&](auto full_tag) {
            constexpr bool FULL = decltype(full_tag)::value;
            const bool vec = FULL || vec_ok;
            uint32_t cw[2 * kTransTileRowBlocks];
            uint32_t sbytes = 0u;
#pragma unroll kTransUnroll
            for (int k = 0; k < kTransTileRowBlocks; ++k) {
                if constexpr (!FULL) {
                    if (k >= nrb) break;
                }
                float x[16];
                const uint16_t* colp = stage + 16 * k * kTransTileCols + c;
#pragma unroll
                for (int i = 0; i < 16; ++i) x[i] = __uint_as_float((uint32_t)colp[i * kTransTileCols] << 16);
                if constexpr (RHT) hadamard16_pairs(x, sign_mask);   // along the group, i.e. down the column
                if constexpr (MODE == 1) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) local_max = max(local_max, __float_as_uint(x[i]) & 0x7FFFFFFFu);
                    continue;
                }
                const float m0 = max3abs(x[0], x[1], x[2]), m1 = max3abs(x[3], x[4], x[5]);
                const float m2 = max3abs(x[6], x[7], x[8]), m3 = max3abs(x[9], x[10], x[11]);
                const float m4 = max3abs(x[12], x[13], x[14]);
                const float gmax = fmaxf(max3abs(m0, m1, m2), max3abs(m3, m4, x[15]));   // G1
                const float tt = __fmul_rn(__fmul_rn(gmax, inv_a6), scale_mul);          // G2
                const uint32_t sb = e4m3_encode(tt);                                     // G3
                const float d = __fmul_rn(e4m3_value(sb), alpha);                        // G5
                const float r = __frcp_rn(d);
                uint32_t sbyte = 0u, c_lo = 0u, c_hi = 0u;
                const int64_t g = (c0 + c) * rblocks + rb0 + k;      // group index in the transposed matrix
                if constexpr (SR) {
                    if (sb != 0u) {
                        const uint64_t i8 = ctr_base + (uint64_t)g * 2u;   // Philox blocks 2g, 2g+1: elements 16g .. 16g+15
                        const uint4 p0 = philox4x32_10((uint32_t)i8, (uint32_t)(i8 >> 32), keys);
                        const uint4 p1 = philox4x32_10((uint32_t)i8 + 1u, (uint32_t)(i8 >> 32), keys);
                        const uint32_t rnd[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
                        encode_body4_sr<HAS_INT>(x, rnd, sb, d, r, sbyte, c_lo, c_hi);
                    }
                } else if ((sb - 8u) >= 118u) {
                    if (sb != 0u) encode_body4<HAS_INT, HAS_INT>(x, sb, d, r, sbyte, c_lo, c_hi);
                } else {
                    encode_body4<HAS_INT, false>(x, sb, d, r, sbyte, c_lo, c_hi);
                }
                if constexpr (EMUL) {
                    // decode the group from its codes (arithmetic of the dequantize kernel) over its own inputs
                    const bool is_int = HAS_INT && (sbyte & 0x80u);
                    const float dd = is_int ? __fmul_rn(d, __uint_as_float(0x3F5B6DB7u)) : d;
                    const float addend = is_int ? -1032.0f : -0.0f;
                    const uint64_t D2 = pack2(dd, dd);
                    uint32_t lo[4], hi[4];
                    dequant_word4<HAS_INT>(c_lo, is_int, addend, D2, lo);
                    dequant_word4<HAS_INT>(c_hi, is_int, addend, D2, hi);
                    uint16_t* colw = stage + 16 * k * kTransTileCols + c;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        colw[(2 * i) * kTransTileCols] = (uint16_t)lo[i];
                        colw[(2 * i + 1) * kTransTileCols] = (uint16_t)(lo[i] >> 16);
                        colw[(8 + 2 * i) * kTransTileCols] = (uint16_t)hi[i];
                        colw[(9 + 2 * i) * kTransTileCols] = (uint16_t)(hi[i] >> 16);
                    }
                    if (!store_codes) continue;
                }
                if (vec) {
                    // k is a runtime index: select the slot without dynamic register indexing
#pragma unroll
                    for (int j = 0; j < kTransTileRowBlocks; ++j)
                        if (j == k) { cw[2 * j] = c_lo; cw[2 * j + 1] = c_hi; }
                    sbytes |= sbyte << (8 * k);
                } else {
                    scales_t[g] = (uint8_t)sbyte;
                    codes_t[g] = make_uint2(c_lo, c_hi);
                }
            }
            if (MODE == 0 && vec && (!EMUL || store_codes)) {
                const int64_t g0 = (c0 + c) * rblocks + rb0;
                store32B<true>(codes_t + g0, reinterpret_cast<const uint32_t(&)[8]>(cw));
                *reinterpret_cast<uint32_t*>(scales_t + g0) = sbytes;
            }
        };
        if (ncols == kTransTileCols && nrb == kTransTileRowBlocks && vec_ok) encode_column(std::true_type{});
        else if (c < ncols) encode_column(std::false_type{});
        if constexpr (EMUL) {
            __syncthreads();                         // the whole tile now holds dequantized values
            uint16_t* dst = out + rb0 * 16 * cols + c0;
            const int chunks_per_row = ncols / 8;
            for (int ch = threadIdx.x; ch < 16 * nrb * chunks_per_row; ch += blockDim.x) {
                const int r = ch / chunks_per_row, q = ch - r * chunks_per_row;
                *reinterpret_cast<uint4*>(dst + (int64_t)r * cols + q * 8) =
                    *reinterpret_cast<const uint4*>(stage + r * kTransTileCols + q * 8);
            }
        }
        __syncthreads();                             // the stage may be overwritten by the next prefetch
        ty = ty_next;
        tx = tx_next;
    }
    if constexpr (MODE == 1) {
        __shared__ uint32_t warp_max[8];
        local_max = __reduce_max_sync(0xFFFFFFFFu, local_max);
        if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = local_max;
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t m = 0u;
#pragma unroll
            for (int w = 0; w < 8; ++w) m = max(m, warp_max[w]);
            atomicMax(amax_slot, ((unsigned long long)amax_gen << 32) | m);
        }
    }
}

#define ABS_TRANS_PARAMS                                                                                              \
    const uint16_t *__restrict__ in, uint2 *__restrict__ codes_t, uint8_t *__restrict__ scales_t,                     \
        const AlphaSrc alpha_src, int64_t rows, int64_t cols, uint32_t sign_mask, unsigned long long *amax_slot,      \
        uint32_t amax_gen, float scale_mul, const PhiloxKeys keys, uint64_t ctr_base,                                   \
        uint16_t *__restrict__ out, bool store_codes
#define ABS_TRANS_ARGS                                                                                                \
    in, codes_t, scales_t, alpha_src, rows, cols, sign_mask, amax_slot, amax_gen, scale_mul, keys,                    \
        ctr_base, out, store_codes

// Round-to-nearest and Hadamard instances are held to the registers of three blocks per SM (what the shared
// memory allows): left alone the compiler takes up to 124 and only two blocks fit.
template <bool HAS_INT, bool FROM_SLOT, bool RHT, int MODE, bool EMUL>
__global__ void __launch_bounds__(256, 3) quantize4_transposed_kernel(ABS_TRANS_PARAMS) {
    quantize4_transposed_body<HAS_INT, FROM_SLOT, RHT, false, MODE, EMUL>(ABS_TRANS_ARGS);
}
// The stochastic-rounding instances measured 3-7 % faster with the compiler's own register choice (about 80,
// no spills) than held to three or to two blocks per SM.
template <bool HAS_INT, bool FROM_SLOT, bool RHT, int MODE, bool EMUL>
__global__ void __launch_bounds__(256) quantize4_transposed_sr_kernel(ABS_TRANS_PARAMS) {
    quantize4_transposed_body<HAS_INT, FROM_SLOT, RHT, true, MODE, EMUL>(ABS_TRANS_ARGS);
}
#undef ABS_TRANS_PARAMS
#undef ABS_TRANS_ARGS

// The kernel instance for a set of options (both wrappers have the same signature).
template <bool HAS_INT, bool FROM_SLOT, bool RHT, bool SR, int MODE, bool EMUL>
constexpr auto transposed_kernel() {
    if constexpr (SR) return &quantize4_transposed_sr_kernel<HAS_INT, FROM_SLOT, RHT, MODE, EMUL>;
    else return &quantize4_transposed_kernel<HAS_INT, FROM_SLOT, RHT, MODE, EMUL>;
}

}  // namespace absq
