// IF4 matrix product on the Blackwell tensor cores (tcgen05): C = A B^T for two IF4 (or NVFP4) operands with the
// arithmetic of the paper's MAC unit (Sec. 5.2): inside a pair of groups the decoded codes are multiplied and
// summed exactly, the sum is scaled by Delta_a * Delta_b, and the factors 1, 6/7 or 36/49 -- none, one or both
// groups stored as integers -- are applied in FP32 on the scale path, here in the epilogue.
//
// How integer groups reach an FP4 tensor core.  An FP4 group is an NVFP4 group (Sec. 3) and goes to
// tcgen05.mma kind::mxf4nvf4 as it is.  An integer code k in -7..7 is not an E2M1 value, but it is the sum of
// two: k = h + l with h in {0, 1, 2, 3, 4, 6} and l in {0, 1} (5 = 4 + 1, 7 = 6 + 1), signs equal.  So every
// operand is split once into three NVFP4 "planes" that share the group scales:
//     F: the codes of the FP groups (integer groups zero)     H, L: the two parts of the integer groups
// and the product is  F_a F_b  +  6/7 (F_a (H_b + L_b) + (H_a + L_a) F_b)  +  36/49 (H_a + L_a)(H_b + L_b),
// nine block-scaled MMAs per K-step into three FP32 accumulators that live in tensor memory side by side
// (3 x 128 columns) and meet only in the epilogue.  Every product and partial sum is exact in the tensor core's
// FP32 accumulation up to its rounding of the running sum, which is what the float64 reference is compared to.
//
// Kernel: persistent, one block of ten warps per SM over the 128 x 128 tiles of C.  One thread feeds the pipeline with
// TMA (cp.async.bulk.tensor.2d, 128-byte swizzle, each load for this CTA alone) and runs ahead into the next tile, one
// thread issues the MMAs, four warps write the scales of every K-step into tensor memory (tcgen05.st), four warps read
// the accumulators back (tcgen05.ld) and write C.  Every mbarrier wait is bounded in time: when a wait runs out the
// block raises an error word, stops issuing, frees its tensor memory and returns.
//
// What bounds it: the rate at which the one MMA stream of a CTA completes -- about 87 cycles per 128 x 128 x 64
// block-scaled MMA against the 64 the tensor pipe counts as active; the loads hide completely under it.
#include "../../include/abs_b200.h"
#include "abs_device.cuh"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <mutex>

namespace absq {

constexpr int kTileM = 128, kTileN = 128;
constexpr int kStageK = 256;                       // elements of K of one TMA box: 128 bytes of packed codes per row
constexpr int kMmaK = 64;                          // K of one tcgen05.mma kind::mxf4nvf4
constexpr int kPlaneBytes = kTileM * kStageK / 2;  // 16 KiB: one box (128 rows x 128 bytes) of one plane of one operand
// A pipeline stage (one K-step) holds KBOXES boxes of each of the PLANES planes of A and of B (the scales do not pass
// through shared memory).  IF4 (three planes, one box: K = 256, 96 KiB) has room for two stages.  Plain NVFP4 issues one
// MMA per K-block, so the hand-overs of a step weigh more: its steps are two boxes long where K allows (K = 512, 64 KiB,
// three stages), else one box (32 KiB, six stages).
template <int PLANES, int KBOXES> constexpr int kStageBytes = 2 * PLANES * KBOXES * kPlaneBytes;
template <int PLANES, int KBOXES> constexpr int kStages = PLANES == 3 ? 2 : (KBOXES == 2 ? 3 : 6);
// Epilogue staging: each of the four epilogue warps turns its 32 rows x 32 columns of a chunk through shared memory
// (rows 36 floats apart: 16-byte aligned and free of bank conflicts for 128-bit accesses both ways).
constexpr int kStagePitch = 36, kStagingBytes = 4 * 32 * kStagePitch * 4;
template <int PLANES, int KBOXES> constexpr int kGemmSmemBytes =
    kStages<PLANES, KBOXES> * kStageBytes<PLANES, KBOXES> + 1024 /* alignment slack */ + 512 /* barriers */ + kStagingBytes;
constexpr uint64_t kWaitLimitNs = 1000000000ull;   // one second: how long an mbarrier wait polls before the block gives up

// ----------------------------------------------------------------------------- operand split

// Splits eight integer codes (two's complement nibbles of one word) into the planes H and L, all nibbles at once:
// sign s, magnitude m = |k|; H = s | e2m1(h), L = s | e2m1(l) with m = h + l, h in {0, 1, 2, 3, 4, 6} and l = 1 for
// m = 5 or 7, l = 2 for m = 8 (the most negative code, which no quantizer writes but dequantize reads as -8), else
// 0.  E2M1 codes of the integers 0, 1, 2, 3, 4, 6 are 0, 2, 4, 5, 6, 7.  No step carries from one nibble into the next.
__device__ __forceinline__ void split_int_word(uint32_t w, uint32_t& h, uint32_t& l) {
    constexpr uint32_t kOnes = 0x11111111u;
    const uint32_t s = w & 0x88888888u, neg = s >> 3;
    const uint32_t m = (w ^ (neg * 15u)) + neg;                      // |k| per nibble, 0 .. 8
    const uint32_t l1 = (m >> 2) & m & kOnes;                         // m = 5 or 7
    const uint32_t l2 = (m >> 3) & kOnes;                             // m = 8
    const uint32_t mh = m - (l1 | (l2 << 1));                         // 0, 1, 2, 3, 4, 6
    const uint32_t c0 = mh & kOnes, c1 = (mh >> 1) & kOnes, c2 = (mh >> 2) & kOnes;
    h = s | ((c2 | c1) << 2) | ((c2 | (c0 & ~c1)) << 1) | (c1 & (c0 | c2));
    l = (((l1 | l2) << 3) & s) | (l1 << 1) | (l2 << 2);
}

// One operand of the product as the split kernel sees it.
struct SplitOperand {
    const uint4* codes;            // [rows, k / 2] bytes as abs_quantize wrote them
    const uint8_t* scales;         // [rows, k / 16] row-major
    uint4 *plane_f, *plane_h, *plane_l;
    uint8_t* sf_tiled;             // magnitudes of the scales in the 128x4-tile layout
    int64_t rows;
    int64_t pairs;                 // rows * k / 32: pairs of groups (16 bytes of codes)
    int64_t sf_items;              // ceil(rows / 128) * ktiles / 4 * 32: one item = 4 rows x 16 scales
    uint32_t gpr, ktiles;          // groups per row (a multiple of 16), gpr / 4
};

// Prepares both operands in one launch.  Code items (IF4 only; an NVFP4 operand is read by the product kernel where
// it lies): 32 codes = two groups -> 16 bytes of each of the planes F, H, L.  Scale items: thread i of a warp reads 16
// scale bytes of each of the rows i, i + 32, i + 64, i + 96 of a 128-row block and writes, for each of four
// consecutive 128x4 tiles, the 16 bytes that tile keeps for those four rows.  Also clears the error word.
__global__ void __launch_bounds__(256) if4_split_kernel(const SplitOperand a, const SplitOperand b, bool has_int,
                                                        int* __restrict__ error) {
    pdl_launch_dependents();
    pdl_wait();
    const int64_t stride = (int64_t)gridDim.x * blockDim.x, first = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (first == 0) { error[0] = 0; error[1] = 0; error[2] = 0; }     // error word, output maximum, ticket
    const int64_t code_items = has_int ? a.pairs + b.pairs : 0;
    for (int64_t i = first; i < code_items; i += stride) {
        const SplitOperand& o = i < a.pairs ? a : b;
        const int64_t p = i < a.pairs ? i : i - a.pairs;
        const uint4 c = __ldg(o.codes + p);
        const uint32_t sb = __ldg(reinterpret_cast<const uint16_t*>(o.scales) + p);
        uint4 f = c, h = make_uint4(0u, 0u, 0u, 0u), l = h;
        if (sb & 0x80u) { f.x = 0u; f.y = 0u; split_int_word(c.x, h.x, l.x); split_int_word(c.y, h.y, l.y); }
        if (sb & 0x8000u) { f.z = 0u; f.w = 0u; split_int_word(c.z, h.z, l.z); split_int_word(c.w, h.w, l.w); }
        o.plane_f[p] = f;
        o.plane_h[p] = h;
        o.plane_l[p] = l;
    }
    const int64_t sf_items = a.sf_items + b.sf_items;
    for (int64_t i = first; i < sf_items; i += stride) {
        const SplitOperand& o = i < a.sf_items ? a : b;
        const int64_t j = i < a.sf_items ? i : i - a.sf_items;
        const uint32_t lane = (uint32_t)(j & 31);
        const int64_t t4 = j >> 5;                                    // (row block, group of four tiles)
        const uint32_t quads = o.ktiles >> 2;
        const int64_t rb = t4 / quads;
        const uint32_t kq = (uint32_t)(t4 - rb * quads);
        uint4 r[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int64_t row = rb * 128 + q * 32 + lane;       // rows beyond the operand (last row block) get zero scales
            r[q] = row < o.rows ? __ldg(reinterpret_cast<const uint4*>(o.scales + row * o.gpr) + kq) : make_uint4(0u, 0u, 0u, 0u);
        }
        uint4* out = reinterpret_cast<uint4*>(o.sf_tiled + ((size_t)rb * o.ktiles + (size_t)kq * 4u) * 512u) + lane;
        constexpr uint32_t kMag = 0x7F7F7F7Fu;
        out[0] = make_uint4(r[0].x & kMag, r[1].x & kMag, r[2].x & kMag, r[3].x & kMag);
        out[32] = make_uint4(r[0].y & kMag, r[1].y & kMag, r[2].y & kMag, r[3].y & kMag);
        out[64] = make_uint4(r[0].z & kMag, r[1].z & kMag, r[2].z & kMag, r[3].z & kMag);
        out[96] = make_uint4(r[0].w & kMag, r[1].w & kMag, r[2].w & kMag, r[3].w & kMag);
    }
}

// ----------------------------------------------------------------------------- PTX building blocks

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Wait for the phase with the given parity, bounded in time (a try_wait may itself sleep for a while, so counting
// polls would not bound it); false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    do {
        if (mbar_try_wait(bar, parity)) return true;
    } while (global_timer_ns() - t0 < kWaitLimitNs);
    return false;
}
// One 2-D tile (inner coordinate x in bytes, outer coordinate y in rows) from a tensor map into shared memory.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :: "r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t columns) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_result), "r"(columns) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_free(uint32_t addr, uint32_t columns) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(addr), "r"(columns) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Arrives on the mbarrier once every tcgen05 operation this thread issued before has completed.
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, 128 x 128 x 64, E2M1 operands, one UE4M3 scale per 16 elements read from tensor memory.
// What happens to the A operand in the tensor core's collector buffer: read from shared memory and dropped, read and
// kept (kFill), taken from the buffer and kept (kUse), taken from the buffer and dropped (kLastUse).  An MMA that
// takes A from the buffer reads only B from shared memory.
enum Collector { kDiscard, kFill, kUse, kLastUse };
template <Collector C = kDiscard>
__device__ __forceinline__ void tc_mma_nvf4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate,
                                            uint32_t sfa_tmem, uint32_t sfb_tmem) {
#define ABS_MMA_NVF4(USAGE)                                                                                              \
    asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0;\n"                                                               \
                 "  tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.block16" USAGE " [%0], %1, %2, %3, [%5], [%6], p; }" \
                 :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate), "r"(sfa_tmem), "r"(sfb_tmem) \
                 : "memory")
    if constexpr (C == kFill) ABS_MMA_NVF4(".collector::a::fill");
    else if constexpr (C == kUse) ABS_MMA_NVF4(".collector::a::use");
    else if constexpr (C == kLastUse) ABS_MMA_NVF4(".collector::a::lastuse");
    else ABS_MMA_NVF4("");
#undef ABS_MMA_NVF4
}
// 32 lanes x 32 columns of 32 bits: thread t of the warp gets columns c .. c+31 of lane (warp % 4) * 32 + t.
__device__ __forceinline__ void tmem_load32(uint32_t addr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(addr) : "memory");
}
// Two FP32 values rounded to nearest even bf16, the first in the low half.
__device__ __forceinline__ uint32_t bf16x2_bits(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ void tmem_load_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 32 lanes x 16 columns of 32 bits: thread t of the warp writes columns c .. c+15 of lane (warp % 4) * 32 + t.
__device__ __forceinline__ void tmem_store16(uint32_t addr, const uint4& a, const uint4& b, const uint4& c, const uint4& d) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 :: "r"(addr), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w), "r"(c.x), "r"(c.y),
                    "r"(c.z), "r"(c.w), "r"(d.x), "r"(d.y), "r"(d.z), "r"(d.w)
                 : "memory");
}
__device__ __forceinline__ void tmem_store_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptors (64 bits): start address, leading / stride byte offsets (all in 16-byte units),
// descriptor version 1 (Blackwell) in bits 46-47, swizzle mode in bits 61-63.
//   operand tiles: K-major rows of 128 bytes, 128-byte swizzle (mode 2), 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t operand_desc(uint32_t smem_addr) {
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
           ((uint64_t)2 << 61);
}
// Instruction descriptor of kind::mxf4nvf4: A and B E2M1 (format 1, bits 7-9 and 10-12), both K-major, N / 8 in bits
// 17-22, scale format UE4M3 (bit 23 = 0), M / 16 in bits 24-28, dense, K = 64 (bit 31 = 0), scale ids 0.
constexpr uint32_t kInstrDesc = (1u << 7) | (1u << 10) | ((uint32_t)(kTileN >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);

// ----------------------------------------------------------------------------- the product kernel

// Tensor memory columns (512 allocated): the accumulators (IF4: three of 128 columns; NVFP4: two, used alternately),
// then the scale slots: 16 columns of A scales and 16 of B scales each (four per MMA of K = 64).
constexpr uint32_t kTmemCols = 512;

struct GemmMaps {
    CUtensorMap a[3], b[3];        // planes F, H, L of A [M, K/2 bytes] and B [N, K/2 bytes], boxes of 128 bytes x 128 rows
};

// Tile t of the (tiles_m x tiles_n) grid of 128 x 128 tiles, walked in bands of eight tile rows, column by column
// inside a band, so that the blocks running at the same time share few rows of A and few of B (L2 reuse).
__device__ __forceinline__ void tile_of(int32_t t, int32_t tiles_m, int32_t tiles_n, int32_t& tm, int32_t& tn) {
    constexpr int32_t kBand = 8;
    const int32_t per_band = kBand * tiles_n, band = t / per_band, in_band = t - band * per_band;
    const int32_t first = band * kBand, rows = min(kBand, tiles_m - first);
    tn = in_band / rows;
    tm = first + (in_band - tn * rows);
}

// PLANES = 3: IF4 operands (nine MMAs per K-step); PLANES = 1: plain NVFP4 (one).  error: device word set to a
// non-zero code when a wait ran out.
//
// Persistent: one block per SM walks the tiles blockIdx.x, blockIdx.x + gridDim.x, ...  Ten warps: warp 0 (one
// thread) feeds the pipeline and runs ahead into the next tile while the current one is finished; warp 1 (one thread)
// issues MMAs; warps 2-5 are the epilogue (warp w reads the 32 accumulator lanes of tensor-memory quarter w % 4);
// warps 6-9 bring the scales: each loads the 128x4 scale tiles of a K-step from global memory into registers and
// writes them to its quarter of tensor memory (tcgen05.st; every quarter holds the same four columns per MMA: rows
// r, r+32, r+64, r+96 of the tile, which is the byte order of the 128x4 tile), two slots used alternately and handed
// over through sf_full / sf_empty barriers -- a tcgen05.cp from shared memory by the MMA thread would stand in the
// MMA queue for some 34 cycles per copy, 270 per K-step.  The accumulators pass between MMA and epilogue through
// acc_full / acc_empty barriers; NVFP4, with one accumulator of 128 columns, alternates between two of them so that a
// tile's epilogue overlaps the next tile's MMAs, IF4 (3 x 128 columns) has room for one set and overlaps the epilogue
// only with the next tile's loads.
// OUT_BF16: C is written as bf16 (round to nearest even of the same FP32 value), else as FP32.
template <int PLANES, bool OUT_BF16, int KBOXES = 1>
__global__ void __launch_bounds__(320, 1)
if4_gemm_kernel(const __grid_constant__ GemmMaps maps, const uint8_t* __restrict__ sfa, const uint8_t* __restrict__ sfb,
                const float* __restrict__ alpha_a, const float* __restrict__ alpha_b, void* __restrict__ c_out, int32_t tiles_m,
                int32_t tiles_n, int32_t k_iters, int32_t m_rows, int* __restrict__ error, int32_t stall_step,
                float* __restrict__ next_alpha, float next_denom) {
    constexpr int planes = PLANES, kStages = absq::kStages<PLANES, KBOXES>, kStageBytes = absq::kStageBytes<PLANES, KBOXES>;
    constexpr int kStepBlocks = KBOXES * (kStageK / kMmaK);          // MMA K-blocks (and scale tiles per operand) of one step
    constexpr int kAccBufs = PLANES == 1 ? 2 : 1;
    extern __shared__ uint8_t gemm_smem_raw[];
    const uint32_t raw = smem_u32(gemm_smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;                    // 128-byte swizzle wants 1024-byte aligned tiles
    // Scale slots in tensor memory: 32 columns each (16 of A scales, 16 of B scales).  IF4 has room for two behind its
    // three accumulators; NVFP4, whose K-steps are only four MMAs long, takes eight behind its two accumulators so
    // that the scale warps can run several steps ahead of the MMAs.
    constexpr uint32_t kSlotCols = 8u * kStepBlocks;                  // 4 columns per K-block and operand
    constexpr uint32_t kSfSlots = PLANES == 1 ? 256u / kSlotCols : 2u, kSfBase = PLANES == 1 ? 2 * kTileN : 3 * kTileN;
    // barriers: full[], empty[] (stages), acc_full[2], acc_empty[2], sf_full[], sf_empty[] (slots); then the tmem address word
    const uint32_t bars = base + kStages * kStageBytes;
    uint32_t* tmem_word = reinterpret_cast<uint32_t*>(gemm_smem_raw + (bars - raw) + 320);
    const uint32_t full0 = bars, empty0 = bars + 64, acc_full0 = bars + 128, acc_empty0 = bars + 144;
    const uint32_t sf_full0 = bars + 192, sf_empty0 = bars + 256;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int32_t num_tiles = tiles_m * tiles_n, n_cols = tiles_n * kTileN;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int i = 0; i < kAccBufs; ++i) { mbar_init(acc_full0 + 8 * i, 1); mbar_init(acc_empty0 + 8 * i, 4); }
        for (int i = 0; i < (int)kSfSlots; ++i) { mbar_init(sf_full0 + 8 * i, 4); mbar_init(sf_empty0 + 8 * i, 1); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) { tmem_alloc(smem_u32(tmem_word), kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_word;
    pdl_wait();

    if (warp == 0) {
        if (lane == 0) {
            // ---- producer: TMA loads of the operand planes
            const uint32_t bytes = (uint32_t)planes * 2u * KBOXES * kPlaneBytes;
            uint32_t it = 0;
            bool ok = true;
            for (int32_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
                int32_t tile_m, tile_n;
                tile_of(t, tiles_m, tiles_n, tile_m, tile_n);
                for (int32_t kt = 0; kt < k_iters; ++kt, ++it) {
                    const uint32_t s = it % kStages;
                    if (!mbar_wait(empty0 + 8 * s, ((it / kStages) & 1u) ^ 1u)) { atomicExch(error, 1); ok = false; break; }
                    const uint32_t st = base + s * kStageBytes, bar = full0 + 8 * s;
                    mbar_expect_tx(bar, bytes);
                    if ((int32_t)it == stall_step) continue;      // self-test only: the bytes announced never arrive
                    for (int p = 0; p < planes; ++p)
                        for (int box = 0; box < KBOXES; ++box) {
                            const int32_t x = (kt * KBOXES + box) * (kStageK / 2);
                            tma_load_2d(st + (p * KBOXES + box) * kPlaneBytes, &maps.a[p], x, tile_m * kTileM, bar);
                            tma_load_2d(st + ((PLANES + p) * KBOXES + box) * kPlaneBytes, &maps.b[p], x, tile_n * kTileN, bar);
                        }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMAs
            uint32_t it = 0, j = 0;
            bool ok = true;
            for (int32_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++j) {
                const uint32_t buf = j % kAccBufs, acc = tmem + buf * kTileN;
                if (!mbar_wait(acc_empty0 + 8 * buf, ((j / kAccBufs) & 1u) ^ 1u)) { atomicExch(error, 4); ok = false; break; }
                tc_fence_after();
                for (int32_t kt = 0; kt < k_iters; ++kt, ++it) {
                    const uint32_t s = it % kStages;
                    const uint32_t slot = it % kSfSlots;
                    if (!mbar_wait(full0 + 8 * s, (it / kStages) & 1u)) { atomicExch(error, 2); ok = false; break; }
                    if (!mbar_wait(sf_full0 + 8 * slot, (it / kSfSlots) & 1u)) { atomicExch(error, 5); ok = false; break; }
                    tc_fence_after();
                    const uint32_t st = base + s * kStageBytes;
                    const uint32_t tsfa = tmem + kSfBase + slot * kSlotCols, tsfb = tsfa + kSlotCols / 2;
                    // the MMAs of a step, one accumulator after the other (K order inside an accumulator is free)
                    // K-block kb of a step lies in box kb / 4 of its plane, 32 bytes per K-block inside the box's 128-byte rows
                    auto desc_a = [&](int p, int kb) {
                        return operand_desc(st + (p * KBOXES + (kb >> 2)) * kPlaneBytes + (kb & 3) * (kMmaK / 2));
                    };
                    auto desc_b = [&](int p, int kb) {
                        return operand_desc(st + ((PLANES + p) * KBOXES + (kb >> 2)) * kPlaneBytes + (kb & 3) * (kMmaK / 2));
                    };
#pragma unroll
                    for (int kb = 0; kb < kStepBlocks; ++kb)
                        tc_mma_nvf4(acc, desc_a(0, kb), desc_b(0, kb), kInstrDesc, !(kt == 0 && kb == 0), tsfa + 4 * kb, tsfb + 4 * kb);   // F F
                    if constexpr (PLANES == 3) {
#pragma unroll
                        for (int kb = 0; kb < kStepBlocks; ++kb) {
                            const uint32_t fa = tsfa + 4 * kb, fb = tsfb + 4 * kb;
                            tc_mma_nvf4<kFill>(acc + kTileN, desc_a(0, kb), desc_b(1, kb), kInstrDesc, !(kt == 0 && kb == 0), fa, fb);   // F H
                            tc_mma_nvf4<kLastUse>(acc + kTileN, desc_a(0, kb), desc_b(2, kb), kInstrDesc, true, fa, fb);                 // F L
                            tc_mma_nvf4(acc + kTileN, desc_a(1, kb), desc_b(0, kb), kInstrDesc, true, fa, fb);                           // H F
                            tc_mma_nvf4(acc + kTileN, desc_a(2, kb), desc_b(0, kb), kInstrDesc, true, fa, fb);                           // L F
                        }
#pragma unroll
                        for (int kb = 0; kb < kStepBlocks; ++kb) {
                            const uint32_t fa = tsfa + 4 * kb, fb = tsfb + 4 * kb;
                            tc_mma_nvf4<kFill>(acc + 2 * kTileN, desc_a(1, kb), desc_b(1, kb), kInstrDesc, !(kt == 0 && kb == 0), fa, fb);  // H H
                            tc_mma_nvf4<kLastUse>(acc + 2 * kTileN, desc_a(1, kb), desc_b(2, kb), kInstrDesc, true, fa, fb);              // H L
                            tc_mma_nvf4<kFill>(acc + 2 * kTileN, desc_a(2, kb), desc_b(1, kb), kInstrDesc, true, fa, fb);                 // L H
                            tc_mma_nvf4<kLastUse>(acc + 2 * kTileN, desc_a(2, kb), desc_b(2, kb), kInstrDesc, true, fa, fb);              // L L
                        }
                    }
                    tc_commit(empty0 + 8 * s);          // the stage's shared memory is free once these MMAs have run
                    tc_commit(sf_empty0 + 8 * slot);    // and so is the slot of scales
                }
                if (ok) tc_commit(acc_full0 + 8 * buf); // and the tile's accumulators are complete
            }
        }
    } else if (warp >= 6) {
        // ---- scales: this warp's copy of every K-step's scale tiles, global memory -> registers -> tensor memory
        // The loads of step it + 1 are in flight while step it waits for its slot and is written.
        const int32_t ktiles = k_iters * kStepBlocks;
        const uint32_t lane_base = tmem + kSfBase + ((uint32_t)((warp & 3) * 32) << 16);
        int32_t t = blockIdx.x, kt = 0;                                   // the step whose tiles are loaded next
        const uint4 *pa = nullptr, *pb = nullptr;
        auto load_next = [&](uint4 (&a)[kStepBlocks], uint4 (&b)[kStepBlocks]) {   // false when there is no further step
            if (t >= num_tiles) return false;
            if (kt == 0) {
                int32_t tile_m, tile_n;
                tile_of(t, tiles_m, tiles_n, tile_m, tile_n);
                pa = reinterpret_cast<const uint4*>(sfa + (size_t)tile_m * ktiles * 512) + lane;
                pb = reinterpret_cast<const uint4*>(sfb + (size_t)tile_n * ktiles * 512) + lane;
            }
#pragma unroll
            for (int kb = 0; kb < kStepBlocks; ++kb) {                     // tile kb of the step: 16 bytes per lane, tiles 512 bytes apart
                a[kb] = __ldg(pa + (kt * kStepBlocks + kb) * 32);
                b[kb] = __ldg(pb + (kt * kStepBlocks + kb) * 32);
            }
            if (++kt == k_iters) { kt = 0; t += gridDim.x; }
            return true;
        };
        // One step of lookahead in registers where a step is one box long; with two-box steps the four scale slots
        // already let these warps run three steps ahead of the MMAs.
        constexpr bool kLookahead = KBOXES == 1;
        uint4 a[kStepBlocks], b[kStepBlocks], an[kLookahead ? kStepBlocks : 1], bn[kLookahead ? kStepBlocks : 1];
        bool more = load_next(a, b);
        for (uint32_t it = 0; more; ++it) {
            if constexpr (kLookahead) more = load_next(an, bn);
            const uint32_t slot = it % kSfSlots;
            bool have = mbar_wait(sf_empty0 + 8 * slot, ((it / kSfSlots) & 1u) ^ 1u);
            if (!have && lane == 0) atomicExch(error, 6);
            have = __all_sync(0xFFFFFFFFu, have);
            if (!have) break;
            tc_fence_after();
#pragma unroll
            for (int g = 0; g < KBOXES; ++g) {
                tmem_store16(lane_base + slot * kSlotCols + 16u * g, a[4 * g], a[4 * g + 1], a[4 * g + 2], a[4 * g + 3]);
                tmem_store16(lane_base + slot * kSlotCols + kSlotCols / 2 + 16u * g, b[4 * g], b[4 * g + 1], b[4 * g + 2], b[4 * g + 3]);
            }
            tmem_store_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(sf_full0 + 8 * slot);
            if constexpr (kLookahead) {
#pragma unroll
                for (int kb = 0; kb < kStepBlocks; ++kb) { a[kb] = an[kb]; b[kb] = bn[kb]; }
            } else {
                more = load_next(a, b);
            }
        }
    } else {
        // ---- epilogue: warp w owns the accumulator lanes (rows of the tile) 32 (w % 4) .. 32 (w % 4) + 31
        const int quarter = warp & 3;
        float* staging = reinterpret_cast<float*>(gemm_smem_raw + (bars - raw) + 512) + (warp - 2) * 32 * kStagePitch;
        const float scale = __fmul_rn(__ldg(alpha_a), __ldg(alpha_b));
        const float c1 = __uint_as_float(0x3F5B6DB7u);                 // fp32(6/7)
        const float c2 = __fdiv_rn(36.0f, 49.0f);
        uint32_t j = 0;
        uint32_t out_max = 0u;                  // bf16 output with next_alpha: largest |C| bit pattern this thread has written
        bool all_tiles = true;
        for (int32_t t = blockIdx.x; t < num_tiles; t += gridDim.x, ++j) {
            int32_t tile_m, tile_n;
            tile_of(t, tiles_m, tiles_n, tile_m, tile_n);
            const uint32_t buf = j % kAccBufs;
            bool have = mbar_wait(acc_full0 + 8 * buf, (j / kAccBufs) & 1u);
            if (!have && lane == 0) atomicExch(error, 3);
            have = __all_sync(0xFFFFFFFFu, have);
            if (!have) { all_tiles = false; break; }
            tc_fence_after();
            const bool own_row_valid = tile_m * kTileM + quarter * 32 + lane < m_rows;   // the row whose values this thread holds
            // this thread's part of every store.  FP32: row (lane / 8) of each group of four rows, 16 bytes at column
            // 4 (lane % 8); bf16: row (lane / 4) of each group of eight rows, 16 bytes at column 8 (lane % 4)
            const int32_t row0 = tile_m * kTileM + quarter * 32 + (OUT_BF16 ? (lane >> 2) : (lane >> 3));
            float* out = reinterpret_cast<float*>(c_out) + (size_t)row0 * (size_t)n_cols + (size_t)tile_n * kTileN + 4 * (lane & 7);
            __nv_bfloat16* out16 = reinterpret_cast<__nv_bfloat16*>(c_out) + (size_t)row0 * (size_t)n_cols + (size_t)tile_n * kTileN +
                                   8 * (lane & 3);
            const uint32_t lane_base = tmem + buf * kTileN + ((uint32_t)(quarter * 32) << 16);
            for (int chunk = 0; chunk < kTileN / 32; ++chunk) {
                uint32_t r0[32], r1[32], r2[32];
                tmem_load32(lane_base + chunk * 32, r0);
                if (planes == 3) {
                    tmem_load32(lane_base + kTileN + chunk * 32, r1);
                    tmem_load32(lane_base + 2 * kTileN + chunk * 32, r2);
                }
                tmem_load_wait();
                if (chunk == kTileN / 32 - 1) {         // everything is in registers: the MMAs of the next tile may start
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acc_empty0 + 8 * buf);
                }
                float v[32];
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) {
                    float acc = __uint_as_float(r0[jj]);
                    if (planes == 3) acc = __fmaf_rn(c2, __uint_as_float(r2[jj]), __fmaf_rn(c1, __uint_as_float(r1[jj]), acc));
                    v[jj] = __fmul_rn(acc, scale);
                }
                // A thread holds 32 columns of ONE row; stored as they are, every store instruction of the warp would
                // touch 32 different rows.  Through shared memory each instruction writes four rows of 128 contiguous bytes.
                if constexpr (!OUT_BF16) {
#pragma unroll
                    for (int jj = 0; jj < 32; jj += 4)
                        *reinterpret_cast<float4*>(staging + lane * kStagePitch + jj) = make_float4(v[jj], v[jj + 1], v[jj + 2], v[jj + 3]);
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 x = *reinterpret_cast<const float4*>(staging + (4 * i + (lane >> 3)) * kStagePitch + 4 * (lane & 7));
                        if (row0 + 4 * i < m_rows)                      // the last row block may be partial
                            *reinterpret_cast<float4*>(out + (size_t)(4 * i) * n_cols + chunk * 32) = x;
                    }
                } else {
                    // 32 bf16 = 64 bytes per row, rows 20 words apart; a store instruction writes eight rows of 64 bytes
                    uint32_t* stg = reinterpret_cast<uint32_t*>(staging);
#pragma unroll
                    for (int jj = 0; jj < 32; jj += 8) {
                        uint4 pk;
                        pk.x = bf16x2_bits(v[jj], v[jj + 1]); pk.y = bf16x2_bits(v[jj + 2], v[jj + 3]);
                        pk.z = bf16x2_bits(v[jj + 4], v[jj + 5]); pk.w = bf16x2_bits(v[jj + 6], v[jj + 7]);
                        *reinterpret_cast<uint4*>(stg + lane * 20 + jj / 2) = pk;
                        if (next_alpha != nullptr && own_row_valid) {
                            const uint32_t w4[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
                            for (int q = 0; q < 4; ++q) out_max = max(out_max, max(w4[q] & 0x7FFFu, (w4[q] >> 16) & 0x7FFFu));
                        }
                    }
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint4 x = *reinterpret_cast<const uint4*>(stg + (8 * i + (lane >> 2)) * 20 + 4 * (lane & 3));
                        if (row0 + 8 * i < m_rows)
                            *reinterpret_cast<uint4*>(out16 + (size_t)(8 * i) * n_cols + chunk * 32) = x;
                    }
                }
                __syncwarp();
            }
        }
        // The global maximum of |C| as written (bf16), for the next quantizer's tensor scale (Eq. 1): every epilogue
        // warp publishes its maximum with an atomic and takes a ticket; the last of all warps converts and writes alpha.
        if (OUT_BF16 && next_alpha != nullptr && all_tiles) {
            const uint32_t wmax = __reduce_max_sync(0xFFFFFFFFu, out_max);
            if (lane == 0) {
                atomicMax(reinterpret_cast<unsigned int*>(error) + 1, wmax);
                __threadfence();
                const int ticket = atomicAdd(error + 2, 1);
                if (ticket == (int)gridDim.x * 4 - 1) {
                    const float A = __uint_as_float(atomicMax(reinterpret_cast<unsigned int*>(error) + 1, 0u) << 16);
                    *next_alpha = (A == 0.0f) ? 1.0f : __fdiv_rn(A, next_denom);
                }
            }
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_free(tmem, kTmemCols);
}

}  // namespace absq

// ----------------------------------------------------------------------------- host side

namespace {

using namespace absq;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled through the runtime's driver entry point (the library does not link libcuda).
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, []() {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// Tensor map of one plane: bytes [rows, row_bytes], box 128 bytes x 128 rows, 128-byte swizzle.  The map covers
// this GPU's own workspace only.
bool plane_map(CUtensorMap* map, void* base, uint64_t rows, uint64_t row_bytes) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {row_bytes, rows};
    const cuuint64_t strides[1] = {row_bytes};
    const cuuint32_t box[2] = {128, 128}, elem[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t round1k(size_t n) { return (n + 1023) & ~(size_t)1023; }

// Launch with programmatic stream serialization: the kernel may become resident while its predecessor in the stream
// drains; both kernels here call pdl_wait() before their first global access.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, int block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
struct GemmLayout {
    size_t plane_a, plane_b, sf_a, sf_b;       // sizes
    size_t off_a, off_b, off_sfa, off_sfb, total;
};
GemmLayout gemm_layout(int64_t m, int64_t n, int64_t k) {
    GemmLayout L;
    L.plane_a = round1k((size_t)m * k / 2);
    L.plane_b = round1k((size_t)n * k / 2);
    L.sf_a = round1k((size_t)((m + kTileM - 1) / kTileM * kTileM) * k / 16);
    L.sf_b = round1k((size_t)n * k / 16);
    L.off_a = 1024;
    L.off_b = L.off_a + 3 * L.plane_a;
    L.off_sfa = L.off_b + 3 * L.plane_b;
    L.off_sfb = L.off_sfa + L.sf_a;
    L.total = L.off_sfb + L.sf_b;
    return L;
}

bool gemm_shape_ok(abs_fmt_t fmt, int64_t m, int64_t n, int64_t k) {
    return (fmt == ABS_FMT_IF4 || fmt == ABS_FMT_NVFP4) && m > 0 && n > 0 && k > 0 && n % kTileN == 0 &&
           k % kStageK == 0 && m < ((int64_t)1 << 30) && n < ((int64_t)1 << 30) && k < ((int64_t)1 << 30);
}

}  // namespace

extern "C" {

size_t abs_matmul_workspace_bytes(abs_fmt_t fmt, int64_t m, int64_t n, int64_t k) {
    if (!gemm_shape_ok(fmt, m, n, k)) return 0;
    return gemm_layout(m, n, k).total;
}

static abs_status_t matmul_impl(abs_fmt_t fmt, const void* a_codes, const void* a_scales, const float* a_alpha, const void* b_codes,
                                const void* b_scales, const float* b_alpha, int64_t m, int64_t n, int64_t k, void* c_f32,
                                void* workspace, size_t workspace_bytes, void* stream, int32_t stall_step, bool out_bf16 = false,
                                float* next_alpha = nullptr, float next_denom = 0.0f) {
    const absq::CallRange range("abs_matmul");
    if (fmt != ABS_FMT_IF4 && fmt != ABS_FMT_NVFP4) return ABS_ERR_FMT;
    if (!gemm_shape_ok(fmt, m, n, k)) return ABS_ERR_SHAPE;
    if (!a_codes || !a_scales || !a_alpha || !b_codes || !b_scales || !b_alpha || !c_f32 || !workspace) return ABS_ERR_NULL;
    const uintptr_t all = (uintptr_t)a_codes | (uintptr_t)a_scales | (uintptr_t)b_codes | (uintptr_t)b_scales | (uintptr_t)c_f32;
    if ((all & 15u) || ((uintptr_t)workspace & 1023u)) return ABS_ERR_ALIGN;
    const GemmLayout L = gemm_layout(m, n, k);
    if (workspace_bytes < L.total) return ABS_ERR_SIZE;
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* ws = (uint8_t*)workspace;
    const bool has_int = fmt == ABS_FMT_IF4;

    GemmMaps maps;
    for (int p = 0; p < 3; ++p) {
        // NVFP4 needs no split: its single plane is the caller's codes
        void* pa = has_int ? (void*)(ws + L.off_a + p * L.plane_a) : const_cast<void*>(a_codes);
        void* pb = has_int ? (void*)(ws + L.off_b + p * L.plane_b) : const_cast<void*>(b_codes);
        if (!plane_map(&maps.a[p], pa, (uint64_t)m, (uint64_t)k / 2) || !plane_map(&maps.b[p], pb, (uint64_t)n, (uint64_t)k / 2))
            return ABS_ERR_CUDA;
    }
    const uint32_t gpr = (uint32_t)(k / 16), ktiles = gpr / 4u;
    SplitOperand so[2];
    for (int op = 0; op < 2; ++op) {
        const int64_t rows = op ? n : m;
        const size_t off = op ? L.off_b : L.off_a, plane = op ? L.plane_b : L.plane_a;
        so[op].codes = (const uint4*)(op ? b_codes : a_codes);
        so[op].scales = (const uint8_t*)(op ? b_scales : a_scales);
        so[op].plane_f = (uint4*)(ws + off);
        so[op].plane_h = (uint4*)(ws + off + plane);
        so[op].plane_l = (uint4*)(ws + off + 2 * plane);
        so[op].sf_tiled = ws + (op ? L.off_sfb : L.off_sfa);
        so[op].rows = rows;
        so[op].pairs = rows * (k / 32);
        so[op].sf_items = (rows + 127) / 128 * (int64_t)(ktiles / 4u) * 32;
        so[op].gpr = gpr;
        so[op].ktiles = ktiles;
    }
    {
        const int64_t items = has_int ? so[0].pairs + so[1].pairs : so[0].sf_items + so[1].sf_items;
        int64_t blocks = (items + 255) / 256;
        if (blocks > 148 * 8) blocks = 148 * 8;
        if (launch_pdl(if4_split_kernel, dim3((unsigned)blocks), 256, 0, s, so[0], so[1], has_int, (int*)ws) != cudaSuccess)
            return ABS_ERR_CUDA;
    }
    // the opt-in to more than 48 KiB of dynamic shared memory is per device
    static std::once_flag attr_once[64];
    static cudaError_t attr_err[64];
    static int sm_count[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ABS_ERR_CUDA;
    std::call_once(attr_once[dev], [dev]() {
        if (cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count[dev] < 1)
            sm_count[dev] = 1;
        attr_err[dev] = cudaSuccess;
#define ABS_GEMM_ATTR(P, O, B)                                                                                         \
    if (attr_err[dev] == cudaSuccess)                                                                                   \
        attr_err[dev] = cudaFuncSetAttribute(if4_gemm_kernel<P, O, B>, cudaFuncAttributeMaxDynamicSharedMemorySize,      \
                                             kGemmSmemBytes<P, B>)
        ABS_GEMM_ATTR(3, false, 1); ABS_GEMM_ATTR(3, true, 1);
        ABS_GEMM_ATTR(1, false, 1); ABS_GEMM_ATTR(1, true, 1);
        ABS_GEMM_ATTR(1, false, 2); ABS_GEMM_ATTR(1, true, 2);
#undef ABS_GEMM_ATTR
    });
    if (attr_err[dev] != cudaSuccess) return ABS_ERR_CUDA;
    const int32_t tiles_m = (int32_t)((m + kTileM - 1) / kTileM), tiles_n = (int32_t)(n / kTileN);
    const int64_t num_tiles = (int64_t)tiles_m * tiles_n;
    const dim3 pgrid((unsigned)(num_tiles < sm_count[dev] ? num_tiles : sm_count[dev]));
    cudaError_t e;
#define ABS_LAUNCH_GEMM(P, O, B)                                                                                        \
    e = launch_pdl(if4_gemm_kernel<P, O, B>, pgrid, 320, kGemmSmemBytes<P, B>, s, maps, (const uint8_t*)(ws + L.off_sfa), \
                   (const uint8_t*)(ws + L.off_sfb), a_alpha, b_alpha, c_f32, tiles_m, tiles_n,                           \
                   (int32_t)(k / (kStageK * B)), (int32_t)m, (int*)ws, stall_step, next_alpha, next_denom)
    const bool long_steps = !has_int && k % (2 * kStageK) == 0;      // NVFP4: K-steps of 512 where K allows
    if (has_int && out_bf16) ABS_LAUNCH_GEMM(3, true, 1);
    else if (has_int) ABS_LAUNCH_GEMM(3, false, 1);
    else if (long_steps && out_bf16) ABS_LAUNCH_GEMM(1, true, 2);
    else if (long_steps) ABS_LAUNCH_GEMM(1, false, 2);
    else if (out_bf16) ABS_LAUNCH_GEMM(1, true, 1);
    else ABS_LAUNCH_GEMM(1, false, 1);
#undef ABS_LAUNCH_GEMM
    if (e != cudaSuccess) return ABS_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
}

abs_status_t abs_matmul(abs_fmt_t fmt, const void* a_codes, const void* a_scales, const float* a_alpha, const void* b_codes,
                        const void* b_scales, const float* b_alpha, int64_t m, int64_t n, int64_t k, float* c_f32,
                        void* workspace, size_t workspace_bytes, void* stream) {
    return matmul_impl(fmt, a_codes, a_scales, a_alpha, b_codes, b_scales, b_alpha, m, n, k, c_f32, workspace, workspace_bytes, stream, -1);
}

abs_status_t abs_matmul_bf16(abs_fmt_t fmt, const void* a_codes, const void* a_scales, const float* a_alpha, const void* b_codes,
                             const void* b_scales, const float* b_alpha, int64_t m, int64_t n, int64_t k, void* c_bf16,
                             void* workspace, size_t workspace_bytes, void* stream) {
    return matmul_impl(fmt, a_codes, a_scales, a_alpha, b_codes, b_scales, b_alpha, m, n, k, c_bf16, workspace, workspace_bytes, stream, -1,
                       true);
}

abs_status_t abs_matmul_bf16_scaled(abs_fmt_t fmt, const void* a_codes, const void* a_scales, const float* a_alpha,
                                    const void* b_codes, const void* b_scales, const float* b_alpha, int64_t m, int64_t n, int64_t k,
                                    void* c_bf16, abs_fmt_t next_fmt, float* next_alpha, void* workspace, size_t workspace_bytes,
                                    void* stream) {
    if (!next_alpha) return ABS_ERR_NULL;
    float m_fp;
    switch (next_fmt) {
        case ABS_FMT_NVFP4: case ABS_FMT_IF4: case ABS_FMT_IF4_BS8: case ABS_FMT_NVFP4_BS8: m_fp = 6.0f; break;
        case ABS_FMT_IF3: case ABS_FMT_IF3_BS8: m_fp = 4.0f; break;
        case ABS_FMT_IF6_E2M3: m_fp = 7.5f; break;
        case ABS_FMT_IF6_E3M2: m_fp = 28.0f; break;
        default: return ABS_ERR_FMT;
    }
    return matmul_impl(fmt, a_codes, a_scales, a_alpha, b_codes, b_scales, b_alpha, m, n, k, c_bf16, workspace, workspace_bytes, stream, -1,
                       true, next_alpha, m_fp * 448.0f);
}

abs_status_t abs_selftest_matmul_stall(abs_fmt_t fmt, const void* a_codes, const void* a_scales, const float* a_alpha,
                                       const void* b_codes, const void* b_scales, const float* b_alpha, int64_t m, int64_t n,
                                       int64_t k, float* c_f32, void* workspace, size_t workspace_bytes, void* stream,
                                       int32_t stall_step) {
    if (stall_step < 0) return ABS_ERR_SHAPE;
    return matmul_impl(fmt, a_codes, a_scales, a_alpha, b_codes, b_scales, b_alpha, m, n, k, c_f32, workspace, workspace_bytes, stream,
                       stall_step);
}

abs_status_t abs_matmul_check(const void* workspace, void* stream) {
    if (!workspace) return ABS_ERR_NULL;
    int word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess ||
        cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess)
        return ABS_ERR_CUDA;
    return word == 0 ? ABS_OK : ABS_ERR_CUDA;
}

}  // extern "C"
