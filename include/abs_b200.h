/*
 * abs_b200.h -- C ABI of the B200 (sm_100a) quantize / dequantize library for the
 * Adaptive Block-Scaled (IF) data types: IF4, IF3, IF6 and plain NVFP4.
 *
 * Data model (paper Sec. 3, Eq. 1-2, Fig. 3a; Sec. 5.1 for the other widths):
 *   - a row-major bf16 matrix [rows, cols], cols a multiple of 16;
 *   - one FP32 tensor scale alpha = max|X| / (M_FP * 448)                      (Eq. 1);
 *   - one E4M3 byte per 16 consecutive row elements, Delta = E4M3(gmax/(alpha*M_FP)) (Eq. 2);
 *     bit 7 of that byte is the type flag: 1 = the group is stored as scaled integers
 *     (pre-scaled by M_INT/M_FP, de-scaled by M_FP/M_INT on the way back), 0 = as the
 *     format's minifloat, in which case an IF4 group is exactly an NVFP4 group   (Sec. 3);
 *   - 16 b-bit codes per group, packed as a little-endian bitstream: code j occupies bits
 *     [b*j, b*j+b) of the group's 2*b bytes (IF4/NVFP4: element 2j in the low nibble of
 *     byte j).  FP codes are sign|exponent|mantissa, integer codes two's complement.
 *
 * Unless a function says otherwise every data pointer is a DEVICE pointer owned by the
 * caller; the library neither frees nor keeps it.  Calls validate on the host, enqueue
 * their kernels on `stream` (a cudaStream_t passed as void*, NULL = default stream) and
 * return without synchronising; execution errors surface at the caller's next sync.
 * Inputs must be finite and the tensor maximum either 0 or at least 2^-100; input and
 * output buffers must not overlap.  All device pointers must be 16-byte aligned.
 * The library keeps a small per-device scratch ring (allocated on the first quantize call
 * on a device, or by abs_init); make that first call outside any stream capture.
 *   - In flight: every call that runs an amax pass (abs_amax, and abs_quantize* without
 *     ABS_F_ALPHA_GIVEN) takes the next of ABS_MAX_INFLIGHT ring slots, chosen on the host.  If
 *     more than ABS_MAX_INFLIGHT such calls are enqueued on a device before the oldest has run,
 *     the oldest loses its maximum: its kernel notices (the slot carries another call's tag),
 *     quantizes with alpha = 1, and raises a flag that makes the NEXT such call on the device
 *     return ABS_ERR_SIZE once, so the overrun cannot pass unseen.
 *   - CUDA graphs: the slot and its tag are kernel arguments fixed at enqueue time, so a captured
 *     call of that kind must not be replayed (a replay would merge its maximum with the previous
 *     replay's).  Inside a graph use ABS_F_ALPHA_GIVEN with an alpha computed outside the graph.
 *     Calls with ABS_F_ALPHA_GIVEN, and every dequantize call, use no scratch and may be captured.
 * There is no CPU fallback: without a CUDA device every compute call returns ABS_ERR_CUDA.
 */
#ifndef ABS_B200_H
#define ABS_B200_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define ABS_API __attribute__((visibility("default")))
#else
#define ABS_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

/* Formats.  (M_FP, M_INT, bits): NVFP4 (6, -, 4); IF4 (6, 7, 4) Sec. 3; IF3 (4, 3, 3),
 * IF6_E2M3 (7.5, 31, 6), IF6_E3M2 (28, 31, 6) Sec. 5.1 footnote and Table 5. */
typedef enum {
    ABS_FMT_NVFP4 = 0,
    ABS_FMT_IF4 = 1,
    ABS_FMT_IF3 = 2,
    ABS_FMT_IF6_E2M3 = 3,
    ABS_FMT_IF6_E3M2 = 4,
    /* Block-size-8 variants (Sec. 5.1, Table 5): one E4M3 scale per 8 values instead of 16; codes are
     * laid out exactly as for the 16-value sibling, the scale array is [rows, cols/8]. */
    ABS_FMT_NVFP4_BS8 = 5,
    ABS_FMT_IF4_BS8 = 6,
    ABS_FMT_IF3_BS8 = 7
} abs_fmt_t;

typedef enum {
    ABS_OK = 0,
    ABS_ERR_NULL = 1,   /* a required pointer is NULL                         */
    ABS_ERR_SHAPE = 2,  /* negative size, or cols not a multiple of 16        */
    ABS_ERR_ALIGN = 3,  /* a device pointer is not 16-byte aligned            */
    ABS_ERR_FMT = 4,    /* unknown format                                     */
    ABS_ERR_FLAGS = 5,  /* unknown flag bit, or a flag the call cannot honour */
    ABS_ERR_CUDA = 6,   /* a CUDA runtime call or a launch failed             */
    ABS_ERR_SIZE = 7    /* workspace too small / size beyond a stated maximum / an earlier call on this device
                           overran the ring of ABS_MAX_INFLIGHT scratch slots (see the top of this file)   */
} abs_status_t;

enum {
    ABS_F_HADAMARD16 = 1u << 0,     /* quantize: 16-point blockwise random Hadamard transform of every
                                       group before the amax pass and the encoding (Sec. 4.1)            */
    ABS_F_STOCHASTIC = 1u << 1,     /* quantize: stochastic rounding of both candidates from
                                       Philox4x32-10(sr_seed, element index) (Sec. 4.1, App. B)          */
    ABS_F_SR_SCALE_17_16 = 1u << 2, /* quantize: group scale target times 17/16 before E4M3 rounding,
                                       the 16/17 factor of Sec. 4.1, so stochastic values never clip     */
    ABS_F_ALPHA_GIVEN = 1u << 3,    /* quantize: *tensor_scale_f32 is an input; the amax pass is skipped */
    ABS_F_OUT_FP32 = 1u << 4,       /* dequantize: write the FP32 products instead of bf16               */
    ABS_F_SCALES_SWIZZLED = 1u << 6, /* quantize / dequantize, ABS_FMT_NVFP4 and ABS_FMT_IF4 only: the scale array uses
                                       the 128x4-tile layout that Blackwell block-scaled tensor-core MMAs read
                                       (see abs_scales_bytes_swizzled) instead of row-major [rows, cols/16]      */
    ABS_F_FP_GROUPS_ONLY = 1u << 7,  /* dequantize (ABS_FMT_IF4, bf16 output): groups stored as integers come out as +0    */
    ABS_F_INT_GROUPS_RAW = 1u << 8,  /* dequantize (ABS_FMT_IF4, bf16 output): FP groups come out as +0 and integer groups as
                                       k * Delta * alpha WITHOUT the 6/7 de-scale.  Both halves are exact in bf16, so
                                       the MAC arithmetic of Sec. 5.2 (factors 1, 6/7, 36/49 applied in FP32 on the
                                       scale path) can be reproduced with four plain bf16 GEMMs                      */
    ABS_F_GROUPS_DOWN_COLUMNS = 1u << 9, /* abs_quantize_dequantize only: groups are 16 consecutive ROWS of one column
                                       (Sec. 4.1: the operands of the weight-gradient product are quantized along the
                                       token dimension); needs rows % 16 == 0                                        */
    ABS_F_INDEX64 = 1u << 5         /* TESTING ONLY (see the last block of this file)                    */
};

#define ABS_MAX_INFLIGHT 1024

typedef struct {
    uint32_t flags;         /* OR of ABS_F_*                                                     */
    uint16_t had_sign_mask; /* Hadamard option: bit i = 1 multiplies element i of each group by -1 */
    uint16_t _pad;          /* must be 0                                                          */
    uint64_t sr_seed;       /* stochastic rounding: Philox key                                    */
    uint64_t sr_index_offset; /* stochastic rounding: index, in the whole tensor, of this call's first element.
                               Element (r, c) of the matrix passed to the call draws the random field of index
                               sr_index_offset + r * cols + c (App. B: one stream over the tensor), so a row shard
                               that starts at row r0 of a [R, cols] tensor passes r0 * cols and gets the bytes the
                               unsharded call gives for those rows.  A multiple of 16 (else ABS_ERR_SHAPE); read
                               only with ABS_F_STOCHASTIC.  For abs_quantize_transposed and the column mode of
                               abs_quantize_dequantize the index runs over the transposed matrix.               */
} abs_opts_t;

/* Sizes of the outputs of abs_quantize: rows*cols*b/8 and rows*cols/16 bytes (rows*cols/8 for the
 * block-size-8 formats); 0 on bad arguments. */
ABS_API size_t abs_codes_bytes(abs_fmt_t fmt, int64_t rows, int64_t cols);
ABS_API size_t abs_scales_bytes(abs_fmt_t fmt, int64_t rows, int64_t cols);
ABS_API const char* abs_status_string(abs_status_t status);

/* Size of the scale array with ABS_F_SCALES_SWIZZLED.  (Sec. 3 notes that a group stored as FP4 is an
 * NVFP4 group; this option stores the scales where NVFP4 tensor-core kernels expect them.)  The scale of
 * row r, group k (k = column / 16) lives at byte
 *     ((r / 128) * ceil(K / 4) + k / 4) * 512 + (r % 32) * 16 + ((r % 128) / 32) * 4 + k % 4,   K = cols / 16,
 * i.e. tiles of 128 rows x 4 scales, 512 bytes each, tiles ordered row-major.  The array is padded to whole
 * tiles: ceil(rows / 128) * ceil(K / 4) * 512 bytes; the library never writes the padding bytes. */
ABS_API size_t abs_scales_bytes_swizzled(abs_fmt_t fmt, int64_t rows, int64_t cols);

/* Allocates the per-device scratch ring of `device` now (synchronous).  Optional: the first
 * quantize call on a device does the same. */
ABS_API abs_status_t abs_init(int device);

/* Quantize (Eq. 1-2, Fig. 3a steps 1-10, Sec. 3 "6/7 method" and sign-bit flag).
 *   in_bf16          [rows, cols] bf16, row-major, leading dimension = cols
 *   codes_u8         out, abs_codes_bytes() bytes, group g at byte offset g*2*b
 *   scales_e4m3      out, abs_scales_bytes() bytes, row-major [rows, cols/16]
 *   tensor_scale_f32 device pointer to one float: out (alpha), or in with ABS_F_ALPHA_GIVEN
 * Launches a grid-wide amax reduction that also writes alpha, then the group-quantize kernel.
 * rows*cols == 0 is ABS_OK and enqueues nothing.  abs_quantize == abs_quantize_ex with no options. */
ABS_API abs_status_t abs_quantize(abs_fmt_t fmt, const void* in_bf16, int64_t rows, int64_t cols, void* codes_u8,
                          void* scales_e4m3, float* tensor_scale_f32, void* stream);
ABS_API abs_status_t abs_quantize_ex(abs_fmt_t fmt, const void* in_bf16, int64_t rows, int64_t cols, void* codes_u8,
                             void* scales_e4m3, float* tensor_scale_f32, const abs_opts_t* opts, void* stream);

/* Quantize the transpose (Sec. 4.1: for the weight-gradient product both operands are quantized along
 * the token dimension, i.e. down the columns of a [tokens, features] matrix).  `in_bf16` is the same
 * row-major [rows, cols] matrix as for abs_quantize; the outputs are exactly what abs_quantize would
 * give for its transpose [cols, rows]: groups are 16 consecutive rows of one column,
 *   codes_t_u8    [cols, rows*b/8]   scales_t_e4m3 [cols, rows/16]   alpha as for abs_quantize.
 * The transpose is never materialised.  rows and cols must be multiples of 16; formats ABS_FMT_IF4 and
 * ABS_FMT_NVFP4; flags accepted: ABS_F_ALPHA_GIVEN, ABS_F_HADAMARD16 (the transform then runs along the
 * groups, i.e. down the columns: the paper's recipe for both operands of the weight-gradient product),
 * ABS_F_STOCHASTIC and ABS_F_SR_SCALE_17_16 (App. B; element indices, hence the random stream, are those of
 * the transposed matrix); any other flag is ABS_ERR_FLAGS.  abs_dequantize(fmt, ..., cols, rows, ...)
 * turns the result back into the transposed matrix. */
ABS_API abs_status_t abs_quantize_transposed(abs_fmt_t fmt, const void* in_bf16, int64_t rows, int64_t cols,
                                             void* codes_t_u8, void* scales_t_e4m3, float* tensor_scale_f32,
                                             const abs_opts_t* opts, void* stream);

/* Quantize and dequantize in one pass: the emulation of Sec. 4.1 (every format studied was emulated by
 * dequantizing the quantized values back to BF16 before each matrix product).  Every format; flags
 * ABS_F_ALPHA_GIVEN and ABS_F_SR_SCALE_17_16, and for ABS_FMT_IF4 / ABS_FMT_NVFP4 also ABS_F_HADAMARD16,
 * ABS_F_STOCHASTIC and ABS_F_GROUPS_DOWN_COLUMNS.
 *   in_bf16          [rows, cols] bf16 (device), as for abs_quantize
 *   out_bf16         out, [rows, cols] bf16 (device): byte for byte what abs_dequantize gives for the result
 *                    of abs_quantize_ex with the same options (with the Hadamard option: the dequantized
 *                    TRANSFORMED values; nothing inverts the transform, as in abs_dequantize)
 *   codes_u8, scales_e4m3   optional outputs as for abs_quantize; pass both or pass NULL for both
 *   tensor_scale_f32 device pointer to one float: out (alpha), or in with ABS_F_ALPHA_GIVEN
 * With ABS_F_GROUPS_DOWN_COLUMNS the groups run down the columns, as in abs_quantize_transposed: out_bf16 is
 * still [rows, cols] in the orientation of the input (element (r, c) is the dequantized value of input element
 * (r, c)), while the optional codes and scales come in the transposed layout of abs_quantize_transposed.
 * Each group is decoded from the registers that hold its codes, so the codes are never read back.  All
 * pointers 16-byte aligned; in_bf16 and out_bf16 must not overlap.  Flags the format does not take:
 * ABS_ERR_FLAGS; more than about 2^31 groups: ABS_ERR_SIZE. */
ABS_API abs_status_t abs_quantize_dequantize(abs_fmt_t fmt, const void* in_bf16, int64_t rows, int64_t cols,
                                             void* out_bf16, void* codes_u8, void* scales_e4m3, float* tensor_scale_f32,
                                             const abs_opts_t* opts, void* stream);

/* Quantize without any allocation.  (The paper has no counterpart: this entry point exists for the
 * way the library is deployed, not for the method.)
 *
 * abs_quantize keeps its amax scratch in device memory that it obtains with cudaMalloc the first time
 * it runs on a device.  Some callers cannot afford that: a serving process that has already handed
 * every free byte of device memory to its own pool, so that a later cudaMalloc simply fails; or a
 * latency-critical loop that must not run into the device-wide synchronisation cudaMalloc implies.
 * For them this variant computes exactly the same outputs as abs_quantize(fmt, ...) with round to
 * nearest and no options, but its amax pass reduces the tensor in chunks of 131072 elements whose
 * partial maxima go to an array that is part of the library image (33 KiB on every GPU that loads
 * the library, held until the process exits).  It calls no cudaMalloc, cudaFree or other allocating
 * routine, and it allocates nothing through any framework.
 *
 *   - Limit: at most ABS_NOALLOC_MAX_ELEMS = 8192 chunks x 131072 = 1 073 741 824 elements; a larger
 *     rows*cols returns ABS_ERR_SIZE and enqueues nothing.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress, with that
 *     device current); make that first call before any stream capture.
 *   - With CUDA's default lazy module loading the first launch of each kernel loads its code onto the
 *     device, which itself needs a little device memory.  A caller whose pool is about to take every
 *     free byte should therefore make one abs_quantize_noalloc call per format it will use, with input
 *     pointers of the alignment it will use (32-byte and 16-byte aligned inputs run different kernel
 *     instances), BEFORE handing out its last memory, or run with CUDA_MODULE_LOADING=EAGER.
 *   - All calls on a device share the one array.  Each call clears the ticket word it needs at zero
 *     itself (a 4-byte cudaMemsetAsync on `stream`) and overwrites every partial maximum it reads, so
 *     stale contents from earlier calls are harmless; but two calls that overlap on the GPU (different
 *     streams, or graphs replayed concurrently) race on the array and produce wrong scales.  Serialise
 *     them, or use abs_quantize on one of the streams.
 * Arguments, layouts, alignment rules and the other status codes are those of abs_quantize. */
#define ABS_NOALLOC_MAX_ELEMS ((int64_t)8192 * 8192 * 16)
ABS_API abs_status_t abs_quantize_noalloc(abs_fmt_t fmt, const void* in_bf16, int64_t rows, int64_t cols,
                                          void* codes_u8, void* scales_e4m3, float* tensor_scale_f32, void* stream);

/* Dequantize (Sec. 3: de-scale integer groups by M_FP/M_INT; Sec. 4.1: product in FP32, then
 * bf16 round-to-nearest-even).  out is bf16 [rows, cols], or float with ABS_F_OUT_FP32 (the only
 * flag accepted).  The Hadamard option is not inverted here. */
ABS_API abs_status_t abs_dequantize(abs_fmt_t fmt, const void* codes_u8, const void* scales_e4m3,
                            const float* tensor_scale_f32, int64_t rows, int64_t cols, void* out_bf16,
                            void* stream);
ABS_API abs_status_t abs_dequantize_ex(abs_fmt_t fmt, const void* codes_u8, const void* scales_e4m3,
                               const float* tensor_scale_f32, int64_t rows, int64_t cols, void* out,
                               const abs_opts_t* opts, void* stream);

/* Eq. 1 alone: the grid-wide amax pass.  Writes max|X| (after the Hadamard option when asked) to
 * *amax_f32 (device).  With it a row-sharded tensor can be quantized on several GPUs: each rank
 * reduces its rows, the ranks exchange one float (max), and each rank calls abs_quantize_ex with
 * ABS_F_ALPHA_GIVEN and alpha = abs_alpha_from_amax(fmt, global max). */
ABS_API abs_status_t abs_amax(const void* in_bf16, int64_t rows, int64_t cols, const abs_opts_t* opts, float* amax_f32,
                      void* stream);
/* Host arithmetic of Eq. 1: amax / (M_FP * 448) in IEEE single precision; 1.0f when amax == 0. */
ABS_API float abs_alpha_from_amax(abs_fmt_t fmt, float amax);

/* Matrix product of two quantized operands on the tensor cores, C = A B^T, with the arithmetic of the paper's MAC
 * unit (Sec. 5.2): the decoded codes of a pair of groups are multiplied and summed exactly, the sum is scaled by
 * Delta_a * Delta_b, and the FP32 factor 1, 6/7 or 36/49 is applied on the scale path when none, one or both of
 * the groups are stored as integers; alpha_a * alpha_b multiplies the result.  FP groups are NVFP4 groups (Sec. 3)
 * and go to the block-scaled FP4 MMA (tcgen05.mma kind::mxf4nvf4) unchanged; an integer code k in -7..7 is the sum
 * of two E2M1 values (5 = 4 + 1, 7 = 6 + 1), so each operand is first split into three NVFP4 planes in the
 * workspace and the three kinds of group pairs accumulate in three FP32 accumulators that meet in the epilogue.
 *   fmt                ABS_FMT_IF4 or ABS_FMT_NVFP4 (both operands)
 *   a_codes, a_scales  A as abs_quantize wrote it: [m, k] quantized along k, scales row-major [m, k/16]; a_alpha its alpha
 *   b_codes, b_scales  B likewise: [n, k]
 *   c_f32              out, [m, n] float, row-major
 *   workspace          device memory, 1024-byte aligned, at least abs_matmul_workspace_bytes(fmt, m, n, k) bytes
 * m is any positive number of rows; n must be a multiple of 128, k a multiple of 256 (ABS_ERR_SHAPE otherwise; abs_matmul_workspace_bytes
 * returns 0).  Asynchronous like the other calls.  Every wait inside the kernel is bounded; if one runs out (it
 * never should) the kernel stops and leaves a non-zero word at the start of the workspace, which
 * abs_matmul_check(workspace, stream) reads back (it synchronises the stream): ABS_OK, or ABS_ERR_CUDA.
 * The workspace belongs to one call at a time: calls that share it must be ordered on one stream (concurrent calls on
 * different streams take a workspace each).  Its contents mean nothing between calls.
 * Single GPU: the tensor maps cover the caller's workspace and operands on the current device only. */
ABS_API size_t abs_matmul_workspace_bytes(abs_fmt_t fmt, int64_t m, int64_t n, int64_t k);
ABS_API abs_status_t abs_matmul(abs_fmt_t fmt, const void* a_codes, const void* a_scales, const float* a_alpha,
                                const void* b_codes, const void* b_scales, const float* b_alpha, int64_t m, int64_t n,
                                int64_t k, float* c_f32, void* workspace, size_t workspace_bytes, void* stream);
/* The same product written as bf16 [m, n]: each entry is the FP32 result of abs_matmul rounded to nearest even, so
 * that it can go straight into the next abs_quantize call. */
ABS_API abs_status_t abs_matmul_bf16(abs_fmt_t fmt, const void* a_codes, const void* a_scales, const float* a_alpha,
                                     const void* b_codes, const void* b_scales, const float* b_alpha, int64_t m, int64_t n,
                                     int64_t k, void* c_bf16, void* workspace, size_t workspace_bytes, void* stream);
/* abs_matmul_bf16 that also prepares the next quantization of its output: the epilogue keeps the largest |C| it writes
 * and the kernel leaves  next_alpha = max|C| / (M_FP(next_fmt) * 448)  (Eq. 1; 1 for an all-zero C) in the device float
 * next_alpha -- the value abs_quantize(next_fmt, C, ...) would compute with its own pass over C.  The next call can then
 * be abs_quantize_ex with ABS_F_ALPHA_GIVEN and tensor_scale_f32 = next_alpha: same bytes, one pass over C less.
 * next_alpha is left unwritten when a wait inside the kernel ran out (abs_matmul_check then reports it). */
ABS_API abs_status_t abs_matmul_bf16_scaled(abs_fmt_t fmt, const void* a_codes, const void* a_scales, const float* a_alpha,
                                            const void* b_codes, const void* b_scales, const float* b_alpha, int64_t m,
                                            int64_t n, int64_t k, void* c_bf16, abs_fmt_t next_fmt, float* next_alpha,
                                            void* workspace, size_t workspace_bytes, void* stream);
ABS_API abs_status_t abs_matmul_check(const void* workspace, void* stream);

/* Host-buffer variants: `*_host` pointers are HOST memory (pinned memory makes the copies
 * asynchronous), `d_workspace` is a device buffer of at least abs_host_workspace_bytes() bytes.
 * Each call copies its inputs to the device, runs the same kernels as above, copies the results
 * back and returns after synchronising `stream`.  abs_dequantize_host works in four row chunks and
 * copies each finished chunk back on a second, library-owned stream (created on first use, one per
 * device, ordered against `stream` by events) while the next chunk is uploaded and decoded; calls
 * on the same device are serialised by the library. */
ABS_API size_t abs_host_workspace_bytes(abs_fmt_t fmt, int64_t rows, int64_t cols);
ABS_API abs_status_t abs_quantize_host(abs_fmt_t fmt, const void* in_bf16_host, int64_t rows, int64_t cols,
                               void* codes_u8_host, void* scales_e4m3_host, float* tensor_scale_f32_host,
                               const abs_opts_t* opts, void* d_workspace, size_t workspace_bytes, void* stream);
ABS_API abs_status_t abs_dequantize_host(abs_fmt_t fmt, const void* codes_u8_host, const void* scales_e4m3_host,
                                 const float* tensor_scale_f32_host, int64_t rows, int64_t cols, void* out_host,
                                 const abs_opts_t* opts, void* d_workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * TESTING AND PROFILING ONLY.  Nothing below (nor ABS_F_INDEX64 above) is part of the method or needed
 * by an application; the test suite and the benchmark use them.
 *   ABS_F_INDEX64: run the kernel instances that index groups with 64-bit integers (otherwise chosen
 *   only beyond 2^31 groups); same results.
 * ------------------------------------------------------------------------------------------------ */

/* Profiling hook (no counterpart in the paper): while both handles (cudaEvent_t as void*) are set,
 * every quantize call records them on its stream immediately before and after the group-quantize
 * kernel, so a caller can time that kernel inside a longer stream of work.  Pass NULLs to switch it
 * off.  Process-wide and not thread-safe: set it only while no other thread is calling the library. */
ABS_API void abs_profile_events(void* quantize_begin, void* quantize_end);

/* Self-test hook: applies one of the device conversions the kernels use to n FP32 values.
 *   kind 0: E4M3 scale byte (Fig. 3a step 2)   kind 1..4: FP element code of NVFP4/IF4 (E2M1),
 *   IF3 (E2M0), IF6_E2M3, IF6_E3M2 (step 4)    kind 5: integer candidate rint(z) & 0xFF (step 7)
 * out_u8[i] = conversion(in_f32[i]).  kind 16 + k (k = 0..4): decode, in_f32[i] holds a code in its
 * low byte as an integer-valued float and out is float: value of E4M3 byte / FP element code. */
ABS_API abs_status_t abs_selftest_convert(int kind, const float* in_f32, int64_t n, void* out, void* stream);

/* Self-test hook for the bounded waits of abs_matmul: the same call, but in every block the loads of pipeline step
 * number `stall_step` (counted from 0 over the block's tiles) are announced and never issued, so the block's waits run
 * out after their limit (one second each, concurrently), the error word is set, the block frees its tensor memory and
 * returns.  Nothing faults and nothing waits without a bound; abs_matmul_check then reports ABS_ERR_CUDA and the next
 * abs_matmul call works normally.  c_f32 is left incomplete. */
ABS_API abs_status_t abs_selftest_matmul_stall(abs_fmt_t fmt, const void* a_codes, const void* a_scales, const float* a_alpha,
                                               const void* b_codes, const void* b_scales, const float* b_alpha, int64_t m,
                                               int64_t n, int64_t k, float* c_f32, void* workspace, size_t workspace_bytes,
                                               void* stream, int32_t stall_step);

#ifdef __cplusplus
}
#endif
#endif /* ABS_B200_H */
