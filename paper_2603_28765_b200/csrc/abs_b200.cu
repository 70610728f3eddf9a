// Host side and C ABI of the B200 IF4 / IF3 / IF6 / NVFP4 quantize-dequantize library: argument
// validation, per-device scratch, kernel selection and launches.
//
// Path (paper Sec. 3): amax_kernel (Eq. 1, grid-wide max) -> group-quantize kernel (Eq. 2 and Fig. 3a
// steps 1-10 per 16-value group, flag in the scale's sign bit, packed codes); the dequantize kernels are
// the inverse (Sec. 3, Sec. 4.1).  Kernels: abs_generic.cuh (amax; every format and option, element by
// element), abs_fast4.cuh (4-bit round-to-nearest quantize and dequantize), abs_opt4.cuh (4-bit with the
// Hadamard / stochastic-rounding options, one-pass emulation), abs_fastx.cuh (IF3, IF6, block size 8),
// abs_trans4.cuh (groups down the columns), abs_device.cuh (building blocks).
#include "../../include/abs_b200.h"
#include "abs_device.cuh"
#include "abs_fast4.cuh"
#include "abs_opt4.cuh"
#include "abs_fastx.cuh"
#include "abs_trans4.cuh"
#include "abs_generic.cuh"

#include <atomic>
#include <mutex>

using namespace absq;

namespace {

constexpr int kMaxDevices = 64;

// Launch with programmatic stream serialization: the kernel may be scheduled while the previous
// kernel of the stream drains; every kernel here calls pdl_wait() before its first global access.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), int grid, int block, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ------------------------------------------------------------------------------------------ host state

constexpr int kHostChunks = 4;        // row chunks of abs_dequantize_host

struct DeviceState {
    std::once_flag once;
    cudaError_t init_err = cudaSuccess;
    uint32_t* ring = nullptr;          // ABS_MAX_INFLIGHT slots of 16 bytes: tagged maximum (u64), ticket (u32), pad
    std::mutex slot_mu;                // guards `next` and the clearing of the ring when the generation wraps
    uint64_t next = 0;                 // calls that took a slot so far; generation = low 32 bits
    uint32_t* overrun_host = nullptr;  // pinned, mapped word a kernel sets when its slot was reused under it
    uint32_t* overrun_dev = nullptr;   // the same word as the device sees it
    int sm_count = 148;
    // abs_dequantize_host: a second stream for the device-to-host copies and the events that order it
    std::mutex host_mu;
    cudaStream_t d2h_stream = nullptr;
    cudaEvent_t chunk_done[kHostChunks] = {};
    cudaEvent_t d2h_done = nullptr;
};
DeviceState g_dev[kMaxDevices];

// Optional CUDA events recorded around the group-quantize kernel (abs_profile_events).
cudaEvent_t g_ev_quant_begin = nullptr, g_ev_quant_end = nullptr;

abs_status_t device_state(DeviceState** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ABS_ERR_CUDA;
    DeviceState& st = g_dev[dev];
    std::call_once(st.once, [&]() {
        st.init_err = cudaMalloc(&st.ring, ABS_MAX_INFLIGHT * 4 * sizeof(uint32_t));
        if (st.init_err == cudaSuccess) st.init_err = cudaMemset(st.ring, 0, ABS_MAX_INFLIGHT * 4 * sizeof(uint32_t));
        if (st.init_err == cudaSuccess) st.init_err = cudaHostAlloc(&st.overrun_host, sizeof(uint32_t), cudaHostAllocMapped);
        if (st.init_err == cudaSuccess) {
            *st.overrun_host = 0u;
            st.init_err = cudaHostGetDevicePointer(&st.overrun_dev, st.overrun_host, 0);
        }
        int sms = 0;
        if (st.init_err == cudaSuccess) st.init_err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms > 0) st.sm_count = sms;
    });
    if (st.init_err != cudaSuccess) return ABS_ERR_CUDA;
    *out = &st;
    return ABS_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int fmt_group(int fmt) { return (fmt >= ABS_FMT_NVFP4_BS8 && fmt <= ABS_FMT_IF3_BS8) ? 8 : 16; }

int fmt_bits(int fmt) {
    switch (fmt) {
        case ABS_FMT_NVFP4: case ABS_FMT_IF4: case ABS_FMT_NVFP4_BS8: case ABS_FMT_IF4_BS8: return 4;
        case ABS_FMT_IF3: case ABS_FMT_IF3_BS8: return 3;
        case ABS_FMT_IF6_E2M3: case ABS_FMT_IF6_E3M2: return 6;
        default: return 0;
    }
}
float fmt_mfp(int fmt) {
    switch (fmt) {
        case ABS_FMT_NVFP4: case ABS_FMT_IF4: case ABS_FMT_NVFP4_BS8: case ABS_FMT_IF4_BS8: return 6.0f;
        case ABS_FMT_IF3: case ABS_FMT_IF3_BS8: return 4.0f;
        case ABS_FMT_IF6_E2M3: return 7.5f;
        default: return 28.0f;
    }
}

constexpr uint32_t kQuantFlags = ABS_F_HADAMARD16 | ABS_F_STOCHASTIC | ABS_F_SR_SCALE_17_16 | ABS_F_ALPHA_GIVEN |
                                 ABS_F_INDEX64 | ABS_F_SCALES_SWIZZLED;

int grid_for(int sm_count, int64_t work_items, int blocks_per_sm) {
    int64_t want = (work_items + kThreads - 1) / kThreads;
    int64_t cap = (int64_t)sm_count * blocks_per_sm;
    return (int)(want < cap ? (want < 1 ? 1 : want) : cap);
}

// Grid of a grid-stride kernel that keeps `resident_per_sm` blocks on every SM: a whole number of waves of
// resident blocks, chosen so that a thread handles about `target_iters` work items.  A few items per thread
// amortise the prologue and keep the prefetch running; several waves let blocks that start later overlap
// their first loads with the arithmetic of the others (measured: about seven items per thread is best for
// the IF4 kernel, 10 % faster than one wave of long-running blocks).
int grid_waves(int sm_count, int64_t work_items, int resident_per_sm, int target_iters) {
    const int64_t want = (work_items + kThreads - 1) / kThreads;
    const int64_t resident = (int64_t)sm_count * resident_per_sm;
    if (want <= resident) return (int)(want < 1 ? 1 : want);
    int64_t waves = (want + (int64_t)target_iters * resident / 2) / ((int64_t)target_iters * resident);
    if (waves < 1) waves = 1;
    const int64_t grid = waves * resident;
    return (int)(grid < want ? grid : want);
}

// Takes the next scratch slot and generation of this device.  Generations grow by one per call; when the
// 32-bit generation wraps (after 2^32 calls) the ring is cleared once, after the device went idle, while the
// mutex keeps other callers out.  Returns ABS_ERR_SIZE (once) if a kernel of an earlier call reported that its
// slot had been reused while it was in flight: that call's scales were computed with alpha = 1.
abs_status_t next_slot(DeviceState& st, unsigned long long** slot, uint32_t* gen) {
    std::lock_guard<std::mutex> lock(st.slot_mu);
    if (*reinterpret_cast<volatile uint32_t*>(st.overrun_host)) {
        *reinterpret_cast<volatile uint32_t*>(st.overrun_host) = 0u;
        return ABS_ERR_SIZE;
    }
    uint32_t g = (uint32_t)++st.next;
    if (g == 0) {
        if (cudaDeviceSynchronize() != cudaSuccess) return ABS_ERR_CUDA;
        if (cudaMemset(st.ring, 0, ABS_MAX_INFLIGHT * 4 * sizeof(uint32_t)) != cudaSuccess) return ABS_ERR_CUDA;
        g = (uint32_t)++st.next;
    }
    *gen = g;
    *slot = reinterpret_cast<unsigned long long*>(st.ring + 4 * (g % ABS_MAX_INFLIGHT));
    return ABS_OK;
}

// ticket = true: the kernel itself writes max |x| (denom == 0) or alpha to `result` (abs_amax).
// ticket = false: the maximum stays in the slot for the quantize kernel of the same call.
abs_status_t launch_amax(int sm_count, const void* in, int64_t ngroups, const abs_opts_t& o, bool ticket,
                         unsigned long long* slot, uint32_t gen, float* result, float denom, cudaStream_t s) {
    const bool rht = o.flags & ABS_F_HADAMARD16;
constexpr int kAmaxRhtBlocksPerSm = kAmaxBlocksPerSm;
    const int grid = grid_for(sm_count, rht ? ngroups : ngroups * 2, rht ? kAmaxRhtBlocksPerSm : kAmaxBlocksPerSm);
    cudaError_t e;
#define ABS_LAUNCH_A(R, T)                                                                                          \
    e = launch_pdl(amax_kernel<R, T>, grid, kThreads, s, (const uint4*)in, ngroups, (uint32_t)o.had_sign_mask, slot, \
                   gen, result, denom)
    if (rht && ticket) ABS_LAUNCH_A(true, true);
    else if (rht) ABS_LAUNCH_A(true, false);
    else if (ticket) ABS_LAUNCH_A(false, true);
    else ABS_LAUNCH_A(false, false);
#undef ABS_LAUNCH_A
    if (e != cudaSuccess) return ABS_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
}

// Groups per thread the grid-stride kernels are launched for (see grid_waves); measured optima, all flat
// within a few per cent around the value.
constexpr int kIf6Iters = 7;   // IF6, IF3 and the integer-bearing block-size-8 round-to-nearest kernels
constexpr int kNvIters = 5;   // groups per thread of the NVFP4 round-to-nearest kernel (5 resident blocks per SM)
constexpr int kDeqIters = 2;   // groups per thread of the 4-bit dequantize kernel
constexpr int kFastIters = 7;   // groups per thread the IF4 round-to-nearest kernel is launched for
constexpr int kOptIters = 12;   // same for the Hadamard / stochastic-rounding kernel

template <int FMT>
// emul_out != nullptr asks for the emulation pass (abs_quantize_dequantize) of the formats handled by the
// kernels of abs_fastx.cuh: bf16 output, codes stored only when emul_store.  *handled tells the caller whether
// a kernel with that ability exists for the format and options.
abs_status_t launch_quantize_fmt(int sm_count, const void* in, int64_t ngroups, void* codes, void* scales,
                                 const AlphaSrc& alpha, const abs_opts_t& o, cudaStream_t s, int64_t cols = 0,
                                 void* emul_out = nullptr, bool emul_store = true, bool* handled = nullptr) {
    if (handled) *handled = false;
    const bool o32 = (reinterpret_cast<uintptr_t>(emul_out) & 31u) == 0;
    const bool rht = o.flags & ABS_F_HADAMARD16, sr = o.flags & ABS_F_STOCHASTIC;
    const float mul = (o.flags & ABS_F_SR_SCALE_17_16) ? 1.0625f : 1.0f;
    const int grid = grid_for(sm_count, ngroups, 64);
    const uint32_t k0 = (uint32_t)o.sr_seed, k1 = (uint32_t)(o.sr_seed >> 32);
    const uint64_t ctr = o.sr_index_offset / 8;      // Philox block of the call's first element (even: offset % 16 == 0)
    const PhiloxKeys pk = philox_keys(o.sr_seed);
    if (g_ev_quant_begin) cudaEventRecord(g_ev_quant_begin, s);
    if constexpr (FMT == ABS_FMT_NVFP4 || FMT == ABS_FMT_IF4) {
        if (emul_out) return ABS_ERR_FLAGS;      // the 4-bit emulation pass is launched by abs_quantize_dequantize
        if (!rht && !sr) {   // the 4-bit round-to-nearest fast path
            const int pgrid = FMT == ABS_FMT_IF4 ? grid_waves(sm_count, ngroups, kFastMinBlocks, kFastIters) : grid_waves(sm_count, ngroups, 5, kNvIters);
            constexpr bool kInt = FMT == ABS_FMT_IF4;
            const bool a32 = (reinterpret_cast<uintptr_t>(in) & 31u) == 0;
            // the kernel looks three grid strides past the current group (next group, and its L2 prefetch)
            const bool i32 = !(o.flags & ABS_F_INDEX64) && ngroups < (int64_t)0x7FFFFFFF - 3 * (int64_t)pgrid * kThreads;
            cudaError_t e;
            const bool swz = o.flags & ABS_F_SCALES_SWIZZLED;
            const uint32_t gpr = swz ? (uint32_t)(cols / 16) : 0u, ktiles = (gpr + 3u) / 4u;
            // L2 prefetch ahead of the loads unless the amax pass of this call has just streamed an input that
            // fits the L2 (about 100 MB of the 126 MB stay resident behind a streaming read)
            const bool pf = !alpha.slot || ngroups * 32 > (int64_t)96 << 20;
#define ABS_LAUNCH_F3(IDX, A32, SLOT, MUL)                                                                           \
    e = swz ? launch_pdl(quantize4_fast_kernel<kInt, IDX, A32, SLOT, MUL, true>, pgrid, kThreads, s,                  \
                         (const uint4*)in, (uint2*)codes, (uint8_t*)scales, alpha, (IDX)ngroups, gpr, ktiles, pf)     \
            : launch_pdl(quantize4_fast_kernel<kInt, IDX, A32, SLOT, MUL, false>, pgrid, kThreads, s,                 \
                         (const uint4*)in, (uint2*)codes, (uint8_t*)scales, alpha, (IDX)ngroups, gpr, ktiles, pf)
#define ABS_LAUNCH_F(IDX, A32)                                                                                       \
    do {                                                                                                             \
        if (alpha.slot && mul != 1.0f) ABS_LAUNCH_F3(IDX, A32, true, true);                                          \
        else if (alpha.slot) ABS_LAUNCH_F3(IDX, A32, true, false);                                                   \
        else if (mul != 1.0f) ABS_LAUNCH_F3(IDX, A32, false, true);                                                  \
        else ABS_LAUNCH_F3(IDX, A32, false, false);                                                                  \
    } while (0)
            if (i32 && a32) ABS_LAUNCH_F(int32_t, true);
            else if (i32) ABS_LAUNCH_F(int32_t, false);
            else if (a32) ABS_LAUNCH_F(int64_t, true);
            else ABS_LAUNCH_F(int64_t, false);
#undef ABS_LAUNCH_F
#undef ABS_LAUNCH_F3
            if (e != cudaSuccess) return ABS_ERR_CUDA;
            if (g_ev_quant_end) cudaEventRecord(g_ev_quant_end, s);
            return cudaGetLastError() == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
        }
    }
    if constexpr (FMT == ABS_FMT_NVFP4 || FMT == ABS_FMT_IF4) {
        // Hadamard / stochastic-rounding options of the 4-bit formats: the packed persistent kernel
        const int ogrid = grid_waves(sm_count, ngroups, opt_blocks_per_sm(sr, rht), kOptIters);
        if (!(o.flags & ABS_F_INDEX64) && ngroups < (int64_t)0x7FFFFFFF - (int64_t)ogrid * kThreads) {
            constexpr bool kInt = FMT == ABS_FMT_IF4;
            const bool a32 = (reinterpret_cast<uintptr_t>(in) & 31u) == 0;
            cudaError_t e;
#define ABS_LAUNCH_O(R, S)                                                                                        \
    e = alpha.slot ? launch_pdl(quantize4_opt_kernel<kInt, R, S, true, false>, ogrid, kThreads, s, (const uint4*)in, \
                                (uint2*)codes, (uint8_t*)scales, alpha, (int32_t)ngroups, mul,                    \
                                (uint32_t)o.had_sign_mask, pk, ctr, a32, (uint4*)nullptr, false, true)             \
                   : launch_pdl(quantize4_opt_kernel<kInt, R, S, false, false>, ogrid, kThreads, s, (const uint4*)in, \
                                (uint2*)codes, (uint8_t*)scales, alpha, (int32_t)ngroups, mul,                    \
                                (uint32_t)o.had_sign_mask, pk, ctr, a32, (uint4*)nullptr, false, true)
            if (rht && sr) ABS_LAUNCH_O(true, true);
            else if (rht) ABS_LAUNCH_O(true, false);
            else ABS_LAUNCH_O(false, true);
#undef ABS_LAUNCH_O
            if (e != cudaSuccess) return ABS_ERR_CUDA;
            if (g_ev_quant_end) cudaEventRecord(g_ev_quant_end, s);
            return cudaGetLastError() == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
        }
    }
    if constexpr (FMT == ABS_FMT_NVFP4_BS8 || FMT == ABS_FMT_IF4_BS8) {
        // block-size-8 variants of the 4-bit formats, round-to-nearest: two groups of 8 per thread
        constexpr bool kInt = FMT == ABS_FMT_IF4_BS8;
        const int bgrid = grid_waves(sm_count, ngroups, kInt ? 4 : 5, kInt ? kIf6Iters : 5);
        if (!rht && !sr && !(o.flags & ABS_F_INDEX64) && ngroups < (int64_t)0x7FFFFFFF - (int64_t)bgrid * kThreads) {
            if (handled) *handled = true;
            const bool a32 = (reinterpret_cast<uintptr_t>(in) & 31u) == 0;
            const cudaError_t e =
                alpha.slot ? (emul_out ? launch_pdl(quantize4_bs8_kernel<kInt, true, true>, bgrid, kThreads, s, (const uint4*)in, (uint2*)codes,
                                        (uint16_t*)scales, alpha, (int32_t)ngroups, mul, a32, (uint4*)emul_out, o32, emul_store) : launch_pdl(quantize4_bs8_kernel<kInt, true, false>, bgrid, kThreads, s, (const uint4*)in, (uint2*)codes,
                                        (uint16_t*)scales, alpha, (int32_t)ngroups, mul, a32, (uint4*)nullptr, false, true))
                           : (emul_out ? launch_pdl(quantize4_bs8_kernel<kInt, false, true>, bgrid, kThreads, s, (const uint4*)in, (uint2*)codes,
                                        (uint16_t*)scales, alpha, (int32_t)ngroups, mul, a32, (uint4*)emul_out, o32, emul_store) : launch_pdl(quantize4_bs8_kernel<kInt, false, false>, bgrid, kThreads, s, (const uint4*)in, (uint2*)codes,
                                        (uint16_t*)scales, alpha, (int32_t)ngroups, mul, a32, (uint4*)nullptr, false, true));
            if (e != cudaSuccess) return ABS_ERR_CUDA;
            if (g_ev_quant_end) cudaEventRecord(g_ev_quant_end, s);
            return cudaGetLastError() == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
        }
    }
    if constexpr (FMT == ABS_FMT_IF6_E2M3 || FMT == ABS_FMT_IF6_E3M2) {
        // 6-bit formats, round-to-nearest
        const int sgrid = grid_waves(sm_count, ngroups, 3, kIf6Iters);
        if (!rht && !sr && !(o.flags & ABS_F_INDEX64) && ngroups < (int64_t)0x7FFFFFFF - (int64_t)sgrid * kThreads) {
            if (handled) *handled = true;
            const bool a32 = (reinterpret_cast<uintptr_t>(in) & 31u) == 0;
            const cudaError_t e =
                alpha.slot ? (emul_out ? launch_pdl(quantize6_fast_kernel<FMT, true, true>, sgrid, kThreads, s, (const uint4*)in, (uint32_t*)codes,
                                        (uint8_t*)scales, alpha, (int32_t)ngroups, mul, a32, (uint4*)emul_out, o32, emul_store) : launch_pdl(quantize6_fast_kernel<FMT, true, false>, sgrid, kThreads, s, (const uint4*)in, (uint32_t*)codes,
                                        (uint8_t*)scales, alpha, (int32_t)ngroups, mul, a32, (uint4*)nullptr, false, true))
                           : (emul_out ? launch_pdl(quantize6_fast_kernel<FMT, false, true>, sgrid, kThreads, s, (const uint4*)in, (uint32_t*)codes,
                                        (uint8_t*)scales, alpha, (int32_t)ngroups, mul, a32, (uint4*)emul_out, o32, emul_store) : launch_pdl(quantize6_fast_kernel<FMT, false, false>, sgrid, kThreads, s, (const uint4*)in, (uint32_t*)codes,
                                        (uint8_t*)scales, alpha, (int32_t)ngroups, mul, a32, (uint4*)nullptr, false, true));
            if (e != cudaSuccess) return ABS_ERR_CUDA;
            if (g_ev_quant_end) cudaEventRecord(g_ev_quant_end, s);
            return cudaGetLastError() == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
        }
    }
    if constexpr (FMT == ABS_FMT_IF3 || FMT == ABS_FMT_IF3_BS8) {
        // IF3 and its block-size-8 variant, round-to-nearest
        constexpr int kG = FMT == ABS_FMT_IF3 ? 16 : 8;
        const int tgrid = grid_waves(sm_count, ngroups, kIf3MinBlocks, kIf6Iters);
        if (!rht && !sr && !(o.flags & ABS_F_INDEX64) && ngroups < (int64_t)0x7FFFFFFF - (int64_t)tgrid * kThreads) {
            if (handled) *handled = true;
            const bool a32 = (reinterpret_cast<uintptr_t>(in) & 31u) == 0;
            const cudaError_t e =
                alpha.slot ? (emul_out ? launch_pdl(quantize3_fast_kernel<kG, true, true>, tgrid, kThreads, s, (const uint4*)in, (uint16_t*)codes,
                                        (uint8_t*)scales, alpha, (int32_t)ngroups, mul, a32, (uint4*)emul_out, o32, emul_store) : launch_pdl(quantize3_fast_kernel<kG, true, false>, tgrid, kThreads, s, (const uint4*)in, (uint16_t*)codes,
                                        (uint8_t*)scales, alpha, (int32_t)ngroups, mul, a32, (uint4*)nullptr, false, true))
                           : (emul_out ? launch_pdl(quantize3_fast_kernel<kG, false, true>, tgrid, kThreads, s, (const uint4*)in, (uint16_t*)codes,
                                        (uint8_t*)scales, alpha, (int32_t)ngroups, mul, a32, (uint4*)emul_out, o32, emul_store) : launch_pdl(quantize3_fast_kernel<kG, false, false>, tgrid, kThreads, s, (const uint4*)in, (uint16_t*)codes,
                                        (uint8_t*)scales, alpha, (int32_t)ngroups, mul, a32, (uint4*)nullptr, false, true));
            if (e != cudaSuccess) return ABS_ERR_CUDA;
            if (g_ev_quant_end) cudaEventRecord(g_ev_quant_end, s);
            return cudaGetLastError() == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
        }
    }
    if (emul_out) return ABS_ERR_FLAGS;          // no emulation kernel for this format / option combination
    cudaError_t eq = cudaSuccess;
#define ABS_LAUNCH_Q(R, S)                                                                                      \
    eq = alpha.slot ? launch_pdl(quantize_kernel<FMT, R, S, true>, grid, kThreads, s, (const uint4*)in,         \
                                 (uint8_t*)codes, (uint8_t*)scales, alpha, ngroups, mul,                        \
                                 (uint32_t)o.had_sign_mask, k0, k1, ctr)                                        \
                    : launch_pdl(quantize_kernel<FMT, R, S, false>, grid, kThreads, s, (const uint4*)in,        \
                                 (uint8_t*)codes, (uint8_t*)scales, alpha, ngroups, mul,                        \
                                 (uint32_t)o.had_sign_mask, k0, k1, ctr)
    if (rht && sr) ABS_LAUNCH_Q(true, true);
    else if (rht) ABS_LAUNCH_Q(true, false);
    else if (sr) ABS_LAUNCH_Q(false, true);
    else ABS_LAUNCH_Q(false, false);
#undef ABS_LAUNCH_Q
    if (g_ev_quant_end) cudaEventRecord(g_ev_quant_end, s);
    return (eq == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ABS_OK : ABS_ERR_CUDA;
}

template <int FMT>
abs_status_t launch_dequantize_fmt(int sm_count, const void* codes, const void* scales, const float* alpha,
                                   int64_t ngroups, void* out, bool fp32, bool index64, cudaStream_t s,
                                   int64_t swz_cols = 0, int sel = 0) {
    const int grid = grid_for(sm_count, ngroups, 64);
    if constexpr (FMT == ABS_FMT_NVFP4 || FMT == ABS_FMT_IF4) {
        if (!fp32) {
            constexpr bool kInt = FMT == ABS_FMT_IF4;
            const int grid = grid_waves(sm_count, ngroups, 8, kDeqIters);    // 31 registers: 8 resident blocks per SM
            const bool a32 = (reinterpret_cast<uintptr_t>(out) & 31u) == 0;
            const bool i32 = !index64 && ngroups < (int64_t)0x7FFFFFFF - (int64_t)grid * kThreads;
            cudaError_t e;
            const bool swz = swz_cols > 0;
            const uint32_t gpr = (uint32_t)(swz_cols / 16), ktiles = (gpr + 3u) / 4u;
#define ABS_LAUNCH_D3(IDX, A32, SW, SE)                                                                              \
    e = launch_pdl(dequantize4_fast_kernel<kInt, IDX, A32, SW, SE>, grid, kThreads, s, (const uint2*)codes,         \
                   (const uint8_t*)scales, alpha, (IDX)ngroups, (uint4*)out, gpr, ktiles)
#define ABS_LAUNCH_D(IDX, A32)                                                                                      \
    do {                                                                                                            \
        if (sel == 1) ABS_LAUNCH_D3(IDX, A32, false, 1);                                                            \
        else if (sel == 2) ABS_LAUNCH_D3(IDX, A32, false, 2);                                                       \
        else if (swz) ABS_LAUNCH_D3(IDX, A32, true, 0);                                                             \
        else ABS_LAUNCH_D3(IDX, A32, false, 0);                                                                     \
    } while (0)
            if (i32 && a32) ABS_LAUNCH_D(int32_t, true);
            else if (i32) ABS_LAUNCH_D(int32_t, false);
            else if (a32) ABS_LAUNCH_D(int64_t, true);
            else ABS_LAUNCH_D(int64_t, false);
#undef ABS_LAUNCH_D
#undef ABS_LAUNCH_D3
            if (e != cudaSuccess) return ABS_ERR_CUDA;
            return cudaGetLastError() == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
        }
    }
    if constexpr (FMT == ABS_FMT_NVFP4_BS8 || FMT == ABS_FMT_IF4_BS8) {
        const int bgrid = grid_waves(sm_count, ngroups, 8, kDeqIters);
        if (!fp32 && !index64 && ngroups < (int64_t)0x7FFFFFFF - (int64_t)bgrid * kThreads) {
            constexpr bool kInt = FMT == ABS_FMT_IF4_BS8;
            const bool a32 = (reinterpret_cast<uintptr_t>(out) & 31u) == 0;
            const cudaError_t e8 =
                a32 ? launch_pdl(dequantize4_bs8_kernel<kInt, true>, bgrid, kThreads, s, (const uint2*)codes,
                                 (const uint16_t*)scales, alpha, (int32_t)ngroups, (uint4*)out)
                    : launch_pdl(dequantize4_bs8_kernel<kInt, false>, bgrid, kThreads, s, (const uint2*)codes,
                                 (const uint16_t*)scales, alpha, (int32_t)ngroups, (uint4*)out);
            return (e8 == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ABS_OK : ABS_ERR_CUDA;
        }
    }
    if constexpr (FMT == ABS_FMT_IF6_E2M3 || FMT == ABS_FMT_IF6_E3M2) {
        const int sgrid = grid_waves(sm_count, ngroups, 8, kDeqIters);
        if (!fp32 && !index64 && ngroups < (int64_t)0x7FFFFFFF - (int64_t)sgrid * kThreads) {
            constexpr ElemKind kEK = Fmt<FMT>::EK;
            const float c_post = Fmt<FMT>::M_FP / Fmt<FMT>::M_INT;         // IEEE single division, as in the generic kernel
            const bool a32 = (reinterpret_cast<uintptr_t>(out) & 31u) == 0;
            const cudaError_t e6 =
                a32 ? launch_pdl(dequantize6_fast_kernel<kEK, true>, sgrid, kThreads, s, (const uint32_t*)codes,
                                 (const uint8_t*)scales, alpha, (int32_t)ngroups, (uint4*)out, c_post)
                    : launch_pdl(dequantize6_fast_kernel<kEK, false>, sgrid, kThreads, s, (const uint32_t*)codes,
                                 (const uint8_t*)scales, alpha, (int32_t)ngroups, (uint4*)out, c_post);
            return (e6 == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ABS_OK : ABS_ERR_CUDA;
        }
    }
    if constexpr (FMT == ABS_FMT_IF3 || FMT == ABS_FMT_IF3_BS8) {
        // 3-bit codes widened to nibbles and decoded like the 4-bit formats
        const int tgrid = grid_waves(sm_count, ngroups, 8, kDeqIters);
        if (!fp32 && !index64 && ngroups < (int64_t)0x7FFFFFFF - (int64_t)tgrid * kThreads) {
            constexpr int kG = FMT == ABS_FMT_IF3 ? 16 : 8;
            const bool a32 = (reinterpret_cast<uintptr_t>(out) & 31u) == 0;
            const cudaError_t e3 =
                a32 ? launch_pdl(dequantize3_fast_kernel<kG, true>, tgrid, kThreads, s, (const uint16_t*)codes,
                                 (const uint8_t*)scales, alpha, (int32_t)ngroups, (uint4*)out)
                    : launch_pdl(dequantize3_fast_kernel<kG, false>, tgrid, kThreads, s, (const uint16_t*)codes,
                                 (const uint8_t*)scales, alpha, (int32_t)ngroups, (uint4*)out);
            return (e3 == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ABS_OK : ABS_ERR_CUDA;
        }
    }
    cudaError_t e;
    if (fp32)
        e = launch_pdl(dequantize_kernel<FMT, true>, grid, kThreads, s, (const uint8_t*)codes, (const uint8_t*)scales, alpha,
                       ngroups, out);
    else
        e = launch_pdl(dequantize_kernel<FMT, false>, grid, kThreads, s, (const uint8_t*)codes, (const uint8_t*)scales, alpha,
                       ngroups, out);
    return (e == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ABS_OK : ABS_ERR_CUDA;
}


// ------------------------------------------------------------------------------------------ no-allocation variant

// Scratch of abs_quantize_noalloc: one partial maximum per block of the chunked amax pass plus, in
// the last 64 words, the ticket counter.  It lives in the library image, so every GPU that loads the
// library holds these 33 KiB until the process exits; nothing is ever allocated for it.
#define ABS_NOALLOC_MAX_CHUNKS 8192          /* partial maxima the array can hold                 */
#define ABS_NOALLOC_CHUNK_GROUPS 8192        /* groups of 16 elements reduced by one block        */
static __device__ __align__(256) uint32_t g_noalloc_scratch[ABS_NOALLOC_MAX_CHUNKS + 64];

// Eq. 1 without atomics on the maximum: block b reduces chunk b and stores its partial maximum in
// scratch[b]; the block that draws the last ticket reduces the partials, writes alpha and sets the
// ticket back to zero.  `scratch` is the device address of g_noalloc_scratch obtained on the host
// with cudaGetSymbolAddress (the array's name is not a device address in host code).
__global__ void __launch_bounds__(kThreads) amax_chunks_kernel(const uint4* __restrict__ in, int64_t ngroups,
                                                               uint32_t* __restrict__ scratch,
                                                               float* __restrict__ result, float denom) {
    const int64_t first = (int64_t)blockIdx.x * ABS_NOALLOC_CHUNK_GROUPS * 2;       // in 128-bit vectors
    int64_t last = first + (int64_t)ABS_NOALLOC_CHUNK_GROUPS * 2;
    if (last > ngroups * 2) last = ngroups * 2;
    uint32_t m0 = 0u, m1 = 0u;
    for (int64_t i = first + threadIdx.x; i < last; i += kThreads) {
        const uint4 v = __ldg(in + i);
        m0 = __vmaxu2(m0, __vmaxu2(v.x & 0x7FFF7FFFu, v.y & 0x7FFF7FFFu));
        m1 = __vmaxu2(m1, __vmaxu2(v.z & 0x7FFF7FFFu, v.w & 0x7FFF7FFFu));
    }
    const uint32_t m = __vmaxu2(m0, m1);
    uint32_t local = __reduce_max_sync(0xFFFFFFFFu, max(m & 0xFFFFu, m >> 16) << 16);
    __shared__ uint32_t warp_max[kThreads / 32];
    __shared__ bool is_last;
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = local;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t bm = 0u;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) bm = max(bm, warp_max[w]);
        scratch[blockIdx.x] = bm;
        __threadfence();
        is_last = atomicAdd(&scratch[ABS_NOALLOC_MAX_CHUNKS], 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    uint32_t all = 0u;
    for (uint32_t b = threadIdx.x; b < gridDim.x; b += kThreads) all = max(all, __ldcg(scratch + b));
    all = __reduce_max_sync(0xFFFFFFFFu, all);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = all;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t bm = 0u;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) bm = max(bm, warp_max[w]);
        const float A = __uint_as_float(bm);
        *result = (A == 0.0f) ? 1.0f : __fdiv_rn(A, denom);                          // Eq. 1
        scratch[ABS_NOALLOC_MAX_CHUNKS] = 0u;
    }
}

struct NoAllocState {
    std::once_flag once;
    cudaError_t err = cudaSuccess;
    uint32_t* scratch = nullptr;     // device address of g_noalloc_scratch on this device
    int sm_count = 148;
};
NoAllocState g_noalloc[kMaxDevices];

abs_status_t check_shape(abs_fmt_t fmt, int64_t rows, int64_t cols) {
    if (fmt_bits((int)fmt) == 0) return ABS_ERR_FMT;
    if (rows < 0 || cols < 0 || (cols % 16) != 0) return ABS_ERR_SHAPE;
    return ABS_OK;
}

}  // namespace

// ------------------------------------------------------------------------------------------ C ABI

static abs_status_t quantize_transposed_impl(abs_fmt_t fmt, const void* in_bf16, int64_t rows, int64_t cols,
                                             void* codes_t_u8, void* scales_t_e4m3, float* tensor_scale_f32,
                                             const abs_opts_t& o, void* stream, void* out_bf16, bool store_codes);

extern "C" {

size_t abs_codes_bytes(abs_fmt_t fmt, int64_t rows, int64_t cols) {
    if (check_shape(fmt, rows, cols) != ABS_OK) return 0;
    return (size_t)rows * (size_t)cols / 16 * (size_t)(2 * fmt_bits((int)fmt));
}

size_t abs_scales_bytes_swizzled(abs_fmt_t fmt, int64_t rows, int64_t cols) {
    if (check_shape(fmt, rows, cols) != ABS_OK || (fmt != ABS_FMT_NVFP4 && fmt != ABS_FMT_IF4)) return 0;
    const size_t k = (size_t)cols / 16;
    return (((size_t)rows + 127) / 128) * ((k + 3) / 4) * 512;
}

size_t abs_scales_bytes(abs_fmt_t fmt, int64_t rows, int64_t cols) {
    if (check_shape(fmt, rows, cols) != ABS_OK) return 0;
    return (size_t)rows * (size_t)cols / (size_t)fmt_group((int)fmt);
}

const char* abs_status_string(abs_status_t status) {
    switch (status) {
        case ABS_OK: return "ok";
        case ABS_ERR_NULL: return "null pointer";
        case ABS_ERR_SHAPE: return "bad shape (negative size or cols not a multiple of 16)";
        case ABS_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case ABS_ERR_FMT: return "unknown format";
        case ABS_ERR_FLAGS: return "unknown or unsupported flag";
        case ABS_ERR_CUDA: return "CUDA error";
        case ABS_ERR_SIZE: return "size beyond the supported maximum, workspace too small, or scratch ring overrun by an earlier call";
        default: return "unknown status";
    }
}

abs_status_t abs_init(int device) {
    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess) return ABS_ERR_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return ABS_ERR_CUDA;
    DeviceState* st = nullptr;
    abs_status_t rc = device_state(&st);
    cudaSetDevice(prev);
    return rc;
}

void abs_profile_events(void* quantize_begin, void* quantize_end) {
    g_ev_quant_begin = (cudaEvent_t)quantize_begin;
    g_ev_quant_end = (cudaEvent_t)quantize_end;
}

float abs_alpha_from_amax(abs_fmt_t fmt, float amax) {
    if (fmt_bits((int)fmt) == 0) return 0.0f;
    volatile float den = fmt_mfp((int)fmt) * 448.0f;
    volatile float a = amax;
    return (a == 0.0f) ? 1.0f : a / den;
}

abs_status_t abs_amax(const void* in_bf16, int64_t rows, int64_t cols, const abs_opts_t* opts, float* amax_f32,
                      void* stream) {
    const CallRange range("abs_amax");
    abs_opts_t o = {0, 0, 0, 0, 0};
    if (opts) o = *opts;
    if (rows < 0 || cols < 0 || (cols % 16) != 0) return ABS_ERR_SHAPE;
    if ((o.flags & ~(uint32_t)ABS_F_HADAMARD16) || o._pad) return ABS_ERR_FLAGS;
    if (!amax_f32) return ABS_ERR_NULL;
    cudaStream_t s = (cudaStream_t)stream;
    if (rows * cols == 0) return cudaMemsetAsync(amax_f32, 0, sizeof(float), s) == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
    if (!in_bf16) return ABS_ERR_NULL;
    if (!aligned16(in_bf16)) return ABS_ERR_ALIGN;
    DeviceState* st = nullptr;
    if (device_state(&st) != ABS_OK) return ABS_ERR_CUDA;
    unsigned long long* slot = nullptr;
    uint32_t gen = 0;
    const abs_status_t rc = next_slot(*st, &slot, &gen);
    if (rc != ABS_OK) return rc;
    return launch_amax(st->sm_count, in_bf16, rows * cols / 16, o, true, slot, gen, amax_f32, 0.0f, s);
}

abs_status_t abs_quantize_ex(abs_fmt_t fmt, const void* in_bf16, int64_t rows, int64_t cols, void* codes_u8,
                             void* scales_e4m3, float* tensor_scale_f32, const abs_opts_t* opts, void* stream) {
    const CallRange range("abs_quantize_ex");
    abs_opts_t o = {0, 0, 0, 0, 0};
    if (opts) o = *opts;
    abs_status_t rc = check_shape(fmt, rows, cols);
    if (rc != ABS_OK) return rc;
    if ((o.flags & ~kQuantFlags) || o._pad) return ABS_ERR_FLAGS;
    if ((o.flags & ABS_F_STOCHASTIC) && (o.sr_index_offset % 16) != 0) return ABS_ERR_SHAPE;
    if ((o.flags & ABS_F_SCALES_SWIZZLED) &&
        ((fmt != ABS_FMT_NVFP4 && fmt != ABS_FMT_IF4) || (o.flags & (ABS_F_HADAMARD16 | ABS_F_STOCHASTIC)) ||
         cols / 16 > 0x7FFFFFFF || rows > 0x7FFFFFFF))
        return ABS_ERR_FLAGS;      // the tiled scale layout exists for the 4-bit round-to-nearest kernels only
    if (rows * cols == 0) return ABS_OK;
    if (!in_bf16 || !codes_u8 || !scales_e4m3 || !tensor_scale_f32) return ABS_ERR_NULL;
    if (!aligned16(in_bf16) || !aligned16(codes_u8) || !aligned16(scales_e4m3) || ((uintptr_t)tensor_scale_f32 & 3u))
        return ABS_ERR_ALIGN;
    DeviceState* st = nullptr;
    if (device_state(&st) != ABS_OK) return ABS_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const int64_t ngroups = rows * cols / 16;
    AlphaSrc src = {tensor_scale_f32, nullptr, 0u, 0.0f, tensor_scale_f32, nullptr};
    if (!(o.flags & ABS_F_ALPHA_GIVEN)) {
        unsigned long long* slot = nullptr;
        uint32_t gen = 0;
        if ((rc = next_slot(*st, &slot, &gen)) != ABS_OK) return rc;
        const float denom = fmt_mfp((int)fmt) * 448.0f;
        rc = launch_amax(st->sm_count, in_bf16, ngroups, o, false, slot, gen, tensor_scale_f32, denom, s);
        if (rc != ABS_OK) return rc;
        src.slot = slot;
        src.gen = gen;
        src.denom = denom;
        src.overrun = st->overrun_dev;
    }
    switch (fmt) {
        case ABS_FMT_NVFP4: return launch_quantize_fmt<0>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        case ABS_FMT_IF4: return launch_quantize_fmt<1>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        case ABS_FMT_IF3: return launch_quantize_fmt<2>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        case ABS_FMT_IF6_E2M3: return launch_quantize_fmt<3>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        case ABS_FMT_IF6_E3M2: return launch_quantize_fmt<4>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        case ABS_FMT_NVFP4_BS8: return launch_quantize_fmt<5>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        case ABS_FMT_IF4_BS8: return launch_quantize_fmt<6>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        default: return launch_quantize_fmt<7>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
    }
}

abs_status_t abs_quantize_dequantize(abs_fmt_t fmt, const void* in_bf16, int64_t rows, int64_t cols, void* out_bf16,
                                     void* codes_u8, void* scales_e4m3, float* tensor_scale_f32, const abs_opts_t* opts,
                                     void* stream) {
    const CallRange range("abs_quantize_dequantize");
    abs_opts_t o = {0, 0, 0, 0, 0};
    if (opts) o = *opts;
    abs_status_t rc = check_shape(fmt, rows, cols);
    if (rc != ABS_OK) return rc;
    const bool four_bit = fmt == ABS_FMT_NVFP4 || fmt == ABS_FMT_IF4;
    if ((o.flags & ~(uint32_t)(ABS_F_HADAMARD16 | ABS_F_STOCHASTIC | ABS_F_SR_SCALE_17_16 | ABS_F_ALPHA_GIVEN |
                               ABS_F_GROUPS_DOWN_COLUMNS)) || o._pad)
        return ABS_ERR_FLAGS;
    if ((o.flags & ABS_F_STOCHASTIC) && (o.sr_index_offset % 16) != 0) return ABS_ERR_SHAPE;
    // IF3, IF6 and the block-size-8 formats: round-to-nearest along the rows only
    if (!four_bit && (o.flags & (ABS_F_HADAMARD16 | ABS_F_STOCHASTIC | ABS_F_GROUPS_DOWN_COLUMNS))) return ABS_ERR_FLAGS;
    if ((o.flags & ABS_F_GROUPS_DOWN_COLUMNS) && (rows % 16) != 0) return ABS_ERR_SHAPE;
    if (rows * cols == 0) return ABS_OK;
    if (!in_bf16 || !out_bf16 || !tensor_scale_f32 || ((codes_u8 == nullptr) != (scales_e4m3 == nullptr))) return ABS_ERR_NULL;
    if (!aligned16(in_bf16) || !aligned16(out_bf16) || !aligned16(codes_u8) || !aligned16(scales_e4m3) ||
        ((uintptr_t)tensor_scale_f32 & 3u))
        return ABS_ERR_ALIGN;
    if (o.flags & ABS_F_GROUPS_DOWN_COLUMNS) {
        abs_opts_t ot = o;
        ot.flags &= ~(uint32_t)ABS_F_GROUPS_DOWN_COLUMNS;
        return quantize_transposed_impl(fmt, in_bf16, rows, cols, codes_u8, scales_e4m3, tensor_scale_f32, ot, stream,
                                        out_bf16, codes_u8 != nullptr);
    }
    DeviceState* st = nullptr;
    if (device_state(&st) != ABS_OK) return ABS_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const int64_t ngroups = rows * cols / 16;
    const bool rht = o.flags & ABS_F_HADAMARD16, sr = o.flags & ABS_F_STOCHASTIC;
    const int grid = grid_waves(st->sm_count, ngroups, opt_blocks_per_sm(sr, rht), (rht || sr) ? kOptIters : kFastIters);
    if (ngroups >= (int64_t)0x7FFFFFFF - (int64_t)grid * kThreads) return ABS_ERR_SIZE;    // 32-bit group indices only
    AlphaSrc src = {tensor_scale_f32, nullptr, 0u, 0.0f, tensor_scale_f32, nullptr};
    if (!(o.flags & ABS_F_ALPHA_GIVEN)) {
        unsigned long long* slot = nullptr;
        uint32_t gen = 0;
        if ((rc = next_slot(*st, &slot, &gen)) != ABS_OK) return rc;
        const float denom = fmt_mfp((int)fmt) * 448.0f;
        rc = launch_amax(st->sm_count, in_bf16, ngroups, o, false, slot, gen, tensor_scale_f32, denom, s);
        if (rc != ABS_OK) return rc;
        src.slot = slot;
        src.gen = gen;
        src.denom = denom;
        src.overrun = st->overrun_dev;
    }
    const bool store = codes_u8 != nullptr;
    if (!four_bit) {
        bool handled = false;
        switch (fmt) {
            case ABS_FMT_IF3: rc = launch_quantize_fmt<2>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols, out_bf16, store, &handled); break;
            case ABS_FMT_IF6_E2M3: rc = launch_quantize_fmt<3>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols, out_bf16, store, &handled); break;
            case ABS_FMT_IF6_E3M2: rc = launch_quantize_fmt<4>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols, out_bf16, store, &handled); break;
            case ABS_FMT_NVFP4_BS8: rc = launch_quantize_fmt<5>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols, out_bf16, store, &handled); break;
            case ABS_FMT_IF4_BS8: rc = launch_quantize_fmt<6>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols, out_bf16, store, &handled); break;
            default: rc = launch_quantize_fmt<7>(st->sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols, out_bf16, store, &handled); break;
        }
        return (!handled && rc == ABS_ERR_FLAGS) ? ABS_ERR_SIZE : rc;
    }
    const float mul = (o.flags & ABS_F_SR_SCALE_17_16) ? 1.0625f : 1.0f;
    const uint64_t ctr = o.sr_index_offset / 8;
    const PhiloxKeys pk = philox_keys(o.sr_seed);
    const bool a32 = (reinterpret_cast<uintptr_t>(in_bf16) & 31u) == 0, o32 = (reinterpret_cast<uintptr_t>(out_bf16) & 31u) == 0;
    cudaError_t e = cudaSuccess;
#define ABS_LAUNCH_E3(I, R, S, SLOT)                                                                                \
    e = launch_pdl(quantize4_opt_kernel<I, R, S, SLOT, true>, grid, kThreads, s, (const uint4*)in_bf16, (uint2*)codes_u8, \
                   (uint8_t*)scales_e4m3, src, (int32_t)ngroups, mul, (uint32_t)o.had_sign_mask, pk, ctr, a32,       \
                   (uint4*)out_bf16, o32, store)
#define ABS_LAUNCH_E2(I, R, S)                                                                                      \
    do {                                                                                                            \
        if (src.slot) ABS_LAUNCH_E3(I, R, S, true);                                                                 \
        else ABS_LAUNCH_E3(I, R, S, false);                                                                         \
    } while (0)
#define ABS_LAUNCH_E(I)                                                                                             \
    do {                                                                                                            \
        if (rht && sr) ABS_LAUNCH_E2(I, true, true);                                                                \
        else if (rht) ABS_LAUNCH_E2(I, true, false);                                                                \
        else if (sr) ABS_LAUNCH_E2(I, false, true);                                                                 \
        else ABS_LAUNCH_E2(I, false, false);                                                                        \
    } while (0)
    if (fmt == ABS_FMT_IF4) ABS_LAUNCH_E(true);
    else ABS_LAUNCH_E(false);
#undef ABS_LAUNCH_E
#undef ABS_LAUNCH_E2
#undef ABS_LAUNCH_E3
    return (e == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ABS_OK : ABS_ERR_CUDA;
}

abs_status_t abs_quantize(abs_fmt_t fmt, const void* in_bf16, int64_t rows, int64_t cols, void* codes_u8,
                          void* scales_e4m3, float* tensor_scale_f32, void* stream) {
    return abs_quantize_ex(fmt, in_bf16, rows, cols, codes_u8, scales_e4m3, tensor_scale_f32, nullptr, stream);
}


abs_status_t abs_quantize_transposed(abs_fmt_t fmt, const void* in_bf16, int64_t rows, int64_t cols,
                                     void* codes_t_u8, void* scales_t_e4m3, float* tensor_scale_f32,
                                     const abs_opts_t* opts, void* stream) {
    const CallRange range("abs_quantize_transposed");
    abs_opts_t o = {0, 0, 0, 0, 0};
    if (opts) o = *opts;
    if (fmt != ABS_FMT_NVFP4 && fmt != ABS_FMT_IF4) return ABS_ERR_FMT;
    if (rows < 0 || cols < 0 || (cols % 16) != 0 || (rows % 16) != 0) return ABS_ERR_SHAPE;
    if ((o.flags & ~(uint32_t)(ABS_F_ALPHA_GIVEN | ABS_F_HADAMARD16 | ABS_F_STOCHASTIC | ABS_F_SR_SCALE_17_16)) || o._pad)
        return ABS_ERR_FLAGS;
    if ((o.flags & ABS_F_STOCHASTIC) && (o.sr_index_offset % 16) != 0) return ABS_ERR_SHAPE;
    if (rows * cols == 0) return ABS_OK;
    if (!in_bf16 || !codes_t_u8 || !scales_t_e4m3 || !tensor_scale_f32) return ABS_ERR_NULL;
    if (!aligned16(in_bf16) || !aligned16(codes_t_u8) || !aligned16(scales_t_e4m3) || ((uintptr_t)tensor_scale_f32 & 3u))
        return ABS_ERR_ALIGN;
    return quantize_transposed_impl(fmt, in_bf16, rows, cols, codes_t_u8, scales_t_e4m3, tensor_scale_f32, o, stream,
                                    nullptr, true);
}

}  // extern "C"

// The transposed tile walk: plain transposed quantize (out == nullptr) or the emulation pass along the columns
// (out = [rows, cols] bf16 in the original orientation; codes stored only when store_codes).  Arguments are
// already validated.
static abs_status_t quantize_transposed_impl(abs_fmt_t fmt, const void* in_bf16, int64_t rows, int64_t cols,
                                             void* codes_t_u8, void* scales_t_e4m3, float* tensor_scale_f32,
                                             const abs_opts_t& o, void* stream, void* out_bf16, bool store_codes) {
    DeviceState* st = nullptr;
    if (device_state(&st) != ABS_OK) return ABS_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const int64_t ngroups = rows * cols / 16;
    const bool rht = o.flags & ABS_F_HADAMARD16;
    const int64_t rblocks = rows / 16;
    const int64_t ntiles = ((cols + kTransTileCols - 1) / kTransTileCols) *
                           ((rblocks + kTransTileRowBlocks - 1) / kTransTileRowBlocks);
    if (ntiles > (int64_t)0x7FFFFFFF) return ABS_ERR_SIZE;      // the kernel indexes tiles with 32 bits
    // 64 KiB of shared memory per block: 3 blocks per SM.  The arithmetic-bound variants (IF4, options) and the
    // emulation pass run best as several waves with about four tiles per block; plain NVFP4 as one wave of
    // persistent blocks.
    const int64_t resident = (int64_t)st->sm_count * 3;
    const bool heavy = fmt == ABS_FMT_IF4 || (o.flags & (ABS_F_HADAMARD16 | ABS_F_STOCHASTIC)) || out_bf16 != nullptr;
    int64_t tgrid = ntiles < resident ? ntiles : resident;
    if (heavy && ntiles > resident) {
        int64_t waves = (ntiles + 2 * resident) / (4 * resident);
        if (waves < 1) waves = 1;
        tgrid = waves * resident < ntiles ? waves * resident : ntiles;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)tgrid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kTransSmemBytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaSuccess;
    const uint16_t* in = (const uint16_t*)in_bf16;
    uint2* ct = (uint2*)codes_t_u8;
    uint8_t* stp = (uint8_t*)scales_t_e4m3;
    const uint32_t mask = o.had_sign_mask;
#define ABS_LAUNCH_TE(I, S, R, Q, M, E, SLOT, GEN)                                                                  \
    do {                                                                                                            \
        e = cudaFuncSetAttribute(transposed_kernel<I, S, R, Q, M, E>(), cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                 kTransSmemBytes);                                                                  \
        if (e == cudaSuccess)                                                                                       \
            e = cudaLaunchKernelEx(&cfg, transposed_kernel<I, S, R, Q, M, E>(), in, ct, stp, src, rows, cols, mask, \
                                   SLOT, GEN, mul, pk, ctr, (uint16_t*)out_bf16, store_codes);                      \
    } while (0)
#define ABS_LAUNCH_T(I, S, R, Q, M, SLOT, GEN)                                                                      \
    do {                                                                                                            \
        if (M == 0 && out_bf16) ABS_LAUNCH_TE(I, S, R, Q, 0, true, SLOT, GEN);                                      \
        else ABS_LAUNCH_TE(I, S, R, Q, M, false, SLOT, GEN);                                                        \
    } while (0)

    const bool sr = o.flags & ABS_F_STOCHASTIC;
    const float mul = (o.flags & ABS_F_SR_SCALE_17_16) ? 1.0625f : 1.0f;
    const uint64_t ctr = o.sr_index_offset / 8;
    const PhiloxKeys pk = philox_keys(o.sr_seed);
    AlphaSrc src = {tensor_scale_f32, nullptr, 0u, 0.0f, tensor_scale_f32, nullptr};
    if (!(o.flags & ABS_F_ALPHA_GIVEN)) {
        unsigned long long* slot = nullptr;
        uint32_t gen = 0;
        const abs_status_t rs = next_slot(*st, &slot, &gen);
        if (rs != ABS_OK) return rs;
        const float denom = 6.0f * 448.0f;
        if (rht) {
            // the maximum is taken over the transformed column groups: same tile walk, MODE 1
            ABS_LAUNCH_T(false, false, true, false, 1, slot, gen);
            if (e != cudaSuccess) return ABS_ERR_CUDA;
        } else {
            abs_status_t rc = launch_amax(st->sm_count, in_bf16, ngroups, o, false, slot, gen, tensor_scale_f32, denom, s);
            if (rc != ABS_OK) return rc;
        }
        src.slot = slot;
        src.gen = gen;
        src.denom = denom;
        src.overrun = st->overrun_dev;
    }
    unsigned long long* no_slot = nullptr;
#define ABS_LAUNCH_T2(I, R, Q)                                                                                      \
    do {                                                                                                            \
        if (src.slot) ABS_LAUNCH_T(I, true, R, Q, 0, no_slot, 0u);                                                  \
        else ABS_LAUNCH_T(I, false, R, Q, 0, no_slot, 0u);                                                          \
    } while (0)
#define ABS_LAUNCH_T3(I)                                                                                            \
    do {                                                                                                            \
        if (rht && sr) ABS_LAUNCH_T2(I, true, true);                                                                \
        else if (rht) ABS_LAUNCH_T2(I, true, false);                                                                \
        else if (sr) ABS_LAUNCH_T2(I, false, true);                                                                 \
        else ABS_LAUNCH_T2(I, false, false);                                                                        \
    } while (0)
    if (fmt == ABS_FMT_IF4) ABS_LAUNCH_T3(true);
    else ABS_LAUNCH_T3(false);
#undef ABS_LAUNCH_T3
#undef ABS_LAUNCH_T2
#undef ABS_LAUNCH_T
#undef ABS_LAUNCH_TE
    return (e == cudaSuccess && cudaGetLastError() == cudaSuccess) ? ABS_OK : ABS_ERR_CUDA;
}

extern "C" {

abs_status_t abs_quantize_noalloc(abs_fmt_t fmt, const void* in_bf16, int64_t rows, int64_t cols, void* codes_u8,
                                  void* scales_e4m3, float* tensor_scale_f32, void* stream) {
    const CallRange range("abs_quantize_noalloc");
    abs_status_t rc = check_shape(fmt, rows, cols);
    if (rc != ABS_OK) return rc;
    if (rows * cols == 0) return ABS_OK;
    if (!in_bf16 || !codes_u8 || !scales_e4m3 || !tensor_scale_f32) return ABS_ERR_NULL;
    if (!aligned16(in_bf16) || !aligned16(codes_u8) || !aligned16(scales_e4m3) || ((uintptr_t)tensor_scale_f32 & 3u))
        return ABS_ERR_ALIGN;
    const int64_t ngroups = rows * cols / 16;
    const int64_t nchunks = (ngroups + ABS_NOALLOC_CHUNK_GROUPS - 1) / ABS_NOALLOC_CHUNK_GROUPS;
    if (nchunks > ABS_NOALLOC_MAX_CHUNKS) return ABS_ERR_SIZE;      // more partial maxima than the static array holds
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ABS_ERR_CUDA;
    NoAllocState& na = g_noalloc[dev];
    std::call_once(na.once, [&]() {
        // The current device is `dev`: the address returned is the array's copy on this device.
        na.err = cudaGetSymbolAddress((void**)&na.scratch, g_noalloc_scratch);
        int sms = 0;
        if (na.err == cudaSuccess) na.err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms > 0) na.sm_count = sms;
    });
    if (na.err != cudaSuccess || na.scratch == nullptr) return ABS_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    // The array keeps whatever the last call left: the ticket must start at zero; the partial maxima
    // need no clearing because every block overwrites its own slot before it draws a ticket.
    if (cudaMemsetAsync(na.scratch + ABS_NOALLOC_MAX_CHUNKS, 0, sizeof(uint32_t), s) != cudaSuccess) return ABS_ERR_CUDA;
    amax_chunks_kernel<<<(int)nchunks, kThreads, 0, s>>>((const uint4*)in_bf16, ngroups, na.scratch, tensor_scale_f32,
                                                        fmt_mfp((int)fmt) * 448.0f);
    if (cudaGetLastError() != cudaSuccess) return ABS_ERR_CUDA;
    const abs_opts_t o = {0, 0, 0, 0, 0};
    const AlphaSrc src = {tensor_scale_f32, nullptr, 0u, 0.0f, tensor_scale_f32, nullptr};   // alpha was written by the chunked pass
    switch (fmt) {
        case ABS_FMT_NVFP4: return launch_quantize_fmt<0>(na.sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        case ABS_FMT_IF4: return launch_quantize_fmt<1>(na.sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        case ABS_FMT_IF3: return launch_quantize_fmt<2>(na.sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        case ABS_FMT_IF6_E2M3: return launch_quantize_fmt<3>(na.sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        case ABS_FMT_IF6_E3M2: return launch_quantize_fmt<4>(na.sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        case ABS_FMT_NVFP4_BS8: return launch_quantize_fmt<5>(na.sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        case ABS_FMT_IF4_BS8: return launch_quantize_fmt<6>(na.sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
        default: return launch_quantize_fmt<7>(na.sm_count, in_bf16, ngroups, codes_u8, scales_e4m3, src, o, s, cols);
    }
}

abs_status_t abs_dequantize_ex(abs_fmt_t fmt, const void* codes_u8, const void* scales_e4m3,
                               const float* tensor_scale_f32, int64_t rows, int64_t cols, void* out,
                               const abs_opts_t* opts, void* stream) {
    const CallRange range("abs_dequantize_ex");
    abs_opts_t o = {0, 0, 0, 0, 0};
    if (opts) o = *opts;
    abs_status_t rc = check_shape(fmt, rows, cols);
    if (rc != ABS_OK) return rc;
    if ((o.flags & ~(uint32_t)(ABS_F_OUT_FP32 | ABS_F_INDEX64 | ABS_F_SCALES_SWIZZLED | ABS_F_FP_GROUPS_ONLY | ABS_F_INT_GROUPS_RAW)) || o._pad)
        return ABS_ERR_FLAGS;
    const uint32_t split = o.flags & (ABS_F_FP_GROUPS_ONLY | ABS_F_INT_GROUPS_RAW);
    if (split && (fmt != ABS_FMT_IF4 || split == (ABS_F_FP_GROUPS_ONLY | ABS_F_INT_GROUPS_RAW) ||
                  (o.flags & (ABS_F_OUT_FP32 | ABS_F_SCALES_SWIZZLED))))
        return ABS_ERR_FLAGS;      // the split exists for IF4 with bf16 output and row-major scales
    if ((o.flags & ABS_F_SCALES_SWIZZLED) &&
        ((fmt != ABS_FMT_NVFP4 && fmt != ABS_FMT_IF4) || (o.flags & ABS_F_OUT_FP32) || cols / 16 > 0x7FFFFFFF || rows > 0x7FFFFFFF))
        return ABS_ERR_FLAGS;
    if (rows * cols == 0) return ABS_OK;
    if (!codes_u8 || !scales_e4m3 || !tensor_scale_f32 || !out) return ABS_ERR_NULL;
    if (!aligned16(codes_u8) || !aligned16(scales_e4m3) || !aligned16(out) || ((uintptr_t)tensor_scale_f32 & 3u))
        return ABS_ERR_ALIGN;
    DeviceState* st = nullptr;
    if (device_state(&st) != ABS_OK) return ABS_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const int64_t ngroups = rows * cols / 16;
    const bool fp32 = o.flags & ABS_F_OUT_FP32, i64 = o.flags & ABS_F_INDEX64;
    const int64_t swz_cols = (o.flags & ABS_F_SCALES_SWIZZLED) ? cols : 0;
    const int sel = (o.flags & ABS_F_FP_GROUPS_ONLY) ? 1 : ((o.flags & ABS_F_INT_GROUPS_RAW) ? 2 : 0);
    switch (fmt) {
        case ABS_FMT_NVFP4: return launch_dequantize_fmt<0>(st->sm_count, codes_u8, scales_e4m3, tensor_scale_f32, ngroups, out, fp32, i64, s, swz_cols);
        case ABS_FMT_IF4: return launch_dequantize_fmt<1>(st->sm_count, codes_u8, scales_e4m3, tensor_scale_f32, ngroups, out, fp32, i64, s, swz_cols, sel);
        case ABS_FMT_IF3: return launch_dequantize_fmt<2>(st->sm_count, codes_u8, scales_e4m3, tensor_scale_f32, ngroups, out, fp32, i64, s);
        case ABS_FMT_IF6_E2M3: return launch_dequantize_fmt<3>(st->sm_count, codes_u8, scales_e4m3, tensor_scale_f32, ngroups, out, fp32, i64, s);
        case ABS_FMT_IF6_E3M2: return launch_dequantize_fmt<4>(st->sm_count, codes_u8, scales_e4m3, tensor_scale_f32, ngroups, out, fp32, i64, s);
        case ABS_FMT_NVFP4_BS8: return launch_dequantize_fmt<5>(st->sm_count, codes_u8, scales_e4m3, tensor_scale_f32, ngroups, out, fp32, i64, s);
        case ABS_FMT_IF4_BS8: return launch_dequantize_fmt<6>(st->sm_count, codes_u8, scales_e4m3, tensor_scale_f32, ngroups, out, fp32, i64, s);
        default: return launch_dequantize_fmt<7>(st->sm_count, codes_u8, scales_e4m3, tensor_scale_f32, ngroups, out, fp32, i64, s);
    }
}

abs_status_t abs_dequantize(abs_fmt_t fmt, const void* codes_u8, const void* scales_e4m3,
                            const float* tensor_scale_f32, int64_t rows, int64_t cols, void* out_bf16, void* stream) {
    return abs_dequantize_ex(fmt, codes_u8, scales_e4m3, tensor_scale_f32, rows, cols, out_bf16, nullptr, stream);
}

// Workspace layout of the host-buffer variants: [input bf16 | codes | scales | alpha], each
// section rounded up to 256 bytes; the dequantize variant reuses the first section for its output.
static size_t round256(size_t n) { return (n + 255) & ~(size_t)255; }

size_t abs_host_workspace_bytes(abs_fmt_t fmt, int64_t rows, int64_t cols) {
    if (check_shape(fmt, rows, cols) != ABS_OK) return 0;
    const size_t n = (size_t)rows * (size_t)cols;
    return round256(n * 4) + round256(abs_codes_bytes(fmt, rows, cols)) + round256(abs_scales_bytes(fmt, rows, cols)) + 256;
}

abs_status_t abs_quantize_host(abs_fmt_t fmt, const void* in_bf16_host, int64_t rows, int64_t cols,
                               void* codes_u8_host, void* scales_e4m3_host, float* tensor_scale_f32_host,
                               const abs_opts_t* opts, void* d_workspace, size_t workspace_bytes, void* stream) {
    const CallRange range("abs_quantize_host");
    abs_status_t rc = check_shape(fmt, rows, cols);
    if (rc != ABS_OK) return rc;
    if (rows * cols == 0) return ABS_OK;
    if (!in_bf16_host || !codes_u8_host || !scales_e4m3_host || !tensor_scale_f32_host || !d_workspace) return ABS_ERR_NULL;
    if (!aligned16(d_workspace)) return ABS_ERR_ALIGN;
    if (workspace_bytes < abs_host_workspace_bytes(fmt, rows, cols)) return ABS_ERR_SIZE;
    const size_t n = (size_t)rows * (size_t)cols;
    const size_t cb = abs_codes_bytes(fmt, rows, cols), sb = abs_scales_bytes(fmt, rows, cols);
    uint8_t* base = (uint8_t*)d_workspace;
    uint8_t* d_in = base;
    uint8_t* d_codes = d_in + round256(n * 4);
    uint8_t* d_scales = d_codes + round256(cb);
    float* d_alpha = (float*)(d_scales + round256(sb));
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemcpyAsync(d_in, in_bf16_host, n * 2, cudaMemcpyHostToDevice, s) != cudaSuccess) return ABS_ERR_CUDA;
    if (opts && (opts->flags & ABS_F_ALPHA_GIVEN))
        if (cudaMemcpyAsync(d_alpha, tensor_scale_f32_host, 4, cudaMemcpyHostToDevice, s) != cudaSuccess) return ABS_ERR_CUDA;
    rc = abs_quantize_ex(fmt, d_in, rows, cols, d_codes, d_scales, d_alpha, opts, stream);
    if (rc != ABS_OK) return rc;
    if (cudaMemcpyAsync(codes_u8_host, d_codes, cb, cudaMemcpyDeviceToHost, s) != cudaSuccess) return ABS_ERR_CUDA;
    if (cudaMemcpyAsync(scales_e4m3_host, d_scales, sb, cudaMemcpyDeviceToHost, s) != cudaSuccess) return ABS_ERR_CUDA;
    if (cudaMemcpyAsync(tensor_scale_f32_host, d_alpha, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return ABS_ERR_CUDA;
    return cudaStreamSynchronize(s) == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
}

abs_status_t abs_dequantize_host(abs_fmt_t fmt, const void* codes_u8_host, const void* scales_e4m3_host,
                                 const float* tensor_scale_f32_host, int64_t rows, int64_t cols, void* out_host,
                                 const abs_opts_t* opts, void* d_workspace, size_t workspace_bytes, void* stream) {
    const CallRange range("abs_dequantize_host");
    abs_status_t rc = check_shape(fmt, rows, cols);
    if (rc != ABS_OK) return rc;
    if (rows * cols == 0) return ABS_OK;
    if (!codes_u8_host || !scales_e4m3_host || !tensor_scale_f32_host || !out_host || !d_workspace) return ABS_ERR_NULL;
    if (!aligned16(d_workspace)) return ABS_ERR_ALIGN;
    if (workspace_bytes < abs_host_workspace_bytes(fmt, rows, cols)) return ABS_ERR_SIZE;
    const size_t n = (size_t)rows * (size_t)cols;
    const size_t cb = abs_codes_bytes(fmt, rows, cols), sb = abs_scales_bytes(fmt, rows, cols);
    const bool fp32 = opts && (opts->flags & ABS_F_OUT_FP32);
    uint8_t* base = (uint8_t*)d_workspace;
    uint8_t* d_out = base;
    uint8_t* d_codes = d_out + round256(n * 4);
    uint8_t* d_scales = d_codes + round256(cb);
    float* d_alpha = (float*)(d_scales + round256(sb));
    cudaStream_t s = (cudaStream_t)stream;
    // Row chunks: the device-to-host copy of one chunk (second stream) overlaps the host-to-device copy and
    // the kernel of the next.  Chunk boundaries are multiples of 16 rows, which keeps every section pointer
    // 16-byte aligned; the tiled scale layout does not split by rows and takes the single-shot path below.
    const int64_t chunk_rows = ((rows + kHostChunks - 1) / kHostChunks + 15) / 16 * 16;
    DeviceState* st = nullptr;
    if (rows >= 16 * kHostChunks && !(opts && (opts->flags & ABS_F_SCALES_SWIZZLED)) && device_state(&st) == ABS_OK) {
        std::lock_guard<std::mutex> lock(st->host_mu);
        if (!st->d2h_stream) {
            // created once per device; the stream pointer is published last, so a failed attempt is retried
            cudaStream_t ns = nullptr;
            bool ok = true;
            for (int i = 0; ok && i < kHostChunks; ++i)
                if (!st->chunk_done[i]) ok = cudaEventCreateWithFlags(&st->chunk_done[i], cudaEventDisableTiming) == cudaSuccess;
            if (ok && !st->d2h_done) ok = cudaEventCreateWithFlags(&st->d2h_done, cudaEventDisableTiming) == cudaSuccess;
            ok = ok && cudaStreamCreateWithFlags(&ns, cudaStreamNonBlocking) == cudaSuccess;
            if (!ok) return ABS_ERR_CUDA;
            st->d2h_stream = ns;
        }
        if (cudaMemcpyAsync(d_alpha, tensor_scale_f32_host, 4, cudaMemcpyHostToDevice, s) != cudaSuccess) return ABS_ERR_CUDA;
        const size_t out_row = (size_t)cols * (fp32 ? 4 : 2);
        int i = 0;
        for (int64_t r0 = 0; r0 < rows; r0 += chunk_rows, ++i) {
            const int64_t nr = rows - r0 < chunk_rows ? rows - r0 : chunk_rows;
            const size_t c0 = abs_codes_bytes(fmt, r0, cols), cn = abs_codes_bytes(fmt, nr, cols);
            const size_t s0 = abs_scales_bytes(fmt, r0, cols), sn = abs_scales_bytes(fmt, nr, cols);
            if (cudaMemcpyAsync(d_codes + c0, (const uint8_t*)codes_u8_host + c0, cn, cudaMemcpyHostToDevice, s) != cudaSuccess ||
                cudaMemcpyAsync(d_scales + s0, (const uint8_t*)scales_e4m3_host + s0, sn, cudaMemcpyHostToDevice, s) != cudaSuccess)
                return ABS_ERR_CUDA;
            rc = abs_dequantize_ex(fmt, d_codes + c0, d_scales + s0, d_alpha, nr, cols, d_out + (size_t)r0 * out_row, opts, stream);
            if (rc != ABS_OK) return rc;
            if (cudaEventRecord(st->chunk_done[i], s) != cudaSuccess ||
                cudaStreamWaitEvent(st->d2h_stream, st->chunk_done[i], 0) != cudaSuccess ||
                cudaMemcpyAsync((uint8_t*)out_host + (size_t)r0 * out_row, d_out + (size_t)r0 * out_row, (size_t)nr * out_row,
                                cudaMemcpyDeviceToHost, st->d2h_stream) != cudaSuccess)
                return ABS_ERR_CUDA;
        }
        if (cudaEventRecord(st->d2h_done, st->d2h_stream) != cudaSuccess || cudaStreamWaitEvent(s, st->d2h_done, 0) != cudaSuccess)
            return ABS_ERR_CUDA;
        return cudaStreamSynchronize(s) == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
    }
    if (cudaMemcpyAsync(d_codes, codes_u8_host, cb, cudaMemcpyHostToDevice, s) != cudaSuccess) return ABS_ERR_CUDA;
    if (cudaMemcpyAsync(d_scales, scales_e4m3_host, sb, cudaMemcpyHostToDevice, s) != cudaSuccess) return ABS_ERR_CUDA;
    if (cudaMemcpyAsync(d_alpha, tensor_scale_f32_host, 4, cudaMemcpyHostToDevice, s) != cudaSuccess) return ABS_ERR_CUDA;
    rc = abs_dequantize_ex(fmt, d_codes, d_scales, d_alpha, rows, cols, d_out, opts, stream);
    if (rc != ABS_OK) return rc;
    if (cudaMemcpyAsync(out_host, d_out, n * (fp32 ? 4 : 2), cudaMemcpyDeviceToHost, s) != cudaSuccess) return ABS_ERR_CUDA;
    return cudaStreamSynchronize(s) == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
}

abs_status_t abs_selftest_convert(int kind, const float* in_f32, int64_t n, void* out, void* stream) {
    if (!((kind >= 0 && kind <= 5) || (kind >= 16 && kind <= 20))) return ABS_ERR_FLAGS;
    if (n < 0) return ABS_ERR_SHAPE;
    if (n == 0) return ABS_OK;
    if (!in_f32 || !out) return ABS_ERR_NULL;
    int64_t blocks = (n + kThreads - 1) / kThreads;
    if (blocks > 148 * 32) blocks = 148 * 32;
    selftest_kernel<<<(int)blocks, kThreads, 0, (cudaStream_t)stream>>>(kind, in_f32, n, out);
    return cudaGetLastError() == cudaSuccess ? ABS_OK : ABS_ERR_CUDA;
}

}  // extern "C"
