// Shared device/host helpers of the CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/cass.h"

#define CASS_CUDA_CHECK(expr)                                  \
    do {                                                       \
        cudaError_t _e = (expr);                               \
        if (_e != cudaSuccess) return CASS_ERR_CUDA;           \
    } while (0)

#define CASS_LAUNCH_CHECK()                                    \
    do {                                                       \
        if (cudaGetLastError() != cudaSuccess) return CASS_ERR_CUDA; \
    } while (0)

// Launch with programmatic stream serialisation: the grid may be scheduled while its predecessor in the stream is
// still running; every kernel launched this way calls pdl_wait() before it touches global memory, which returns
// once the predecessor has completed and its writes are visible.
#define CASS_PDL_LAUNCH(kernel_, grid_, block_, smem_, stream_, ...)                                              \
    do {                                                                                                    \
        cudaLaunchConfig_t _cfg = {};                                                                       \
        _cfg.gridDim = (grid_); _cfg.blockDim = (block_); _cfg.dynamicSmemBytes = (smem_); _cfg.stream = (stream_); \
        cudaLaunchAttribute _at[1];                                                                         \
        _at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                                     \
        _at[0].val.programmaticStreamSerializationAllowed = cass::pdl_enabled();                            \
        _cfg.attrs = _at; _cfg.numAttrs = 1;                                                                \
        if (cudaLaunchKernelEx(&_cfg, kernel_, __VA_ARGS__) != cudaSuccess) return CASS_ERR_CUDA;            \
    } while (0)

#include <cstdlib>

namespace cass {

// CASS_NO_PDL=1 in the environment turns the overlap off (plain stream order), e.g. to read per-kernel times from a trace.
inline int pdl_enabled() {
    static int v = -1;
    if (v < 0) {
        const char* e = std::getenv("CASS_NO_PDL");
        v = (e && e[0] == '1') ? 0 : 1;
    }
    return v;
}

constexpr int kRowsPerBlock = 32;          // rows (or tokens) interleaved in one superblock
constexpr int kGroupCols = 8;              // kept columns per bitmap-walk group
constexpr int kGroupCodes = 4;             // codewords per unary-walk group
constexpr int kMaxVerifyRows = 16;         // rows of one sequence in one verification call; also the margin kept at the end of a cache
constexpr int kMaxBatch = 8;               // sequences per session
constexpr int kMaxRows = 64;               // rows of all sequences in one call

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
__host__ __device__ inline size_t align_up(size_t a, size_t b) { return (a + b - 1) / b * b; }

// ---- sign + mantissa fields of the speculation data ----------------------------------------------------
// A field is the sign bit followed by the 7-t kept mantissa bits (F = 8-t bits); a 32-bit word holds 32/F
// fields and no field straddles words.  When F divides 32 field j is stored float-aligned and rotated: sign at
// bit 31 and mantissa from bit 22 downwards, that pattern rotated right by F*j (the patterns of one word are
// disjoint), so that one rotate-left and one mask put both where a binary32 (or, after >> 16, a bf16) value
// keeps them.  Otherwise fields are packed from the most significant end.
__host__ __device__ inline bool field_rotated(int t) { return 32 % (8 - t) == 0; }

__device__ __forceinline__ uint32_t field_bits_in_word(uint32_t field, int j, int t) {
    const int F = 8 - t;
    if (field_rotated(t)) {
        uint32_t canon = ((field >> (7 - t)) << 31) | ((field & ((1u << (7 - t)) - 1u)) << (16 + t));
        return __funnelshift_r(canon, canon, (F * j) & 31);
    }
    return field << (32 - F * (j + 1));
}

// Sign and mantissa of field j of `word`, already at their bf16 positions (bit 15, bits 6..t).
__device__ __forceinline__ uint32_t field_sign_mant_bf16(uint32_t word, int j, int t) {
    const int F = 8 - t;
    if (field_rotated(t)) {
        uint32_t canon = __funnelshift_l(word, word, (F * j) & 31);
        return (canon >> 16) & (0x8000u | (0x7Fu & ~((1u << t) - 1u)));
    }
    uint32_t f = (word >> (32 - F * (j + 1))) & ((1u << F) - 1u);
    return ((f >> (F - 1)) << 15) | ((f & ((1u << (F - 1)) - 1u)) << t);
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

__device__ __forceinline__ uint16_t float_to_bf16_bits(float f) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}

__device__ __forceinline__ float round_bf16(float f) { return __bfloat162float(__float2bfloat16_rn(f)); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ int warp_max_i(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ int warp_min_i(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ uint32_t lanemask_lt() {
    uint32_t m;
    asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}

// ---- mbarrier + bulk async copy (TMA, one destination CTA) --------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait: gives up after ~2^22 polls and reports failure so that the kernel can flag an error
// and leave instead of spinning forever.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    for (uint32_t i = 0; i < (1u << 22); ++i) {
        if (mbar_try_wait(bar, parity)) return true;
    }
    return false;
}

// Global -> shared bulk copy; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Programmatic dependent launch: let the next kernel start / wait for the previous kernel's memory.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Which kernel classes release their successor (griddepcontrol.launch_dependents) before they finish (bit per class:
// 0 small operators, 1 KV encoder, 2 draft attention, 3 attention merge, 4 verification attention, 5 verification
// GEMM).  A kernel outside the mask releases its successor when it exits; every kernel still starts with
// griddepcontrol.wait, and the draft GEMV does its set-up (barriers, table, first weight copy) before that wait.
// Measured on the full model (ms per speculative step / plain tokens per s): none 25.5 / 249, small operators + GEMM
// 25.7 / 252, all but the KV encoder about the same, with the KV encoder 26.6 / 224, all 27.1 / 226: an early release
// mostly lets the successor's CTAs take SM resources while they wait, so the default releases nothing early.
#ifndef CASS_PDL_EARLY_MASK
#define CASS_PDL_EARLY_MASK 0x00
#endif
template <int CLS>
__device__ __forceinline__ void pdl_early() {
    if constexpr ((CASS_PDL_EARLY_MASK >> CLS) & 1) pdl_launch_dependents();
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

}  // namespace cass
