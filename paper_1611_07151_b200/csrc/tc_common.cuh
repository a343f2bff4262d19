// Device helpers shared by the tensor-core kernels: the bounded mbarrier wait and the fp32 -> bf16 packing.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "ptx_sm100.cuh"
#include "sqn_internal.h"

namespace sqn {

constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // about two seconds

// Bounded mbarrier wait.  Polls back to back at first (hand-offs between the roles take a few
// hundred cycles), backs off with nanosleep on long waits, and gives up after `limit` cycles:
// the CTA then records SQN_ERR_TIMEOUT and every role leaves its loop.
__device__ __forceinline__ bool wait_bar_limit(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, long long limit)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t i = 1;; ++i) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > limit) {
                *abort_flag = 1;
                if (status) atomicExch(status, (int)SQN_ERR_TIMEOUT);
                return false;
            }
        }
        if (i > 4096u) __nanosleep(128);
    }
}
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status)
{
    return wait_bar_limit(bar, parity, abort_flag, status, WAIT_LIMIT_CYCLES);
}

// The 16-bit storage type of the tensor-core paths is bf16, or fp16 where `f16` is set (same size, same layouts).
// two fp32 values -> packed pair, round to nearest even
__device__ __forceinline__ uint32_t pack_x2(float lo, float hi, int f16)
{
    uint32_t d;
    if (f16) asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    else asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
// max(.,0) and the conversion of two values in one instruction
__device__ __forceinline__ uint32_t pack_relu_x2(float lo, float hi, int f16)
{
    uint32_t d;
    if (f16) asm("cvt.rn.relu.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    else asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// maximum of three values in one instruction
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
// fp32 -> 16 bits (round to nearest even), with max(., 0) folded into the conversion when relu is set
__device__ __forceinline__ unsigned short to_16_bits(float v, int relu, int f16)
{
    unsigned short h;
    if (f16) {
        if (relu) asm("cvt.rn.relu.f16.f32 %0, %1;" : "=h"(h) : "f"(v));
        else asm("cvt.rn.f16.f32 %0, %1;" : "=h"(h) : "f"(v));
    } else {
        if (relu) asm("cvt.rn.relu.bf16.f32 %0, %1;" : "=h"(h) : "f"(v));
        else asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(h) : "f"(v));
    }
    return h;
}
// 1.0 twice
__device__ __forceinline__ uint32_t one_x2(int f16) { return f16 ? 0x3c003c00u : 0x3f803f80u; }
// b as {hi, lo} with hi + lo = b to 16 (bf16) or 22 (fp16) bits below its leading bit
__device__ __forceinline__ uint32_t bias_hi_lo(float b, int f16)
{
    if (f16) {
        const __half hi = __float2half_rn(b);
        const __half lo = __float2half_rn(b - __half2float(hi));
        return (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
    }
    const __nv_bfloat16 hi = __float2bfloat16_rn(b);
    const __nv_bfloat16 lo = __float2bfloat16_rn(b - __bfloat162float(hi));
    return (uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(lo) << 16);
}
// Bias row of the bias MMAs: one 32-byte row {hi, lo, 0, ...} per output layer in the 32-byte swizzle.
__device__ __forceinline__ void bias_row(uint4* rows, int c, float b, int f16)
{
    const int u = (c >> 2) & 1;
    rows[2 * c + u] = make_uint4(bias_hi_lo(b, f16), 0u, 0u, 0u);
    rows[2 * c + (u ^ 1)] = make_uint4(0u, 0u, 0u, 0u);
}

}  // namespace sqn
