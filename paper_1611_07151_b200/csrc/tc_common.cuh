// Device helpers shared by the tensor-core kernels: the bounded mbarrier wait and the fp32 -> bf16 packing.
#pragma once

#include <cuda_bf16.h>

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

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// max(.,0) and round-to-nearest-even conversion of two values in one instruction
__device__ __forceinline__ uint32_t pack_relu_bf16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// maximum of three values in one instruction
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
// fp32 -> bf16 (round to nearest even), with max(., 0) folded into the conversion when relu is set
__device__ __forceinline__ unsigned short to_bf16_bits(float v, int relu)
{
    unsigned short h;
    if (relu) asm("cvt.rn.relu.bf16.f32 %0, %1;" : "=h"(h) : "f"(v));
    else asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(h) : "f"(v));
    return h;
}


}  // namespace sqn
