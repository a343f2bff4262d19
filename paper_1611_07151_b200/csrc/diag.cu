// Diagnostics of the tensor-core kernels' shared machinery, reachable through the C ABI: a bounded wait that runs out,
// and the issue rate of tcgen05.mma as a function of its N (the measurement the kernels' role layout rests on).
#include <cuda.h>
#include <cuda_bf16.h>

#include "ptx_sm100.cuh"
#include "sqn_internal.h"
#include "tc_common.cuh"

namespace sqn {
namespace {

using namespace ptx;

// One CTA with the roles' skeleton of the kernels above -- barriers, a TMEM allocation, a bounded wait -- whose wait
// is for an mbarrier that nothing ever arrives on: the wait runs out after `limit` cycles, the CTA records
// SQN_ERR_TIMEOUT in the status word, frees its TMEM and returns like any other.
__global__ void __launch_bounds__(64, 1) wait_timeout_kernel(long long limit, int* status)
{
    __shared__ unsigned long long bar;
    __shared__ unsigned tmem_base_s;
    __shared__ volatile int abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_base_s), 32);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) {
        // the whole warp waits, as the MMA issuers do; every lane sees the time-out
        const bool ok = __all_sync(0xffffffffu, wait_bar_limit(smem_u32(&bar), 0u, &abort_flag, status, limit));
        if (ok && lane == 0) atomicExch(status, (int)SQN_ERR_CUDA);        // (cannot happen: nothing arrives)
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base_s, 32);
    }
}


// `iters` MMAs of M = 128, K = 16, the given N (bf16 operands: zeros in shared memory, rows of `row_bytes` in the
// matching swizzle) issued back to back by one elected thread of `issuers` warps (1 or 2, each with its own accumulator),
// one commit per warp at the end, bounded wait for it.  out[3 * (2 * block + warp)] = {clocks until the last MMA was
// issued, clocks until all had completed, 1 if the wait ended in time}.
__global__ void __launch_bounds__(128, 1) mma_rate_kernel(int iters, int n, int row_bytes, int issuers, long long* out, int* status)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    __shared__ unsigned long long bars[2];
    __shared__ unsigned tmem_base_s;
    __shared__ volatile int abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (uint32_t i = threadIdx.x; i < 96u * 1024u / 16u; i += blockDim.x)
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(base + 16u * i), "r"(0u) : "memory");
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars[0]), 1);
        mbar_init(smem_u32(&bars[1]), 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(smem_u32(&tmem_base_s), 512); tmem_relinquish(); }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    if (warp < issuers) {
        // each issuer: A = 128 rows at its 48 KB half of the buffer, B = n rows 16 KB further on (both inside the 96 KB)
        const uint32_t idesc = make_idesc_bf16(128, (uint32_t)n);
        const uint64_t da = make_kmajor_desc(base + (uint32_t)warp * 48u * 1024u, (uint32_t)row_bytes, 8u * (uint32_t)row_bytes);
        const uint64_t db = make_kmajor_desc(base + (uint32_t)warp * 48u * 1024u + 16384u, (uint32_t)row_bytes, 8u * (uint32_t)row_bytes);
        const uint32_t d = tmem_base + (uint32_t)warp * 256u;
        const uint32_t bar = smem_u32(&bars[warp]);
        __syncwarp();
        const long long t0 = clock64();
        if (elect_one()) {
            for (int i = 0; i < iters; ++i) mma_bf16_ss(d, da, db, idesc, i ? 1u : 0u);
            mma_commit(bar);
        }
        __syncwarp();
        const long long t_issue = clock64();
        const bool ok = __all_sync(0xffffffffu, wait_bar_limit(bar, 0u, &abort_flag, status, 2000000000LL));
        const long long t1 = clock64();
        if (lane == 0) {
            long long* o = out + 3 * (2 * (int)blockIdx.x + warp);
            o[0] = t_issue - t0;
            o[1] = t1 - t0;
            o[2] = ok ? 1 : 0;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) { __syncwarp(); tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}

}  // namespace

int launch_wait_timeout_selftest(long long limit_cycles, cudaStream_t stream)
{
    int* status = device_status_word();
    if (!status) return SQN_ERR_CUDA;
    wait_timeout_kernel<<<1, 64, 0, stream>>>(limit_cycles, status);
    note_launch();
    return cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}


int launch_mma_rate_selftest(int n, int row_bytes, int issuers, int iters, long long* out, cudaStream_t stream)
{
    int* status = device_status_word();
    if (!status) return SQN_ERR_CUDA;
    static const cudaError_t attr_rc = cudaFuncSetAttribute(mma_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
    if (attr_rc != cudaSuccess) return SQN_ERR_CUDA;
    int sms = 0, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms <= 0) return SQN_ERR_CUDA;
    mma_rate_kernel<<<sms, 128, 98 * 1024, stream>>>(iters, n, row_bytes, issuers, out, status);
    note_launch();
    return cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}

}  // namespace sqn
