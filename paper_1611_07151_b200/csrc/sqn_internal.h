// Internal declarations shared by the library's translation units.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "sqn.h"

namespace sqn {

// One convolution layer as the kernels see it (validated by the caller).
struct ConvDesc {
    const void* in;       // [N][H][W][Cin]
    const void* w;        // [Cout][K][K][Cin]
    const float* bias;    // [Cout]
    void* out;            // [N][OH][OW][out_c_total], written at out_c_offset
    int N, Cin, H, W, Cout, K, S, pad, OH, OW;
    int out_c_offset, out_c_total, relu;
    int pool;             // 1: out receives the 3x3/stride-2 max-pool of the layer's output (bf16 path only)
    int params_static;    // 1: kernels and bias are not written by earlier work on the stream (a net's own parameters), so
                          //    a chained launch may fetch them before the kernel ahead of it has finished
    int f16;              // tensor-core paths: 1 = activations and kernels are fp16, 0 = bf16
    int stem_prepacked;   // 1 (stem only): in and w already have the stem kernel's own layouts, see sqn_pack_stem_input
};

// Launch counter (host side): every kernel launch goes through note_launch().
void note_launch(int n = 1);

// Device status word shared by all kernels (0 = fine, else an sqn_status).
int* device_status_word();

// fp32 path: register-tiled FFMA implicit GEMM, any (K, S, pad, Cin, Cout).
int launch_conv_f32(const ConvDesc& d, cudaStream_t stream);

// bf16 path: tcgen05/TMEM implicit GEMM fed by TMA.
// Returns SQN_ERR_UNSUPPORTED for shapes outside its family.
int conv_bf16_supported(const ConvDesc& d);
int launch_conv_bf16(const ConvDesc& d, cudaStream_t stream);
// Two independent layers in one launch (first `big`'s CTAs, then `small`'s); SQN_ERR_UNSUPPORTED if they share no
// kernel variant.
int launch_conv_bf16_pair(const ConvDesc& small, const ConvDesc& big, cudaStream_t stream);
int launch_conv_bf16_pool4(const ConvDesc* four, cudaStream_t stream);   // four pooled layers over one input, one launch
// n (1 or 2) pooled 3x3 layers, each with a pooled 1x1 layer on the same input riding on its patches: one launch
int launch_conv_bf16_pool_riders(const ConvDesc* big, const ConvDesc* rider, int n, cudaStream_t stream);
bool conv_bf16_pool_fits(const ConvDesc& d);   // true when the layer can run with its max-pool fused (d.pool = 1)
int launch_conv_bf16_uncached(const ConvDesc& d, cudaStream_t stream);   // no plan cache, no allocation
// Stem (7x7/2 on 3 layers): needs scratch for the repacked input and kernels.
size_t stem_bf16_workspace_bytes(int N, int H, int W, int Cout);
int launch_stem_pack_bf16(const ConvDesc& d, void* workspace, size_t workspace_bytes, cudaStream_t stream);
int launch_stem_conv_bf16(const ConvDesc& d, void* workspace, size_t workspace_bytes, cudaStream_t stream);
// The stem on operands the caller packed offline (d.in = [N][Hp][Wp][4], d.w = [Cout][7][8][4] with the bias folded in).
int launch_stem_conv_bf16_prepacked(const ConvDesc& d, cudaStream_t stream);
inline int stem_packed_rows(int H) { return (H + 1) / 2 * 2; }
inline int stem_packed_cols(int W) { return (W + 2) / 2 * 2; }

// The whole fire layer (squeeze, both expands) in one launch, the squeeze map kept in shared memory; SQN_ERR_UNSUPPORTED
// where that kernel does not apply.  SQN_FUSED_FIRE=0 in the environment turns it off.
bool fused_fire_enabled();
int launch_fire_fused_bf16(const ConvDesc& dsq, const ConvDesc& d1, const ConvDesc& d3, cudaStream_t stream);
// Both expands on a stored squeeze map with the same kernel's expand pipeline (SQN_ERR_UNSUPPORTED where it does not apply).
int launch_fire_expands_bf16(const ConvDesc& d1, const ConvDesc& d3, cudaStream_t stream);

// 1x1 convolution + ReLU + global average in one launch (the map is not stored): logits[n][m], fp32.
// SQN_FUSED_HEAD=0 in the environment turns its use by squeezenet_forward off.
bool fused_head_enabled();
int launch_conv_avgpool_bf16(const ConvDesc& d, float* logits, cudaStream_t stream);

// A kernel whose bounded wait runs out (see sqn_selftest_wait_timeout).
int launch_wait_timeout_selftest(long long limit_cycles, cudaStream_t stream);
// tcgen05.mma issue rate (see sqn_selftest_mma_rate); out: 6 values per SM.
int launch_mma_rate_selftest(int n, int row_bytes, int issuers, int iters, long long* out, cudaStream_t stream);

// Pooling / head.
int launch_maxpool3x3s2(const void* in, void* out, int C, int H, int W, int N, int dtype, cudaStream_t stream);
int launch_avgpool_softmax(const void* in, float* logits, float* probs, int C, int H, int W, int N, int dtype,
                           cudaStream_t stream);
int launch_softmax(const float* logits, float* probs, int C, int N, cudaStream_t stream);

// Chained launches.  A kernel launched through launch_chained() may be scheduled while the kernel before it
// in the stream is still running (programmatic stream serialisation): its blocks take the SMs the earlier
// grid frees and do their on-chip set-up there.  Every such kernel calls chain_wait() before its first
// access to global memory; that returns once the earlier grid has finished and its writes are visible, so
// the data dependences of a plain launch are kept.  chain_release() lets the grid after this one start its
// own set-up early.  SQN_CHAINED_LAUNCH=0 in the environment turns the attribute off (plain launches).
bool chained_launch_enabled();

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                  Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chained_launch_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#ifdef __CUDACC__
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// Debug build (-DSQN_DEBUG): index checks in the kernels.  A failed check records SQN_ERR_DEBUG in the status word and
// the guarded access is skipped; nothing traps.  In the normal build the checks compile to nothing.
#ifdef __CUDACC__
#ifdef SQN_DEBUG
__device__ __forceinline__ bool sqn_dbg_ok(bool cond, int* status)
{
    if (!cond && status) atomicExch(status, (int)SQN_ERR_DEBUG);
    return cond;
}
#else
__device__ __forceinline__ bool sqn_dbg_ok(bool, int*) { return true; }
#endif
#endif

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace sqn
