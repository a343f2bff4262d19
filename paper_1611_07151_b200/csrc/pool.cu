// Pooling layers and the classifier head (paper Section III-E), NHWC.
//   max pooling 3x3 / stride 2, no padding: one thread per output pixel and group of layers,
//   128-bit loads and stores along the layer dimension (memory bound: one read, one write);
//   global average pooling + softmax: one block per image.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "sqn_internal.h"

namespace sqn {
namespace {

__device__ __forceinline__ float4 max4(float4 a, float4 b)
{
    return make_float4(fmaxf(a.x, b.x), fmaxf(a.y, b.y), fmaxf(a.z, b.z), fmaxf(a.w, b.w));
}

// fp32, C % 4 == 0: each thread produces 4 layers of one output pixel.
__global__ void maxpool_f32_v4(const float* __restrict__ in, float* __restrict__ out, int C4, int H, int W, int OH,
                               int OW, long long total)
{
    chain_release();
    chain_wait();
    const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int c4 = (int)(idx % C4);
    long long r = idx / C4;
    const int ow = (int)(r % OW); r /= OW;
    const int oh = (int)(r % OH);
    const long long n = r / OH;
    const float4* src = reinterpret_cast<const float4*>(in) + ((n * H + 2 * oh) * W + 2 * ow) * C4 + c4;
    float4 m = __ldg(src);
#pragma unroll
    for (int i = 0; i < 3; ++i)
#pragma unroll
        for (int j = 0; j < 3; ++j) m = max4(m, __ldg(src + ((long long)i * W + j) * C4));
    reinterpret_cast<float4*>(out)[idx] = m;
}

// fp32, any C: one thread per output element.
__global__ void maxpool_f32_s(const float* __restrict__ in, float* __restrict__ out, int C, int H, int W, int OH,
                              int OW, long long total)
{
    chain_release();
    chain_wait();
    const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int c = (int)(idx % C);
    long long r = idx / C;
    const int ow = (int)(r % OW); r /= OW;
    const int oh = (int)(r % OH);
    const long long n = r / OH;
    const float* src = in + ((n * H + 2 * oh) * W + 2 * ow) * C + c;
    float m = __ldg(src);
    for (int i = 0; i < 3; ++i)
        for (int j = 0; j < 3; ++j) m = fmaxf(m, __ldg(src + ((long long)i * W + j) * C));
    out[idx] = m;
}

// 16-bit element types of the tensor-core paths: scalar type, packed pair
struct Bf16 { typedef __nv_bfloat16 T; typedef __nv_bfloat162 T2; };
struct Fp16 { typedef __half T; typedef __half2 T2; };
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_f32(__half v) { return __half2float(v); }
__device__ __forceinline__ void from_f32(float f, __nv_bfloat16* o) { *o = __float2bfloat16(f); }
__device__ __forceinline__ void from_f32(float f, __half* o) { *o = __float2half(f); }

template <typename E>
__device__ __forceinline__ uint32_t bmax2(uint32_t a, uint32_t b)
{
    typename E::T2 x = *reinterpret_cast<typename E::T2*>(&a);
    typename E::T2 y = *reinterpret_cast<typename E::T2*>(&b);
    typename E::T2 m = __hmax2(x, y);
    return *reinterpret_cast<uint32_t*>(&m);
}

// 16-bit types, C % 8 == 0: each thread produces 8 layers (16 bytes) of one output pixel.
template <typename E>
__global__ void maxpool_bf16_v8(const uint4* __restrict__ in, uint4* __restrict__ out, int C8, int H, int W, int OH,
                                int OW, long long total)
{
    chain_release();
    chain_wait();
    // last output first: the end of the input map is what the layer before left in the L2
    const long long idx = total - 1 - (blockIdx.x * (long long)blockDim.x + threadIdx.x);
    if (idx < 0) return;
    const int c8 = (int)(idx % C8);
    long long r = idx / C8;
    const int ow = (int)(r % OW); r /= OW;
    const int oh = (int)(r % OH);
    const long long n = r / OH;
    const uint4* src = in + ((n * H + 2 * oh) * W + 2 * ow) * C8 + c8;
    uint4 m = __ldg(src);
#pragma unroll
    for (int i = 0; i < 3; ++i)
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            const uint4 v = __ldg(src + ((long long)i * W + j) * C8);
            m.x = bmax2<E>(m.x, v.x); m.y = bmax2<E>(m.y, v.y); m.z = bmax2<E>(m.z, v.z); m.w = bmax2<E>(m.w, v.w);
        }
    out[idx] = m;
}

template <typename E>
__global__ void maxpool_bf16_s(const typename E::T* __restrict__ in, typename E::T* __restrict__ out, int C, int H,
                               int W, int OH, int OW, long long total)
{
    chain_release();
    chain_wait();
    const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int c = (int)(idx % C);
    long long r = idx / C;
    const int ow = (int)(r % OW); r /= OW;
    const int oh = (int)(r % OH);
    const long long n = r / OH;
    const typename E::T* src = in + ((n * H + 2 * oh) * W + 2 * ow) * C + c;
    float m = to_f32(src[0]);
    for (int i = 0; i < 3; ++i)
        for (int j = 0; j < 3; ++j) m = fmaxf(m, to_f32(src[((long long)i * W + j) * C]));
    from_f32(m, &out[idx]);
}

// Global average: block (x = group of 128 layers, y = image), 256 threads = 64 layer pairs x 4 pixel
// quarters.  Consecutive threads read consecutive 4- or 8-byte words of a pixel; the quarters are combined
// in shared memory.  Small batches still get C/128 blocks per image.
template <int MODE>        // 0: fp32, 1: bf16, 2: fp16
__global__ void __launch_bounds__(256) global_avgpool_kernel(const void* __restrict__ in_, float* __restrict__ logits,
                                                             int C, int HW)
{
    chain_release();
    chain_wait();
    __shared__ float part[4][128];
    const int n = blockIdx.y;
    const int tid = threadIdx.x;
    const int quarter = tid >> 6;
    const int c = blockIdx.x * 128 + 2 * (tid & 63);
    const int p_lo = quarter * HW / 4, p_hi = (quarter + 1) * HW / 4;
    float s0 = 0.f, s1 = 0.f, t0 = 0.f, t1 = 0.f, u0 = 0.f, u1 = 0.f, v0 = 0.f, v1 = 0.f;
    if (c < C) {
        const bool pair = (c + 1 < C) && (C % 2 == 0);
        auto ld = [&](int p, float& a, float& b) {
            if (MODE == 1) {
                const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(in_) + ((size_t)n * HW + p) * C + c;
                if (pair) {
                    const __nv_bfloat162 w = *reinterpret_cast<const __nv_bfloat162*>(src);
                    a += __low2float(w); b += __high2float(w);
                } else {
                    a += __bfloat162float(src[0]);
                    if (c + 1 < C) b += __bfloat162float(src[1]);
                }
            } else if (MODE == 2) {
                const __half* src = static_cast<const __half*>(in_) + ((size_t)n * HW + p) * C + c;
                if (pair) {
                    const __half2 w = *reinterpret_cast<const __half2*>(src);
                    a += __low2float(w); b += __high2float(w);
                } else {
                    a += __half2float(src[0]);
                    if (c + 1 < C) b += __half2float(src[1]);
                }
            } else {
                const float* src = static_cast<const float*>(in_) + ((size_t)n * HW + p) * C + c;
                if (pair) {
                    const float2 w = __ldg(reinterpret_cast<const float2*>(src));
                    a += w.x; b += w.y;
                } else {
                    a += __ldg(src);
                    if (c + 1 < C) b += __ldg(src + 1);
                }
            }
        };
        int p = p_lo;
        for (; p + 4 <= p_hi; p += 4) { ld(p, s0, s1); ld(p + 1, t0, t1); ld(p + 2, u0, u1); ld(p + 3, v0, v1); }
        for (; p < p_hi; ++p) ld(p, s0, s1);
    }
    part[quarter][2 * (tid & 63)] = (s0 + t0) + (u0 + v0);
    part[quarter][2 * (tid & 63) + 1] = (s1 + t1) + (u1 + v1);
    __syncthreads();
    if (tid < 128) {
        const int cc = blockIdx.x * 128 + tid;
        if (cc < C)
            logits[(size_t)n * C + cc] = ((part[0][tid] + part[1][tid]) + (part[2][tid] + part[3][tid])) / (float)HW;
    }
}

// Global average of a 16-bit map with C % 8 == 0: block (x = group of 128 layers, y = image), 256 threads =
// 16 groups of 8 layers (one 16-byte load per pixel) x 16 pixel slices, four loads in flight per thread.
template <typename E>
__global__ void __launch_bounds__(256) global_avgpool_bf16_v8(const uint4* __restrict__ in, float* __restrict__ logits,
                                                              int C, int HW)
{
    chain_release();
    chain_wait();
    __shared__ float part[16][129];
    const int n = gridDim.y - 1 - blockIdx.y, tid = threadIdx.x;      // last image first (still in the L2)
    const int g = tid & 15, slice = tid >> 4;
    const int c0 = blockIdx.x * 128 + 8 * g;
    float acc[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = 0.f;
    if (c0 < C) {
        const int C8 = C >> 3;
        const uint4* src = in + (size_t)n * HW * C8 + (c0 >> 3);
        auto add = [&](const uint4& v) {
            const typename E::T2* h = reinterpret_cast<const typename E::T2*>(&v);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                acc[2 * k] += __low2float(h[k]);
                acc[2 * k + 1] += __high2float(h[k]);
            }
        };
        int p = slice;
        for (; p + 48 < HW; p += 64) {
            const uint4 v0 = __ldg(src + (size_t)p * C8), v1 = __ldg(src + (size_t)(p + 16) * C8);
            const uint4 v2 = __ldg(src + (size_t)(p + 32) * C8), v3 = __ldg(src + (size_t)(p + 48) * C8);
            add(v0); add(v1); add(v2); add(v3);
        }
        for (; p < HW; p += 16) add(__ldg(src + (size_t)p * C8));
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) part[slice][8 * g + k] = acc[k];
    __syncthreads();
    if (tid < 128) {
        const int c = blockIdx.x * 128 + tid;
        if (c < C) {
            float s = 0.f;
#pragma unroll
            for (int q = 0; q < 16; ++q) s += part[q][tid];
            logits[(size_t)n * C + c] = s / (float)HW;
        }
    }
}

// Softmax over the C logits of one image per block.
__global__ void __launch_bounds__(256) softmax_kernel(const float* __restrict__ logits, float* __restrict__ probs, int C)
{
    chain_release();
    chain_wait();
    extern __shared__ float z[];
    __shared__ float red[8];
    const int n = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float m = -INFINITY;
    for (int c = tid; c < C; c += 256) { z[c] = logits[(size_t)n * C + c]; m = fmaxf(m, z[c]); }
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) red[warp] = m;
    __syncthreads();
    m = red[0];
    for (int i = 1; i < 8; ++i) m = fmaxf(m, red[i]);
    __syncthreads();
    float s = 0.f;
    for (int c = tid; c < C; c += 256) {
        const float e = expf(z[c] - m);
        z[c] = e;
        s += e;
    }
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) red[warp] = s;
    __syncthreads();
    s = 0.f;
    for (int i = 0; i < 8; ++i) s += red[i];
    const float r = 1.0f / s;
    for (int c = tid; c < C; c += 256) probs[(size_t)n * C + c] = z[c] * r;
}

}  // namespace

int launch_maxpool3x3s2(const void* in, void* out, int C, int H, int W, int N, int dtype, cudaStream_t stream)
{
    const int OH = (H - 3) / 2 + 1, OW = (W - 3) / 2 + 1;
    const int threads = 256;
    if (dtype == SQN_F32) {
        if (C % 4 == 0) {
            const long long total = (long long)N * OH * OW * (C / 4);
            launch_chained(maxpool_f32_v4, dim3((unsigned)((total + threads - 1) / threads)), dim3(threads), 0, stream,
                           static_cast<const float*>(in), static_cast<float*>(out), C / 4, H, W, OH, OW, total);
        } else {
            const long long total = (long long)N * OH * OW * C;
            launch_chained(maxpool_f32_s, dim3((unsigned)((total + threads - 1) / threads)), dim3(threads), 0, stream,
                           static_cast<const float*>(in), static_cast<float*>(out), C, H, W, OH, OW, total);
        }
    } else {
        const bool f16 = dtype == SQN_F16;
        if (C % 8 == 0) {
            const long long total = (long long)N * OH * OW * (C / 8);
            const dim3 grid((unsigned)((total + threads - 1) / threads));
            if (f16) launch_chained(maxpool_bf16_v8<Fp16>, grid, dim3(threads), 0, stream, static_cast<const uint4*>(in),
                                    static_cast<uint4*>(out), C / 8, H, W, OH, OW, total);
            else launch_chained(maxpool_bf16_v8<Bf16>, grid, dim3(threads), 0, stream, static_cast<const uint4*>(in),
                                static_cast<uint4*>(out), C / 8, H, W, OH, OW, total);
        } else {
            const long long total = (long long)N * OH * OW * C;
            const dim3 grid((unsigned)((total + threads - 1) / threads));
            if (f16) launch_chained(maxpool_bf16_s<Fp16>, grid, dim3(threads), 0, stream, static_cast<const __half*>(in),
                                    static_cast<__half*>(out), C, H, W, OH, OW, total);
            else launch_chained(maxpool_bf16_s<Bf16>, grid, dim3(threads), 0, stream, static_cast<const __nv_bfloat16*>(in),
                                static_cast<__nv_bfloat16*>(out), C, H, W, OH, OW, total);
        }
    }
    note_launch();
    return cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}

int launch_avgpool_softmax(const void* in, float* logits, float* probs, int C, int H, int W, int N, int dtype,
                           cudaStream_t stream)
{
    const dim3 grid((unsigned)((C + 127) / 128), (unsigned)N);
    if (dtype == SQN_F32) launch_chained(global_avgpool_kernel<0>, grid, dim3(256), 0, stream, in, logits, C, H * W);
    else if (C % 8 == 0 && aligned16(in)) {
        if (dtype == SQN_F16)
            launch_chained(global_avgpool_bf16_v8<Fp16>, grid, dim3(256), 0, stream, static_cast<const uint4*>(in), logits, C, H * W);
        else
            launch_chained(global_avgpool_bf16_v8<Bf16>, grid, dim3(256), 0, stream, static_cast<const uint4*>(in), logits, C, H * W);
    } else if (dtype == SQN_F16) launch_chained(global_avgpool_kernel<2>, grid, dim3(256), 0, stream, in, logits, C, H * W);
    else launch_chained(global_avgpool_kernel<1>, grid, dim3(256), 0, stream, in, logits, C, H * W);
    note_launch();
    if (cudaGetLastError() != cudaSuccess) return SQN_ERR_CUDA;
    if (probs) return launch_softmax(logits, probs, C, N, stream);
    return SQN_OK;
}

int launch_softmax(const float* logits, float* probs, int C, int N, cudaStream_t stream)
{
    launch_chained(softmax_kernel, dim3((unsigned)N), dim3(256), (size_t)C * sizeof(float), stream, logits, probs, C);
    note_launch();
    return cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}

}  // namespace sqn
