// 1x1 convolution + ReLU + global average pooling in one kernel (bf16 operands, fp32 everywhere else): the classifier
// head of the network (conv10 and the average of Section III-E of the paper).  The convolution's output map is never
// stored: only the per-layer means leave the SM.
//
// The GEMM is taken with the layers on the accumulator's rows: D[layer][pixel] = sum_k W[layer][k] * X[pixel][k].
// A CTA owns one tile of 128 output layers, whose kernels (128 x Cin) stay in shared memory; it walks images, for each
// streaming the image's pixels (N = all HW pixels of the image, rounded up to 16; K-major as they lie in NHWC memory)
// through a ring of TMA boxes.  An epilogue thread owns one output layer and sees every pixel of the image in its
// accumulator row: it adds the bias, applies the ReLU and sums in registers -- no exchange between threads, no atomics,
// the same order of additions whatever the launch shape.  Two accumulators alternate, so the sums of image i are taken
// while the MMAs of image i + 1 run.  The CTAs that work on the same image (one per layer tile) are neighbours in the
// grid and run at the same time, so the image's pixels come from HBM once and from the L2 after that.
// Warps: 0 TMA producer, 1 MMA issuer, 2..5 epilogue (one per TMEM lane quadrant).  Every mbarrier wait is bounded.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <string>

#include "ptx_sm100.cuh"
#include "sqn_internal.h"
#include "tc_common.cuh"
#include "tc_host.h"

namespace sqn {
namespace {

using namespace ptx;

constexpr int CH_THREADS = 32 * 6;
constexpr int CH_MAX_STAGES = 8;
constexpr size_t CH_SMEM_LIMIT = 227 * 1024;

struct HeadParams {
    int N, HW, Cin, Cout;
    int NP;                          // pixels per MMA: HW rounded up to a multiple of 16
    int chunks;                      // reduction chunks of 64 layers
    int n_tiles;                     // tiles of 128 output layers
    int groups;                      // CTAs per layer tile; group g takes images g, g + groups, ...
    int stages;
    int relu;
    int f16;                         // 1: fp16 operands, 0: bf16
    int b_early;
    unsigned x_tile, x_bytes;        // ring slot size / bytes one pixel box delivers
    unsigned off_x, off_ctl;         // (the kernels start at offset 0: `chunks` tiles of 128 rows x 128 bytes)
    float inv_hw;
    const float* bias;
    float* logits;                   // [N][Cout]
    int* status;
};

struct HeadShared {
    unsigned long long full[CH_MAX_STAGES];
    unsigned long long empty[CH_MAX_STAGES];
    unsigned long long w_full;
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned tmem_base;
    volatile int abort_flag;
};

__global__ void __launch_bounds__(CH_THREADS, 1)
conv_head_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                 const __grid_constant__ HeadParams p)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - raw);
    HeadShared* sh = reinterpret_cast<HeadShared*>(base_ptr + p.off_ctl);
    const uint32_t smW = base, smX = base + p.off_x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = (int)blockIdx.x % p.n_tiles, grp = (int)blockIdx.x / p.n_tiles;
    constexpr uint32_t W_TILE = 128u * 128u;            // one reduction chunk of the kernels: 128 rows of 128 bytes

    auto load_kernels = [&]() {
        const uint32_t bar = smem_u32(&sh->w_full);
        mbar_arrive_expect_tx(bar, (uint32_t)p.chunks * W_TILE);        // (rows past Cout are filled with zeros and counted)
        for (int ch = 0; ch < p.chunks; ++ch) tma_load_2d(smW + (uint32_t)ch * W_TILE, &tmW, bar, ch * 64, tile * 128);
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&sh->full[s]), 1);
            mbar_init(smem_u32(&sh->empty[s]), 1);
        }
        mbar_init(smem_u32(&sh->w_full), 1);
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&sh->tmem_full[a]), 1);
            mbar_init(smem_u32(&sh->tmem_empty[a]), 4);
        }
        sh->abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmX);
        prefetch_tensormap(&tmW);
        if (p.b_early) load_kernels();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&sh->tmem_base), 512);
        tmem_relinquish();
        chain_release();            // (only once this CTA holds its TMEM: see conv_tc_body)
    }
    chain_wait();       // the grid ahead has finished: global memory may be read and written from here on
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    volatile int* abort_flag = &sh->abort_flag;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer: the images' pixels, chunk by chunk
        if (lane == 0) {
            if (!p.b_early) load_kernels();
            bool ok = true;
            int st = 0, issued = 0;
            uint32_t ph = 0;
            for (int n = grp; n < p.N && ok; n += p.groups)
                for (int ch = 0; ch < p.chunks; ++ch) {
                    if (!wait_bar(smem_u32(&sh->empty[st]), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    const uint32_t full = smem_u32(&sh->full[st]);
                    mbar_arrive_expect_tx(full, p.x_bytes);
                    tma_load_2d(smX + (uint32_t)st * p.x_tile, &tmX, full, ch * 64, n * p.HW);
                    ++issued;
                    if (++st == p.stages) { st = 0; ph ^= 1u; }
                }
            if (!ok) {      // give the copies already issued a bounded chance to land before the CTA exits
                int pending = issued < p.stages ? issued : p.stages;
                while (pending-- > 0) {
                    if (st == 0) { st = p.stages; ph ^= 1u; }
                    --st;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(smem_u32(&sh->full[st]), ph)) {
                        if (clock64() - t0 > WAIT_LIMIT_CYCLES / 8) break;
                        __nanosleep(100);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc = make_idesc_bf16(128, (uint32_t)p.NP, (uint32_t)p.f16);
        const uint32_t hi = (uint32_t)(make_kmajor_desc(0, 128u, 1024u) >> 32);
        const uint32_t smW16 = smW >> 4, smX16 = smX >> 4, x_tile16 = p.x_tile >> 4;
        bool ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->w_full), 0u, abort_flag, p.status));
        int st = 0, as = 0;
        uint32_t ph = 0, aph = 0;
        for (int n = grp; n < p.N && ok; n += p.groups) {
            ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->tmem_empty[as]), aph ^ 1u, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(as * 256);
            for (int ch = 0; ch < p.chunks; ++ch) {
                ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->full[st]), ph, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
                    const uint64_t da = ((uint64_t)hi << 32) | (uint64_t)((smW16 + (uint32_t)ch * (W_TILE >> 4)) | 0x10000u);
                    const uint64_t db = ((uint64_t)hi << 32) | (uint64_t)((smX16 + (uint32_t)st * x_tile16) | 0x10000u);
                    mma_bf16_ss(d_tmem, da, db, idesc, ch ? 1u : 0u);
                    mma_bf16_ss(d_tmem, da + 2u, db + 2u, idesc, 1u);
                    mma_bf16_ss(d_tmem, da + 4u, db + 4u, idesc, 1u);
                    mma_bf16_ss(d_tmem, da + 6u, db + 6u, idesc, 1u);
                    mma_commit(smem_u32(&sh->empty[st]));               // pixel slot free once these MMAs have read it
                    if (ch == p.chunks - 1) mma_commit(smem_u32(&sh->tmem_full[as]));
                }
                __syncwarp();
                if (++st == p.stages) { st = 0; ph ^= 1u; }
            }
            if (!ok) break;
            if (++as == 2) { as = 0; aph ^= 1u; }
        }
    } else {
        // -------------------------------------------------------------------- epilogue: one output layer per thread
        const int q = warp & 3;
        const int layer = tile * 128 + q * 32 + lane;
        const bool live = layer < p.Cout;
        const float b = live ? __ldg(p.bias + layer) : 0.f;
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        bool ok = true;
        int as = 0;
        uint32_t aph = 0;
        for (int n = grp; n < p.N && ok; n += p.groups) {
            ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->tmem_full[as]), aph, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
            const uint32_t ta = tmem_base + lane_base + (uint32_t)(as * 256);
            // four partial sums; the pixels are taken 16 at a time with the next 16 already requested
            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
            auto add16 = [&](const uint32_t (&v)[16], int c0) {
#pragma unroll
                for (int j = 0; j < 16; j += 4) {
                    float t0 = __uint_as_float(v[j]) + b, t1 = __uint_as_float(v[j + 1]) + b;
                    float t2 = __uint_as_float(v[j + 2]) + b, t3 = __uint_as_float(v[j + 3]) + b;
                    if (p.relu) { t0 = fmaxf(t0, 0.f); t1 = fmaxf(t1, 0.f); t2 = fmaxf(t2, 0.f); t3 = fmaxf(t3, 0.f); }
                    // (columns past the image's last pixel belong to the next image: left out)
                    if (c0 + j < p.HW) s0 += t0;
                    if (c0 + j + 1 < p.HW) s1 += t1;
                    if (c0 + j + 2 < p.HW) s2 += t2;
                    if (c0 + j + 3 < p.HW) s3 += t3;
                }
            };
            uint32_t va[16], vb[16];
            tmem_ld_x16(ta, va);
            for (int c0 = 0; c0 < p.NP; c0 += 32) {
                tmem_ld_wait();
                const bool second = c0 + 16 < p.NP;
                if (second) tmem_ld_x16(ta + (uint32_t)(c0 + 16), vb);
                add16(va, c0);
                if (second) {
                    tmem_ld_wait();
                    if (c0 + 32 < p.NP) tmem_ld_x16(ta + (uint32_t)(c0 + 32), va);
                    add16(vb, c0 + 16);
                }
            }
            // accumulator read: hand it back to the MMA issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->tmem_empty[as]));
            if (++as == 2) { as = 0; aph ^= 1u; }
            if (live && sqn_dbg_ok(n < p.N && layer < p.Cout, p.status)) p.logits[(size_t)n * p.Cout + layer] = ((s0 + s1) + (s2 + s3)) * p.inv_hw;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

struct HeadPlan {
    CUtensorMap x, w;
    HeadParams p;
    int grid;
    size_t smem;
};

struct HeadKey {
    const void *in, *w, *bias, *out;
    int v[8];
};

std::mutex g_head_mu;
std::map<std::string, HeadPlan> g_head_plans;

int build_head_plan(const ConvDesc& d, float* logits, HeadPlan* plan)
{
    HeadParams& p = plan->p;
    std::memset(&p, 0, sizeof(p));
    const int HW = d.H * d.W;
    if (d.K != 1 || d.S != 1 || d.pad != 0) return SQN_ERR_UNSUPPORTED;
    if (d.Cin % 64 != 0 || HW > 256 || d.Cout < 1) return SQN_ERR_UNSUPPORTED;
    if ((long long)d.N * HW > 0x7fffffffLL / 2) return SQN_ERR_UNSUPPORTED;
    p.N = d.N; p.HW = HW; p.Cin = d.Cin; p.Cout = d.Cout;
    p.NP = (HW + 15) / 16 * 16;
    p.chunks = d.Cin / 64;
    p.n_tiles = (d.Cout + 127) / 128;
    p.relu = d.relu;
    p.f16 = d.f16;
    p.b_early = d.params_static ? 1 : 0;
    p.bias = d.bias;
    p.logits = logits;
    p.inv_hw = 1.0f / (float)HW;
    p.status = device_status_word();
    p.x_bytes = (unsigned)p.NP * 128u;
    p.x_tile = (p.x_bytes + 1023u) / 1024u * 1024u;
    const size_t w_bytes = (size_t)p.chunks * 128 * 128;
    if (w_bytes >= (1u << 20)) return SQN_ERR_UNSUPPORTED;       // one mbarrier transaction count
    if (CH_SMEM_LIMIT < 1024 + w_bytes + 1024 + 2 * (size_t)p.x_tile) return SQN_ERR_UNSUPPORTED;
    int stages = (int)((CH_SMEM_LIMIT - 1024 - w_bytes - 1024) / p.x_tile);
    if (stages > CH_MAX_STAGES) stages = CH_MAX_STAGES;
    p.stages = stages;
    p.off_x = (unsigned)w_bytes;
    p.off_ctl = p.off_x + (unsigned)stages * p.x_tile;
    static_assert(sizeof(HeadShared) <= 1024, "control block");
    plan->smem = 1024 + (size_t)p.off_ctl + 1024;
    // one CTA per (layer tile, group of images); the CTAs of a group sit next to each other in the grid
    int groups = sm_count() / p.n_tiles;
    if (groups < 1) groups = 1;
    if (groups > d.N) groups = d.N;
    p.groups = groups;
    plan->grid = groups * p.n_tiles;
    {
        // the map as a flat list of pixels [Cin][N*HW]; a box is one reduction chunk of NP pixels (the last few of them
        // the next image's, or zeros past the end)
        cuuint64_t dims[2] = {(cuuint64_t)d.Cin, (cuuint64_t)d.N * HW};
        cuuint64_t str[1] = {(cuuint64_t)d.Cin * 2};
        cuuint32_t box[2] = {64, (cuuint32_t)p.NP};
        if (!tmap_encode_16(&plan->x, 2, d.in, dims, str, box, 128, p.f16)) return SQN_ERR_CUDA;
    }
    {
        cuuint64_t dims[2] = {(cuuint64_t)d.Cin, (cuuint64_t)d.Cout};
        cuuint64_t str[1] = {(cuuint64_t)d.Cin * 2};
        cuuint32_t box[2] = {64, 128};
        if (!tmap_encode_16(&plan->w, 2, d.w, dims, str, box, 128, p.f16)) return SQN_ERR_CUDA;
    }
    return SQN_OK;
}

}  // namespace

bool fused_head_enabled()
{
    const char* v = std::getenv("SQN_FUSED_HEAD");        // read at every call: tests switch it
    return !(v && v[0] == '0');
}

// logits[n][m] = mean over the map of relu(bias[m] + 1x1 convolution): one launch, no map stored.
// SQN_ERR_UNSUPPORTED where the kernel does not apply (more than 256 pixels per image, Cin not a multiple of 64).
int launch_conv_avgpool_bf16(const ConvDesc& d, float* logits, cudaStream_t stream)
{
    HeadKey k;
    std::memset(&k, 0, sizeof(k));
    k.in = d.in; k.w = d.w; k.bias = d.bias; k.out = logits;
    int dev = 0;
    cudaGetDevice(&dev);
    const int v[8] = {d.N, d.Cin, d.H, d.W, d.Cout, d.relu | (d.params_static << 1) | (d.f16 << 2), dev, d.K | (d.S << 8) | (d.pad << 16)};
    std::memcpy(k.v, v, sizeof(v));
    const std::string key(reinterpret_cast<const char*>(&k), sizeof(k));
    HeadPlan plan;
    bool have = false;
    {
        std::lock_guard<std::mutex> lock(g_head_mu);
        auto it = g_head_plans.find(key);
        if (it != g_head_plans.end()) { plan = it->second; have = true; }
    }
    if (!have) {
        const int rc = build_head_plan(d, logits, &plan);
        if (rc != SQN_OK) return rc;
        std::lock_guard<std::mutex> lock(g_head_mu);
        if (g_head_plans.size() > 1024) g_head_plans.clear();
        g_head_plans[key] = plan;
    }
    static const cudaError_t attr_rc =
        cudaFuncSetAttribute(conv_head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CH_SMEM_LIMIT);
    if (attr_rc != cudaSuccess) return SQN_ERR_CUDA;
    const cudaError_t rc = launch_chained(conv_head_kernel, dim3((unsigned)plan.grid), dim3(CH_THREADS), plan.smem, stream, plan.x,
                                          plan.w, plan.p);
    if (rc != cudaSuccess) return SQN_ERR_CUDA;
    note_launch();
    return cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}

}  // namespace sqn
