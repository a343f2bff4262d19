// bf16 convolution layer on the 5th-generation tensor cores: implicit GEMM, operands staged in
// shared memory by TMA, accumulators in TMEM (tcgen05.mma), fused bias + ReLU + bf16 store.
//
// GEMM view (Section II of the paper): rows = output pixels, columns = output layers,
// reduction = (kernel row, kernel column, input layer).  The im2col matrix is never built:
// for every kernel tap the producer issues one TMA box load of the activation tensor whose
// start coordinate is the tile origin shifted by the tap; coordinates outside the map are
// filled with zeros by the TMA unit, which is exactly the zero padding of the layer.  With
// NHWC activations the box rows are the input layers of one pixel, contiguous in memory and
// K-major for the MMA.  A tile of output pixels is a (columns x rows x images) box, so the
// output tile is again a box and is written with one TMA store per 16/32/64-layer chunk
// straight into the layer slice [c_off, c_off+Cout) of the destination tensor; the TMA unit
// clips the parts of edge tiles that fall outside the map.
//
// One persistent CTA per SM, 6 warps:
//   warp 0 (one thread)  TMA producer: ring of `stages` {A box, B box} slots, full/empty mbarriers
//   warp 1 (one thread)  MMA issuer: tcgen05.mma 128 x BN x 16, commits free the slots;
//                        two accumulators in TMEM so tile i+1 is multiplied while tile i drains
//   warps 2..5           epilogue: tcgen05.ld (one output pixel per thread), +bias, ReLU, ->bf16,
//                        swizzled staging tile in shared memory, TMA store
// Every mbarrier wait is bounded: when it runs out the CTA records SQN_ERR_TIMEOUT in the
// device status word, drains its outstanding copies, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstring>
#include <map>
#include <mutex>
#include <string>

#include "ptx_sm100.cuh"
#include "sqn_internal.h"

namespace sqn {
namespace {

using namespace ptx;

constexpr int TILE_M = 128;            // MMA M: TMEM lanes
constexpr int NUM_THREADS = 192;
constexpr int MAX_STAGES = 8;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // about two seconds
constexpr size_t SMEM_LIMIT = 227 * 1024;

struct TcParams {
    int tiles_w, tiles_h, tiles_i;   // output-pixel tiles: columns, rows, images
    int BW, BH, BI;                  // box extents, BW*BH*BI <= 128
    int n_tiles, BN;                 // output-layer tiles and their width (multiple of 16, <= 256)
    int Cout;
    int taps, taps_w, pad;           // kernel taps, taps per kernel row, zero padding
    int chunks, BKc;                 // reduction chunks per tap, elements per chunk (16/32/64)
    int k_per_tap;                   // reduction elements per tap in the kernel matrix
    int stem;                        // 1: 7x7 stride-2 stem on the repacked input (tap = kernel row)
    int c_off;                       // first output layer inside the destination tensor
    int relu;
    int stages;
    int CW;                          // layers per TMA store (16/32/64)
    int bn_pad;                      // TMEM column stride between the two accumulators
    unsigned tmem_cols;
    unsigned a_bytes, b_bytes;       // bytes one stage's two boxes deliver
    unsigned a_tile, b_tile;         // shared-memory bytes reserved per stage for A and B
    const float* bias;
    int* status;
};

struct Shared {                       // small control block placed after the tiles
    unsigned long long full[MAX_STAGES];
    unsigned long long empty[MAX_STAGES];
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned tmem_base;
    volatile int abort_flag;
};

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t i = 1;; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 31u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
                *abort_flag = 1;
                if (status) atomicExch(status, (int)SQN_ERR_TIMEOUT);
                return false;
            }
            __nanosleep(40);
        }
    }
}

// AND-reduction of a predicate over the 128 epilogue threads (named barrier 2).
__device__ __forceinline__ bool epilogue_vote(bool ok)
{
    uint32_t all;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 2, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(all)
        : "r"((uint32_t)ok)
        : "memory");
    return all != 0;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmO, const TcParams p)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - raw);

    const uint32_t smA = base;
    const uint32_t smB = smA + (uint32_t)p.stages * p.a_tile;
    const uint32_t smStage = smB + (uint32_t)p.stages * p.b_tile;          // epilogue staging, 128 x BN bf16
    const uint32_t stage_bytes = (uint32_t)TILE_M * p.BN * 2u;
    float* bias_s = reinterpret_cast<float*>(base_ptr + (smStage - base) + stage_bytes);
    Shared* sh = reinterpret_cast<Shared*>(reinterpret_cast<unsigned char*>(bias_s) + 256 * sizeof(float));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t row_bytes = (uint32_t)p.BKc * 2u;
    const int items = p.taps * p.chunks;
    const int m_tiles = p.tiles_w * p.tiles_h * p.tiles_i;
    const int total_tiles = m_tiles * p.n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&sh->full[s]), 1);
            mbar_init(smem_u32(&sh->empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&sh->tmem_full[a]), 1);
            mbar_init(smem_u32(&sh->tmem_empty[a]), 4);
        }
        sh->abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
        prefetch_tensormap(&tmO);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&sh->tmem_base), p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    volatile int* abort_flag = &sh->abort_flag;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            int it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const int nt = t % p.n_tiles;
                const int mt = t / p.n_tiles;
                const int w0 = (mt % p.tiles_w) * p.BW;
                const int h0 = ((mt / p.tiles_w) % p.tiles_h) * p.BH;
                const int i0 = (mt / (p.tiles_w * p.tiles_h)) * p.BI;
                const int n0 = nt * p.BN;
                for (int i = 0; i < items; ++i, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
                    if (!wait_bar(smem_u32(&sh->empty[s]), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    const int tap = i / p.chunks;
                    const int x = (i - tap * p.chunks) * p.BKc;
                    const uint32_t full = smem_u32(&sh->full[s]);
                    mbar_arrive_expect_tx(full, p.a_bytes + p.b_bytes);
                    if (p.stem) {
                        // tap = kernel row kh = 2a + b: input rows are split into (pair, parity)
                        tma_load_5d(smA + s * p.a_tile, &tmA, full, 0, w0, h0 + (tap >> 1), tap & 1, i0);
                    } else {
                        const int kh = tap / p.taps_w;
                        const int kw = tap - kh * p.taps_w;
                        tma_load_5d(smA + s * p.a_tile, &tmA, full, x, w0 + kw - p.pad, h0 + kh - p.pad, i0, 0);
                    }
                    tma_load_2d(smB + s * p.b_tile, &tmB, full, tap * p.k_per_tap + x, n0);
                }
            }
            if (!ok) {
                // give the copies already issued a bounded chance to land before the CTA exits
                const int pending = it < p.stages ? it : p.stages;
                for (int j = 1; j <= pending; ++j) {
                    const int q = it - j;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(smem_u32(&sh->full[q % p.stages]), (uint32_t)(q / p.stages) & 1u)) {
                        if (clock64() - t0 > WAIT_LIMIT_CYCLES / 8) break;
                        __nanosleep(100);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(TILE_M, (uint32_t)p.BN);
            const int ksteps = p.BKc / 16;
            int it = 0, ti = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++ti) {
                const int as = ti & 1;
                const uint32_t aph = (uint32_t)(ti >> 1) & 1u;
                if (!wait_bar(smem_u32(&sh->tmem_empty[as]), aph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(as * p.bn_pad);
                for (int i = 0; i < items; ++i, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
                    if (!wait_bar(smem_u32(&sh->full[s]), ph, abort_flag, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t adesc = make_kmajor_desc(smA + s * p.a_tile, row_bytes);
                    const uint64_t bdesc = make_kmajor_desc(smB + s * p.b_tile, row_bytes);
                    for (int k = 0; k < ksteps; ++k) {
                        // 16 bf16 = 32 bytes further along the row: +2 in the (>>4) address field
                        mma_bf16_ss(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc,
                                    (i > 0 || k > 0) ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&sh->empty[s]));        // slot free once these MMAs have read it
                }
                if (ok) mma_commit(smem_u32(&sh->tmem_full[as]));   // accumulator complete
            }
        }
    } else {
        // -------------------------------------------------------------------- epilogue
        const int q = warp & 3;                        // TMEM lane quadrant this warp may read
        const int row = q * 32 + lane;                 // output pixel within the tile
        const int et = threadIdx.x - 64;               // 0..127
        const bool store_thread = (et == 0);
        const uint32_t cw_bytes = (uint32_t)p.CW * 2u;             // bytes per staging row
        const uint32_t chunk_bytes = (uint32_t)TILE_M * cw_bytes;  // one store chunk
        // TMA swizzle of width cw_bytes: 16-byte unit index XOR (row-derived bits)
        const uint32_t sw = cw_bytes == 128 ? (uint32_t)(row & 7)
                          : cw_bytes == 64 ? (uint32_t)((row >> 1) & 3) : (uint32_t)((row >> 2) & 1);
        int ti = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++ti) {
            const int nt = t % p.n_tiles;
            const int mt = t / p.n_tiles;
            const int w0 = (mt % p.tiles_w) * p.BW;
            const int h0 = ((mt / p.tiles_w) % p.tiles_h) * p.BH;
            const int i0 = (mt / (p.tiles_w * p.tiles_h)) * p.BI;
            const int n0 = nt * p.BN;
            const int as = ti & 1;
            const uint32_t aph = (uint32_t)(ti >> 1) & 1u;

            // staging and bias buffers are free once the previous tile's stores have read them
            if (store_thread) tma_store_wait_read();
            for (int c = et; c < p.BN; c += 128) bias_s[c] = (n0 + c < p.Cout) ? __ldg(p.bias + n0 + c) : 0.f;
            asm volatile("bar.sync 1, 128;" ::: "memory");

            // all 128 epilogue threads take the same decision, so nobody is left alone at a barrier
            if (!epilogue_vote(wait_bar(smem_u32(&sh->tmem_full[as]), aph, abort_flag, p.status))) { ok = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * p.bn_pad);
            for (int c = 0; c < p.BN; c += 16) {
                uint32_t v[16];
                tmem_ld_x16(taddr + (uint32_t)c, v);
                tmem_ld_wait();
                uint32_t o[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float a = __uint_as_float(v[2 * j]) + bias_s[c + 2 * j];
                    float b = __uint_as_float(v[2 * j + 1]) + bias_s[c + 2 * j + 1];
                    if (p.relu) { a = fmaxf(a, 0.f); b = fmaxf(b, 0.f); }
                    o[j] = pack_bf16x2(a, b);
                }
                const int chunk = c / p.CW;
                const int u0 = (c - chunk * p.CW) / 8;           // first of two 16-byte units
                const uint32_t rbase = smStage + (uint32_t)chunk * chunk_bytes + (uint32_t)row * cw_bytes;
                const uint32_t a0 = rbase + ((((uint32_t)u0) ^ sw) << 4);
                const uint32_t a1 = rbase + ((((uint32_t)u0 + 1u) ^ sw) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a0), "r"(o[0]), "r"(o[1]), "r"(o[2]),
                             "r"(o[3]) : "memory");
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a1), "r"(o[4]), "r"(o[5]), "r"(o[6]),
                             "r"(o[7]) : "memory");
            }
            // accumulator drained: hand it back to the MMA issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->tmem_empty[as]));
            // staging tile complete and visible to the TMA unit
            fence_proxy_async_smem();
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (store_thread) {
                for (int chunk = 0; chunk * p.CW < p.BN; ++chunk) {
                    if (n0 + chunk * p.CW >= p.Cout) break;
                    tma_store_4d(&tmO, smStage + (uint32_t)chunk * chunk_bytes, p.c_off + n0 + chunk * p.CW, w0, h0, i0);
                }
                tma_store_commit();
            }
        }
        if (store_thread) tma_store_wait_all();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

// ---------------------------------------------------------------------------- stem repack
// Input [N][H][W][3] bf16 -> [N][Hp][Wp][4] bf16, zero in the fourth layer and in the padding
// column/row, so that every pixel is 8 bytes and two pixels are one 16-byte TMA stride.
__global__ void stem_pack_input(const __nv_bfloat16* __restrict__ in, uint2* __restrict__ out, int N, int H, int W,
                                int Hp, int Wp)
{
    const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    const long long total = (long long)N * Hp * Wp;
    if (idx >= total) return;
    const int x = (int)(idx % Wp);
    const int y = (int)((idx / Wp) % Hp);
    const long long n = idx / ((long long)Wp * Hp);
    uint2 v = make_uint2(0u, 0u);
    if (x < W && y < H) {
        const unsigned short* src = reinterpret_cast<const unsigned short*>(in) + ((n * H + y) * W + x) * 3;
        v.x = (unsigned)src[0] | ((unsigned)src[1] << 16);
        v.y = (unsigned)src[2];
    }
    out[idx] = v;
}

// Kernels [Cout][7][7][3] bf16 -> [Cout][7][8][4] bf16 (zero for the eighth column and fourth layer).
__global__ void stem_pack_weights(const unsigned short* __restrict__ w, unsigned short* __restrict__ out, int Cout)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= Cout * 224) return;
    const int c = idx & 3;
    const int px = (idx >> 2) & 7;
    const int kh = (idx >> 5) % 7;
    const int m = idx / 224;
    out[idx] = (px < 7 && c < 3) ? w[((m * 7 + kh) * 7 + px) * 3 + c] : (unsigned short)0;
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

CUtensorMapSwizzle swizzle_for_bytes(unsigned row_bytes)
{
    return row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
         : row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
}

bool encode(CUtensorMap* m, int rank, const void* ptr, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
            const cuuint32_t* box, unsigned inner_bytes)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint32_t ones[5] = {1, 1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(ptr), dims, strides_bytes, box,
              ones, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for_bytes(inner_bytes), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Box of output pixels (columns x rows x images, at most 128) that wastes the fewest MMA rows.
void choose_box(int W, int H, int N, int* BW, int* BH, int* BI)
{
    double best = -1.0;
    *BW = 1; *BH = 1; *BI = 1;
    for (int bw = 1; bw <= W && bw <= TILE_M; ++bw) {
        for (int bh = 1; bh <= H && bw * bh <= TILE_M; ++bh) {
            int bi = 1;
            if (bw == W && bh == H) bi = TILE_M / (W * H) < N ? TILE_M / (W * H) : N;
            if (bi < 1) bi = 1;
            const double tiles = (double)((W + bw - 1) / bw) * ((H + bh - 1) / bh) * ((N + bi - 1) / bi);
            const double eff = (double)W * H * N / (tiles * TILE_M);
            if (eff > best + 1e-9 || (eff > best - 1e-9 && bw > *BW)) { best = eff; *BW = bw; *BH = bh; *BI = bi; }
        }
    }
}

struct Plan {
    CUtensorMap a, b, o;
    TcParams p;
    int grid;
    size_t smem;
};

int num_sms()
{
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

// Builds tensor maps and kernel parameters.  For the stem, a_ptr / w_ptr are the repacked
// tensors ([N][Hp][Wp][4] and [Cout][7][8][4]).
int build_plan(const ConvDesc& d, bool stem, const void* a_ptr, const void* w_ptr, int Hp, int Wp, Plan* plan)
{
    TcParams& p = plan->p;
    std::memset(&p, 0, sizeof(p));
    p.stem = stem ? 1 : 0;
    p.Cout = d.Cout;
    p.c_off = d.out_c_offset;
    p.relu = d.relu;
    p.bias = d.bias;
    p.status = device_status_word();
    if (stem) {
        p.taps = 7; p.taps_w = 1; p.pad = 0; p.BKc = 32; p.chunks = 1; p.k_per_tap = 32;
    } else {
        p.taps = d.K * d.K; p.taps_w = d.K; p.pad = d.pad;
        p.BKc = d.Cin % 64 == 0 ? 64 : (d.Cin % 32 == 0 ? 32 : 16);
        p.chunks = d.Cin / p.BKc;
        p.k_per_tap = d.Cin;
    }
    const unsigned row_bytes = (unsigned)p.BKc * 2u;

    // output-pixel tiling; a 1x1 layer is tiled over the flattened pixel index
    const bool flat = !stem && d.K == 1 && d.pad == 0;
    long long OWl = d.OW, OHl = d.OH, NIl = d.N;
    if (flat) { OWl = (long long)d.N * d.OH * d.OW; OHl = 1; NIl = 1; }
    if (OWl > 0x7fffffffLL) return SQN_ERR_UNSUPPORTED;
    const int OW = (int)OWl, OH = (int)OHl, NI = (int)NIl;
    if (flat) { p.BW = OW < TILE_M ? OW : TILE_M; p.BH = 1; p.BI = 1; }
    else choose_box(OW, OH, NI, &p.BW, &p.BH, &p.BI);
    p.tiles_w = (OW + p.BW - 1) / p.BW;
    p.tiles_h = (OH + p.BH - 1) / p.BH;
    p.tiles_i = (NI + p.BI - 1) / p.BI;
    const int rows = p.BW * p.BH * p.BI;

    p.BN = d.Cout <= 256 ? d.Cout : 256;
    p.n_tiles = (d.Cout + p.BN - 1) / p.BN;
    p.bn_pad = (p.BN + 31) / 32 * 32;
    unsigned cols = 32;
    while (cols < 2u * (unsigned)p.bn_pad) cols *= 2;
    p.tmem_cols = cols;
    p.CW = p.BN % 64 == 0 ? 64 : (p.BN % 32 == 0 ? 32 : 16);

    p.a_tile = (unsigned)TILE_M * row_bytes;
    p.b_tile = ((unsigned)p.BN * row_bytes + 1023u) / 1024u * 1024u;
    p.a_bytes = (unsigned)rows * row_bytes;
    p.b_bytes = (unsigned)p.BN * row_bytes;
    const size_t fixed = 1024 /*alignment slack*/ + (size_t)TILE_M * p.BN * 2 + 256 * sizeof(float) + sizeof(Shared) + 64;
    int stages = (int)((SMEM_LIMIT - fixed) / (p.a_tile + p.b_tile));
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    if (stages < 2) return SQN_ERR_UNSUPPORTED;
    p.stages = stages;
    plan->smem = fixed + (size_t)stages * (p.a_tile + p.b_tile);

    const long long total = (long long)p.tiles_w * p.tiles_h * p.tiles_i * p.n_tiles;
    if (total > 0x7fffffffLL) return SQN_ERR_UNSUPPORTED;
    plan->grid = (int)(total < num_sms() ? total : num_sms());

    // ---- tensor maps
    if (stem) {
        // [32 window elements][OW windows, 16 B apart][row pairs][row parity][image]
        const cuuint64_t row_pitch = (cuuint64_t)Wp * 8;
        cuuint64_t dims[5] = {32, (cuuint64_t)d.OW, (cuuint64_t)(Hp / 2), 2, (cuuint64_t)d.N};
        cuuint64_t str[4] = {16, 2 * row_pitch, row_pitch, (cuuint64_t)Hp * row_pitch};
        cuuint32_t box[5] = {32, (cuuint32_t)p.BW, (cuuint32_t)p.BH, 1, (cuuint32_t)p.BI};
        if (!encode(&plan->a, 5, a_ptr, dims, str, box, row_bytes)) return SQN_ERR_CUDA;
    } else if (flat) {
        cuuint64_t dims[5] = {(cuuint64_t)d.Cin, (cuuint64_t)OW, 1, 1, 1};
        const cuuint64_t s1 = (cuuint64_t)d.Cin * 2;
        cuuint64_t str[4] = {s1, s1 * OW, s1 * OW, s1 * OW};
        cuuint32_t box[5] = {(cuuint32_t)p.BKc, (cuuint32_t)p.BW, 1, 1, 1};
        if (!encode(&plan->a, 5, a_ptr, dims, str, box, row_bytes)) return SQN_ERR_CUDA;
    } else {
        cuuint64_t dims[5] = {(cuuint64_t)d.Cin, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)d.N, 1};
        const cuuint64_t s1 = (cuuint64_t)d.Cin * 2;
        cuuint64_t str[4] = {s1, s1 * d.W, s1 * d.W * d.H, s1 * d.W * d.H * d.N};
        cuuint32_t box[5] = {(cuuint32_t)p.BKc, (cuuint32_t)p.BW, (cuuint32_t)p.BH, (cuuint32_t)p.BI, 1};
        if (!encode(&plan->a, 5, a_ptr, dims, str, box, row_bytes)) return SQN_ERR_CUDA;
    }
    {
        const cuuint64_t kdim = (cuuint64_t)p.taps * p.k_per_tap;
        cuuint64_t dims[2] = {kdim, (cuuint64_t)d.Cout};
        cuuint64_t str[1] = {kdim * 2};
        cuuint32_t box[2] = {(cuuint32_t)p.BKc, (cuuint32_t)p.BN};
        if (!encode(&plan->b, 2, w_ptr, dims, str, box, row_bytes)) return SQN_ERR_CUDA;
    }
    {
        // extent of the layer dimension stops at the end of this layer's slice so that a
        // partial last tile is clipped instead of spilling into the neighbouring slice
        const cuuint64_t s1 = (cuuint64_t)d.out_c_total * 2;
        cuuint64_t dims[4] = {(cuuint64_t)(d.out_c_offset + d.Cout), (cuuint64_t)OW, (cuuint64_t)OH, (cuuint64_t)NI};
        cuuint64_t str[3] = {s1, s1 * OW, s1 * OW * OH};
        cuuint32_t box[4] = {(cuuint32_t)p.CW, (cuuint32_t)p.BW, (cuuint32_t)p.BH, (cuuint32_t)p.BI};
        if (!encode(&plan->o, 4, d.out, dims, str, box, (unsigned)p.CW * 2u)) return SQN_ERR_CUDA;
    }
    return SQN_OK;
}

int launch_plan(const Plan& plan, cudaStream_t stream)
{
    static std::once_flag once;
    static cudaError_t attr_rc = cudaSuccess;
    std::call_once(once, [] {
        attr_rc = cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT);
    });
    if (attr_rc != cudaSuccess) return SQN_ERR_CUDA;
    conv_tc_kernel<<<plan.grid, NUM_THREADS, plan.smem, stream>>>(plan.a, plan.b, plan.o, plan.p);
    note_launch();
    return cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}

// Plans are cached by the full request: encoding three tensor maps costs microseconds that a
// batch-1 forward would notice.
struct PlanKey {
    const void *in, *w, *bias, *out, *ws;
    int v[14];
};

std::mutex g_plan_mu;
std::map<std::string, Plan> g_plans;

int cached_plan(const ConvDesc& d, bool stem, const void* a_ptr, const void* w_ptr, int Hp, int Wp, const void* ws,
                Plan* out)
{
    PlanKey k;
    std::memset(&k, 0, sizeof(k));
    k.in = d.in; k.w = d.w; k.bias = d.bias; k.out = d.out; k.ws = ws;
    const int v[14] = {d.N, d.Cin, d.H, d.W, d.Cout, d.K, d.S, d.pad, d.out_c_offset, d.out_c_total, d.relu,
                       stem ? 1 : 0, Hp, Wp};
    std::memcpy(k.v, v, sizeof(v));
    int dev = 0;
    cudaGetDevice(&dev);
    std::string key(reinterpret_cast<const char*>(&k), sizeof(k));
    key.push_back((char)dev);
    {
        std::lock_guard<std::mutex> lock(g_plan_mu);
        auto it = g_plans.find(key);
        if (it != g_plans.end()) { *out = it->second; return SQN_OK; }
    }
    Plan plan;
    const int rc = build_plan(d, stem, a_ptr, w_ptr, Hp, Wp, &plan);
    if (rc != SQN_OK) return rc;
    {
        std::lock_guard<std::mutex> lock(g_plan_mu);
        if (g_plans.size() > 4096) g_plans.clear();
        g_plans[key] = plan;
    }
    *out = plan;
    return SQN_OK;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

int conv_bf16_supported(const ConvDesc& d)
{
    if (d.S != 1) return SQN_ERR_UNSUPPORTED;
    if (d.K > 7) return SQN_ERR_UNSUPPORTED;
    if (d.Cin % 16 != 0) return SQN_ERR_UNSUPPORTED;
    if (d.Cout <= 256 ? (d.Cout % 16 != 0) : (d.Cout % 8 != 0)) return SQN_ERR_UNSUPPORTED;
    if (d.out_c_offset % 8 != 0 || d.out_c_total % 8 != 0) return SQN_ERR_ALIGN;
    if (d.K == 1 && d.pad != 0) return SQN_ERR_UNSUPPORTED;
    return SQN_OK;
}

int launch_conv_bf16(const ConvDesc& d, cudaStream_t stream)
{
    Plan plan;
    const int rc = cached_plan(d, false, d.in, d.w, 0, 0, nullptr, &plan);
    if (rc != SQN_OK) return rc;
    return launch_plan(plan, stream);
}

size_t stem_bf16_workspace_bytes(int N, int H, int W, int Cout)
{
    const int Hp = (H + 1) / 2 * 2, Wp = (W + 2) / 2 * 2;
    return align_up((size_t)N * Hp * Wp * 8, 1024) + align_up((size_t)Cout * 224 * 2, 1024);
}

namespace {
int stem_check(const ConvDesc& d, void* workspace, size_t workspace_bytes)
{
    if (d.Cout % 16 != 0 || d.Cout > 256) return SQN_ERR_UNSUPPORTED;
    if (d.out_c_offset % 8 != 0 || d.out_c_total % 8 != 0) return SQN_ERR_ALIGN;
    if (!workspace || workspace_bytes < stem_bf16_workspace_bytes(d.N, d.H, d.W, d.Cout)) return SQN_ERR_WORKSPACE;
    if (!aligned16(workspace)) return SQN_ERR_ALIGN;
    return SQN_OK;
}
}  // namespace

// Repack of the stem's input and kernels into the workspace (two small launches).
int launch_stem_pack_bf16(const ConvDesc& d, void* workspace, size_t workspace_bytes, cudaStream_t stream)
{
    const int rc = stem_check(d, workspace, workspace_bytes);
    if (rc != SQN_OK) return rc;
    const int Hp = (d.H + 1) / 2 * 2, Wp = (d.W + 2) / 2 * 2;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    uint2* pin = reinterpret_cast<uint2*>(ws);
    unsigned short* pw = reinterpret_cast<unsigned short*>(ws + align_up((size_t)d.N * Hp * Wp * 8, 1024));
    const long long total = (long long)d.N * Hp * Wp;
    stem_pack_input<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(d.in), pin,
                                                                        d.N, d.H, d.W, Hp, Wp);
    stem_pack_weights<<<(d.Cout * 224 + 255) / 256, 256, 0, stream>>>(static_cast<const unsigned short*>(d.w), pw,
                                                                       d.Cout);
    note_launch(2);
    return cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}

// The stem convolution itself, on the repacked tensors left in the workspace by the call above.
int launch_stem_conv_bf16(const ConvDesc& d, void* workspace, size_t workspace_bytes, cudaStream_t stream)
{
    int rc = stem_check(d, workspace, workspace_bytes);
    if (rc != SQN_OK) return rc;
    const int Hp = (d.H + 1) / 2 * 2, Wp = (d.W + 2) / 2 * 2;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    Plan plan;
    rc = cached_plan(d, true, ws, ws + align_up((size_t)d.N * Hp * Wp * 8, 1024), Hp, Wp, workspace, &plan);
    if (rc != SQN_OK) return rc;
    return launch_plan(plan, stream);
}

}  // namespace sqn
