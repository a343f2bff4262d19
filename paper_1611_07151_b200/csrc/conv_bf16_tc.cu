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
// Persistent CTAs (one per SM, or two light ones), warp roles:
//   warp 0 (one thread)  TMA producer: ring of `stages` {A box, B box} slots, full/empty mbarriers
//   warp 1 (one lane)    MMA issuer: tcgen05.mma 128 x BN x 16, commits free the slots; the last MMA of a
//                        tile adds the bias (ones x bias rows); two accumulators in TMEM so tile i+1 is
//                        multiplied while tile i drains
//   4*SPLIT warps        epilogue: tcgen05.ld (one output pixel per thread), ReLU, ->bf16,
//                        swizzled staging tile in shared memory
//   last warp            TMA stores of the staged chunks
// Every mbarrier wait is bounded: when it runs out the CTA records SQN_ERR_TIMEOUT in the
// device status word, drains its outstanding copies, frees its TMEM and returns.
//
// Kernels in this file: conv_tc_kernel (one layer), conv_tc_kernel2 (two independent layers, e.g. the two
// expands of a fire layer, in one grid), conv_pool_kernel / conv_pool_kernel2 / conv_pool_kernel4 (convolution with the following
// 3x3/2 max-pool: output layers on the TMEM lanes, pool taken in registers), stem_pack (repack of the stem's
// 3-layer input and kernels).  The kernel bodies are __device__ functions of (tensor maps, parameters, CTA index).
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <cstddef>
#include <mutex>
#include <string>

#include "ptx_sm100.cuh"
#include "sqn_internal.h"
#include "tc_common.cuh"
#include "tc_host.h"

namespace sqn {
namespace {

using namespace ptx;

constexpr int TILE_M = 128;            // MMA M: TMEM lanes
// Threads per CTA: producer warp, MMA warp, 4*SPLIT epilogue warps, store warp.  SPLIT = 2: one CTA per SM
// (large tiles, kernels resident in up to 227 KB); SPLIT = 1: two lighter CTAs per SM, i.e. two MMA issuers,
// two producers and two store threads per SM, for the layers whose tiles are small.
__host__ __device__ constexpr int threads_for(int split) { return 96 + 128 * split; }
constexpr int MAX_STAGES = 8;
constexpr int MAX_STG = 4;             // staging ring slots
constexpr int MAX_TAB = 448;           // MMAs per tile in patch mode
constexpr int PARAM_TAB = 160;         // ... of which this many can be tabulated in the kernel parameters
constexpr size_t CTL_BYTES = 4096;
constexpr size_t CTL_BYTES_NO_TAB = 1024;   // control block without the shared-memory MMA table
constexpr size_t SMEM_LIMIT = 227 * 1024;
constexpr size_t SMEM_LIMIT_2CTA = 113 * 1024;     // two CTAs share an SM's 228 KB (1 KB reserved each)

struct TcParams {
    int tiles_w, tiles_h, tiles_i;   // output-pixel tiles: columns, rows, images
    int BW, BH, BI;                  // box extents, BW*BH*BI <= 128
    int n_tiles, BN;                 // output-layer tiles and their width (multiple of 16, <= 256)
    int total_tiles;
    int reverse;                     // 1: tiles are taken from the last to the first (see build_plan_cfg)
    int grid;                        // CTAs working on this layer (the launch may hold a second layer's CTAs as well)
    int g_nt, g_tw, g_th, g_ti;      // `grid` written in the mixed radix (n_tiles, tiles_w, tiles_h, tiles_i)
    int Cout;
    int taps, taps_w, pad;           // kernel taps, taps per kernel row, zero padding
    int chunks, BKc;                 // reduction chunks per tap, elements per chunk (16/32/64)
    int k_per_tap;                   // reduction elements per tap in the kernel matrix
    int patch;                       // 1: one input patch per tile serves every tap (see below)
    int taps_h;                      // kernel rows
    unsigned tap_h_bytes, tap_w_bytes;   // patch bytes to skip per kernel row / kernel column
    int a_lines;                     // 1 (stem): the patch is whole input lines, not swizzled; MMA row j of a line
                                     // starts 16 bytes (two pixels of four layers) after row j-1, so rows overlap
    int h_mul;                       // input rows per output row (2 for the stride-2 stem)
    unsigned sbo_bytes;              // patch bytes between consecutive groups of 8 output pixels
    unsigned patch_tile;             // shared-memory bytes reserved per reduction chunk of a patch
    int c_off;                       // first output layer inside the destination tensor
    int relu;
    int stages;                      // A (or A+B) ring slots
    int b_resident;                  // 1: all kernel tiles are loaded once and stay in shared memory
    int bias_in_k;                   // 1 (stem): the bias sits in two unused places of the repacked kernels and meets a
                                     // constant 1 in the fourth layer of the repacked image: no bias MMA
    int b_early;                     // 1: kernels and bias are not written by the kernel this launch is chained to, so
                                     // they are fetched before the wait for that kernel (0 for the stem: its kernels
                                     // are repacked by the launch before it)
    int CW;                          // layers per TMA store (16/32/64)
    int nstg;                        // staging ring slots (2 or 4)
    int bn_pad;                      // TMEM column stride between the two accumulators
    unsigned tmem_cols;
    unsigned a_bytes, b_bytes;       // bytes one item's A box / B box delivers
    unsigned a_tile, b_tile;         // shared-memory bytes reserved per A / B tile
    unsigned off_b, off_stg, off_bias, off_ones, off_ctl;   // byte offsets from the 1024-aligned base
    // fused 3x3/stride-2 max-pool (conv_pool_kernel): a CTA walks the tiles of a strip of output rows from
    // left to right and emits pooled pixels directly
    int pool;                        // 1: write max-pooled output instead of the convolution's own
    int h_step;                      // output rows between consecutive tile rows (BH, or 30 when pooling)
    int PW_out, PH_out;              // pooled extents
    int pool_ctot;                   // layers per pixel of the pooled tensor
    __nv_bfloat16* pool_out;
    int npix;                        // conv_pool_kernel: pixels per tile, 256 or 128
    int two_issuers;                 // ... 1 (no rider): warp 18 issues the odd tiles' MMAs (the ring then has an even number of slots)
    int f16;                         // 1: the 16-bit type is fp16, 0: bf16
    // conv_pool_kernel: a second layer, 1x1 on the same input with as many output layers, that rides on this layer's
    // patches: its MMAs read the centre of the same patch and fill an accumulator of their own, and the epilogue pools
    // both (the 1x1 expand of a fire layer beside the 3x3 expand)
    int rider;
    int r_nmma;                      // the rider's MMAs per tile
    unsigned r_off_b, r_off_bias;    // its kernels (chunks tiles of Cout rows) and bias rows in shared memory
    unsigned r_b_bytes;              // bytes of its kernels
    int r_c_off;                     // its first output layer in the pooled tensor
    const float* r_bias;
    uint2 r_ptab[8];                 // per MMA {patch offset, kernel offset from r_off_b}, 16-byte units
    const float* bias;
    int* status;
    // patch mode, at most PARAM_TAB MMAs per tile: per MMA {A offset from the stage base, B offset from the
    // kernel region} in 16-byte units.  Read from the constant bank, i.e. with warp-uniform loads.
    int use_ptab;
    uint2 ptab[PARAM_TAB];
};

struct Shared {                       // control block placed after the tiles
    unsigned long long full[MAX_STAGES];
    unsigned long long empty[MAX_STAGES];
    unsigned long long b_full;
    unsigned long long tmem_full[4];      // (conv_pool_kernel with a rider: two accumulators per layer)
    unsigned long long tmem_empty[4];
    unsigned long long stg_full[MAX_STG];
    unsigned long long stg_free[MAX_STG];
    unsigned tmem_base;
    volatile int abort_flag;
    uint2 mma_tab[MAX_TAB + 1];           // patch mode: per MMA, {A offset from the stage base, B address} in 16-byte units
};

// Position of a tile in (output-layer tile, column tile, row tile, image tile) digits.  A CTA
// walks tiles bid, bid + grid, ...; the step is added digit by digit, so the
// loops below contain no integer division.
struct TileCoord { int nt, tw, th, ti; };

__device__ __forceinline__ void tile_first(const TcParams& p, int t, TileCoord& c)
{
    if (p.pool) {                 // t is a strip: (row tile, image)
        c.nt = 0; c.tw = 0;
        c.th = t % p.tiles_h;
        c.ti = t / p.tiles_h;
        return;
    }
    if (p.reverse) t = p.total_tiles - 1 - t;
    c.nt = t % p.n_tiles;
    const int mt = t / p.n_tiles;
    c.tw = mt % p.tiles_w;
    const int r = mt / p.tiles_w;
    c.th = r % p.tiles_h;
    c.ti = r / p.tiles_h;
}
__device__ __forceinline__ void tile_next(const TcParams& p, TileCoord& c)
{
    int carry = 0;
    if (p.pool) {                 // left to right inside the strip, then this CTA's next strip
        if (++c.tw < p.tiles_w) return;
        c.tw = 0;
        c.th += p.g_th;
        if (c.th >= p.tiles_h) { c.th -= p.tiles_h; carry = 1; }
        c.ti += p.g_ti + carry;
        return;
    }
    if (p.reverse) {              // the same step downwards, with borrows
        c.nt -= p.g_nt;
        if (c.nt < 0) { c.nt += p.n_tiles; carry = 1; }
        c.tw -= p.g_tw + carry; carry = 0;
        if (c.tw < 0) { c.tw += p.tiles_w; carry = 1; }
        c.th -= p.g_th + carry; carry = 0;
        if (c.th < 0) { c.th += p.tiles_h; carry = 1; }
        c.ti -= p.g_ti + carry;
        return;
    }
    c.nt += p.g_nt;
    if (c.nt >= p.n_tiles) { c.nt -= p.n_tiles; carry = 1; }
    c.tw += p.g_tw + carry; carry = 0;
    if (c.tw >= p.tiles_w) { c.tw -= p.tiles_w; carry = 1; }
    c.th += p.g_th + carry; carry = 0;
    if (c.th >= p.tiles_h) { c.th -= p.tiles_h; carry = 1; }
    c.ti += p.g_ti + carry;
}
// Number of tiles CTA `bid` of the layer's `grid` CTAs processes (it takes tiles, or strips of tiles_w tiles,
// bid + k*grid).
__device__ __forceinline__ int tiles_of_cta(const TcParams& p, int bid)
{
    const int units = p.pool ? p.tiles_h * p.tiles_i : p.total_tiles;
    if (bid >= units) return 0;
    const int mine = (units - bid + p.grid - 1) / p.grid;
    return p.pool ? mine * p.tiles_w : mine;
}

// Every kernel tile of the layer, once, into the resident region (one mbarrier counts all of them).
__device__ __forceinline__ void load_resident_kernels(const TcParams& p, const CUtensorMap& tmB, uint32_t smB, uint32_t bar, int items)
{
    mbar_arrive_expect_tx(bar, (uint32_t)items * p.b_bytes);
    int tap = 0, ch = 0;
    for (int i = 0; i < items; ++i) {
        tma_load_2d(smB + (uint32_t)i * p.b_tile, &tmB, bar, tap * p.k_per_tap + ch * p.BKc, 0);
        if (++ch == p.chunks) { ch = 0; ++tap; }
    }
}

// Bias rows of the bias MMA: one 32-byte row {hi, lo, 0, ...} per output layer, hi + lo = the fp32 bias.
template <int NUM_THREADS>
__device__ __forceinline__ void fill_bias_rows(const TcParams& p, unsigned char* base_ptr)
{
    uint4* rows = reinterpret_cast<uint4*>(base_ptr + p.off_bias);
    for (int c = threadIdx.x; c < p.n_tiles * p.BN; c += NUM_THREADS) bias_row(rows, c, c < p.Cout ? __ldg(p.bias + c) : 0.f, p.f16);
}

// HC: output layers per epilogue piece (8, 16 or 32; a store chunk CW is two pieces), fixed at compile time so
// that the conversion loop is straight-line code.
template <int SPLIT, int HC, bool F16>
__device__ __forceinline__ void conv_tc_body(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmO,
                                             const TcParams& p, const int bid)
{
    constexpr int NUM_THREADS = threads_for(SPLIT);
    constexpr int EPI_WARPS = 4 * SPLIT;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - raw);

    const uint32_t smA = base;
    const uint32_t smB = base + p.off_b;
    const uint32_t smStg = base + p.off_stg;
    Shared* sh = reinterpret_cast<Shared*>(base_ptr + p.off_ctl);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t row_bytes = (uint32_t)p.BKc * 2u;
    const int items = p.taps * p.chunks;
    const int nchunks = p.BN / p.CW;
    const int my_tiles = tiles_of_cta(p, bid);

    // The launch is chained to the kernel before it in the stream: this block may be running while
    // that grid drains.  Up to chain_wait() below it touches only its own shared memory, TMEM, the
    // kernel parameters and, when b_early is set, the layer's kernels and bias (which that grid does not
    // write): a CTA that starts in the tail of the layer before has its kernels resident by the time
    // the first input tile may be read.  The grid after this one is let go by warp 1 once this CTA
    // holds its TMEM (see below).
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&sh->full[s]), 1);
            mbar_init(smem_u32(&sh->empty[s]), 1);
        }
        mbar_init(smem_u32(&sh->b_full), 1);
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&sh->tmem_full[a]), 1);
            mbar_init(smem_u32(&sh->tmem_empty[a]), EPI_WARPS);
        }
        for (int b = 0; b < p.nstg; ++b) {
            mbar_init(smem_u32(&sh->stg_full[b]), EPI_WARPS);
            mbar_init(smem_u32(&sh->stg_free[b]), 1);
        }
        sh->abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
        prefetch_tensormap(&tmO);
        if (p.b_resident && p.b_early) load_resident_kernels(p, tmB, smB, smem_u32(&sh->b_full), items);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&sh->tmem_base), p.tmem_cols);
        tmem_relinquish();
        // Only now may the next grid in the stream be scheduled: every CTA of a grid that has let its
        // dependents go already holds its TMEM, so a CTA waiting in tcgen05.alloc can only be waiting for
        // columns of grids that do not wait for it.
        chain_release();
    }
    if (p.patch && !p.use_ptab) {
        // operand addresses of every MMA of a tile, in issue order (tap-major, then chunk, then k-step)
        const int ksteps = p.BKc / 16;
        for (int e = threadIdx.x; e < items * ksteps; e += NUM_THREADS) {
            const int k = e % ksteps, it = e / ksteps;
            const int ch = it % p.chunks, tap = it / p.chunks;
            const int kw = tap % p.taps_w, kh = tap / p.taps_w;
            const uint32_t a_off = (uint32_t)ch * p.patch_tile + (uint32_t)kh * p.tap_h_bytes + (uint32_t)kw * p.tap_w_bytes;
            sh->mma_tab[e] = make_uint2((a_off >> 4) + 2u * k, ((smB + (uint32_t)it * p.b_tile) >> 4) + 2u * k);
        }
    }
    // The bias is added by the tensor core: the last MMA of every tile multiplies a tile of ones
    // (128 rows, K = 16: ones in the first two places) by the bias rows (one per output layer:
    // {hi, lo, 0, ...} with hi + lo = bias to 16 bits below its leading bit).  Both tiles have
    // 32-byte rows in the 32-byte swizzle: 16-byte unit u of row r sits at unit u ^ ((r >> 2) & 1).
    {
        uint4* ones = reinterpret_cast<uint4*>(base_ptr + p.off_ones);
        for (int r = threadIdx.x; r < TILE_M; r += NUM_THREADS) {
            const int u = (r >> 2) & 1;
            ones[2 * r + u] = make_uint4(one_x2(p.f16), 0u, 0u, 0u);
            ones[2 * r + (u ^ 1)] = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    if (p.b_early) fill_bias_rows<NUM_THREADS>(p, base_ptr);
    chain_wait();       // the earlier grid has finished: global memory may be read and written from here on
    if (!p.b_early) fill_bias_rows<NUM_THREADS>(p, base_ptr);
    fence_proxy_async_smem();           // the MMA reads the ones and the bias rows through the async proxy
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    volatile int* abort_flag = &sh->abort_flag;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            bool ok = true;
            // every kernel tile, once: they stay in shared memory for all tiles of this CTA
            if (p.b_resident && !p.b_early) load_resident_kernels(p, tmB, smB, smem_u32(&sh->b_full), items);
            const uint32_t tx = p.b_resident ? p.a_bytes : p.a_bytes + p.b_bytes;
            int s = 0, issued = 0;
            uint32_t ph = 0;
            TileCoord tc;
            tile_first(p, bid, tc);
            for (int it = 0; it < my_tiles && ok; ++it, tile_next(p, tc)) {
                const int w0 = tc.tw * p.BW, h0 = tc.th * p.h_step, i0 = tc.ti * p.BI, n0 = tc.nt * p.BN;
                if (p.patch) {
                    // one box per reduction chunk covers the tile plus its halo; every tap reads from it
                    if (!wait_bar(smem_u32(&sh->empty[s]), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    const uint32_t full = smem_u32(&sh->full[s]);
                    mbar_arrive_expect_tx(full, p.a_bytes);
                    if (p.a_lines)     // stem: 22 pixels of (2*BH+5) input lines, starting at pixel 2*w0 of line 2*h0
                        tma_load_5d(smA + (uint32_t)s * p.a_tile, &tmA, full, 8 * w0, 2 * h0, i0, 0, 0);
                    else
                        for (int ch = 0; ch < p.chunks; ++ch)
                            tma_load_5d(smA + (uint32_t)s * p.a_tile + (uint32_t)ch * p.patch_tile, &tmA, full, ch * p.BKc,
                                        w0 - p.pad, h0 * p.h_mul - p.pad, i0, 0);
                    ++issued;
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                    continue;
                }
                int tap = 0, kh = 0, kw = 0, ch = 0;
                for (int i = 0; i < items; ++i) {
                    if (!wait_bar(smem_u32(&sh->empty[s]), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    const uint32_t full = smem_u32(&sh->full[s]);
                    const int x = ch * p.BKc;
                    mbar_arrive_expect_tx(full, tx);
                    tma_load_5d(smA + (uint32_t)s * p.a_tile, &tmA, full, x, w0 + kw - p.pad, h0 + kh - p.pad, i0, 0);
                    if (!p.b_resident)
                        tma_load_2d(smB + (uint32_t)s * p.b_tile, &tmB, full, tap * p.k_per_tap + x, n0);
                    ++issued;
                    if (++ch == p.chunks) {
                        ch = 0; ++tap;
                        if (++kw == p.taps_w) { kw = 0; ++kh; }
                    }
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
            }
            if (!ok) {
                // give the copies already issued a bounded chance to land before the CTA exits
                int pending = issued < p.stages ? issued : p.stages;
                while (pending-- > 0) {
                    if (s == 0) { s = p.stages; ph ^= 1u; }
                    --s;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(smem_u32(&sh->full[s]), ph)) {
                        if (clock64() - t0 > WAIT_LIMIT_CYCLES / 8) break;
                        __nanosleep(100);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // The whole warp walks the loop converged (all lanes wait on the barriers) and one elected
        // lane issues the MMAs and their commits.  With the operand offsets read from the kernel
        // parameters everything the issuing instruction needs is warp-uniform, which is what lets the
        // MMAs go out back to back (about 55 clocks each for N <= 128, the tensor pipe's own rate; a
        // single diverged thread reading a shared-memory table needs about 100).
        const uint32_t idesc = make_idesc_bf16(TILE_M, (uint32_t)p.BN, (uint32_t)p.f16);
        const int ksteps = p.BKc / 16;
        const uint32_t hiA = p.a_lines ? (uint32_t)(make_kmajor_desc_plain(0, 16u, p.sbo_bytes) >> 32)
                                       : (uint32_t)(make_kmajor_desc(0, row_bytes, p.patch ? p.sbo_bytes : 8u * row_bytes) >> 32);
        const uint32_t hiB = (uint32_t)(make_kmajor_desc(0, row_bytes, 8u * row_bytes) >> 32);
        const uint32_t a_tile16 = p.a_tile >> 4, b_tile16 = p.b_tile >> 4;
        const uint32_t smA16 = smA >> 4, smB16 = smB >> 4;
        const int nmma = items * ksteps;
        // bias MMA: ones tile x bias rows of the tile's output layers (32 bytes = 2 address units per row)
        const uint64_t bias_da = make_kmajor_desc(base + p.off_ones, 32u, 256u);
        const uint64_t bias_db0 = make_kmajor_desc(base + p.off_bias, 32u, 256u);
        bool ok = true;
        if (p.b_resident) ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->b_full), 0u, abort_flag, p.status));
        int s = 0, as = 0;
        uint32_t ph = 0, aph = 0;
        TileCoord tc;
        tile_first(p, bid, tc);
        for (int it = 0; it < my_tiles && ok; ++it, tile_next(p, tc)) {
            const uint64_t bias_db = bias_db0 + (uint64_t)(2 * tc.nt * p.BN);
            ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->tmem_empty[as]), aph ^ 1u, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(as * p.bn_pad);
            if (p.patch) {
                ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->full[s]), ph, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
                // output pixel (g, j) of the tile reads patch row g*(rows per line) + j + tap offset
                const uint32_t a_base = smA16 + (uint32_t)s * a_tile16;
                if (elect_one()) {
                    if (p.use_ptab) {
                        uint32_t acc = 0u;
#pragma unroll 2
                        for (int e = 0; e < nmma; ++e) {
                            const uint2 o = p.ptab[e];
                            mma_bf16_ss(d_tmem, ((uint64_t)hiA << 32) | (uint64_t)((a_base + o.x) | 0x10000u),
                                        ((uint64_t)hiB << 32) | (uint64_t)((smB16 + o.y) | 0x10000u), idesc, acc);
                            acc = 1u;
                        }
                    } else {
                        uint2 o = sh->mma_tab[0];
                        uint32_t acc = 0u;
#pragma unroll 2
                        for (int e = 1; e <= nmma; ++e) {
                            const uint2 nxt = sh->mma_tab[e];        // one entry ahead (the table has a spare slot)
                            mma_bf16_ss(d_tmem, ((uint64_t)hiA << 32) | (uint64_t)((a_base + o.x) | 0x10000u),
                                        ((uint64_t)hiB << 32) | (uint64_t)(o.y | 0x10000u), idesc, acc);
                            acc = 1u;
                            o = nxt;
                        }
                    }
                    mma_commit(smem_u32(&sh->empty[s]));            // patch slot free once these MMAs have read it
                    if (!p.bias_in_k) mma_bf16_ss(d_tmem, bias_da, bias_db, idesc, 1u);
                    mma_commit(smem_u32(&sh->tmem_full[as]));       // accumulator complete
                }
                __syncwarp();
                if (++s == p.stages) { s = 0; ph ^= 1u; }
            } else {
                uint32_t bres16 = smB16;
                for (int i = 0; i < items; ++i, bres16 += b_tile16) {
                    ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->full[s]), ph, abort_flag, p.status));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a16 = smA16 + (uint32_t)s * a_tile16;
                    const uint32_t b16 = p.b_resident ? bres16 : smB16 + (uint32_t)s * b_tile16;
                    if (elect_one()) {
                        // ksteps MMAs of K = 16 (32 bytes = 2 address units along the row)
                        const uint64_t da = ((uint64_t)hiA << 32) | (uint64_t)(a16 | 0x10000u);
                        const uint64_t db = ((uint64_t)hiB << 32) | (uint64_t)(b16 | 0x10000u);
                        mma_bf16_ss(d_tmem, da, db, idesc, i > 0 ? 1u : 0u);
                        if (ksteps >= 2) mma_bf16_ss(d_tmem, da + 2, db + 2, idesc, 1u);
                        if (ksteps == 4) {
                            mma_bf16_ss(d_tmem, da + 4, db + 4, idesc, 1u);
                            mma_bf16_ss(d_tmem, da + 6, db + 6, idesc, 1u);
                        }
                        mma_commit(smem_u32(&sh->empty[s]));        // slot free once these MMAs have read it
                        if (i == items - 1) {
                            mma_bf16_ss(d_tmem, bias_da, bias_db, idesc, 1u);
                            mma_commit(smem_u32(&sh->tmem_full[as]));           // accumulator complete
                        }
                    }
                    __syncwarp();
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
            }
            if (++as == 2) { as = 0; aph ^= 1u; }
        }
    } else if (warp < 2 + EPI_WARPS) {
        // -------------------------------------------------------------------- epilogue
        // 4*SPLIT warps: warp w reads TMEM lane quadrant w % 4 (one output pixel per thread) and, of
        // every chunk of CW layers, the piece(s) given by (w - 2) / 4.  TMEM -> registers (bias already added by the last MMA), ReLU, -> bf16,
        // into a slot of the staging ring (TMA-swizzled rows); the store warp sends the slot to
        // global memory while the next chunk is converted.
        const int q = warp & 3;
        constexpr int PIECES = SPLIT < 2 ? 2 : SPLIT;  // a chunk is converted in this many pieces
        constexpr int NH = PIECES / SPLIT;             // pieces each thread converts per chunk (2 when SPLIT == 1)
        const int half0 = ((warp - 2) >> 2) * NH;      // first piece of this warp
        const int row = q * 32 + lane;
        const uint32_t cw_bytes = (uint32_t)p.CW * 2u;
        const uint32_t slot_bytes = (uint32_t)TILE_M * cw_bytes;
        const uint32_t sw = cw_bytes == 128 ? (uint32_t)(row & 7)
                          : cw_bytes == 64 ? (uint32_t)((row >> 1) & 3) : (uint32_t)((row >> 2) & 1);
        constexpr int hc = HC;                         // layers per piece: 8, 16 or 32 (CW / PIECES)
        bool ok = true;
        int as = 0, sb = 0;
        uint32_t aph = 0, sph = 0;
        TileCoord tc;
        tile_first(p, bid, tc);
        for (int it = 0; it < my_tiles && ok; ++it, tile_next(p, tc)) {
            const int n0 = tc.nt * p.BN;
            ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->tmem_full[as]), aph, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * p.bn_pad);
            for (int chunk = 0; chunk < nchunks; ++chunk) {
                const int c0 = chunk * p.CW;
                if (n0 + c0 >= p.Cout) break;
                uint32_t v[NH][32];
#pragma unroll
                for (int h = 0; h < NH; ++h) {
                    const uint32_t ta = taddr + (uint32_t)(c0 + (half0 + h) * hc);
                    if (hc == 32) {
                        tmem_ld_x16(ta, *reinterpret_cast<uint32_t(*)[16]>(&v[h][0]));
                        tmem_ld_x16(ta + 16u, *reinterpret_cast<uint32_t(*)[16]>(&v[h][16]));
                    } else if (hc == 16) {
                        tmem_ld_x16(ta, *reinterpret_cast<uint32_t(*)[16]>(&v[h][0]));
                    } else {
                        tmem_ld_x8(ta, *reinterpret_cast<uint32_t(*)[8]>(&v[h][0]));
                    }
                }
                ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->stg_free[sb]), sph ^ 1u, abort_flag, p.status));
                tmem_ld_wait();
                if (!ok) break;
                const uint32_t rbase = smStg + (uint32_t)sb * slot_bytes + (uint32_t)row * cw_bytes;
#pragma unroll
                for (int h = 0; h < NH; ++h) {
                    const int col_h = (half0 + h) * hc;
                    const uint32_t u_h = (uint32_t)(col_h >> 3);       // first 16-byte unit of this half-chunk
                    uint32_t o[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        if (2 * j < hc) {
                            const float f0 = __uint_as_float(v[h][2 * j]), f1 = __uint_as_float(v[h][2 * j + 1]);
                            o[j] = p.relu ? pack_relu_x2(f0, f1, F16) : pack_x2(f0, f1, F16);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {                       // 8 layers = one 16-byte unit
                        if (8 * u < hc) {
                            const uint32_t addr = rbase + (((u_h + (uint32_t)u) ^ sw) << 4);
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(o[4 * u]),
                                         "r"(o[4 * u + 1]), "r"(o[4 * u + 2]), "r"(o[4 * u + 3]));
                        }
                    }
                }
                fence_proxy_async_smem();             // staging rows visible to the TMA unit
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh->stg_full[sb]));
                if (++sb == p.nstg) { sb = 0; sph ^= 1u; }
            }
            if (!ok) break;
            // accumulator drained: hand it back to the MMA issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->tmem_empty[as]));
            if (++as == 2) { as = 0; aph ^= 1u; }
        }
    } else {
        // ----------------------------------------------------------------- store issuer
        if (lane == 0) {
            const uint32_t slot_bytes = (uint32_t)TILE_M * (uint32_t)p.CW * 2u;
            bool ok = true;
            int sb = 0, pend = 0, fb = 0;       // next slot, stores whose slot is not yet released, next slot to release
            uint32_t sph = 0;
            TileCoord tc;
            tile_first(p, bid, tc);
            for (int it = 0; it < my_tiles && ok; ++it, tile_next(p, tc)) {
                const int w0 = tc.tw * p.BW, h0 = tc.th * p.h_step, i0 = tc.ti * p.BI, n0 = tc.nt * p.BN;
                for (int chunk = 0; chunk < nchunks; ++chunk) {
                    const int c0 = chunk * p.CW;
                    if (n0 + c0 >= p.Cout) break;
                    if (!wait_bar(smem_u32(&sh->stg_full[sb]), sph, abort_flag, p.status)) { ok = false; break; }
                    if (sqn_dbg_ok(n0 + c0 < p.Cout && w0 < p.tiles_w * p.BW && h0 < p.tiles_h * p.BH && i0 < p.tiles_i * p.BI && sb < p.nstg, p.status))
                    tma_store_4d(&tmO, smStg + (uint32_t)sb * slot_bytes, p.c_off + n0 + c0, w0, h0, i0);
                    tma_store_commit();
                    if (++sb == p.nstg) { sb = 0; sph ^= 1u; }
                    // a slot is free again once its store has finished reading shared memory:
                    // keep nstg-1 stores in flight, release the oldest
                    if (++pend == p.nstg) {
                        if (p.nstg == 4) asm volatile("cp.async.bulk.wait_group.read 3;" ::: "memory");
                        else if (p.nstg == 3) asm volatile("cp.async.bulk.wait_group.read 2;" ::: "memory");
                        else asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                        mbar_arrive(smem_u32(&sh->stg_free[fb]));
                        if (++fb == p.nstg) fb = 0;
                        --pend;
                    }
                }
            }
            tma_store_wait_all();
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

// One layer per launch, or two independent layers that read the same input (the two expands of a fire layer):
// the first p0.grid CTAs work on the first, the others on the second, so the second fills the tail of the first
// and the pair costs one launch.
template <int SPLIT, int HC>
__global__ void __launch_bounds__(threads_for(SPLIT), SPLIT == 1 ? 2 : 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmO, const __grid_constant__ TcParams p)
{
    // (the 16-bit type is a compile-time constant of the body: the epilogue's conversion loop is straight-line code)
    if (p.f16) conv_tc_body<SPLIT, HC, true>(tmA, tmB, tmO, p, (int)blockIdx.x);
    else conv_tc_body<SPLIT, HC, false>(tmA, tmB, tmO, p, (int)blockIdx.x);
}

template <int SPLIT, int HC>
__global__ void __launch_bounds__(threads_for(SPLIT), SPLIT == 1 ? 2 : 1)
conv_tc_kernel2(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
                const __grid_constant__ CUtensorMap tmO0, const __grid_constant__ TcParams p0,
                const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1,
                const __grid_constant__ CUtensorMap tmO1, const __grid_constant__ TcParams p1)
{
    if (p0.f16) {
        if ((int)blockIdx.x < p0.grid) conv_tc_body<SPLIT, HC, true>(tmA0, tmB0, tmO0, p0, (int)blockIdx.x);
        else conv_tc_body<SPLIT, HC, true>(tmA1, tmB1, tmO1, p1, (int)blockIdx.x - p0.grid);
    } else {
        if ((int)blockIdx.x < p0.grid) conv_tc_body<SPLIT, HC, false>(tmA0, tmB0, tmO0, p0, (int)blockIdx.x);
        else conv_tc_body<SPLIT, HC, false>(tmA1, tmB1, tmO1, p1, (int)blockIdx.x - p0.grid);
    }
}

// ------------------------------------------------------------------- convolution + 3x3/2 max-pool
// The same implicit GEMM with the roles of the operands exchanged: D[layer][pixel] = sum_k W[layer][k] * X[pixel][k].
// The kernels of the layer are the A operand (M = 128 rows = output layers, resident in shared memory), the 256
// pixels of a tile (8 columns x 32 rows, pixel = 8 * row + column) are the B operand, read from the shared-memory
// patch through the same shifted descriptors as in conv_tc_kernel, and the accumulator has the output layers on the
// TMEM lanes and the pixels on its 256 columns.  An epilogue thread therefore owns one output layer and sees all
// pixels of the tile: the 3x3/2 max-pool is taken in its registers and nothing of it goes through shared memory.
// One MMA covers 256 pixels, so a tile needs half as many instructions (and per-tile hand-overs) per pixel as the
// 128-pixel tiles of conv_tc_kernel, which is what bounds these layers with few output layers.
// A CTA walks a strip of 32 output rows (strips 30 rows apart: 15 pooled rows) from left to right; tile k emits the
// pooled columns 4k-1 .. 4k+2, the vertical maxima of its last two columns are carried to tile k+1 in registers.
// Warps: 0 TMA producer, 1 MMA issuer, 18 the rider's MMA issuer, 2..17 epilogue (lane quadrant = warp % 4; the four
// groups of four warps take four (128-pixel tiles: two) pooled rows of the strip each, the last group one fewer).
// The bias is added by one more MMA (bias rows {hi, lo} x tile of ones).  Lanes past the last output layer compute on
// whatever follows the kernels in shared memory and are never read.
// With a rider (a 1x1 layer on the same input) the tiles are 128 pixels: the layer's tiles take three accumulators of
// 128 columns in turn, the rider's the fourth, and the rider's MMAs come from a warp of their own -- with one thread
// issuing both, and one accumulator for the layer, the layer's MMAs, its pooling and the rider's MMAs ran one after
// the other (fire4 + pool4: 84 us; 75 us so).
constexpr int POOLT_THREADS = 64 + 512 + 32;
constexpr int POOLT_RIDER_WARP = 18;           // issues the rider's MMAs (idle without a rider)
__host__ __device__ constexpr int poolt_rows(int npix) { return npix / 8; }                 // output rows per tile
__host__ __device__ constexpr int poolt_prows(int npix) { return (npix / 8 - 2) / 2; }      // pooled rows per strip

// NPIX = 256 (8 x 32 pixels per tile, 15 pooled rows per strip) where the layer's kernels leave room for the larger
// patches, else 128 (8 x 16 pixels, 7 pooled rows).
// CTOT: the layers per pixel of the pooled tensor as a compile-time constant (0: read from the parameters) -- the
// four stores of a pooled row then differ by immediate offsets.
template <int NPIX, bool F16, int CTOT>
__device__ __forceinline__ void conv_pool_body(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB2,
                                               const TcParams& p, const int bid)
{
    constexpr int PROWS = poolt_prows(NPIX);          // 15 or 7
    constexpr int PR = (PROWS + 3) / 4;               // pooled rows per epilogue group: 4 or 2
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - raw);
    const uint32_t smA = base + p.off_stg;          // pixel patches (ring of p.stages slots)
    const uint32_t smB = base + p.off_b;            // the layer's kernels
    Shared* sh = reinterpret_cast<Shared*>(base_ptr + p.off_ctl);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t row_bytes = (uint32_t)p.BKc * 2u;
    const int items = p.taps * p.chunks;
    const int nmma = items * (p.BKc / 16);
    const int my_tiles = tiles_of_cta(p, bid);
    const int n_acc = p.rider ? 3 : 2;              // accumulators of the layer itself
    // every kernel tile of the layer (and of its rider), once: one mbarrier counts them all
    auto load_kernels = [&]() {
        const uint32_t bar = smem_u32(&sh->b_full);
        mbar_arrive_expect_tx(bar, (uint32_t)items * p.b_bytes + (p.rider ? p.r_b_bytes : 0u));
        int tap = 0, ch = 0;
        for (int i = 0; i < items; ++i) {
            tma_load_2d(smB + (uint32_t)i * p.b_tile, &tmB, bar, tap * p.k_per_tap + ch * p.BKc, 0);
            if (++ch == p.chunks) { ch = 0; ++tap; }
        }
        if (p.rider)
            for (int c = 0; c < p.chunks; ++c) tma_load_2d(base + p.r_off_b + (uint32_t)c * p.b_tile, &tmB2, bar, c * p.BKc, 0);
    };
    auto fill_bias = [&]() {
        fill_bias_rows<POOLT_THREADS>(p, base_ptr);
        if (p.rider) {
            uint4* rows = reinterpret_cast<uint4*>(base_ptr + p.r_off_bias);
            for (int c = threadIdx.x; c < TILE_M; c += POOLT_THREADS) bias_row(rows, c, c < p.Cout ? __ldg(p.r_bias + c) : 0.f, p.f16);
        }
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&sh->full[s]), 1);
            mbar_init(smem_u32(&sh->empty[s]), p.rider ? 2 : 1);      // (a rider's issuer reads the patch too)
        }
        mbar_init(smem_u32(&sh->b_full), 1);
        for (int a = 0; a < 4; ++a) {
            mbar_init(smem_u32(&sh->tmem_full[a]), 1);
            mbar_init(smem_u32(&sh->tmem_empty[a]), 4 * ((p.Cout + 31) / 32));     // the epilogue warps that have output layers
        }
        sh->abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
        if (p.b_early) load_kernels();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&sh->tmem_base), p.tmem_cols);
        tmem_relinquish();
        // Only now may the next grid in the stream be scheduled: every CTA of a grid that has let its
        // dependents go already holds its TMEM, so a CTA waiting in tcgen05.alloc can only be waiting for
        // columns of grids that do not wait for it.
        chain_release();
    }
    {
        // tile of ones for the bias MMA: 256 rows of 32 bytes in the 32-byte swizzle, ones in the first two places
        uint4* ones = reinterpret_cast<uint4*>(base_ptr + p.off_ones);
        for (int r = threadIdx.x; r < NPIX; r += POOLT_THREADS) {
            const int u = (r >> 2) & 1;
            ones[2 * r + u] = make_uint4(one_x2(p.f16), 0u, 0u, 0u);
            ones[2 * r + (u ^ 1)] = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    if (p.b_early) fill_bias();
    chain_wait();       // the earlier grid has finished: its output may be read from here on
    if (!p.b_early) fill_bias();
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    volatile int* abort_flag = &sh->abort_flag;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer: one patch per tile
        if (lane == 0) {
            if (!p.b_early) load_kernels();
            bool ok = true;
            int s = 0, issued = 0;
            uint32_t ph = 0;
            TileCoord tc;
            tile_first(p, bid, tc);
            for (int it = 0; it < my_tiles; ++it, tile_next(p, tc)) {
                const int w0 = tc.tw * p.BW, h0 = tc.th * p.h_step, i0 = tc.ti;
                if (!wait_bar(smem_u32(&sh->empty[s]), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                const uint32_t full = smem_u32(&sh->full[s]);
                mbar_arrive_expect_tx(full, p.a_bytes);
                if (p.a_lines)
                    tma_load_5d(smA + (uint32_t)s * p.a_tile, &tmA, full, 8 * w0, 2 * h0, i0, 0, 0);
                else
                    for (int ch = 0; ch < p.chunks; ++ch)
                        tma_load_5d(smA + (uint32_t)s * p.a_tile + (uint32_t)ch * p.patch_tile, &tmA, full, ch * p.BKc,
                                    w0 - p.pad, h0 - p.pad, i0, 0);
                ++issued;
                if (++s == p.stages) { s = 0; ph ^= 1u; }
            }
            if (!ok) {
                int pending = issued < p.stages ? issued : p.stages;
                while (pending-- > 0) {
                    if (s == 0) { s = p.stages; ph ^= 1u; }
                    --s;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(smem_u32(&sh->full[s]), ph)) {
                        if (clock64() - t0 > WAIT_LIMIT_CYCLES / 8) break;
                        __nanosleep(100);
                    }
                }
            }
        }
    } else if (warp == 1 || (warp == POOLT_RIDER_WARP && p.two_issuers)) {
        // ------------------------------------------------------------------ MMA issuer(s)
        // Between a tile's last MMA and the next tile's first the issuing thread spends some 500 clocks on barriers,
        // fences and commits, more than the tensor pipe's queue holds: without a rider the warp that would issue the
        // rider's MMAs takes the odd tiles, so that one thread's hand-shakes fall into the other's MMAs.  Each issuer
        // keeps count of ring slot and accumulator of all tiles.  A wait on a barrier must not be two phases ahead of
        // it: with an even number of ring slots and two accumulators an issuer only meets slots and accumulators whose
        // previous tile was its own.
        const int step = p.two_issuers ? 2 : 1, first = warp == 1 ? 0 : 1;
        const uint32_t idesc = make_idesc_bf16(TILE_M, NPIX, (uint32_t)p.f16);
        const uint32_t hiX = p.a_lines ? (uint32_t)(make_kmajor_desc_plain(0, 16u, p.sbo_bytes) >> 32)
                                       : (uint32_t)(make_kmajor_desc(0, row_bytes, p.sbo_bytes) >> 32);
        const uint32_t hiW = (uint32_t)(make_kmajor_desc(0, row_bytes, 8u * row_bytes) >> 32);
        const uint32_t a_tile16 = p.a_tile >> 4, smA16 = smA >> 4, smB16 = smB >> 4;
        const uint64_t bias_desc = make_kmajor_desc(base + p.off_bias, 32u, 256u);
        const uint64_t ones_desc = make_kmajor_desc(base + p.off_ones, 32u, 256u);
        bool ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->b_full), 0u, abort_flag, p.status));
        // The tiles take the layer's accumulators in turn: two, or with a rider (128-pixel tiles) three, the rider's few
        // MMAs going to the fourth.  From the commit of a tile's MMAs to the issuer seeing its accumulator free again
        // (MMA drain, the epilogue's wake-up and TMEM loads, the way back) is about as long as two such tiles' MMAs.
        // The rider's MMAs are issued by a warp of their own: with 64 clocks per MMA issuing, not the tensor pipe, is
        // what a single thread is bound by.
        int s = first, as = first;              // (two issuers: at least two ring slots, two accumulators)
        uint32_t ph = 0, aph = 0;
        for (int it = first; it < my_tiles && ok; it += step) {
            ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->tmem_empty[as]), aph ^ 1u, abort_flag, p.status));
            if (!ok) break;
            ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->full[s]), ph, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(as * NPIX);
            const uint32_t x_base = smA16 + (uint32_t)s * a_tile16;
            if (elect_one()) {
                uint32_t acc = 0u;
#pragma unroll 2
                for (int e = 0; e < nmma; ++e) {
                    const uint2 o = p.ptab[e];
                    mma_bf16_ss(d_tmem, ((uint64_t)hiW << 32) | (uint64_t)((smB16 + o.y) | 0x10000u),
                                ((uint64_t)hiX << 32) | (uint64_t)((x_base + o.x) | 0x10000u), idesc, acc);
                    acc = 1u;
                }
                mma_commit(smem_u32(&sh->empty[s]));                // patch slot free once these MMAs (and the rider's) have read it
                if (!p.bias_in_k) mma_bf16_ss(d_tmem, bias_desc, ones_desc, idesc, 1u);
                mma_commit(smem_u32(&sh->tmem_full[as]));           // accumulator complete
            }
            __syncwarp();
            as += step;
            if (as >= n_acc) { as -= n_acc; aph ^= 1u; }
            s += step;
            if (s >= p.stages) { s -= p.stages; ph ^= 1u; }
        }
    } else if (warp == POOLT_RIDER_WARP) {
        // ------------------------------------------------------------------ the rider's MMA issuer
        // the rider's tile from the same patch (its centre tap), into an accumulator of the rider's own
        if (p.rider) {
            const uint32_t idesc = make_idesc_bf16(TILE_M, NPIX, (uint32_t)p.f16);
            const uint32_t hiX = (uint32_t)(make_kmajor_desc(0, row_bytes, p.sbo_bytes) >> 32);
            const uint32_t hiW = (uint32_t)(make_kmajor_desc(0, row_bytes, 8u * row_bytes) >> 32);
            const uint32_t a_tile16 = p.a_tile >> 4, smA16 = smA >> 4, smR16 = (base + p.r_off_b) >> 4;
            const uint64_t bias_desc = make_kmajor_desc(base + p.r_off_bias, 32u, 256u);
            const uint64_t ones_desc = make_kmajor_desc(base + p.off_ones, 32u, 256u);
            bool ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->b_full), 0u, abort_flag, p.status));
            int s = 0;
            uint32_t ph = 0;
            for (int it = 0; it < my_tiles && ok; ++it) {
                const int ar = 3;
                const uint32_t aph = (uint32_t)it & 1u;
                ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->tmem_empty[ar]), aph ^ 1u, abort_flag, p.status));
                if (!ok) break;
                ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->full[s]), ph, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
                const uint32_t d2 = tmem_base + (uint32_t)(ar * NPIX);
                const uint32_t x_base = smA16 + (uint32_t)s * a_tile16;
                if (elect_one()) {
                    uint32_t acc = 0u;
                    for (int e = 0; e < p.r_nmma; ++e) {
                        const uint2 o = p.r_ptab[e];
                        mma_bf16_ss(d2, ((uint64_t)hiW << 32) | (uint64_t)((smR16 + o.y) | 0x10000u),
                                    ((uint64_t)hiX << 32) | (uint64_t)((x_base + o.x) | 0x10000u), idesc, acc);
                        acc = 1u;
                    }
                    mma_commit(smem_u32(&sh->empty[s]));
                    mma_bf16_ss(d2, bias_desc, ones_desc, idesc, 1u);
                    mma_commit(smem_u32(&sh->tmem_full[ar]));
                }
                __syncwarp();
                if (++s == p.stages) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp < POOLT_RIDER_WARP) {
        // -------------------------------------------------------------------- epilogue: pool in registers
        // group g = (warp - 2) / 4 takes the pooled rows PR*g .. PR*g + PR-1 of the strip (group 3: one fewer), i.e.
        // the rows 2*PR*g .. 2*PR*g + 2*PR of the tile = accumulator columns 16*PR*g .. 16*PR*g + 16*PR + 7
        const int q = warp & 3, grp = (warp - 2) >> 2;
        const int m = q * 32 + lane;
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        const bool live = m < p.Cout, warp_live = q * 32 < p.Cout;
        const bool warp_full = q * 32 + 32 <= p.Cout && p.relu != 0;      // (and the layer has a ReLU: the common case's stores carry no predicates)
        const int ctot = CTOT ? CTOT : p.pool_ctot;
        const int row_stride = p.PW_out * ctot;                    // elements between pooled rows
        float carry[PR][2], carry2[PR][2];              // (carry2: the rider's)
#pragma unroll
        for (int r = 0; r < PR; ++r) carry[r][0] = carry[r][1] = carry2[r][0] = carry2[r][1] = 0.f;
        bool ok = true;
        int eas = 0;
        uint32_t eaph = 0;
        TileCoord tc;
        tile_first(p, bid, tc);
        // accumulator `as` -> pooled pixels of one layer; `cr` carries the vertical maxima of the tile's last two columns
        auto pool_tile = [&](float (&cr)[PR][2], const int c_off, const int as, const uint32_t aph) {
            ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->tmem_full[as]), aph, abort_flag, p.status));
            if (!ok) return;
            tc_fence_after();
            const uint32_t taddr = tmem_base + lane_base + (uint32_t)(as * NPIX) + (uint32_t)(grp * 16 * PR);
            const int pw0 = tc.tw * 4 - 1, ph0 = tc.th * PROWS + grp * PR;
            unsigned short* dst0 = reinterpret_cast<unsigned short*>(p.pool_out) +
                                   (((size_t)tc.ti * p.PH_out + ph0) * p.PW_out + pw0) * ctot + c_off + m;
            const bool first = pw0 >= 0 && pw0 < p.PW_out, last3 = pw0 + 3 < p.PW_out, last2 = pw0 + 2 < p.PW_out,
                       last1 = pw0 + 1 < p.PW_out;
            const bool inner = warp_full && pw0 >= 0 && last3;       // all four pooled columns of the tile exist (the same for the whole warp)
            // One pooled row per step: its three tile rows are the last row of the step before (still in registers) and
            // two new ones (16 accumulator columns).  The load of step r + 1 is issued before the maxima of step r are
            // taken, so that only the first load's latency is exposed; three buffers rotate (the step before, this one,
            // the one in flight).  The last group has one pooled row -- one step -- fewer.
            const int nsteps = grp == 3 ? PR - 1 : PR;
            uint32_t row0[8], buf[3][16];
            tmem_ld_x8(taddr, row0);
            tmem_ld_x16(taddr + 8u, buf[0]);
            tmem_ld_wait_x8(row0);
            tmem_ld_wait_x16(buf[0]);
            auto release = [&]() {          // accumulator in registers: hand it back to the MMA issuer
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh->tmem_empty[as]));
            };
            if (nsteps == 1) release();
#pragma unroll
            for (int r = 0; r < PR; ++r) {
                if (r >= nsteps) break;
                const bool more = r + 1 < nsteps;
                if (more) tmem_ld_x16(taddr + 8u + (uint32_t)(16 * (r + 1)), buf[(r + 1) % 3]);
                const uint32_t* top = r == 0 ? &row0[0] : &buf[(r + 2) % 3][8];         // (row 2r: the last row of the step before)
                const uint32_t(&cur)[16] = buf[r % 3];
                float c[8];
#pragma unroll
                for (int j = 0; j < 8; ++j)                             // vertical maximum of rows 2r, 2r+1, 2r+2, column j
                    c[j] = max3(__uint_as_float(top[j]), __uint_as_float(cur[j]), __uint_as_float(cur[8 + j]));
                const float o0 = max3(cr[r][0], cr[r][1], c[0]), o1 = max3(c[0], c[1], c[2]),
                            o2 = max3(c[2], c[3], c[4]), o3 = max3(c[4], c[5], c[6]);
                cr[r][0] = c[6];
                cr[r][1] = c[7];
                if (inner) {
                    if (ph0 + r < p.PH_out && sqn_dbg_ok(tc.ti < p.tiles_i && c_off + m < ctot, p.status)) {
                        // (two values per conversion: a single-value conversion costs the pipe as much as the pair)
                        unsigned short* dst = dst0 + r * row_stride;
                        const uint32_t o01 = pack_relu_x2(o0, o1, F16), o23 = pack_relu_x2(o2, o3, F16);
                        dst[0] = (unsigned short)(o01 & 0xffffu);
                        dst[ctot] = (unsigned short)(o01 >> 16);
                        dst[2 * ctot] = (unsigned short)(o23 & 0xffffu);
                        dst[3 * ctot] = (unsigned short)(o23 >> 16);
                    }
                } else if (live && ph0 + r < p.PH_out && sqn_dbg_ok(tc.ti < p.tiles_i && c_off + m < ctot, p.status)) {
                    unsigned short* dst = dst0 + r * row_stride;
                    if (first) dst[0] = to_16_bits(o0, p.relu, F16);
                    if (last1) dst[ctot] = to_16_bits(o1, p.relu, F16);
                    if (last2) dst[2 * ctot] = to_16_bits(o2, p.relu, F16);
                    if (last3) dst[3 * ctot] = to_16_bits(o3, p.relu, F16);
                }
                if (more) {
                    tmem_ld_wait_x16(buf[(r + 1) % 3]);
                    if (r + 2 == nsteps) release();                     // that was the accumulator's last load
                }
            }
        };
        // (warps whose lanes lie past the last output layer have nothing to do and are not counted by tmem_empty)
        for (int it = 0; it < my_tiles && ok && warp_live; ++it, tile_next(p, tc)) {
            pool_tile(carry, p.c_off, eas, eaph);
            if (++eas == n_acc) { eas = 0; eaph ^= 1u; }
            if (p.rider && ok) pool_tile(carry2, p.r_c_off, 3, (uint32_t)it & 1u);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

// (tile size, 16-bit type and -- for the pooled tensors of SqueezeNet -- the layers per pixel are compile-time constants of the body)
template <int NPIX>
__device__ __forceinline__ void pool_body(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB2, const TcParams& p,
                                          const int bid)
{
    if (p.f16) conv_pool_body<NPIX, true, 0>(tmA, tmB, tmB2, p, bid);
    else if (p.pool_ctot == 256) conv_pool_body<NPIX, false, 256>(tmA, tmB, tmB2, p, bid);
    else if (NPIX == 256 && p.pool_ctot == 96) conv_pool_body<NPIX, false, 96>(tmA, tmB, tmB2, p, bid);
    else if (NPIX == 128 && p.pool_ctot == 512) conv_pool_body<NPIX, false, 512>(tmA, tmB, tmB2, p, bid);
    else conv_pool_body<NPIX, false, 0>(tmA, tmB, tmB2, p, bid);
}

__global__ void __launch_bounds__(POOLT_THREADS, 1)
conv_pool_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ TcParams p)
{
    if (p.npix == 256) pool_body<256>(tmA, tmB, tmB2, p, (int)blockIdx.x);
    else pool_body<128>(tmA, tmB, tmB2, p, (int)blockIdx.x);
}

// Two pooled layers (each possibly with its rider) over the same input in one launch (see conv_tc_kernel2).
__global__ void __launch_bounds__(POOLT_THREADS, 1)
conv_pool_kernel2(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
                  const __grid_constant__ CUtensorMap tmR0, const __grid_constant__ TcParams p0,
                  const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1,
                  const __grid_constant__ CUtensorMap tmR1, const __grid_constant__ TcParams p1)
{
    if (p0.npix == 256) {           // (both layers have the same tile size)
        if ((int)blockIdx.x < p0.grid) pool_body<256>(tmA0, tmB0, tmR0, p0, (int)blockIdx.x);
        else pool_body<256>(tmA1, tmB1, tmR1, p1, (int)blockIdx.x - p0.grid);
    } else {
        if ((int)blockIdx.x < p0.grid) pool_body<128>(tmA0, tmB0, tmR0, p0, (int)blockIdx.x);
        else pool_body<128>(tmA1, tmB1, tmR1, p1, (int)blockIdx.x - p0.grid);
    }
}

// Four pooled layers over the same input in one launch (the two 128-layer slices of both expands of fire8).
__global__ void __launch_bounds__(POOLT_THREADS, 1)
conv_pool_kernel4(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
                  const __grid_constant__ TcParams p0, const __grid_constant__ CUtensorMap tmA1,
                  const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ TcParams p1,
                  const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2,
                  const __grid_constant__ TcParams p2, const __grid_constant__ CUtensorMap tmA3,
                  const __grid_constant__ CUtensorMap tmB3, const __grid_constant__ TcParams p3)
{
    int b = (int)blockIdx.x;                       // (all four layers have 128-pixel tiles)
    if (b < p0.grid) { pool_body<128>(tmA0, tmB0, tmB0, p0, b); return; }
    b -= p0.grid;
    if (b < p1.grid) { pool_body<128>(tmA1, tmB1, tmB1, p1, b); return; }
    b -= p1.grid;
    if (b < p2.grid) { pool_body<128>(tmA2, tmB2, tmB2, p2, b); return; }
    pool_body<128>(tmA3, tmB3, tmB3, p3, b - p2.grid);
}

// ---------------------------------------------------------------------------- stem repack
// Input [N][H][W][3] bf16 -> [N][Hp][Wp][4] bf16, 1.0 in the fourth layer of the image's pixels, zero in the padding
// column/row, so that every pixel is 8 bytes and two pixels are one 16-byte unit.
// A block repacks PACK_ROWS rows: each row (6*W bytes, only 2-byte aligned) is brought into shared memory with
// 16-byte loads from the enclosing aligned range -- all loads of a thread are issued before the first is used, so a
// block has its whole input in flight at once -- then every thread writes four pixels (32 bytes) at a time.
// Loads never leave [in, in + in_elems): the units that straddle an end of the tensor are read by halfwords.
constexpr int PACK_ROWS = 16;
// The blocks past the first `row_blocks` repack the layer's kernels [Cout][7][7][3] -> [Cout][7][8][4] (zero for
// the eighth column and fourth layer, except that the fourth layer of the first two pixels of the first kernel row
// holds the bias as hi + lo: with the constant 1 of the repacked image the convolution itself adds the bias), so that the stem needs one repack launch.
__global__ void __launch_bounds__(256) stem_pack(const __nv_bfloat16* __restrict__ in, uint4* __restrict__ out, int N, int H, int W,
                                                 int Hp, int Wp, long long in_elems, int pitch, int row_blocks,
                                                 const unsigned short* __restrict__ w, unsigned short* __restrict__ w_out, int Cout,
                                                 const float* __restrict__ bias, int f16)
{
    chain_release();
    chain_wait();
    if ((int)blockIdx.x >= row_blocks) {
        const int idx = ((int)blockIdx.x - row_blocks) * 256 + (int)threadIdx.x;
        if (idx >= Cout * 224) return;
        const int c = idx & 3;
        const int px = (idx >> 2) & 7;
        const int kh = (idx >> 5) % 7;
        const int m = idx / 224;
        unsigned short v = (px < 7 && c < 3) ? w[((m * 7 + kh) * 7 + px) * 3 + c] : (unsigned short)0;
        if (c == 3 && kh == 0 && px < 2) {          // fourth layer of the first two pixels of the first kernel row: bias hi, lo
            const uint32_t hl = bias_hi_lo(__ldg(bias + m), f16);
            v = px == 0 ? (unsigned short)(hl & 0xffffu) : (unsigned short)(hl >> 16);
        }
        w_out[idx] = v;
        return;
    }
    extern __shared__ __align__(16) unsigned short rows_s[];
    constexpr int RPT = PACK_ROWS / 4;                             // rows per thread group (64 threads share a row)
    const int r0 = threadIdx.x >> 6, i = threadIdx.x & 63;
    // over N * Hp, last rows first: the stem kernel that follows starts with the first rows, then still in the L2
    const long long row_base = ((long long)row_blocks - 1 - blockIdx.x) * PACK_ROWS;
    const long long total_rows = (long long)N * Hp;
    const unsigned long long lo = reinterpret_cast<unsigned long long>(in), hi = lo + 2ull * (unsigned long long)in_elems;
    int shift[RPT];                                                // halfwords between the aligned start and the row
    const int row_units = pitch / 8;                               // 16-byte units staged per row
    for (int u0 = 0; u0 < row_units; u0 += 128) {                  // (one round for rows up to 2 KB)
        uint4 v[RPT][2];
#pragma unroll
        for (int k = 0; k < RPT; ++k) {
            const long long rowid = row_base + r0 + 4 * k;
            const int y = rowid < total_rows ? (int)(rowid % Hp) : H;
            const long long n = rowid < total_rows ? rowid / Hp : 0;
            shift[k] = 0;
            v[k][0] = v[k][1] = make_uint4(0u, 0u, 0u, 0u);
            if (y < H) {
                const unsigned long long b0 = lo + 6ull * (unsigned long long)((n * H + y) * W);
                const unsigned long long a0 = b0 & ~15ull;
                shift[k] = (int)((b0 - a0) >> 1);
                const int units = (2 * shift[k] + 6 * W + 15) / 16;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int u = u0 + i + 64 * h;
                    if (u >= units) continue;
                    const unsigned long long a = a0 + 16ull * u;
                    if (a >= lo && a + 16 <= hi) {
                        v[k][h] = __ldg(reinterpret_cast<const uint4*>(a));
                    } else {
                        unsigned short e[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const unsigned long long ah = a + 2ull * j;
                            e[j] = (ah >= lo && ah + 2 <= hi) ? __ldg(reinterpret_cast<const unsigned short*>(ah)) : (unsigned short)0;
                        }
                        v[k][h] = make_uint4((unsigned)e[0] | ((unsigned)e[1] << 16), (unsigned)e[2] | ((unsigned)e[3] << 16),
                                             (unsigned)e[4] | ((unsigned)e[5] << 16), (unsigned)e[6] | ((unsigned)e[7] << 16));
                    }
                }
            }
        }
#pragma unroll
        for (int k = 0; k < RPT; ++k) {
            uint4* rs = reinterpret_cast<uint4*>(rows_s + (size_t)(r0 + 4 * k) * pitch);
            if (u0 + i < row_units) rs[u0 + i] = v[k][0];
            if (u0 + i + 64 < row_units) rs[u0 + i + 64] = v[k][1];
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < RPT; ++k) {
        const long long rowid = row_base + r0 + 4 * k;
        if (rowid >= total_rows) continue;
        const int y = (int)(rowid % Hp);
        const long long n = rowid / Hp;
        const unsigned short* rs = rows_s + (size_t)(r0 + 4 * k) * pitch;
        for (int x0 = 4 * i; x0 < Wp; x0 += 256) {
            unsigned short e[12];
#pragma unroll
            for (int j = 0; j < 12; ++j) e[j] = (y < H && x0 + j / 3 < W) ? rs[shift[k] + 3 * x0 + j] : (unsigned short)0;
            uint4* dst = out + ((n * Hp + y) * Wp + x0) / 2;           // two pixels per 16 bytes (Wp is even)
            // fourth layer of a pixel of the image: 1.0 (it meets the bias in the repacked kernels), else 0
            unsigned one[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) one[q] = (y < H && x0 + q < W) ? (one_x2(f16) & 0xffff0000u) : 0u;
            dst[0] = make_uint4((unsigned)e[0] | ((unsigned)e[1] << 16), (unsigned)e[2] | one[0],
                                (unsigned)e[3] | ((unsigned)e[4] << 16), (unsigned)e[5] | one[1]);
            if (x0 + 2 < Wp)
                dst[1] = make_uint4((unsigned)e[6] | ((unsigned)e[7] << 16), (unsigned)e[8] | one[2],
                                    (unsigned)e[9] | ((unsigned)e[10] << 16), (unsigned)e[11] | one[3]);
        }
    }
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
         : row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
         : row_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
}

thread_local int t_f16 = 0;      // element type of the tensor maps being encoded: 0 bf16, 1 fp16

bool encode(CUtensorMap* m, int rank, const void* ptr, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
            const cuuint32_t* box, unsigned inner_bytes)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint32_t ones[5] = {1, 1, 1, 1, 1};
    return fn(m, t_f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(ptr), dims, strides_bytes, box,
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
    CUtensorMap r;   // the rider's kernels (conv_pool_kernel), else a copy of b
    TcParams p;
    int grid;
    int halves;      // 1 = two light CTAs per SM, 2 = one CTA per SM
    int split;       // epilogue warps / 4 of the kernel variant: 1 or 2
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
// Shared-memory layout for one candidate (store chunk width, staging slots); returns the number
// of A stages that fit (0 if the candidate does not fit at all).
thread_local size_t t_smem_limit = SMEM_LIMIT;   // budget the layout search below works against
thread_local int t_pool_npix = 256;              // conv_pool_kernel: pixels per tile the plan is built for (256 or 128)
thread_local const ConvDesc* t_rider = nullptr;  // conv_pool_kernel: the 1x1 layer that rides on the plan's layer (see TcParams::rider)
thread_local int t_force_cw = 0;                 // != 0: only layouts with this store chunk width (see launch_conv_bf16_pair)

int fit_stages(TcParams& p, size_t a_tile, bool want_resident, int cw, int nstg, bool smem_tab, size_t* smem_bytes)
{
    const size_t SMEM_LIMIT = t_smem_limit;
    const int items = p.taps * p.chunks;
    const size_t slot = (size_t)TILE_M * cw * 2;
    // bias rows (32 bytes per output layer) followed by the tile of ones (128 rows of 32 bytes)
    const size_t bias_rows = ((size_t)p.n_tiles * p.BN * 32 + 1023) / 1024 * 1024;
    const size_t bias_bytes = bias_rows + (size_t)TILE_M * 32;
    // the MMA operand table at the end of the control block is only needed when it does not fit the parameters
    const size_t ctl_bytes = smem_tab ? CTL_BYTES : CTL_BYTES_NO_TAB;
    static_assert(sizeof(Shared) <= CTL_BYTES && offsetof(Shared, mma_tab) <= CTL_BYTES_NO_TAB, "control block");
    if (SMEM_LIMIT < 1024 + bias_bytes + ctl_bytes) return 0;
    const size_t avail = SMEM_LIMIT - 1024 /*alignment slack*/ - bias_bytes - ctl_bytes;
    const size_t stg_bytes = (size_t)nstg * slot;
    const size_t b_all = (size_t)items * p.b_tile;
    int stages;
    size_t b_region;
    if (want_resident) {
        if (p.n_tiles != 1 || b_all + stg_bytes + 2 * a_tile > avail) return 0;
        stages = (int)((avail - b_all - stg_bytes) / a_tile);
        if (stages > MAX_STAGES) stages = MAX_STAGES;
        b_region = b_all;
    } else {
        if (stg_bytes + 2 * (a_tile + p.b_tile) > avail) return 0;
        stages = (int)((avail - stg_bytes) / (a_tile + p.b_tile));
        if (stages > MAX_STAGES) stages = MAX_STAGES;
        b_region = (size_t)stages * p.b_tile;
    }
    p.b_resident = want_resident ? 1 : 0;
    p.stages = stages;
    p.CW = cw;
    p.nstg = nstg;
    p.a_tile = (unsigned)a_tile;
    p.off_b = (unsigned)((size_t)stages * a_tile);
    p.off_stg = p.off_b + (unsigned)b_region;
    p.off_bias = p.off_stg + (unsigned)stg_bytes;
    p.off_ones = p.off_bias + (unsigned)bias_rows;
    p.off_ctl = p.off_bias + (unsigned)bias_bytes;
    *smem_bytes = 1024 + (size_t)p.off_ctl + ctl_bytes;
    return stages;
}

// Tries the staging candidates in order of preference; true when one gives at least min_stages.
bool choose_layout(TcParams& p, size_t a_tile, bool want_resident, int min_stages, bool smem_tab, size_t* smem_bytes)
{
    static const int cand[][2] = {{64, 4}, {64, 3}, {32, 4}, {64, 2}, {32, 3}, {32, 2}, {16, 4}, {16, 2}};
    for (const auto& c : cand) {
        if (p.BN % c[0] != 0 || (t_force_cw != 0 && c[0] != t_force_cw)) continue;
        if (fit_stages(p, a_tile, want_resident, c[0], c[1], smem_tab, smem_bytes) >= min_stages) return true;
    }
    return false;
}

// Shared memory of conv_pool_kernel: the layer's kernels (tiles of Cout rows; an MMA reads 128 rows from a tile's
// start, the rows past Cout come from the tiles and patches behind it), the patch ring, bias rows, the tile of ones,
// the control block.
int pool_issuers_env();

bool pool_layout(TcParams& p, size_t a_tile, size_t* smem_bytes)
{
    const size_t items = (size_t)p.taps * p.chunks;
    const size_t w_bytes = items * p.b_tile;
    // (a rider adds its kernels -- one tile of Cout rows per reduction chunk -- and its bias rows)
    const size_t r_bytes = p.rider ? (size_t)p.chunks * p.b_tile + (size_t)TILE_M * 32 : 0;
    const size_t fixed = 1024 /*alignment slack*/ + w_bytes + r_bytes + (size_t)TILE_M * 32 + (size_t)p.npix * 32 + CTL_BYTES_NO_TAB;
    if (t_smem_limit < fixed + 2 * a_tile) return false;
    size_t stages = (t_smem_limit - fixed) / a_tile;
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    p.two_issuers = p.rider ? 0 : 1;
    if (pool_issuers_env() == 1) p.two_issuers = 0;
    if (p.two_issuers) stages &= ~(size_t)1;        // (an even number of ring slots: see the issuers)
    // the 128-row read of the last kernel tile must stay inside the patch ring
    if ((size_t)TILE_M * p.BKc * 2 > p.b_tile + stages * a_tile) return false;
    p.stages = (int)stages;
    p.a_tile = (unsigned)a_tile;
    p.b_resident = 1;
    p.off_b = 0;
    p.off_stg = (unsigned)w_bytes;
    p.off_bias = p.off_stg + (unsigned)(stages * a_tile);
    p.off_ones = p.off_bias + (unsigned)TILE_M * 32;
    p.off_ctl = p.off_ones + (unsigned)p.npix * 32;
    if (p.rider) {
        p.r_off_bias = p.off_ctl;
        p.r_off_b = p.r_off_bias + (unsigned)TILE_M * 32;
        p.off_ctl = p.r_off_b + (unsigned)((size_t)p.chunks * p.b_tile);
        // (the 128-row read of the rider's last kernel tile ends inside the control block or the slack behind it)
    }
    *smem_bytes = 1024 + (size_t)p.off_ctl + CTL_BYTES_NO_TAB;
    return true;
}

// Builds tensor maps and kernel parameters.  For the stem, a_ptr / w_ptr are the repacked
// tensors ([N][Hp][Wp][4] and [Cout][7][8][4]).
int build_plan_cfg(const ConvDesc& d, bool stem, const void* a_ptr, const void* w_ptr, int Hp, int Wp, int halves,
                   Plan* plan)
{
    TcParams& p = plan->p;
    std::memset(&p, 0, sizeof(p));
    plan->halves = halves;
    plan->split = halves;
    t_smem_limit = halves == 1 ? SMEM_LIMIT_2CTA : SMEM_LIMIT;
    p.f16 = d.f16;
    t_f16 = d.f16;
    p.Cout = d.Cout;
    p.c_off = d.out_c_offset;
    p.relu = d.relu;
    p.bias = d.bias;
    p.status = device_status_word();
    p.h_mul = 1;
    p.b_early = (d.params_static && (!stem || d.stem_prepacked)) ? 1 : 0;   // (the stem's kernels are otherwise repacked by the launch before it)
    p.bias_in_k = stem ? 1 : 0;
    p.pool = d.pool ? 1 : 0;
    if (p.pool && (d.OH < 3 || d.OW < 3 || d.Cout % 32 != 0 || d.Cout > TILE_M)) return SQN_ERR_UNSUPPORTED;
    const ConvDesc* rider = p.pool ? t_rider : nullptr;
    if (rider) {
        if (stem || d.Cout != TILE_M || rider->Cout != d.Cout || rider->Cin != d.Cin || rider->K != 1 || rider->S != 1 || rider->pad != 0 ||
            rider->in != d.in || rider->H != d.H || rider->W != d.W || rider->N != d.N || rider->out != d.out ||
            rider->out_c_total != d.out_c_total || rider->relu != d.relu || !rider->pool || rider->out_c_offset % 8 != 0)
            return SQN_ERR_UNSUPPORTED;
        p.rider = 1;
    }
    if (stem) {
        p.taps = 7; p.taps_h = 7; p.taps_w = 1; p.pad = 0; p.BKc = 32; p.chunks = 1; p.k_per_tap = 32;
    } else {
        p.taps = d.K * d.K; p.taps_h = d.K; p.taps_w = d.K; p.pad = d.pad;
        p.BKc = d.Cin % 64 == 0 ? 64 : (d.Cin % 32 == 0 ? 32 : 16);
        p.chunks = d.Cin / p.BKc;
        p.k_per_tap = d.Cin;
    }
    const unsigned row_bytes = (unsigned)p.BKc * 2u;

    p.BN = d.Cout <= 256 ? d.Cout : 256;
    p.n_tiles = (d.Cout + p.BN - 1) / p.BN;
    p.bn_pad = (p.BN + 31) / 32 * 32;
    unsigned cols = 32;
    while (cols < 2u * (unsigned)p.bn_pad) cols *= 2;
    p.tmem_cols = cols;
    if (halves == 1 && (cols > 256 || d.pool)) return SQN_ERR_UNSUPPORTED;   // two CTAs share the SM's 512 TMEM columns
    p.b_tile = ((unsigned)p.BN * row_bytes + 1023u) / 1024u * 1024u;
    p.b_bytes = (unsigned)p.BN * row_bytes;
    if (p.pool) {
        // conv_pool_kernel: the kernels are the M = 128 operand; their tiles hold Cout rows and the rows past them
        // belong to whatever follows in shared memory
        p.npix = t_pool_npix;
        if (p.rider && p.npix != 128) return SQN_ERR_UNSUPPORTED;      // (three accumulators for the layer, one for the rider: 4 x 128 columns)
        p.tmem_cols = (p.rider ? 4u : 2u) * (unsigned)p.npix;
        p.b_tile = (unsigned)p.BN * row_bytes;
    }

    // output-pixel tiling; a 1x1 layer is tiled over the flattened pixel index
    const bool flat = !stem && d.K == 1 && d.pad == 0 && !d.pool;      // (a pooled 1x1 layer needs the 8x16 spatial tiles)
    long long OWl = d.OW, OHl = d.OH, NIl = d.N;
    if (flat) { OWl = (long long)d.N * d.OH * d.OW; OHl = 1; NIl = 1; }
    if (OWl > 0x7fffffffLL) return SQN_ERR_UNSUPPORTED;
    const int OW = (int)OWl, OH = (int)OHl, NI = (int)NIl;

    // Patch mode (stem and KxK stride-1 layers whose kernels fit in shared memory): the tile is
    // 8 output columns x BH <= 16 output rows of one image, so that each group of 8 MMA rows is a
    // run of 8 consecutive patch rows and consecutive groups are a constant number of bytes apart.
    int patch_w = 0, patch_h = 0;     // TMA box extents of the patch (lines of patch_w rows)
    bool patch_ok = false;
    if (!flat && p.n_tiles == 1) {
        const int th = (OH + 15) / 16;
        const int bh = p.pool ? poolt_rows(p.npix) : (OH + th - 1) / th;   // pooling: 32 (16) rows give 15 (7) pooled rows
        const unsigned last_group = p.pool ? poolt_rows(p.npix) - 1 : 15;  // the MMA reads 16 (pooling: 32 or 16) groups of 8 pixels
        unsigned patch_bytes;              // bytes one patch box delivers per reduction chunk
        if (stem) {
            // Input lines 2*h0 .. 2*h0 + 2*BH+4, 22 pixels (176 bytes) of each, stored as they are.  Output pixel
            // (g, j) of the tile and kernel row kh read the 64 bytes at line 2g + kh, byte 16j: in the MMA's
            // unswizzled K-major layout that is a row pitch of 16 bytes inside a group of eight rows (the
            // 16-byte columns of the core matrices are then 16 bytes apart as well) and two lines between groups.
            const unsigned line_bytes = (2u * 7u + 8u) * 8u;
            patch_w = 8; patch_h = 2 * bh + 5;
            p.a_lines = 1;
            p.tap_h_bytes = line_bytes; p.tap_w_bytes = 0; p.sbo_bytes = 2u * line_bytes; p.h_mul = 2;
            patch_bytes = (unsigned)patch_h * line_bytes;
            p.patch_tile = ((2u * last_group + 7u) * line_bytes + 1023u) / 1024u * 1024u;
        } else {
            patch_w = 8 + d.K - 1; patch_h = bh + d.K - 1;
            p.tap_h_bytes = (unsigned)patch_w * row_bytes; p.tap_w_bytes = row_bytes; p.sbo_bytes = (unsigned)patch_w * row_bytes;
            int max_rows = (int)last_group * patch_w + 8 + (d.K - 1) * patch_w + (d.K - 1);
            if (max_rows < patch_w * patch_h) max_rows = patch_w * patch_h;
            patch_bytes = (unsigned)(patch_w * patch_h) * row_bytes;
            p.patch_tile = ((unsigned)max_rows * row_bytes + 1023u) / 1024u * 1024u;
        }
        const int nmma = p.taps * p.chunks * (p.BKc / 16);
        if (patch_h <= 256 && p.sbo_bytes < (1u << 18) && nmma <= (p.pool ? PARAM_TAB : MAX_TAB) &&
            (p.pool ? pool_layout(p, (size_t)p.chunks * p.patch_tile, &plan->smem)
                    : choose_layout(p, (size_t)p.chunks * p.patch_tile, true, 2, nmma > PARAM_TAB, &plan->smem))) {
            patch_ok = true;
            p.patch = 1;
            p.BW = 8; p.BH = bh; p.BI = 1;
            p.a_bytes = (unsigned)p.chunks * patch_bytes;
        }
    }
    if (!patch_ok) {
        if (stem || p.pool) return SQN_ERR_UNSUPPORTED;
        p.patch = 0;
        p.h_mul = 1;
        if (flat) { p.BW = OW < TILE_M ? OW : TILE_M; p.BH = 1; p.BI = 1; }
        else choose_box(OW, OH, NI, &p.BW, &p.BH, &p.BI);
        p.a_bytes = (unsigned)(p.BW * p.BH * p.BI) * row_bytes;
        const size_t a_tile = (size_t)TILE_M * row_bytes;
        if (!choose_layout(p, a_tile, true, 3, false, &plan->smem) && !choose_layout(p, a_tile, false, 3, false, &plan->smem) &&
            !choose_layout(p, a_tile, false, 2, false, &plan->smem))
            return SQN_ERR_UNSUPPORTED;
    }
    p.use_ptab = 0;
    if (p.patch && p.taps * p.chunks * (p.BKc / 16) <= PARAM_TAB) {
        // operand offsets of every MMA of a tile, in issue order (tap-major, then chunk, then k-step)
        p.use_ptab = 1;
        const int ksteps = p.BKc / 16;
        int e = 0;
        for (int kh = 0; kh < p.taps_h; ++kh)
            for (int kw = 0; kw < p.taps_w; ++kw)
                for (int ch = 0; ch < p.chunks; ++ch)
                    for (int k = 0; k < ksteps; ++k, ++e) {
                        const unsigned it = (unsigned)((kh * p.taps_w + kw) * p.chunks + ch);
                        const unsigned a_off = (unsigned)ch * p.patch_tile + (unsigned)kh * p.tap_h_bytes + (unsigned)kw * p.tap_w_bytes;
                        p.ptab[e].x = (a_off >> 4) + 2u * k;
                        p.ptab[e].y = ((it * p.b_tile) >> 4) + 2u * k;
                    }
    }
    if (plan->smem > t_smem_limit) return SQN_ERR_UNSUPPORTED;
    if (rider) {
        // the rider's MMAs read the centre of the patch (the layer's own padding shifted away)
        const int ksteps = p.BKc / 16;
        p.r_nmma = p.chunks * ksteps;
        if (!p.patch || p.r_nmma > 8) return SQN_ERR_UNSUPPORTED;
        int e = 0;
        for (int ch = 0; ch < p.chunks; ++ch)
            for (int k = 0; k < ksteps; ++k, ++e) {
                const unsigned a_off = (unsigned)ch * p.patch_tile + (unsigned)p.pad * p.tap_h_bytes + (unsigned)p.pad * p.tap_w_bytes;
                p.r_ptab[e].x = (a_off >> 4) + 2u * k;
                p.r_ptab[e].y = (((unsigned)ch * p.b_tile) >> 4) + 2u * k;
            }
        p.r_b_bytes = (unsigned)p.chunks * p.b_bytes;
        p.r_c_off = rider->out_c_offset;
        p.r_bias = rider->bias;
    }
    p.tiles_w = (OW + p.BW - 1) / p.BW;
    p.tiles_h = (OH + p.BH - 1) / p.BH;
    p.tiles_i = (NI + p.BI - 1) / p.BI;
    p.h_step = p.BH;
    if (p.pool) {
        p.PW_out = (d.OW - 3) / 2 + 1;
        p.PH_out = (d.OH - 3) / 2 + 1;
        p.h_step = 2 * poolt_prows(p.npix);
        p.tiles_h = (p.PH_out + poolt_prows(p.npix) - 1) / poolt_prows(p.npix);
        const int tw_pool = (p.PW_out + 1 + 3) / 4;            // tile k emits pooled columns 4k-1 .. 4k+2
        if (tw_pool > p.tiles_w) p.tiles_w = tw_pool;
        p.pool_out = static_cast<__nv_bfloat16*>(d.out);
        p.pool_ctot = d.out_c_total;
    }

    const long long total = (long long)p.tiles_w * p.tiles_h * p.tiles_i * p.n_tiles;
    if (total > 0x7fffffffLL) return SQN_ERR_UNSUPPORTED;
    p.total_tiles = (int)total;
    // A 1x1 layer over a map larger than a third of the L2 walks its tiles backwards: the layer before it wrote the
    // map front to back, so its last part is still in the L2 and is read from there before it is evicted.
    p.reverse = (!p.patch && p.taps == 1 && !p.pool && (size_t)d.N * d.H * d.W * d.Cin * 2 > ((size_t)40 << 20)) ? 1 : 0;
    const long long ctas = (long long)num_sms() * (halves == 1 ? 2 : 1);
    const long long units = p.pool ? (long long)p.tiles_h * p.tiles_i : total;
    plan->grid = (int)(units < ctas ? units : ctas);
    p.grid = plan->grid;
    if (p.pool) {
        p.g_nt = 0; p.g_tw = 0;
        p.g_th = plan->grid % p.tiles_h;
        p.g_ti = plan->grid / p.tiles_h;
    } else {
        int g = plan->grid;
        p.g_nt = g % p.n_tiles; g /= p.n_tiles;
        p.g_tw = g % p.tiles_w; g /= p.tiles_w;
        p.g_th = g % p.tiles_h; g /= p.tiles_h;
        p.g_ti = g;
    }

    // ---- tensor maps
    if (stem) {
        // [4 layers x Wp pixels of a line][input lines][image]; the patch box is 22 pixels x (2*BH+5) lines,
        // unswizzled, so a line lands in shared memory as it is in global memory
        const cuuint64_t row_pitch = (cuuint64_t)Wp * 8;
        cuuint64_t dims[5] = {(cuuint64_t)Wp * 4, (cuuint64_t)Hp, (cuuint64_t)d.N, 1, 1};
        cuuint64_t str[4] = {row_pitch, (cuuint64_t)Hp * row_pitch, (cuuint64_t)Hp * row_pitch * d.N,
                             (cuuint64_t)Hp * row_pitch * d.N};
        cuuint32_t box[5] = {(2 * 7 + 8) * 4, (cuuint32_t)patch_h, 1, 1, 1};
        if (!encode(&plan->a, 5, a_ptr, dims, str, box, 0)) return SQN_ERR_CUDA;
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
        cuuint32_t box[5] = {(cuuint32_t)p.BKc, (cuuint32_t)(p.patch ? patch_w : p.BW),
                             (cuuint32_t)(p.patch ? patch_h : p.BH), (cuuint32_t)p.BI, 1};
        if (!encode(&plan->a, 5, a_ptr, dims, str, box, row_bytes)) return SQN_ERR_CUDA;
    }
    {
        const cuuint64_t kdim = (cuuint64_t)p.taps * p.k_per_tap;
        cuuint64_t dims[2] = {kdim, (cuuint64_t)d.Cout};
        cuuint64_t str[1] = {kdim * 2};
        cuuint32_t box[2] = {(cuuint32_t)p.BKc, (cuuint32_t)p.BN};
        if (!encode(&plan->b, 2, w_ptr, dims, str, box, row_bytes)) return SQN_ERR_CUDA;
    }
    plan->r = plan->b;
    if (rider) {
        cuuint64_t dims[2] = {(cuuint64_t)d.Cin, (cuuint64_t)rider->Cout};
        cuuint64_t str[1] = {(cuuint64_t)d.Cin * 2};
        cuuint32_t box[2] = {(cuuint32_t)p.BKc, (cuuint32_t)p.BN};
        if (!encode(&plan->r, 2, rider->w, dims, str, box, row_bytes)) return SQN_ERR_CUDA;
    }
    if (!p.pool) {                  // (conv_pool_kernel writes the pooled map with plain stores)
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

// Two light CTAs per SM when the layer's tiles, kernels and accumulators fit twice; else one CTA per SM.
int build_plan(const ConvDesc& d, bool stem, const void* a_ptr, const void* w_ptr, int Hp, int Wp, Plan* plan)
{
    // Measured on B200 over the SqueezeNet shapes: two light CTAs per SM (two independent producer / MMA /
    // epilogue chains) win for patch-mode layers up to 64 output layers and for 1x1 layers whose light layout
    // still has three A stages; with fewer stages (large kernels resident) or wider tiles the deep rings of
    // the single CTA win.
    if (build_plan_cfg(d, stem, a_ptr, w_ptr, Hp, Wp, 1, plan) == SQN_OK) {
        const TcParams& p = plan->p;
        if ((p.patch && p.BN <= 64) || (!p.patch && p.taps == 1 && p.stages >= 3)) return SQN_OK;
    }
    if (d.pool) {       // the larger tiles where the layer's kernels leave room for their patches
        t_pool_npix = 256;
        int rc = build_plan_cfg(d, stem, a_ptr, w_ptr, Hp, Wp, 2, plan);
        if (rc != SQN_OK) {
            t_pool_npix = 128;
            rc = build_plan_cfg(d, stem, a_ptr, w_ptr, Hp, Wp, 2, plan);
            t_pool_npix = 256;
        }
        return rc;
    }
    return build_plan_cfg(d, stem, a_ptr, w_ptr, Hp, Wp, 2, plan);
}

template <int SPLIT, int HC>
cudaError_t launch_variant(const Plan& plan, cudaStream_t stream)
{
    static const cudaError_t attr_rc =
        cudaFuncSetAttribute(conv_tc_kernel<SPLIT, HC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(SPLIT == 1 ? SMEM_LIMIT_2CTA : SMEM_LIMIT));
    if (attr_rc != cudaSuccess) return attr_rc;
    return launch_chained(conv_tc_kernel<SPLIT, HC>, dim3((unsigned)plan.grid), dim3(threads_for(SPLIT)), plan.smem,
                          stream, plan.a, plan.b, plan.o, plan.p);
}

int launch_plan(const Plan& plan, cudaStream_t stream)
{
    cudaError_t rc;
    const int hc = plan.p.CW / 2;
    if (plan.p.pool) {
        static const cudaError_t attr_rc =
            cudaFuncSetAttribute(conv_pool_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT);
        rc = attr_rc != cudaSuccess ? attr_rc
           : launch_chained(conv_pool_kernel, dim3((unsigned)plan.grid), dim3(POOLT_THREADS), plan.smem, stream, plan.a, plan.b, plan.r,
                            plan.p);
    }
    else if (plan.split == 1)
        rc = hc == 32 ? launch_variant<1, 32>(plan, stream)
           : hc == 16 ? launch_variant<1, 16>(plan, stream) : launch_variant<1, 8>(plan, stream);
    else
        rc = hc == 32 ? launch_variant<2, 32>(plan, stream)
           : hc == 16 ? launch_variant<2, 16>(plan, stream) : launch_variant<2, 8>(plan, stream);
    if (rc != cudaSuccess) return SQN_ERR_CUDA;
    note_launch();
    return cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}

template <int SPLIT, int HC>
cudaError_t launch_variant2(const Plan& a, const Plan& b, cudaStream_t stream)
{
    static const cudaError_t attr_rc =
        cudaFuncSetAttribute(conv_tc_kernel2<SPLIT, HC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(SPLIT == 1 ? SMEM_LIMIT_2CTA : SMEM_LIMIT));
    if (attr_rc != cudaSuccess) return attr_rc;
    return launch_chained(conv_tc_kernel2<SPLIT, HC>, dim3((unsigned)(a.grid + b.grid)), dim3(threads_for(SPLIT)),
                          a.smem > b.smem ? a.smem : b.smem, stream, a.a, a.b, a.o, a.p, b.a, b.b, b.o, b.p);
}

// Two plans of the same kernel variant in one launch: the first a.grid CTAs run `a`, the others `b`.
int launch_plan2(const Plan& a, const Plan& b, cudaStream_t stream)
{
    cudaError_t rc;
    const size_t smem = a.smem > b.smem ? a.smem : b.smem;
    if (a.p.pool != b.p.pool) return SQN_ERR_UNSUPPORTED;
    if (a.p.pool) {
        if (a.p.npix != b.p.npix) return SQN_ERR_UNSUPPORTED;
        static const cudaError_t attr_rc =
            cudaFuncSetAttribute(conv_pool_kernel2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT);
        rc = attr_rc != cudaSuccess ? attr_rc
           : launch_chained(conv_pool_kernel2, dim3((unsigned)(a.grid + b.grid)), dim3(POOLT_THREADS), smem, stream, a.a, a.b,
                            a.r, a.p, b.a, b.b, b.r, b.p);
    } else {
        const int hc = a.p.CW / 2;
        if (a.split != b.split || a.p.CW != b.p.CW) return SQN_ERR_UNSUPPORTED;
        if (a.split == 1)
            rc = hc == 32 ? launch_variant2<1, 32>(a, b, stream)
               : hc == 16 ? launch_variant2<1, 16>(a, b, stream) : launch_variant2<1, 8>(a, b, stream);
        else
            rc = hc == 32 ? launch_variant2<2, 32>(a, b, stream)
               : hc == 16 ? launch_variant2<2, 16>(a, b, stream) : launch_variant2<2, 8>(a, b, stream);
    }
    if (rc != cudaSuccess) return SQN_ERR_CUDA;
    note_launch();
    return cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}

// Plans are cached by the full request: encoding three tensor maps costs microseconds that a
// batch-1 forward would notice.
struct PlanKey {
    const void *in, *w, *bias, *out, *ws;
    const void *rw, *rbias;     // the rider's kernels and bias (conv_pool_kernel), else null
    int v[14];
    int r_c_off;
};

std::mutex g_plan_mu;
std::map<std::string, Plan> g_plans;

// SQN_POOL_ISSUERS in the environment (tuning aid: 1 or 2 issuer warps for a pooled convolution without a rider), 0 if unset
int pool_issuers_env()
{
    const char* v = std::getenv("SQN_POOL_ISSUERS");
    const int n = v ? std::atoi(v) : 0;
    return n == 1 || n == 2 ? n : 0;
}

// force_halves / force_cw != 0: the plan of that kernel variant (CTAs per SM, store chunk width) instead of the
// layer's own best one, so that it can share a launch with another layer's plan.
int cached_plan(const ConvDesc& d, bool stem, const void* a_ptr, const void* w_ptr, int Hp, int Wp, const void* ws,
                Plan* out, int force_halves = 0, int force_cw = 0)
{
    PlanKey k;
    std::memset(&k, 0, sizeof(k));
    k.in = d.in; k.w = d.w; k.bias = d.bias; k.out = d.out; k.ws = ws;
    if (t_rider) { k.rw = t_rider->w; k.rbias = t_rider->bias; k.r_c_off = t_rider->out_c_offset + 1; }
    const int v[14] = {d.N, d.Cin, d.H, d.W, d.Cout, d.K, d.S, d.pad, d.out_c_offset, d.out_c_total, d.relu | (d.pool << 1) | (d.params_static << 2) | (d.stem_prepacked << 3) | (d.f16 << 4),
                       (stem ? 1 : 0) | (force_halves << 4) | ((force_cw & 0xffff) << 8) | (pool_issuers_env() << 24), Hp, Wp};
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
    int rc;
    if (force_halves != 0) {
        t_force_cw = force_cw < 0 ? 0 : force_cw;
        t_pool_npix = force_cw == -128 ? 128 : 256;       // (pooled layers: the tile size instead of a chunk width)
        rc = build_plan_cfg(d, stem, a_ptr, w_ptr, Hp, Wp, force_halves, &plan);
        t_force_cw = 0;
        t_pool_npix = 256;
    } else {
        rc = build_plan(d, stem, a_ptr, w_ptr, Hp, Wp, &plan);
    }
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

bool tmap_encode_16(CUtensorMap* m, int rank, const void* ptr, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
                    const cuuint32_t* box, unsigned inner_bytes, int f16)
{
    t_f16 = f16;
    return encode(m, rank, ptr, dims, strides_bytes, box, inner_bytes);
}
int sm_count() { return num_sms(); }

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

// Tuning aid: SQN_TC_VARIANT="<CTAs per SM: 1|2>,<store chunk width: 16|32|64>" in the environment (read at every
// call, so a sweep can change it between calls) makes single-layer launches use that kernel variant instead of the
// layer's own choice; SQN_ERR_UNSUPPORTED where the variant does not fit.  `bench.py --variants` sweeps it per
// layer, the analogue of the paper's thread-granularity study (Section III-D, Tables 1 and 3).
int launch_conv_bf16(const ConvDesc& d, cudaStream_t stream)
{
    Plan plan;
    int ctas = 0, cw = 0;
    const char* v = d.pool ? nullptr : std::getenv("SQN_TC_VARIANT");
    if (v && std::sscanf(v, "%d,%d", &ctas, &cw) == 2 && (ctas == 1 || ctas == 2) && (cw == 16 || cw == 32 || cw == 64)) {
        const int rc = cached_plan(d, false, d.in, d.w, 0, 0, nullptr, &plan, ctas == 1 ? 2 : 1, cw);
        if (rc != SQN_OK) return SQN_ERR_UNSUPPORTED;
        return launch_plan(plan, stream);
    }
    const int rc = cached_plan(d, false, d.in, d.w, 0, 0, nullptr, &plan);
    if (rc != SQN_OK) return rc;
    return launch_plan(plan, stream);
}

// Two layers that do not depend on one another (the two expands of a fire layer: same input, disjoint layer slices
// of one output tensor) in ONE launch.  `big` keeps its own best kernel variant and takes the first CTAs, `small` is
// planned for the same variant.  SQN_ERR_UNSUPPORTED when no common variant exists: the caller launches them one
// after the other.
int launch_conv_bf16_pair(const ConvDesc& small, const ConvDesc& big, cudaStream_t stream)
{
    if (small.pool != big.pool) return SQN_ERR_UNSUPPORTED;
    Plan pb, ps;
    int rc = cached_plan(big, false, big.in, big.w, 0, 0, nullptr, &pb);
    if (rc != SQN_OK) return rc;
    rc = cached_plan(small, false, small.in, small.w, 0, 0, nullptr, &ps);
    if (rc != SQN_OK) return rc;
    if (big.pool && ps.p.npix != pb.p.npix) {          // both with the smaller tiles
        if (cached_plan(big, false, big.in, big.w, 0, 0, nullptr, &pb, 2, -128) != SQN_OK ||
            cached_plan(small, false, small.in, small.w, 0, 0, nullptr, &ps, 2, -128) != SQN_OK)
            return SQN_ERR_UNSUPPORTED;
    }
    if (!big.pool && (ps.split != pb.split || ps.p.CW != pb.p.CW)) {
        rc = cached_plan(small, false, small.in, small.w, 0, 0, nullptr, &ps, pb.halves, pb.p.CW);
        if (rc != SQN_OK) return SQN_ERR_UNSUPPORTED;
    }
    return launch_plan2(pb, ps, stream);
}

// Four pooled layers that read the same input (two slices of each expand of a fire layer) in ONE launch, in the order
// given (the heavy ones first); all with the 128-pixel tiles.  SQN_ERR_UNSUPPORTED if one of them cannot be planned so.
int launch_conv_bf16_pool4(const ConvDesc* d, cudaStream_t stream)
{
    Plan pl[4];
    size_t smem = 0;
    int grid = 0;
    for (int i = 0; i < 4; ++i) {
        if (!d[i].pool || cached_plan(d[i], false, d[i].in, d[i].w, 0, 0, nullptr, &pl[i], 2, -128) != SQN_OK || pl[i].p.npix != 128)
            return SQN_ERR_UNSUPPORTED;
        if (pl[i].smem > smem) smem = pl[i].smem;
        grid += pl[i].grid;
    }
    static const cudaError_t attr_rc =
        cudaFuncSetAttribute(conv_pool_kernel4, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT);
    if (attr_rc != cudaSuccess) return SQN_ERR_CUDA;
    const cudaError_t rc = launch_chained(conv_pool_kernel4, dim3((unsigned)grid), dim3(POOLT_THREADS), smem, stream, pl[0].a, pl[0].b,
                                          pl[0].p, pl[1].a, pl[1].b, pl[1].p, pl[2].a, pl[2].b, pl[2].p, pl[3].a, pl[3].b, pl[3].p);
    if (rc != cudaSuccess) return SQN_ERR_CUDA;
    note_launch();
    return cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}

// Pooled 3x3 layers each with a pooled 1x1 layer on the same input riding on its patches (both expands of a fire layer
// followed by a max-pool; n = 1, or 2 for two slices of the output layers): ONE launch, one pass over the input, the
// 1x1 layer's few MMAs hidden behind the 3x3 layer's.  SQN_ERR_UNSUPPORTED where the kernels of both do not fit.
int launch_conv_bf16_pool_riders(const ConvDesc* big, const ConvDesc* rider, int n, cudaStream_t stream)
{
    if (n < 1 || n > 2) return SQN_ERR_UNSUPPORTED;
    Plan pl[2];
    for (int i = 0; i < n; ++i) {
        if (!big[i].pool || !rider[i].pool) return SQN_ERR_UNSUPPORTED;
        t_rider = &rider[i];
        int rc = cached_plan(big[i], false, big[i].in, big[i].w, 0, 0, nullptr, &pl[i], 2, -128);      // (the 128-pixel tiles)
        if (rc == SQN_OK && n == 2 && i == 1 && pl[1].p.npix != pl[0].p.npix)
            rc = SQN_ERR_UNSUPPORTED;
        t_rider = nullptr;
        if (rc != SQN_OK) return rc == SQN_ERR_CUDA ? rc : SQN_ERR_UNSUPPORTED;
        if (!pl[i].p.rider) return SQN_ERR_UNSUPPORTED;
    }
    return n == 1 ? launch_plan(pl[0], stream) : launch_plan2(pl[0], pl[1], stream);
}

// Host-only feasibility test of the fused max-pool for a layer (shared-memory budget, shape rules).
bool conv_bf16_pool_fits(const ConvDesc& d)
{
    if (!d.pool || conv_bf16_supported(d) != SQN_OK) return false;
    Plan plan;
    return cached_plan(d, false, d.in, d.w, 0, 0, nullptr, &plan) == SQN_OK;
}

// Same launch without touching the plan cache: the tensor maps are encoded into a stack object on
// every call, so nothing is allocated on the host or on the device.
int launch_conv_bf16_uncached(const ConvDesc& d, cudaStream_t stream)
{
    Plan plan;
    const int rc = build_plan(d, false, d.in, d.w, 0, 0, &plan);
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

// Repack of the stem's input and kernels into the workspace (one launch).
int launch_stem_pack_bf16(const ConvDesc& d, void* workspace, size_t workspace_bytes, cudaStream_t stream)
{
    const int rc = stem_check(d, workspace, workspace_bytes);
    if (rc != SQN_OK) return rc;
    const int Hp = (d.H + 1) / 2 * 2, Wp = (d.W + 2) / 2 * 2;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    uint4* pin = reinterpret_cast<uint4*>(ws);
    unsigned short* pw = reinterpret_cast<unsigned short*>(ws + align_up((size_t)d.N * Hp * Wp * 8, 1024));
    const long long rows = (long long)d.N * Hp;
    const int pitch = (3 * d.W + 23) / 8 * 8;                  // halfwords per staged row: the row, its lead-in, a full last unit
    const int row_blocks = (int)((rows + PACK_ROWS - 1) / PACK_ROWS), w_blocks = (d.Cout * 224 + 255) / 256;
    const cudaError_t e = launch_chained(stem_pack, dim3((unsigned)(row_blocks + w_blocks)), dim3(256),
                                         (size_t)PACK_ROWS * pitch * 2, stream, static_cast<const __nv_bfloat16*>(d.in), pin,
                                         d.N, d.H, d.W, Hp, Wp, (long long)d.N * d.H * d.W * 3, pitch, row_blocks,
                                         static_cast<const unsigned short*>(d.w), pw, d.Cout, d.bias, d.f16);
    note_launch(1);
    return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}

// The stem convolution itself, on the repacked tensors left in the workspace by the call above.
int launch_stem_conv_bf16(const ConvDesc& d, void* workspace, size_t workspace_bytes, cudaStream_t stream)
{
    int rc = stem_check(d, workspace, workspace_bytes);
    if (rc != SQN_OK) return rc;
    const int Hp = stem_packed_rows(d.H), Wp = stem_packed_cols(d.W);
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    Plan plan;
    rc = cached_plan(d, true, ws, ws + align_up((size_t)d.N * Hp * Wp * 8, 1024), Hp, Wp, workspace, &plan);
    if (rc != SQN_OK) return rc;
    return launch_plan(plan, stream);
}

int launch_stem_conv_bf16_prepacked(const ConvDesc& d, cudaStream_t stream)
{
    if (!d.stem_prepacked) return SQN_ERR_BADARG;
    if (d.Cout % 16 != 0 || d.Cout > 256) return SQN_ERR_UNSUPPORTED;
    if (d.out_c_offset % 8 != 0 || d.out_c_total % 8 != 0) return SQN_ERR_ALIGN;
    Plan plan;
    const int rc = cached_plan(d, true, d.in, d.w, stem_packed_rows(d.H), stem_packed_cols(d.W), nullptr, &plan);
    if (rc != SQN_OK) return rc;
    return launch_plan(plan, stream);
}

}  // namespace sqn
