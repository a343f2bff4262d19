// Fire layer (paper Section II: one squeeze layer feeding two expand layers) as ONE kernel, bf16 on the tensor cores:
// the squeeze map never leaves the SM.  Section III-C of the paper has every layer write its output in the order
// the next layer reads, so that nothing is repacked between layers; here the squeeze layer writes its output
// straight into the shared-memory operand of the two expand layers, so that nothing is stored between them at all.
//
// Work item = a band of R output rows of one image.  For a band the CTA
//   1. squeezes the band's input rows and one halo row above and below (1x1 convolution: rows of the flat pixel
//      index are the M = 128 operand, read by TMA as they lie in memory; the squeeze kernels stay in shared
//      memory), and the squeeze epilogue writes the result -- bias added, ReLU, rounded to bf16 -- as a flat array of
//      pixels with a pitch of P = W + 2 pixels per image row: "the patch".  The two extra columns and the rows
//      outside the image are the zero padding of the 3x3 expand and stay zero;
//   2. runs both expands on the patch.  Output tile t = RT image rows = RT*P <= 128 consecutive patch pixels (the two
//      padding pixels of every row compute garbage that is never stored).  Kernel tap (kh, kw) of the 3x3 expand is
//      one MMA whose A descriptor starts (kh*P + kw) pixels further into the patch; the 1x1 expand is the centre
//      tap.  Where both expands fit one accumulator twice over, the 1x1 kernels are appended to the centre tap's and
//      one MMA of N = e3 + e1 serves both (one job per tile); else the 3x3 and the 1x1 expand of a tile are two jobs.
//      The expand epilogue converts an accumulator chunk by chunk into staging tiles of RT rows x W pixels (the
//      padding pixels dropped) that TMA stores send to the layer slices of the output tensor.
// The two steps are two pipelines that run side by side, each with its own MMA issuer, TMEM accumulators and
// epilogue warps -- issuing an MMA costs tens of clocks whatever its size, and with the small N of these layers one
// issuing thread would be the limit:
//   squeeze:  TMA producer -> input ring -> squeeze issuer -> 2 accumulators -> 4 epilogue warps -> patch
//   expand:   patch -> expand issuer -> 2 or 3 accumulators -> 8 epilogue warps -> staging ring -> store warp
// With two patches (where shared memory allows) the squeeze pipeline works on the CTA's next band while the expand
// pipeline works on this one; patch_ready / patch_free barriers hand a patch back and forth.
// Every mbarrier wait is bounded (see wait_bar).
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
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

constexpr int FF_SEPI_WARPS = 4;           // squeeze epilogue warps (one per TMEM lane quadrant)
constexpr int FF_EEPI_WARPS = 8;           // expand epilogue warps: two groups of four (one warp per quadrant)
constexpr int FF_ISSUERS = 2;              // MMA issuer warps per pipeline: they take the pipeline's jobs in turn
constexpr int FF_W_SMMA = 1, FF_W_EMMA = FF_W_SMMA + FF_ISSUERS, FF_W_STORE = FF_W_EMMA + FF_ISSUERS;      // first warp of each role
constexpr int FF_W_SEPI = FF_W_STORE + 1, FF_W_EEPI = FF_W_SEPI + FF_SEPI_WARPS;
constexpr int FF_THREADS = 32 * (FF_W_EEPI + FF_EEPI_WARPS);
constexpr int FF_MAX_STAGES = 16;
constexpr int FF_MAX_STG = 4;
constexpr int FF_MAX_EMMA = 48;            // MMAs of one expand tile: 10 taps x at most 4 k-steps, + spare
constexpr int FF_MAX_ESLOTS = 4;
constexpr size_t FF_SMEM_LIMIT = 227 * 1024;

struct FireParams {
    int H, W, P, N;                  // map extent, patch pitch (W + 2), images
    int Cin, s, e1, e3;
    int RT, R, NB;                   // image rows per expand tile, rows per band, bands per image
    int items, grid;
    int chunks_in, BKc_in, ksteps_in;   // squeeze reduction: chunks, elements per chunk, MMAs per chunk
    int src_tma;                     // 1: no squeeze pipeline -- the patch is loaded by TMA from a stored squeeze map
    int chunks_s, BKs, ksteps_s;     // expand reduction per tap: chunks_s chunks of BKs layers (s = chunks_s * BKs), BKs / 16 MMAs each
    int CS, e3p, e1p;                // the output layers are split over CS CTAs ("parts") of e3p + e1p layers each
    int CW;                          // output layers per store chunk (32 or 64)
    int f16;                         // 1: the 16-bit type is fp16, 0: bf16
    int stages, nstg;
    int s_issuers;                   // squeeze issuer warps at work: 2 where the input ring holds two tiles' chunks, else 1
    int npatch;                      // patches in shared memory: 1, 2, or (flat expands, where they fit) 3
    // expand jobs of a tile: one (both expands in one accumulator) or two (3x3, then 1x1)
    int njobs;
    int job_e0[2], job_en[2];        // the job's MMAs: entries [e0, en) of etab
    int job_chunk0[2], job_nchunks[2];   // its store chunks (chunk c = accumulator-order columns [CW*c, CW*c + CW) of the part)
    unsigned job_bias16[2];          // its bias rows, in 16-byte units from off_bias_e
    unsigned job_idesc[2];           // instruction descriptor of its bias MMA (all of its columns)
    int s_slot_cols;                 // TMEM: two squeeze accumulators of s_slot_cols columns, then eslots expand
    int eslots, eslot_cols;          //       accumulators of eslot_cols columns
    unsigned tmem_cols;
    int c_tot;                       // layers per pixel of the output tensor
    int b_early;                     // kernels and bias may be fetched before the wait for the grid ahead
    unsigned rb_in, rb_s;            // bytes per row of the input / squeeze-kernel tiles and of the patch / expand-kernel tiles (2 * BKs)
    unsigned x_bytes;                // bytes one input box delivers
    unsigned w_bytes;                // bytes of all kernel tiles together
    unsigned off_wsq, wsq_tile;      // squeeze kernels: chunks_in tiles of s rows
    unsigned off_we;                 // expand kernels: centre tap, 1x1, then the other eight taps
    unsigned off_w3[9][3], off_w1c[3];   // ... offsets from off_we of the tiles of (tap, chunk) and of the 1x1 kernels' chunks
    unsigned off_patch, patch_bytes; // one or two patches of patch_bytes each,
    unsigned patch_chunk;            // ... each made of chunks_s arrays of patch_chunk bytes (rows of BKs layers)
    unsigned patch_box_bytes;        // bytes one patch box delivers (src_tma)
    unsigned off_x, x_tile;
    unsigned off_stg, stg_slot;
    unsigned off_bias_s, off_bias_e, off_ones, off_ctl;
    const float *bias_sq, *bias_e1, *bias_e3;
    int* status;
    uint2 etab[FF_MAX_EMMA];         // per expand MMA: {A offset from the tile's first patch pixel, B offset from off_we}, 16-byte units
    unsigned eidesc[FF_MAX_EMMA];    // ... and its instruction descriptor (N differs between the MMAs of a job)
};

struct FireShared {
    unsigned long long full[FF_MAX_STAGES];
    unsigned long long empty[FF_MAX_STAGES];
    unsigned long long w_full;
    unsigned long long s_full[2], s_empty[2];
    unsigned long long e_full[FF_MAX_ESLOTS], e_empty[FF_MAX_ESLOTS];
    unsigned long long patch_ready[4], patch_free[4];
    unsigned long long stg_full[FF_MAX_STG];
    unsigned long long stg_free[FF_MAX_STG];
    unsigned tmem_base;
    volatile int abort_flag;
};

// A band of an image: rows [y0, y0 + rows) are produced, input rows [ylo, yhi) are squeezed.
struct Band { int n, y0, rows, ylo, npx, n_s, n_e; };

__device__ __forceinline__ Band band_of(const FireParams& p, int item)
{
    Band b;
    b.n = item / p.NB;
    const int k = item - b.n * p.NB;
    b.y0 = k * p.R;
    b.rows = p.H - b.y0 < p.R ? p.H - b.y0 : p.R;
    b.ylo = b.y0 > 0 ? b.y0 - 1 : 0;
    const int yhi = b.y0 + b.rows + 1 < p.H ? b.y0 + b.rows + 1 : p.H;
    b.npx = (yhi - b.ylo) * p.W;
    b.n_s = (b.npx + 127) >> 7;
    b.n_e = (b.rows + p.RT - 1) / p.RT;
    return b;
}

// 16-byte unit `u` of row `r` of a tile with `rb`-byte rows written by TMA with the swizzle of that width (tile base
// aligned to 1024 bytes): the unit index is XORed with address bits 7.. of the row.
__device__ __forceinline__ uint32_t swz(uint32_t r, uint32_t rb)
{
    return rb == 128 ? (r & 7u) : rb == 64 ? ((r >> 1) & 3u) : ((r >> 2) & 1u);
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// 16 accumulator columns -> ReLU, bf16 -> two 16-byte units at unit index u0, u0 + 1 of a swizzled row
template <bool F16>
__device__ __forceinline__ void store16(const uint32_t* v, uint32_t rbase, uint32_t u0, uint32_t sw)
{
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) o[j] = pack_relu_x2(__uint_as_float(v[8 * u + 2 * j]), __uint_as_float(v[8 * u + 2 * j + 1]), F16);
        st_shared_v4(rbase + (((u0 + (uint32_t)u) ^ sw) << 4), o[0], o[1], o[2], o[3]);
    }
}

template <bool F16>
__global__ void __launch_bounds__(FF_THREADS, 1)
fire_fused_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmWsq,
                  const __grid_constant__ CUtensorMap tmW3, const __grid_constant__ CUtensorMap tmW1,
                  const __grid_constant__ CUtensorMap tmO, const __grid_constant__ FireParams p)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - raw);
    FireShared* sh = reinterpret_cast<FireShared*>(base_ptr + p.off_ctl);
    const uint32_t smWsq = base + p.off_wsq, smWe = base + p.off_we, smPatch = base + p.off_patch;
    const uint32_t smX = base + p.off_x, smStg = base + p.off_stg;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // CTA -> (part of the output layers, first band); it walks the bands bid, bid + gstep, ...
    const int part = (int)blockIdx.x % p.CS;
    const int bid = (int)blockIdx.x / p.CS, gstep = p.grid / p.CS;
    const int nbuf = p.npatch;

    auto load_kernels = [&]() {          // every kernel tile of the layer (this CTA's part of it), once; one mbarrier counts them all
        const uint32_t bar = smem_u32(&sh->w_full);
        mbar_arrive_expect_tx(bar, p.w_bytes);
        if (!p.src_tma)
            for (int ch = 0; ch < p.chunks_in; ++ch)
                tma_load_2d(smWsq + (uint32_t)ch * p.wsq_tile, &tmWsq, bar, ch * p.BKc_in, 0);
        for (int tap = 0; tap < 9; ++tap)
            for (int ch = 0; ch < p.chunks_s; ++ch)
                tma_load_2d(smWe + p.off_w3[tap][ch], &tmW3, bar, tap * p.s + ch * p.BKs, part * p.e3p);
        for (int ch = 0; ch < p.chunks_s; ++ch) tma_load_2d(smWe + p.off_w1c[ch], &tmW1, bar, ch * p.BKs, part * p.e1p);
    };
    auto fill_bias = [&]() {
        if (!p.src_tma) {
            uint4* rs = reinterpret_cast<uint4*>(base_ptr + p.off_bias_s);
            for (int c = threadIdx.x; c < p.s; c += FF_THREADS) bias_row(rs, c, __ldg(p.bias_sq + c), p.f16);
        }
        uint4* re = reinterpret_cast<uint4*>(base_ptr + p.off_bias_e);
        for (int c = threadIdx.x; c < p.e3p + p.e1p; c += FF_THREADS)
            bias_row(re, c, c < p.e3p ? __ldg(p.bias_e3 + part * p.e3p + c) : __ldg(p.bias_e1 + part * p.e1p + c - p.e3p), p.f16);
    };

    // Up to chain_wait() this block touches only its own shared memory, TMEM, the kernel parameters and, when
    // b_early is set, the layer's kernels and bias (see conv_tc_body).
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&sh->full[s]), 1);
            mbar_init(smem_u32(&sh->empty[s]), 1);
        }
        mbar_init(smem_u32(&sh->w_full), 1);
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&sh->s_full[a]), 1);
            mbar_init(smem_u32(&sh->s_empty[a]), FF_SEPI_WARPS);
        }
        for (int a = 0; a < 4; ++a) {
            mbar_init(smem_u32(&sh->patch_ready[a]), p.src_tma ? 1 : FF_SEPI_WARPS);
            mbar_init(smem_u32(&sh->patch_free[a]), FF_ISSUERS);
        }
        for (int a = 0; a < FF_MAX_ESLOTS; ++a) {
            mbar_init(smem_u32(&sh->e_full[a]), 1);
            mbar_init(smem_u32(&sh->e_empty[a]), FF_EEPI_WARPS);
        }
        for (int b = 0; b < p.nstg; ++b) {
            mbar_init(smem_u32(&sh->stg_full[b]), FF_EEPI_WARPS / 2);      // one group of the expand epilogue
            mbar_init(smem_u32(&sh->stg_free[b]), 1);
        }
        sh->abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmX);
        prefetch_tensormap(&tmWsq);
        prefetch_tensormap(&tmW3);
        prefetch_tensormap(&tmW1);
        prefetch_tensormap(&tmO);
        if (p.b_early) load_kernels();
    }
    if (warp == FF_W_SMMA) {
        tmem_alloc(smem_u32(&sh->tmem_base), p.tmem_cols);
        tmem_relinquish();
        chain_release();            // (only once this CTA holds its TMEM: see conv_tc_body)
    }
    // the patches start as zeros: their two padding columns and the rows outside the image are never written
    for (uint32_t i = threadIdx.x; i < (uint32_t)nbuf * p.patch_bytes / 16u; i += FF_THREADS)
        st_shared_v4(smPatch + 16u * i, 0u, 0u, 0u, 0u);
    {
        // tile of ones for the bias MMAs: 128 rows of 32 bytes in the 32-byte swizzle, ones in the first two places
        uint4* ones = reinterpret_cast<uint4*>(base_ptr + p.off_ones);
        for (int r = threadIdx.x; r < 128; r += FF_THREADS) {
            const int u = (r >> 2) & 1;
            ones[2 * r + u] = make_uint4(one_x2(p.f16), 0u, 0u, 0u);
            ones[2 * r + (u ^ 1)] = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    if (p.b_early) fill_bias();
    chain_wait();       // the grid ahead has finished: global memory may be read and written from here on
    if (!p.b_early) fill_bias();
    fence_proxy_async_smem();           // the MMAs read patch, ones and bias rows through the async proxy
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    volatile int* abort_flag = &sh->abort_flag;
    const uint32_t tmem_e = tmem_base + (uint32_t)(2 * p.s_slot_cols);      // first expand accumulator (s_slot_cols = 0 without a squeeze pipeline)

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer: input tiles of the squeeze
        if (lane == 0 && p.src_tma) {
            // the patch of a band straight from the stored squeeze map: one box per chunk of layers, one pixel to the left
            // of and one row above the band; what lies outside the map is filled with zeros, which is the padding
            if (!p.b_early) load_kernels();
            bool ok = true;
            int buf = 0, j = 0, loaded = 0;
            uint32_t fph = 0;
            for (int item = bid; item < p.items && ok; item += gstep, ++j) {
                const Band b = band_of(p, item);
                if (j >= nbuf && !wait_bar(smem_u32(&sh->patch_free[buf]), fph, abort_flag, p.status)) { ok = false; break; }
                const uint32_t bar = smem_u32(&sh->patch_ready[buf]);
                mbar_arrive_expect_tx(bar, (uint32_t)p.chunks_s * p.patch_box_bytes);
                for (int ch = 0; ch < p.chunks_s; ++ch)
                    tma_load_5d(smPatch + (uint32_t)buf * p.patch_bytes + (uint32_t)ch * p.patch_chunk, &tmX, bar, ch * p.BKs, -1,
                                b.y0 - 1, b.n, 0);
                ++loaded;
                if (++buf == nbuf) { buf = 0; if (j >= nbuf) fph ^= 1u; }
            }
            if (!ok) {      // give the boxes already issued a bounded chance to land before the CTA exits
                for (int k = 0; k < nbuf && k < loaded; ++k) {
                    const int jj = loaded - 1 - k;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(smem_u32(&sh->patch_ready[jj % nbuf]), (uint32_t)(jj / nbuf) & 1u)) {
                        if (clock64() - t0 > WAIT_LIMIT_CYCLES / 8) break;
                        __nanosleep(100);
                    }
                }
            }
        } else if (lane == 0) {
            if (!p.b_early) load_kernels();
            bool ok = true;
            int st = 0, issued = 0;
            uint32_t ph = 0;
            for (int item = bid; item < p.items && ok; item += gstep) {
                const Band b = band_of(p, item);
                const int px0 = (b.n * p.H + b.ylo) * p.W;
                for (int t = 0; t < b.n_s && ok; ++t)
                    for (int ch = 0; ch < p.chunks_in; ++ch) {
                        if (!wait_bar(smem_u32(&sh->empty[st]), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                        const uint32_t full = smem_u32(&sh->full[st]);
                        mbar_arrive_expect_tx(full, p.x_bytes);
                        tma_load_2d(smX + (uint32_t)st * p.x_tile, &tmX, full, ch * p.BKc_in, px0 + 128 * t);
                        ++issued;
                        if (++st == p.stages) { st = 0; ph ^= 1u; }
                    }
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
    } else if (warp < FF_W_EMMA) {
        // ------------------------------------------------------------------ squeeze issuers
        // Issuing an MMA and the hand-shakes around it cost the issuing thread far more clocks than these small MMAs
        // cost the tensor core, so two warps take the squeeze tiles in turn (issuer w fills accumulator w).  Each
        // warp walks the loops converged; one elected lane issues the MMAs and their commits.
        const int w = warp - FF_W_SMMA;
        const uint32_t idesc_s = make_idesc_bf16(128, (uint32_t)p.s, (uint32_t)p.f16);
        const uint32_t hi_in = (uint32_t)(make_kmajor_desc(0, p.rb_in, 8u * p.rb_in) >> 32);
        const uint64_t ones_desc = make_kmajor_desc(base + p.off_ones, 32u, 256u);
        const uint64_t bias_s_desc = make_kmajor_desc(base + p.off_bias_s, 32u, 256u);
        const uint32_t smX16 = smX >> 4, x_tile16 = p.x_tile >> 4, smWsq16 = smWsq >> 4, wsq_tile16 = p.wsq_tile >> 4;
        bool ok = !p.src_tma && __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->w_full), 0u, abort_flag, p.status));
        int st = 0, as = 0;                     // tile k goes to accumulator k & 1 and, with two issuers, to issuer k & 1
        uint32_t ph = 0, aph = 0;
        for (int item = bid; item < p.items && ok; item += gstep) {
            const Band b = band_of(p, item);
            for (int t = 0; t < b.n_s && ok; ++t) {
                if ((p.s_issuers == 2 ? as : 0) != w) {         // the other issuer's tile: step over its input slots
                    st += p.chunks_in;
                    while (st >= p.stages) { st -= p.stages; ph ^= 1u; }
                    if (++as == 2) { as = 0; aph ^= 1u; }
                    continue;
                }
                ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->s_empty[as]), aph ^ 1u, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(as * p.s_slot_cols);
                for (int ch = 0; ch < p.chunks_in; ++ch) {
                    ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->full[st]), ph, abort_flag, p.status));
                    if (!ok) break;
                    tc_fence_after();
                    if (elect_one()) {
                        const uint64_t da = ((uint64_t)hi_in << 32) | (uint64_t)((smX16 + (uint32_t)st * x_tile16) | 0x10000u);
                        const uint64_t db = ((uint64_t)hi_in << 32) | (uint64_t)((smWsq16 + (uint32_t)ch * wsq_tile16) | 0x10000u);
                        mma_bf16_ss(d_tmem, da, db, idesc_s, ch ? 1u : 0u);
                        mma_bf16_ss(d_tmem, da + 2u, db + 2u, idesc_s, 1u);
                        if (p.ksteps_in == 4) {
                            mma_bf16_ss(d_tmem, da + 4u, db + 4u, idesc_s, 1u);
                            mma_bf16_ss(d_tmem, da + 6u, db + 6u, idesc_s, 1u);
                        }
                        mma_commit(smem_u32(&sh->empty[st]));           // input slot free once these MMAs have read it
                        if (ch == p.chunks_in - 1) {
                            mma_bf16_ss(d_tmem, ones_desc, bias_s_desc, idesc_s, 1u);
                            mma_commit(smem_u32(&sh->s_full[as]));
                        }
                    }
                    __syncwarp();
                    if (++st == p.stages) { st = 0; ph ^= 1u; }
                }
                if (!ok) break;
                if (++as == 2) { as = 0; aph ^= 1u; }
            }
        }
    } else if (warp < FF_W_STORE) {
        // ------------------------------------------------------------------ expand issuers (the jobs in turn)
        const int w = warp - FF_W_EMMA;
        const uint32_t hi_s = (uint32_t)(make_kmajor_desc(0, p.rb_s, 8u * p.rb_s) >> 32);
        const uint64_t ones_desc = make_kmajor_desc(base + p.off_ones, 32u, 256u);
        const uint64_t bias_e_desc = make_kmajor_desc(base + p.off_bias_e, 32u, 256u);
        const uint32_t smWe16 = smWe >> 4, patch16 = smPatch >> 4;
        const uint32_t tile_step16 = ((uint32_t)(p.RT * p.P) * p.rb_s) >> 4;      // patch units between expand tiles
        bool ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->w_full), 0u, abort_flag, p.status));
        int es = 0, turn = 0;
        uint32_t eph = 0;
        int buf = 0;
        uint32_t rph = 0;                       // parity of patch_ready[buf] for the band at hand
        for (int item = bid; item < p.items && ok; item += gstep) {
            const Band b = band_of(p, item);
            // the band's patch is complete once every squeeze epilogue warp has passed the band's last squeeze tile
            ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->patch_ready[buf]), rph, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
            for (int t = 0; t < b.n_e && ok; ++t) {
                const uint32_t a_base = patch16 + (uint32_t)buf * (p.patch_bytes >> 4) + (uint32_t)t * tile_step16;
                for (int job = 0; job < p.njobs; ++job, turn ^= 1) {
                    if (turn == w) {
                        ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->e_empty[es]), eph ^ 1u, abort_flag, p.status));
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t d_tmem = tmem_e + (uint32_t)(es * p.eslot_cols);
                        if (elect_one()) {
                            uint32_t acc = 0u;
                            const int en = p.job_en[job];
#pragma unroll 2
                            for (int e = p.job_e0[job]; e < en; ++e) {
                                const uint2 o = p.etab[e];
                                mma_bf16_ss(d_tmem, ((uint64_t)hi_s << 32) | (uint64_t)((a_base + o.x) | 0x10000u),
                                            ((uint64_t)hi_s << 32) | (uint64_t)((smWe16 + o.y) | 0x10000u), p.eidesc[e], acc);
                                acc = 1u;
                            }
                            mma_bf16_ss(d_tmem, ones_desc, bias_e_desc + (uint64_t)p.job_bias16[job], p.job_idesc[job], 1u);
                            mma_commit(smem_u32(&sh->e_full[es]));
                        }
                        __syncwarp();
                    }
                    if (++es == p.eslots) { es = 0; eph ^= 1u; }
                }
            }
            if (!ok) break;
            // the patch may be overwritten once the MMAs of both issuers have read it
            if (elect_one()) mma_commit(smem_u32(&sh->patch_free[buf]));
            __syncwarp();
            if (++buf == nbuf) { buf = 0; rph ^= 1u; }
        }
    } else if (warp == FF_W_STORE) {
        // ----------------------------------------------------------------- store issuer
        if (lane == 0) {
            bool ok = true;
            int sb = 0, pend = 0, fb = 0;       // next slot, stores whose slot is not yet released, next slot to release
            uint32_t sph = 0;
            const int nchunks = p.job_chunk0[p.njobs - 1] + p.job_nchunks[p.njobs - 1];
            for (int item = bid; item < p.items && ok; item += gstep) {
                const Band b = band_of(p, item);
                for (int t = 0; t < b.n_e && ok; ++t)
                    for (int chunk = 0; chunk < nchunks; ++chunk) {
                        if (!wait_bar(smem_u32(&sh->stg_full[sb]), sph, abort_flag, p.status)) { ok = false; break; }
                        // accumulator-order columns [0, e3p) are the part's 3x3 layers (output layers e1 + ..), the rest its 1x1 layers
                        const int col = chunk * p.CW;
                        const int cc = col < p.e3p ? p.e1 + part * p.e3p + col : part * p.e1p + col - p.e3p;
                        if (sqn_dbg_ok(cc >= 0 && cc + p.CW <= p.e1 + p.e3 && b.y0 + t * p.RT < p.H && b.n < p.N, p.status))
                        tma_store_4d(&tmO, smStg + (uint32_t)sb * p.stg_slot, cc, 0, b.y0 + t * p.RT, b.n);
                        tma_store_commit();
                        if (++sb == p.nstg) { sb = 0; sph ^= 1u; }
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
    } else if (warp < FF_W_EEPI) {
        // -------------------------------------------------------------------- squeeze epilogue
        // warp w reads TMEM lane quadrant w % 4: one input pixel per thread, all s layers of it
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        const int sidx = (warp - FF_W_SEPI) * 32 + lane;                 // index among the squeeze epilogue threads
        bool ok = !p.src_tma;
        int as = 0, j = 0, buf = 0;
        uint32_t aph = 0, fph = 0;              // fph: parity of patch_free[buf] for the patch's previous band
        for (int item = bid; item < p.items && ok; item += gstep, ++j) {
            const Band b = band_of(p, item);
            const uint32_t patch = smPatch + (uint32_t)buf * p.patch_bytes;
            for (int t = 0; t < b.n_s; ++t) {
                ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->s_full[as]), aph, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
                const uint32_t ta = tmem_base + lane_base + (uint32_t)(as * p.s_slot_cols);
                uint32_t v[64];
                tmem_ld_x16(ta, *reinterpret_cast<uint32_t(*)[16]>(&v[0]));
                if (p.s >= 32) tmem_ld_x16(ta + 16u, *reinterpret_cast<uint32_t(*)[16]>(&v[16]));
                if (p.s == 64) {
                    tmem_ld_x16(ta + 32u, *reinterpret_cast<uint32_t(*)[16]>(&v[32]));
                    tmem_ld_x16(ta + 48u, *reinterpret_cast<uint32_t(*)[16]>(&v[48]));
                }
                tmem_ld_wait();
                // accumulator in registers: hand it back to the issuer
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh->s_empty[as]));
                if (++as == 2) { as = 0; aph ^= 1u; }
                if (t == 0 && j >= nbuf) {
                    // the expand MMAs of the band that used this patch before must have read it
                    ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->patch_free[buf]), fph, abort_flag, p.status));
                    if (!ok) break;
                }
                const int g = t * 128 + row;                      // pixel of the band's input rows
                if (g < b.npx) {
                    const int yy = g / p.W, xx = g - yy * p.W;
                    const uint32_t pr = (uint32_t)((yy + b.ylo - b.y0 + 1) * p.P + xx + 1);
                    if (!sqn_dbg_ok((pr + 1u) * p.rb_s <= p.patch_chunk, p.status)) continue;      // (the row lies inside the patch)
                    const uint32_t rbase = patch + pr * p.rb_s;
                    const uint32_t sw = swz(pr, p.rb_s);
                    store16<F16>(&v[0], rbase, 0u, sw);
                    if (p.s >= 32) store16<F16>(&v[16], rbase, 2u, sw);
                    if (p.s == 64) {
                        store16<F16>(&v[32], rbase, 4u, sw);
                        store16<F16>(&v[48], rbase, 6u, sw);
                    }
                }
            }
            if (!ok) break;
            {
                // patch rows that lie outside the image (above its first band, below its last) hold what an earlier band left
                const uint32_t row_units = ((uint32_t)p.P * p.rb_s) >> 4;
                if (b.y0 == 0)
                    for (uint32_t i = (uint32_t)sidx; i < row_units; i += 32u * FF_SEPI_WARPS) st_shared_v4(patch + 16u * i, 0u, 0u, 0u, 0u);
                if (b.y0 + b.rows == p.H) {
                    const uint32_t a0 = patch + (uint32_t)((b.rows + 1) * p.P) * p.rb_s;
                    for (uint32_t i = (uint32_t)sidx; i < row_units; i += 32u * FF_SEPI_WARPS) st_shared_v4(a0 + 16u * i, 0u, 0u, 0u, 0u);
                }
            }
            fence_proxy_async_smem();             // patch visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->patch_ready[buf]));
            if (++buf == nbuf) { buf = 0; if (j >= nbuf) fph ^= 1u; }
        }
    } else {
        // -------------------------------------------------------------------- expand epilogue
        // Two groups of four warps (one warp per TMEM lane quadrant, one M row per thread) take the store chunks in
        // turn, so that two chunks are converted at a time: a chunk is a chain of latencies (TMEM load, wait for the
        // staging slot, conversion, proxy fence, hand-over) far longer than its instructions.
        const int q = warp & 3, grp = (warp - FF_W_EEPI) >> 2;
        const int row = q * 32 + lane;
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        // M row -> (image row r of the tile, patch column c); the staging tile drops the padding columns
        const int r_e = row / p.P, c_e = row - r_e * p.P;
        const bool e_valid = c_e < p.W && r_e < p.RT;
        const uint32_t stg_row = (uint32_t)(r_e * p.W + c_e);
        const uint32_t stg_off = stg_row * (uint32_t)(p.CW * 2);
        const uint32_t sw_e = swz(stg_row, (uint32_t)(p.CW * 2));
        bool ok = true;
        int es = 0, sb = 0, turn = 0;           // turn: the group whose chunk the next one is
        uint32_t eph = 0, sph = 0;
        for (int item = bid; item < p.items && ok; item += gstep) {
            const Band b = band_of(p, item);
            for (int t = 0; t < b.n_e && ok; ++t)
                for (int job = 0; job < p.njobs; ++job) {
                    ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->e_full[es]), eph, abort_flag, p.status));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t ta0 = tmem_e + lane_base + (uint32_t)(es * p.eslot_cols);
                    for (int chunk = 0; chunk < p.job_nchunks[job]; ++chunk, turn ^= 1) {
                        if (turn == grp) {
                            uint32_t v[64];
                            const uint32_t ta = ta0 + (uint32_t)(chunk * p.CW);
                            tmem_ld_x16(ta, *reinterpret_cast<uint32_t(*)[16]>(&v[0]));
                            tmem_ld_x16(ta + 16u, *reinterpret_cast<uint32_t(*)[16]>(&v[16]));
                            if (p.CW == 64) {
                                tmem_ld_x16(ta + 32u, *reinterpret_cast<uint32_t(*)[16]>(&v[32]));
                                tmem_ld_x16(ta + 48u, *reinterpret_cast<uint32_t(*)[16]>(&v[48]));
                            }
                            ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->stg_free[sb]), sph ^ 1u, abort_flag, p.status));
                            tmem_ld_wait();
                            if (!ok) break;
                            if (e_valid && sqn_dbg_ok(stg_off + (uint32_t)(p.CW * 2) <= p.stg_slot && sb < p.nstg, p.status)) {
                                const uint32_t rbase = smStg + (uint32_t)sb * p.stg_slot + stg_off;
                                store16<F16>(&v[0], rbase, 0u, sw_e);
                                store16<F16>(&v[16], rbase, 2u, sw_e);
                                if (p.CW == 64) {
                                    store16<F16>(&v[32], rbase, 4u, sw_e);
                                    store16<F16>(&v[48], rbase, 6u, sw_e);
                                }
                            }
                            fence_proxy_async_smem();             // staging rows visible to the TMA unit
                            __syncwarp();
                            if (lane == 0) mbar_arrive(smem_u32(&sh->stg_full[sb]));
                        }
                        if (++sb == p.nstg) { sb = 0; sph ^= 1u; }
                    }
                    if (!ok) break;
                    // this group's part of the accumulator is in its staging tiles: hand it back to the issuers
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&sh->e_empty[es]));
                    if (++es == p.eslots) { es = 0; eph ^= 1u; }
                }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == FF_W_SMMA) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

// ------------------------------------------------------------------------------ host side
struct FirePlan {
    CUtensorMap x, wsq, w3, w1, o;
    FireParams p;
    size_t smem;
};

inline size_t up1k(size_t v) { return (v + 1023) / 1024 * 1024; }

// Shared-memory layout for one choice of band height R, number of patches (2: the next band's patch is made while the
// expands run on this one; 1: they take turns) and, with a squeeze pipeline, input chunk width.  Fills the offsets;
// returns 0 if it does not fit, else 1 + the depth of the input ring (1 when there is no squeeze pipeline).
int fire_layout(FireParams& p, int R, int patches, int BKc_in, size_t* smem_bytes)
{
    const int s = p.s, W = p.W, H = p.H;
    p.R = R;
    p.NB = (H + R - 1) / R;
    p.items = p.N * p.NB;
    p.npatch = patches;
    size_t cur = 0;
    p.w_bytes = 0;
    p.off_wsq = 0;
    if (!p.src_tma) {
        p.BKc_in = BKc_in;
        p.chunks_in = p.Cin / BKc_in;
        p.ksteps_in = BKc_in / 16;
        p.rb_in = (unsigned)BKc_in * 2u;
        p.x_bytes = 128u * p.rb_in;
        p.wsq_tile = (unsigned)up1k((size_t)s * p.rb_in);
        cur += (size_t)p.chunks_in * p.wsq_tile;
        p.w_bytes += (unsigned)((size_t)p.chunks_in * s * p.rb_in);
    }
    p.off_we = (unsigned)cur;
    {
        // per chunk of layers: the centre tap's kernels, then the 1x1 expand's directly behind them (one B operand of
        // e3p + e1p rows); then the other eight taps
        const unsigned t3 = (unsigned)p.e3p * p.rb_s, t1 = (unsigned)p.e1p * p.rb_s;
        unsigned o = 0;
        for (int ch = 0; ch < p.chunks_s; ++ch) {
            p.off_w3[4][ch] = o; o += t3;
            p.off_w1c[ch] = o; o += t1;
            o = (unsigned)up1k(o);
        }
        for (int tap = 0; tap < 9; ++tap)
            if (tap != 4)
                for (int ch = 0; ch < p.chunks_s; ++ch) { p.off_w3[tap][ch] = o; o += (unsigned)up1k(t3); }
        cur += o;
        p.w_bytes += (unsigned)p.chunks_s * (9u * t3 + t1);
        if (p.w_bytes >= (1u << 20)) return 0;  // one mbarrier transaction count
    }
    p.off_patch = (unsigned)cur;
    {
        const int t_max = R / p.RT;
        size_t rows = (size_t)(R + 2) * p.P;
        const size_t reach = (size_t)(t_max - 1) * p.RT * p.P + 2 * p.P + 2 + 128;     // last row an expand MMA reads
        if (reach > rows) rows = reach;
        p.patch_chunk = (unsigned)up1k(rows * p.rb_s);
        p.patch_bytes = (unsigned)p.chunks_s * p.patch_chunk;
        p.patch_box_bytes = (unsigned)((size_t)(R + 2) * p.P * p.rb_s);
        cur += (size_t)patches * p.patch_bytes;
    }
    p.off_bias_s = (unsigned)cur; cur += up1k((size_t)s * 32);
    p.off_bias_e = (unsigned)cur; cur += up1k((size_t)(p.e1p + p.e3p) * 32);
    p.off_ones = (unsigned)cur; cur += 128 * 32;
    p.off_ctl = (unsigned)cur; cur += 1024;
    static_assert(sizeof(FireShared) <= 1024, "control block");
    p.stg_slot = (unsigned)up1k((size_t)p.RT * W * p.CW * 2);
    const size_t fixed = 1024 /*alignment slack*/ + cur;
    if (p.src_tma) {
        if (fixed + 2 * p.stg_slot > FF_SMEM_LIMIT) return 0;
        p.nstg = fixed + 4 * p.stg_slot <= FF_SMEM_LIMIT ? 4 : 2;
        p.stages = 1;                       // (no input ring; its barriers are still initialised)
        p.s_issuers = 1;
        p.off_x = (unsigned)cur;
        p.x_tile = 0;
        p.off_stg = (unsigned)cur; cur += (size_t)p.nstg * p.stg_slot;
        *smem_bytes = 1024 + cur;
        return 1;
    }
    p.x_tile = (unsigned)up1k(p.x_bytes);
    if (fixed + 2 * p.stg_slot + 2 * p.x_tile > FF_SMEM_LIMIT) return 0;
    // input ring first (it feeds the memory-bound part), then staging slots
    size_t left = FF_SMEM_LIMIT - fixed;
    p.nstg = 2;
    left -= 2 * p.stg_slot;
    int stages = (int)(left / p.x_tile);
    // The ring must hold what is in flight between this SM and memory (about 100 KB at full bandwidth); only beyond
    // that are two more staging slots worth their shared memory.
    if (left >= 2 * p.stg_slot + (size_t)128 * 1024) {
        p.nstg = 4;
        left -= 2 * p.stg_slot;
        stages = (int)(left / p.x_tile);
    }
    if (stages > FF_MAX_STAGES) stages = FF_MAX_STAGES;
    if (stages < 2) return 0;
    p.stages = stages;
    // Two issuers wait on the ring's barriers out of step; a wait must never be two phases ahead of its barrier
    // (its parity would match a phase long past), which holds when the ring is at least two tiles deep.
    p.s_issuers = stages >= 2 * p.chunks_in ? 2 : 1;
    p.off_x = (unsigned)cur; cur += (size_t)stages * p.x_tile;
    p.off_stg = (unsigned)cur; cur += (size_t)p.nstg * p.stg_slot;
    *smem_bytes = 1024 + cur;
    return *smem_bytes <= FF_SMEM_LIMIT ? 1 + stages : 0;
}

// Band heights to try, best first: SQN_FIRE_BAND in the environment (tuning aid, read at every call) names one;
// else 14 rows for maps of 40 rows and more (four equal bands for 55 rows), 8 for 20 rows and more, else the whole
// image; with so few images that this leaves SMs idle, one tile.  A band is a whole number of expand tiles.
// Winners of the band-height sweep at batch 256 (`bench.py --kernel fireN` under SQN_FIRE_BAND = 4 ... 28), frozen per
// layer shape: {H, Cin, s, e1 + e3, rows}.  Shapes not listed take the rule below.
struct BandChoice { int H, Cin, s, e, R; };
const BandChoice kBandTable[] = {
    {55, 96, 16, 128, 14},      // fire2: 66.6 us (8 rows: 66.9, 28 rows: 76.2)
    {55, 128, 16, 128, 4},      // fire3: 71.7 us (14 rows: 77.8, 28 rows: 91.2)
    {27, 256, 32, 256, 16},     // fire5: 51.5 us (8 rows: 51.9, 12 rows: 59.7)
};

int band_candidates(int H, int RT, int N, int Cin, int s, int e, int* out)
{
    int n = 0;
    auto add = [&](int R) {
        if (R > H) R = H;
        R = (R + RT - 1) / RT * RT;
        for (int i = 0; i < n; ++i)
            if (out[i] == R) return;
        out[n++] = R;
    };
    if (const char* v = std::getenv("SQN_FIRE_BAND")) {
        const int r = std::atoi(v);
        if (r > 0) { add(r); return n; }
    }
    // few images: bands of one tile, so that as many CTAs as possible have work (the layer is latency-bound then)
    const int pref = H >= 40 ? 14 : H >= 20 ? 8 : H;
    if ((long long)N * ((H + pref - 1) / pref) < sm_count()) { add(RT); add(2 * RT); }
    else
        for (const BandChoice& c : kBandTable)
            if (c.H == H && c.Cin == Cin && c.s == s && c.e == e) add(c.R);
    if (H >= 40) { add(14); add(8); }
    else if (H >= 20) { add(8); add(12); add(16); }
    else add(H);
    add(2 * RT);
    add(RT);
    return n;
}

// Plan for a fire layer: with dsq the whole layer (squeeze pipeline in the kernel), without it the two expands on a
// stored squeeze map (the patch comes by TMA).
int build_fire_plan(const ConvDesc* dsq, const ConvDesc& d1, const ConvDesc& d3, FirePlan* plan)
{
    FireParams& p = plan->p;
    std::memset(&p, 0, sizeof(p));
    const int H = d1.H, W = d1.W, N = d1.N, s = d1.Cin, e1 = d1.Cout, e3 = d3.Cout;
    const int Cin = dsq ? dsq->Cin : 0;
    p.src_tma = dsq ? 0 : 1;
    if (s % 16 != 0 || e1 % 32 != 0 || e3 % 32 != 0) return SQN_ERR_UNSUPPORTED;
    if (W + 2 > 128 || H < 1) return SQN_ERR_UNSUPPORTED;
    if (d1.out != d3.out || d1.out_c_total != d3.out_c_total || d1.out_c_offset != 0 || d3.out_c_offset != e1 ||
        d1.out_c_total % 8 != 0)
        return SQN_ERR_UNSUPPORTED;
    if ((long long)N * H * W > 0x7fffffffLL / 2) return SQN_ERR_UNSUPPORTED;
    if ((dsq && dsq->f16 != d1.f16) || d1.f16 != d3.f16) return SQN_ERR_UNSUPPORTED;
    p.f16 = d1.f16;
    p.H = H; p.W = W; p.P = W + 2; p.N = N; p.Cin = Cin; p.s = s; p.e1 = e1; p.e3 = e3;
    p.RT = 128 / p.P;
    p.BKs = s % 64 == 0 ? 64 : s % 32 == 0 ? 32 : 16;
    p.chunks_s = s / p.BKs;
    p.ksteps_s = p.BKs / 16;
    p.rb_s = (unsigned)p.BKs * 2u;
    if (p.chunks_s > 3) return SQN_ERR_UNSUPPORTED;
    if (dsq) {
        // the squeeze epilogue writes one swizzled row per patch pixel
        if (p.chunks_s != 1 || Cin % 32 != 0) return SQN_ERR_UNSUPPORTED;
    }
    p.tmem_cols = 512;
    p.c_tot = d1.out_c_total;
    p.b_early = ((!dsq || dsq->params_static) && d1.params_static && d3.params_static) ? 1 : 0;
    p.bias_sq = dsq ? dsq->bias : nullptr; p.bias_e1 = d1.bias; p.bias_e3 = d3.bias;
    p.status = device_status_word();
    p.s_slot_cols = dsq ? (s < 32 ? 32 : s) : 0;

    // ---- over how many CTAs the output layers are split (the kernels of a part must fit in shared memory beside the
    // patches), accumulators, shared-memory layout
    bool found = false;
    bool combined = false;
    // (first the splits whose parts are whole 64-layer store chunks: half as many chunk hand-overs in the epilogue)
    const char* csv = std::getenv("SQN_FIRE_CS");           // (tuning aid, read when a plan is built: forces the split)
    const int force_cs = csv && !dsq ? std::atoi(csv) : 0;
    for (int round = 0; round < 2 && !found; ++round)
    for (int cs = 1; cs <= (dsq ? 1 : 4) && !found; ++cs) {
        if (force_cs > 0 && cs != force_cs) continue;
        if (e1 % (32 * cs) != 0 || e3 % (32 * cs) != 0) continue;
        p.CS = cs; p.e3p = e3 / cs; p.e1p = e1 / cs;
        p.CW = (p.e3p % 64 == 0 && p.e1p % 64 == 0) ? 64 : 32;
        if ((p.CW == 64) != (round == 0)) continue;
        if (9 * p.chunks_s * p.ksteps_s + p.chunks_s * p.ksteps_s > FF_MAX_EMMA) continue;
        // TMEM: two squeeze accumulators (if any), then the expand accumulators.  Both expands in one accumulator (the
        // 1x1 kernels ride on the centre tap) where two such accumulators fit, else two jobs per tile over three
        // (or two) accumulators of max(e1p, e3p) columns.
        combined = p.e3p + p.e1p <= 256 && 2 * p.s_slot_cols + 2 * (p.e1p + p.e3p) <= 512 && ((unsigned)p.e3p * p.rb_s) % 256u == 0;
        if (combined) {
            p.njobs = 1; p.eslot_cols = p.e1p + p.e3p;
        } else {
            p.njobs = 2;
            p.eslot_cols = p.e1p > p.e3p ? p.e1p : p.e3p;
            if (p.eslot_cols > 256) continue;
        }
        // as many expand accumulators as the 512 columns hold (up to four): an issuer that finds the next one still
        // with the epilogue stands idle, and a tile's epilogue is a longer chain of latencies than its MMAs
        p.eslots = (512 - 2 * p.s_slot_cols) / p.eslot_cols;
        if (p.eslots > FF_MAX_ESLOTS) p.eslots = FF_MAX_ESLOTS;
        if (const char* v = std::getenv("SQN_FIRE_ESLOTS")) {          // (tuning aid, read when a plan is built)
            const int n = std::atoi(v);
            if (n >= 2 && n < p.eslots) p.eslots = n;
        }
        if (p.eslots < 2) continue;
        // two patches with (if there is one) an input ring of 32 KB or more and three slots or more, else one patch
        // under the same condition, else whatever fits
        int cand[8];
        const int nc = band_candidates(H, p.RT, N, Cin, s, e1 + e3, cand);
        // (flat expands: a third patch first -- the box of band j + 2 can only be requested once band j's MMAs are
        // done, and with two patches the request's latency shows in the issuers' waits; SQN_FIRE_PATCHES=2 tuning aid)
        const char* pv = std::getenv("SQN_FIRE_PATCHES");
        const int max_patches = !dsq ? (pv && std::atoi(pv) >= 2 && std::atoi(pv) <= 4 ? std::atoi(pv) : 3) : 2;
        for (int pass = 0; pass < 3 && !found; ++pass)
            for (int i = 0; i < nc && !found; ++i)
                for (int patches = (pass == 1 ? 1 : max_patches); patches >= (pass == 0 ? 2 : 1) && !found; --patches)
                    for (int bk = 64; bk >= 32 && !found; bk -= 32) {
                        if (dsq && Cin % bk != 0) continue;
                        if (!dsq && bk != 64) continue;
                        const int fit = fire_layout(p, cand[i], patches, bk, &plan->smem);
                        if (fit == 0) continue;
                        const int st = fit - 1;
                        if (pass == 2 || !dsq || (st >= 3 && (size_t)st * p.x_tile >= 32 * 1024)) found = true;
                    }
    }
    if (!found) return SQN_ERR_UNSUPPORTED;

    // ---- MMAs of an expand tile
    {
        int e = 0;
        auto tap_mmas = [&](int tap, const unsigned* b_off, int ncols) {        // b_off: the tile of each chunk
            const int kh = tap / 3, kw = tap % 3;
            for (int ch = 0; ch < p.chunks_s; ++ch)
                for (int k = 0; k < p.ksteps_s; ++k, ++e) {
                    p.etab[e].x = (((unsigned)ch * p.patch_chunk + (unsigned)(kh * p.P + kw) * p.rb_s) >> 4) + 2u * k;
                    p.etab[e].y = (b_off[ch] >> 4) + 2u * k;
                    p.eidesc[e] = make_idesc_bf16(128, (unsigned)ncols, (unsigned)p.f16);
                }
        };
        if (combined) {
            // centre tap first: its B operand is the centre tap's kernels followed by the 1x1 kernels, and the tile's
            // first MMA overwrites all e3p + e1p columns (with several chunks the later centre-tap MMAs add to all of
            // them as well); the other taps add to the first e3p
            p.job_e0[0] = 0;
            tap_mmas(4, p.off_w3[4], p.e3p + p.e1p);
            for (int tap = 0; tap < 9; ++tap)
                if (tap != 4) tap_mmas(tap, p.off_w3[tap], p.e3p);
            p.job_en[0] = e;
            p.job_chunk0[0] = 0; p.job_nchunks[0] = (p.e1p + p.e3p) / p.CW;
            p.job_bias16[0] = 0; p.job_idesc[0] = make_idesc_bf16(128, (unsigned)(p.e3p + p.e1p), (unsigned)p.f16);
        } else {
            p.job_e0[0] = 0;
            for (int tap = 0; tap < 9; ++tap) tap_mmas(tap, p.off_w3[tap], p.e3p);
            p.job_en[0] = e;
            p.job_chunk0[0] = 0; p.job_nchunks[0] = p.e3p / p.CW;
            p.job_bias16[0] = 0; p.job_idesc[0] = make_idesc_bf16(128, (unsigned)p.e3p, (unsigned)p.f16);
            p.job_e0[1] = e;
            tap_mmas(4, p.off_w1c, p.e1p);              // the 1x1 expand reads the centre pixel
            p.job_en[1] = e;
            p.job_chunk0[1] = p.e3p / p.CW; p.job_nchunks[1] = p.e1p / p.CW;
            p.job_bias16[1] = (unsigned)p.e3p * 2u;     // bias rows are 32 bytes each, the 3x3 expand's come first
            p.job_idesc[1] = make_idesc_bf16(128, (unsigned)p.e1p, (unsigned)p.f16);
        }
    }
    // CS consecutive CTAs work on the same bands, one part of the output layers each; such a group takes bands g,
    // g + groups, ...: with a group count that shares no factor with the bands per image every group meets all bands
    // of an image in turn (they differ in height: the last one is shorter)
    int g = sm_count() / p.CS;
    if (g < 1) return SQN_ERR_UNSUPPORTED;
    if (p.items <= g) g = p.items;
    else
        while (g > 1 && std::__gcd(g, p.NB) != 1) --g;
    p.grid = g * p.CS;

    // ---- tensor maps
    if (dsq) {
        {
            // input as a flat list of pixels: [Cin][N*H*W], boxes of 128 pixels
            const cuuint64_t npx = (cuuint64_t)N * H * W;
            cuuint64_t dims[2] = {(cuuint64_t)Cin, npx};
            cuuint64_t str[1] = {(cuuint64_t)Cin * 2};
            cuuint32_t box[2] = {(cuuint32_t)p.BKc_in, 128};
            if (!tmap_encode_16(&plan->x, 2, dsq->in, dims, str, box, p.rb_in, p.f16)) return SQN_ERR_CUDA;
        }
        {
            cuuint64_t dims[2] = {(cuuint64_t)Cin, (cuuint64_t)s};
            cuuint64_t str[1] = {(cuuint64_t)Cin * 2};
            cuuint32_t box[2] = {(cuuint32_t)p.BKc_in, (cuuint32_t)s};
            if (!tmap_encode_16(&plan->wsq, 2, dsq->w, dims, str, box, p.rb_in, p.f16)) return SQN_ERR_CUDA;
        }
    } else {
        // the squeeze map [s][W][H][N]: a patch box is P pixels x (R + 2) rows of one chunk of layers
        if (p.R + 2 > 256) return SQN_ERR_UNSUPPORTED;
        const cuuint64_t s1 = (cuuint64_t)s * 2;
        cuuint64_t dims[5] = {(cuuint64_t)s, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N, 1};
        cuuint64_t str[4] = {s1, s1 * W, s1 * W * H, s1 * W * H * N};
        cuuint32_t box[5] = {(cuuint32_t)p.BKs, (cuuint32_t)p.P, (cuuint32_t)(p.R + 2), 1, 1};
        if (!tmap_encode_16(&plan->x, 5, d1.in, dims, str, box, p.rb_s, p.f16)) return SQN_ERR_CUDA;
        plan->wsq = plan->x;            // (not read)
    }
    {
        cuuint64_t dims[2] = {(cuuint64_t)9 * s, (cuuint64_t)e3};
        cuuint64_t str[1] = {(cuuint64_t)9 * s * 2};
        cuuint32_t box[2] = {(cuuint32_t)p.BKs, (cuuint32_t)p.e3p};
        if (!tmap_encode_16(&plan->w3, 2, d3.w, dims, str, box, p.rb_s, p.f16)) return SQN_ERR_CUDA;
    }
    {
        cuuint64_t dims[2] = {(cuuint64_t)s, (cuuint64_t)e1};
        cuuint64_t str[1] = {(cuuint64_t)s * 2};
        cuuint32_t box[2] = {(cuuint32_t)p.BKs, (cuuint32_t)p.e1p};
        if (!tmap_encode_16(&plan->w1, 2, d1.w, dims, str, box, p.rb_s, p.f16)) return SQN_ERR_CUDA;
    }
    {
        const cuuint64_t s1 = (cuuint64_t)p.c_tot * 2;
        cuuint64_t dims[4] = {(cuuint64_t)(e1 + e3), (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
        cuuint64_t str[3] = {s1, s1 * W, s1 * W * H};
        cuuint32_t box[4] = {(cuuint32_t)p.CW, (cuuint32_t)W, (cuuint32_t)p.RT, 1};
        if (!tmap_encode_16(&plan->o, 4, d1.out, dims, str, box, (unsigned)p.CW * 2u, p.f16)) return SQN_ERR_CUDA;
    }
    return SQN_OK;
}

struct FireKey {
    const void *in, *wsq, *w1, *w3, *bsq, *b1, *b3, *out;
    int v[12];
};

std::mutex g_fire_mu;
std::map<std::string, FirePlan> g_fire_plans;

int launch_fire(const ConvDesc* dsq, const ConvDesc& d1, const ConvDesc& d3, cudaStream_t stream)
{
    if (d1.K != 1 || d3.K != 3 || d3.pad != 1 || d1.S != 1 || d3.S != 1 || !d1.relu || !d3.relu || d1.pool || d3.pool ||
        d1.in != d3.in || d1.Cin != d3.Cin || d1.H != d3.H || d1.W != d3.W || d1.N != d3.N)
        return SQN_ERR_UNSUPPORTED;
    if (dsq && (dsq->K != 1 || dsq->S != 1 || !dsq->relu || dsq->pool || d1.in != dsq->out || d1.Cin != dsq->Cout ||
                d1.H != dsq->H || d1.W != dsq->W || d1.N != dsq->N))
        return SQN_ERR_UNSUPPORTED;
    FireKey k;
    std::memset(&k, 0, sizeof(k));
    k.in = dsq ? dsq->in : d1.in; k.wsq = dsq ? dsq->w : nullptr; k.w1 = d1.w; k.w3 = d3.w; k.bsq = dsq ? dsq->bias : nullptr;
    k.b1 = d1.bias; k.b3 = d3.bias; k.out = d1.out;
    int dev = 0;
    cudaGetDevice(&dev);
    const char* bv = std::getenv("SQN_FIRE_BAND");
    const char* ev = std::getenv("SQN_FIRE_ESLOTS");
    const char* cv = std::getenv("SQN_FIRE_CS");
    const char* pv = std::getenv("SQN_FIRE_PATCHES");
    const int band = (bv ? std::atoi(bv) : 0) + 1000 * (ev ? std::atoi(ev) : 0) + 100000 * (cv ? std::atoi(cv) : 0) + 1000000 * (pv ? std::atoi(pv) : 0);
    const int v[12] = {d1.N, dsq ? dsq->Cin : -1, d1.H, d1.W, d1.Cin, d1.Cout, d3.Cout, d1.out_c_total,
                       (dsq ? dsq->params_static : 0) | (d1.params_static << 1) | (d3.params_static << 2), dev, band, d1.f16};
    std::memcpy(k.v, v, sizeof(v));
    const std::string key(reinterpret_cast<const char*>(&k), sizeof(k));
    FirePlan plan;
    bool have = false;
    {
        std::lock_guard<std::mutex> lock(g_fire_mu);
        auto it = g_fire_plans.find(key);
        if (it != g_fire_plans.end()) { plan = it->second; have = true; }
    }
    if (!have) {
        const int rc = build_fire_plan(dsq, d1, d3, &plan);
        if (rc != SQN_OK) return rc;
        std::lock_guard<std::mutex> lock(g_fire_mu);
        if (g_fire_plans.size() > 1024) g_fire_plans.clear();
        g_fire_plans[key] = plan;
    }
    // (the 16-bit type is a compile-time constant of the kernel: the epilogues' conversion loops are straight-line code)
    static const cudaError_t attr_rc0 =
        cudaFuncSetAttribute(fire_fused_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FF_SMEM_LIMIT);
    static const cudaError_t attr_rc1 =
        cudaFuncSetAttribute(fire_fused_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FF_SMEM_LIMIT);
    if (attr_rc0 != cudaSuccess || attr_rc1 != cudaSuccess) return SQN_ERR_CUDA;
    const cudaError_t rc = launch_chained(plan.p.f16 ? fire_fused_kernel<true> : fire_fused_kernel<false>, dim3((unsigned)plan.p.grid),
                                          dim3(FF_THREADS), plan.smem, stream, plan.x, plan.wsq, plan.w3, plan.w1, plan.o, plan.p);
    if (rc != cudaSuccess) return SQN_ERR_CUDA;
    note_launch();
    return cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}

}  // namespace

bool fused_fire_enabled()
{
    const char* v = std::getenv("SQN_FUSED_FIRE");        // read at every call: tests switch it
    return !(v && v[0] == '0');
}

// The whole fire layer in one launch; SQN_ERR_UNSUPPORTED where the kernel does not apply (the caller then launches
// the squeeze and the expands separately).
int launch_fire_fused_bf16(const ConvDesc& dsq, const ConvDesc& d1, const ConvDesc& d3, cudaStream_t stream)
{
    return launch_fire(&dsq, d1, d3, stream);
}

// Both expands of a fire layer on a stored squeeze map in one launch of the same kernel (its expand pipeline alone, the
// patch loaded by TMA, the output layers split over up to four CTAs so that each CTA's kernels stay in shared memory).
int launch_fire_expands_bf16(const ConvDesc& d1, const ConvDesc& d3, cudaStream_t stream)
{
    return launch_fire(nullptr, d1, d3, stream);
}

}  // namespace sqn
