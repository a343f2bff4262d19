// fp32 convolution layer: implicit GEMM on the FP32 pipes (FFMA), register tiled.
//
// GEMM view of the layer (Section II of the paper: every output pixel is the sum over
// input layers of a KxK kernel applied to a window): rows = output pixels (n, h, w),
// columns = output layers, reduction index k = (i*K + j)*Cin + c.  With NHWC activations
// and OHWI kernels the reduction index is contiguous in memory for both operands, so both
// tiles are read with 128-bit loads and transposed into shared memory.  Each thread owns
// an 8 x TN block of the output tile (the paper's "thread granularity" g, Section III-D,
// carried to two dimensions: a loaded window value is reused TN times, a kernel value 8 times).
#include "sqn_internal.h"

namespace sqn {
namespace {

constexpr int BK = 16;          // reduction elements per shared-memory tile
constexpr int NTHREADS = 256;
constexpr int TBL_MAX = 1024;   // scalar path: reduction-index decode table entries held in shared memory

struct F32Params {
    const float* in;
    const float* w;
    const float* bias;
    float* out;
    int* status;
    int N, Cin, H, W, Cout, K, S, pad, OH, OW;
    int M;      // N*OH*OW
    int Kdim;   // K*K*Cin
    int out_c_offset, out_c_total, relu;
};

__host__ __device__ constexpr int ld_for(int bn) { return bn <= 32 ? 32 : (bn <= 64 ? 64 : 128); }

// Rows of the transposed tiles are padded by PADF floats: the compute loop then reads them at addresses that differ
// from a per-thread base by compile-time offsets only (no index arithmetic between the FFMAs), and the four k-groups a
// warp stores at once fall into two banks' worth of conflicts at most (the stores are 1.5 % of the instructions).
constexpr int PADF = 4;

template <int BM, int BN, int VN, int QN, bool VEC>
__global__ void __launch_bounds__(NTHREADS, 2) conv_f32_kernel(const F32Params p)
{
    constexpr int TN = VN * QN;
    constexpr int TX = BN / TN;
    constexpr int TY = NTHREADS / TX;
    constexpr int TM = BM / TY;
    static_assert(TM == 8, "thread tile is 8 rows");
    static_assert(TX * TN == BN && TY * TM == BM, "tile shape");
    constexpr int LDB = ld_for(BN);

    __shared__ __align__(16) float As[2][BK][BM + PADF];
    __shared__ __align__(16) float Bs[2][BK][LDB + PADF];
    __shared__ int tbl_off[VEC ? 1 : TBL_MAX];
    __shared__ int tbl_hw[VEC ? 1 : TBL_MAX];

    const int tid = threadIdx.x;
    const int tx = tid % TX;
    const int ty = tid / TX;
    const int m0 = blockIdx.x * BM;
    const int n0 = blockIdx.y * BN;
    const int OHW = p.OH * p.OW;
    const bool use_tbl = !VEC && p.Kdim <= TBL_MAX;

    if (!VEC && use_tbl) {
        for (int k = tid; k < p.Kdim; k += NTHREADS) {
            const int c = k % p.Cin;
            const int t = k / p.Cin;
            const int kw = t % p.K;
            const int kh = t / p.K;
            tbl_off[k] = (kh * p.W + kw) * p.Cin + c;
            tbl_hw[k] = (kh << 16) | kw;
        }
        __syncthreads();
    }

    // ---- global -> register staging -------------------------------------------------
    constexpr int A_LOADS = VEC ? BM / 64 : BM * BK / NTHREADS;
    constexpr int B_LOADS_V = (BN + 63) / 64;
    constexpr int B_LOADS_S = BN / 16;

    // rows this thread stages
    const float* a_base[VEC ? A_LOADS : 1];
    int a_ih0[VEC ? A_LOADS : 1], a_iw0[VEC ? A_LOADS : 1];
    bool a_ok[VEC ? A_LOADS : 1];
    {
        constexpr int NR = VEC ? A_LOADS : 1;
#pragma unroll
        for (int j = 0; j < NR; ++j) {
            const int row = VEC ? (tid >> 2) + 64 * j : tid % BM;
            const int m = m0 + row;
            a_ok[j] = m < p.M;
            const int mm = a_ok[j] ? m : 0;
            const int n = mm / OHW;
            const int r = mm - n * OHW;
            const int oh = r / p.OW;
            const int ow = r - oh * p.OW;
            a_ih0[j] = oh * p.S - p.pad;
            a_iw0[j] = ow * p.S - p.pad;
            a_base[j] = p.in + (size_t)n * p.H * p.W * p.Cin;
        }
    }

    // vector path: this thread's position in the reduction index, kept incrementally
    int vk = (tid & 3) * 4, vc = 0, vkw = 0, vkh = 0;
    if (VEC) {
        vc = vk % p.Cin;
        const int t = vk / p.Cin;
        vkw = t % p.K;
        vkh = t / p.K;
    }

    float4 ra4[VEC ? A_LOADS : 1];
    float4 rb4[VEC ? B_LOADS_V : 1];
    float ra1[VEC ? 1 : A_LOADS];
    float rb1[VEC ? 1 : B_LOADS_S];

    auto load_tile = [&](int k0) {
        if (VEC) {
            const bool kin = vk < p.Kdim;
#pragma unroll
            for (int j = 0; j < A_LOADS; ++j) {
                const int ih = a_ih0[j] + vkh, iw = a_iw0[j] + vkw;
                const bool ok = kin && a_ok[j] && (unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.W;
                ra4[j] = ok ? __ldg(reinterpret_cast<const float4*>(a_base[j] + ((size_t)ih * p.W + iw) * p.Cin + vc))
                            : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < B_LOADS_V; ++j) {
                const int n = (tid >> 2) + 64 * j;
                const bool ok = kin && n < BN && (n0 + n) < p.Cout;
                rb4[j] = ok ? __ldg(reinterpret_cast<const float4*>(p.w + (size_t)(n0 + n) * p.Kdim + vk))
                            : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            // advance to the next tile
            vk += BK;
            vc += BK;
            while (vc >= p.Cin) {
                vc -= p.Cin;
                if (++vkw == p.K) { vkw = 0; ++vkh; }
            }
        } else {
            constexpr int KSTEP = NTHREADS / BM;
            const int kk0 = tid / BM;
#pragma unroll
            for (int j = 0; j < A_LOADS; ++j) {
                const int k = k0 + kk0 + KSTEP * j;
                float v = 0.f;
                if (k < p.Kdim && a_ok[0]) {
                    int off, kh, kw;
                    if (use_tbl) {
                        off = tbl_off[k];
                        const int hw = tbl_hw[k];
                        kh = hw >> 16;
                        kw = hw & 0xffff;
                    } else {
                        const int c = k % p.Cin;
                        const int t = k / p.Cin;
                        kw = t % p.K;
                        kh = t / p.K;
                        off = (kh * p.W + kw) * p.Cin + c;
                    }
                    const int ih = a_ih0[0] + kh, iw = a_iw0[0] + kw;
                    if ((unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.W)
                        v = __ldg(a_base[0] + ((ptrdiff_t)a_ih0[0] * p.W + a_iw0[0]) * p.Cin + off);
                }
                ra1[j] = v;
            }
            const int kk = tid & 15;
#pragma unroll
            for (int j = 0; j < B_LOADS_S; ++j) {
                const int n = (tid >> 4) + 16 * j;
                const int k = k0 + kk;
                rb1[j] = (k < p.Kdim && (n0 + n) < p.Cout) ? __ldg(p.w + (size_t)(n0 + n) * p.Kdim + k) : 0.f;
            }
        }
    };

    auto store_tile = [&](int buf) {
        if (VEC) {
            const int k4 = tid & 3;
#pragma unroll
            for (int j = 0; j < A_LOADS; ++j) {
                const int row = (tid >> 2) + 64 * j;
                As[buf][4 * k4 + 0][row] = ra4[j].x;
                As[buf][4 * k4 + 1][row] = ra4[j].y;
                As[buf][4 * k4 + 2][row] = ra4[j].z;
                As[buf][4 * k4 + 3][row] = ra4[j].w;
            }
#pragma unroll
            for (int j = 0; j < B_LOADS_V; ++j) {
                const int n = (tid >> 2) + 64 * j;
                if (n < BN) {
                    const int col = n;
                    Bs[buf][4 * k4 + 0][col] = rb4[j].x;
                    Bs[buf][4 * k4 + 1][col] = rb4[j].y;
                    Bs[buf][4 * k4 + 2][col] = rb4[j].z;
                    Bs[buf][4 * k4 + 3][col] = rb4[j].w;
                }
            }
        } else {
            constexpr int KSTEP = NTHREADS / BM;
            const int kk0 = tid / BM;
            const int row = tid % BM;
#pragma unroll
            for (int j = 0; j < A_LOADS; ++j) {
                const int kk = kk0 + KSTEP * j;
                As[buf][kk][row] = ra1[j];
            }
            const int kk = tid & 15;
#pragma unroll
            for (int j = 0; j < B_LOADS_S; ++j) {
                const int n = (tid >> 4) + 16 * j;
                Bs[buf][kk][n] = rb1[j];
            }
        }
    };

    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

    const int ntiles = (p.Kdim + BK - 1) / BK;
    load_tile(0);
    store_tile(0);
    __syncthreads();

    for (int t = 0; t < ntiles; ++t) {
        const int buf = t & 1;
        if (t + 1 < ntiles) load_tile((t + 1) * BK);

#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[TM], b[TN];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const float4 v = *reinterpret_cast<const float4*>(&As[buf][kk][q * (BM / 2) + ty * 4]);
                a[4 * q + 0] = v.x; a[4 * q + 1] = v.y; a[4 * q + 2] = v.z; a[4 * q + 3] = v.w;
            }
#pragma unroll
            for (int q = 0; q < QN; ++q) {
                const int cb = q * (BN / QN) + tx * VN;
                if (VN == 4) {
                    const float4 v = *reinterpret_cast<const float4*>(&Bs[buf][kk][cb]);
                    b[q * VN + 0] = v.x; b[q * VN + 1] = v.y; b[q * VN + 2] = v.z; b[q * VN + 3] = v.w;
                } else if (VN == 2) {
                    const float2 v = *reinterpret_cast<const float2*>(&Bs[buf][kk][cb]);
                    b[q * VN + 0] = v.x; b[q * VN + 1] = v.y;
                } else {
                    b[q * VN] = Bs[buf][kk][cb];
                }
            }
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }

        if (t + 1 < ntiles) {
            store_tile(buf ^ 1);
            __syncthreads();
        }
    }

    // ---- epilogue: bias, ReLU, store into the layer slice of the NHWC output -----------
    const bool vec_store = (VN > 1) && (p.Cout % VN == 0) && (p.out_c_offset % VN == 0) && (p.out_c_total % VN == 0);
#pragma unroll
    for (int q = 0; q < QN; ++q) {
        const int col0 = n0 + q * (BN / QN) + tx * VN;
        float bv[VN];
#pragma unroll
        for (int j = 0; j < VN; ++j) bv[j] = (col0 + j < p.Cout) ? __ldg(p.bias + col0 + j) : 0.f;
#pragma unroll
        for (int i = 0; i < TM; ++i) {
            const int row = (i >> 2) * (BM / 2) + ty * 4 + (i & 3);
            const int m = m0 + row;
            if (m >= p.M) continue;
            float v[VN];
#pragma unroll
            for (int j = 0; j < VN; ++j) {
                v[j] = acc[i][q * VN + j] + bv[j];
                if (p.relu) v[j] = fmaxf(v[j], 0.f);
            }
            if (!sqn_dbg_ok(m >= 0 && p.out_c_offset + col0 >= 0 && p.out_c_offset + (col0 < p.Cout ? col0 : 0) < p.out_c_total, p.status)) continue;
            float* dst = p.out + (size_t)m * p.out_c_total + p.out_c_offset + col0;
            if (vec_store && col0 + VN <= p.Cout) {
                if (VN == 4) *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
                else if (VN == 2) *reinterpret_cast<float2*>(dst) = make_float2(v[0], v[1]);
            } else {
#pragma unroll
                for (int j = 0; j < VN; ++j)
                    if (col0 + j < p.Cout) dst[j] = v[j];
            }
        }
    }
}

template <int BM, int BN, int VN, int QN>
int launch_cfg(const F32Params& p, bool vec, cudaStream_t stream)
{
    dim3 grid((p.M + BM - 1) / BM, (p.Cout + BN - 1) / BN, 1);
    if (vec) conv_f32_kernel<BM, BN, VN, QN, true><<<grid, NTHREADS, 0, stream>>>(p);
    else conv_f32_kernel<BM, BN, VN, QN, false><<<grid, NTHREADS, 0, stream>>>(p);
    note_launch();
    return cudaGetLastError() == cudaSuccess ? SQN_OK : SQN_ERR_CUDA;
}

}  // namespace

int launch_conv_f32(const ConvDesc& d, cudaStream_t stream)
{
    F32Params p;
    p.in = static_cast<const float*>(d.in);
    p.w = static_cast<const float*>(d.w);
    p.bias = d.bias;
    p.out = static_cast<float*>(d.out);
    p.status = device_status_word();
    p.N = d.N; p.Cin = d.Cin; p.H = d.H; p.W = d.W; p.Cout = d.Cout; p.K = d.K; p.S = d.S; p.pad = d.pad;
    p.OH = d.OH; p.OW = d.OW;
    const long long M = (long long)d.N * d.OH * d.OW;
    const long long Kdim = (long long)d.K * d.K * d.Cin;
    if (M <= 0 || M > 0x7fffffffLL - 512 || Kdim > 0x7fffffffLL - 64) return SQN_ERR_UNSUPPORTED;
    if ((long long)d.H * d.W * d.Cin > 0x7fffffffLL) return SQN_ERR_UNSUPPORTED;
    p.M = (int)M;
    p.Kdim = (int)Kdim;
    p.out_c_offset = d.out_c_offset; p.out_c_total = d.out_c_total; p.relu = d.relu;

    const bool vec = (d.Cin % 4 == 0);
    // output-layer tile: the candidate that wastes the fewest padded columns, larger on ties
    const int cand[6] = {128, 96, 64, 48, 32, 16};
    int best = 128;
    long long best_waste = -1;
    for (int i = 0; i < 6; ++i) {
        const int bn = cand[i];
        const long long waste = (long long)((d.Cout + bn - 1) / bn) * bn - d.Cout;
        if (best_waste < 0 || waste < best_waste) { best_waste = waste; best = bn; }
    }
    // Small layers (a batch of one image): that tile would give the GPU a handful of CTAs.  When it leaves SMs
    // idle, the tile with the least estimated time is taken instead: rounds of CTAs per SM x tile area / relative
    // FFMA efficiency of the thread tile (8 x TN: fewer output layers per thread mean more shared-memory loads per
    // FFMA).  The sum over the reduction index runs in the same order for every tile shape, so the values do not
    // depend on this choice.
    int sms = 148;
    {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    auto ctas_of = [&](int tm, int tn) { return ((M + tm - 1) / tm) * (long long)((d.Cout + tn - 1) / tn); };
    int bm = best <= 32 ? 256 : 128, bn = best;
    if (ctas_of(bm, bn) < sms) {
        static const struct { int bm, bn; double eff; } shapes[9] = {
            {128, 128, 1.0}, {128, 96, 0.95}, {128, 64, 0.85}, {64, 128, 0.85}, {128, 48, 0.75},
            {256, 32, 0.85}, {64, 64, 0.6},   {256, 16, 0.6},  {64, 32, 0.4}};
        double best_t = -1.0;
        for (const auto& sh : shapes) {
            const long long c = ctas_of(sh.bm, sh.bn);
            const double t = (double)((c + sms - 1) / sms) * sh.bm * sh.bn / sh.eff;
            if (best_t < 0 || t < best_t) { best_t = t; bm = sh.bm; bn = sh.bn; }
        }
    }
    switch (bm * 1000 + bn) {
        case 128128: return launch_cfg<128, 128, 4, 2>(p, vec, stream);
        case 128096: return launch_cfg<128, 96, 2, 3>(p, vec, stream);
        case 128064: return launch_cfg<128, 64, 4, 1>(p, vec, stream);
        case 128048: return launch_cfg<128, 48, 1, 3>(p, vec, stream);
        case 256032: return launch_cfg<256, 32, 4, 1>(p, vec, stream);
        case 256016: return launch_cfg<256, 16, 2, 1>(p, vec, stream);
        case 64128: return launch_cfg<64, 128, 4, 1>(p, vec, stream);
        case 64064: return launch_cfg<64, 64, 2, 1>(p, vec, stream);
        default: return launch_cfg<64, 32, 1, 1>(p, vec, stream);
    }
}

}  // namespace sqn
