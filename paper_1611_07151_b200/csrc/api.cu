// C-ABI entry points: argument validation, dispatch, the fire layer and the SqueezeNet v1.0
// forward composition, host-side layout helpers.  No device memory is allocated here.
#include <atomic>
#include <cstdlib>
#include <cmath>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

#include <cuda_fp16.h>

#include "sqn_internal.h"

namespace sqn {

static std::atomic<unsigned long long> g_launches{0};
void note_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }
bool chained_launch_enabled()
{
    static const bool on = [] {
        const char* v = std::getenv("SQN_CHAINED_LAUNCH");
        return !(v && v[0] == '0');
    }();
    return on;
}

// The two expands of a fire layer go out as one launch (bf16) unless SQN_PAIR_LAUNCH=0.
bool pair_launch_enabled()
{
    static const bool on = [] {
        const char* v = std::getenv("SQN_PAIR_LAUNCH");
        return !(v && v[0] == '0');
    }();
    return on;
}

__device__ int g_device_status;   // written by kernels whose bounded waits run out

int* device_status_word()
{
    static std::mutex mu;
    static int* ptrs[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
        ptrs[dev] = static_cast<int*>(p);
    }
    return ptrs[dev];
}

namespace {

inline bool is16(int dtype) { return dtype == SQN_BF16 || dtype == SQN_F16; }      // the tensor-core paths
inline bool valid_dtype(int dtype) { return dtype == SQN_F32 || is16(dtype); }
inline size_t esize(int dtype) { return is16(dtype) ? 2 : 4; }
inline int out_extent(int H, int K, int S, int pad) { return (H + 2 * pad - K) / S + 1; }

inline uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);   // NaN stays NaN
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}
inline float bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}
// fp32 <-> the 16-bit storage type `dtype` (bf16 or fp16), round to nearest even
inline uint16_t f32_to_16(float f, int dtype)
{
    if (dtype == SQN_F16) {
        const __half h = __float2half_rn(f);
        uint16_t u;
        std::memcpy(&u, &h, 2);
        return u;
    }
    return f32_to_bf16_rne(f);
}
inline float f16bits_to_f32(uint16_t u, int dtype)
{
    if (dtype == SQN_F16) {
        __half h;
        std::memcpy(&h, &u, 2);
        return __half2float(h);
    }
    return bf16_to_f32(u);
}

// Validates one convolution request and fills the descriptor.
int make_conv_desc(const void* in, const void* w, const void* bias, void* out, int Cin, int Cout, int H, int W, int K,
                   int S, int pad, int batch, int relu, int c_off, int c_total, ConvDesc* d)
{
    if (!in || !w || !bias || !out) return SQN_ERR_BADARG;
    if (Cin <= 0 || Cout <= 0 || H <= 0 || W <= 0 || K <= 0 || S <= 0 || pad < 0 || batch <= 0) return SQN_ERR_BADARG;
    if (H + 2 * pad < K || W + 2 * pad < K) return SQN_ERR_BADARG;
    if (c_total == 0) { c_total = Cout; if (c_off != 0) return SQN_ERR_BADARG; }
    if (c_off < 0 || c_off + Cout > c_total) return SQN_ERR_BADARG;
    if (!aligned16(in) || !aligned16(w) || !aligned16(out) || (reinterpret_cast<uintptr_t>(bias) & 3u))
        return SQN_ERR_ALIGN;
    d->in = in; d->w = w; d->bias = static_cast<const float*>(bias); d->out = out;
    d->N = batch; d->Cin = Cin; d->H = H; d->W = W; d->Cout = Cout; d->K = K; d->S = S; d->pad = pad;
    d->OH = out_extent(H, K, S, pad); d->OW = out_extent(W, K, S, pad);
    d->out_c_offset = c_off; d->out_c_total = c_total; d->relu = relu ? 1 : 0;
    d->pool = 0;
    d->params_static = 0;
    d->stem_prepacked = 0;
    d->f16 = 0;
    return SQN_OK;
}

inline bool is_stem_shape(const ConvDesc& d) { return d.K == 7 && d.S == 2 && d.pad == 0 && d.Cin == 3; }

int run_conv(const ConvDesc& d_in, int dtype, void* ws, size_t ws_bytes, cudaStream_t stream)
{
    if (dtype == SQN_F32) return d_in.pool ? SQN_ERR_UNSUPPORTED : launch_conv_f32(d_in, stream);
    if (!is16(dtype)) return SQN_ERR_BADARG;
    ConvDesc d = d_in;
    d.f16 = dtype == SQN_F16 ? 1 : 0;
    if (is_stem_shape(d)) {
        const int rc = launch_stem_pack_bf16(d, ws, ws_bytes, stream);
        return rc != SQN_OK ? rc : launch_stem_conv_bf16(d, ws, ws_bytes, stream);
    }
    const int rc = conv_bf16_supported(d);
    if (rc != SQN_OK) return rc;
    return launch_conv_bf16(d, stream);
}

// The two expands of a fire layer (same input, disjoint layer slices of one output): one launch where the bf16
// kernels have a common variant, else two.  *paired tells which.
int run_expands(const ConvDesc& d1_in, const ConvDesc& d3_in, int dtype, cudaStream_t stream, bool* paired)
{
    if (paired) *paired = false;
    ConvDesc d1 = d1_in, d3 = d3_in;
    d1.f16 = d3.f16 = dtype == SQN_F16 ? 1 : 0;
    if (is16(dtype) && fused_fire_enabled() && !d1.pool && !d3.pool) {
        const int rc = launch_fire_expands_bf16(d1, d3, stream);     // flat-patch kernel, kernels resident per CTA
        if (rc == SQN_OK) {
            if (paired) *paired = true;
            return SQN_OK;
        }
        if (rc != SQN_ERR_UNSUPPORTED) return rc;
    }
    if (is16(dtype) && pair_launch_enabled() && conv_bf16_supported(d1) == SQN_OK && conv_bf16_supported(d3) == SQN_OK) {
        const int rc = launch_conv_bf16_pair(d1, d3, stream);
        if (rc == SQN_OK) {
            if (paired) *paired = true;
            return SQN_OK;
        }
        if (rc != SQN_ERR_UNSUPPORTED) return rc;
    }
    const int rc = run_conv(d1, dtype, nullptr, 0, stream);
    return rc != SQN_OK ? rc : run_conv(d3, dtype, nullptr, 0, stream);
}

}  // namespace
}  // namespace sqn

using namespace sqn;

// ------------------------------------------------------------------------- convolution
extern "C" int conv_forward_ex(const void* in, const void* weights, const void* bias, void* out, int numInputLayers,
                               int numOutputLayers, int H, int W, int K, int S, int pad, int batch,
                               const sqn_conv_opts* opts)
{
    sqn_conv_opts o;
    if (opts) o = *opts;
    else { std::memset(&o, 0, sizeof(o)); o.dtype = SQN_F32; o.relu = 1; }
    if (!valid_dtype(o.dtype)) return SQN_ERR_BADARG;
    ConvDesc d;
    const int rc = make_conv_desc(in, weights, bias, out, numInputLayers, numOutputLayers, H, W, K, S, pad, batch,
                                  o.relu, o.out_c_offset, o.out_c_total, &d);
    if (rc != SQN_OK) return rc;
    if (o.fuse_global_avgpool) {
        if (o.fuse_maxpool || o.out_c_total != 0) return SQN_ERR_BADARG;
        if (!is16(o.dtype)) return SQN_ERR_UNSUPPORTED;
        d.f16 = o.dtype == SQN_F16 ? 1 : 0;
        return launch_conv_avgpool_bf16(d, static_cast<float*>(out), static_cast<cudaStream_t>(o.stream));
    }
    if (o.fuse_maxpool) {
        if (d.OH < 3 || d.OW < 3) return SQN_ERR_BADARG;
        d.pool = 1;
    }
    return run_conv(d, o.dtype, o.workspace, o.workspace_bytes, static_cast<cudaStream_t>(o.stream));
}

extern "C" int conv_forward(const void* in, const void* weights, const void* bias, void* out, int numInputLayers,
                            int numOutputLayers, int H, int W, int K, int S, int pad, int batch)
{
    return conv_forward_ex(in, weights, bias, out, numInputLayers, numOutputLayers, H, W, K, S, pad, batch, nullptr);
}

extern "C" int conv_workspace_bytes(int Cin, int Cout, int H, int W, int K, int S, int pad, int batch, int dtype,
                                    size_t* bytes)
{
    if (!bytes || Cin <= 0 || Cout <= 0 || H <= 0 || W <= 0 || K <= 0 || S <= 0 || pad < 0 || batch <= 0)
        return SQN_ERR_BADARG;
    if (!valid_dtype(dtype)) return SQN_ERR_BADARG;
    *bytes = 0;
    if (is16(dtype) && K == 7 && S == 2 && pad == 0 && Cin == 3) *bytes = stem_bf16_workspace_bytes(batch, H, W, Cout);
    return SQN_OK;
}

// ------------------------------------------------------------------------------- fire
extern "C" int fire_forward(const void* in, const void* w_sq, const void* b_sq, const void* w_e1, const void* b_e1,
                            const void* w_e3, const void* b_e3, void* squeeze_scratch, void* out, int Cin, int s,
                            int e1, int e3, int H, int W, int batch, int dtype, void* stream)
{
    if (!valid_dtype(dtype)) return SQN_ERR_BADARG;
    if (!squeeze_scratch) return SQN_ERR_BADARG;
    if (e1 <= 0 || e3 <= 0) return SQN_ERR_BADARG;
    ConvDesc dsq, d1, d3;
    int rc = make_conv_desc(in, w_sq, b_sq, squeeze_scratch, Cin, s, H, W, 1, 1, 0, batch, 1, 0, 0, &dsq);
    if (rc != SQN_OK) return rc;
    rc = make_conv_desc(squeeze_scratch, w_e1, b_e1, out, s, e1, H, W, 1, 1, 0, batch, 1, 0, e1 + e3, &d1);
    if (rc != SQN_OK) return rc;
    rc = make_conv_desc(squeeze_scratch, w_e3, b_e3, out, s, e3, H, W, 3, 1, 1, batch, 1, e1, e1 + e3, &d3);
    if (rc != SQN_OK) return rc;
    dsq.f16 = d1.f16 = d3.f16 = dtype == SQN_F16 ? 1 : 0;
    if (is16(dtype)) {
        if ((rc = conv_bf16_supported(dsq)) != SQN_OK) return rc;
        if ((rc = conv_bf16_supported(d1)) != SQN_OK) return rc;
        if ((rc = conv_bf16_supported(d3)) != SQN_OK) return rc;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (is16(dtype) && fused_fire_enabled()) {
        rc = launch_fire_fused_bf16(dsq, d1, d3, st);       // one kernel, squeeze_scratch stays untouched
        if (rc != SQN_ERR_UNSUPPORTED) return rc;
    }
    if ((rc = run_conv(dsq, dtype, nullptr, 0, st)) != SQN_OK) return rc;
    return run_expands(d1, d3, dtype, st, nullptr);
}

// ------------------------------------------------- fire layer without any allocation
// Scratch for fire_forward_static: lives in the library image, one copy per GPU that loads it.
constexpr size_t kStaticFireScratchBytes = (size_t)8 << 20;
static __device__ __align__(256) unsigned char g_fire_static_scratch[kStaticFireScratchBytes];

// Device address of the array above on the current device.  In host code the array's name is only a
// handle for the runtime, not an address a kernel may use, so the address is looked up once per
// device (with that device current) and remembered.
static void* fire_static_scratch_ptr()
{
    static std::mutex mu;
    static void* ptrs[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_fire_static_scratch) != cudaSuccess) return nullptr;
        ptrs[dev] = p;
    }
    return ptrs[dev];
}

extern "C" int fire_forward_static(const void* in, const void* w_sq, const void* b_sq, const void* w_e1,
                                   const void* b_e1, const void* w_e3, const void* b_e3, void* out, int Cin, int s,
                                   int e1, int e3, int H, int W, int batch, int dtype, void* stream)
{
    if (!valid_dtype(dtype)) return SQN_ERR_BADARG;
    if (e1 <= 0 || e3 <= 0 || s <= 0 || H <= 0 || W <= 0 || batch <= 0) return SQN_ERR_BADARG;
    // the squeeze map must fit the built-in scratch
    // (checked factor by factor: the product of four ints can wrap a 64-bit word)
    unsigned long long need = esize(dtype);
    for (const int f : {batch, H, W, s}) {
        need *= (unsigned long long)f;
        if (need > kStaticFireScratchBytes) return SQN_ERR_WORKSPACE;
    }
    void* scratch = fire_static_scratch_ptr();
    if (!scratch) return SQN_ERR_CUDA;
    ConvDesc dsq, d1, d3;
    int rc = make_conv_desc(in, w_sq, b_sq, scratch, Cin, s, H, W, 1, 1, 0, batch, 1, 0, 0, &dsq);
    if (rc != SQN_OK) return rc;
    rc = make_conv_desc(scratch, w_e1, b_e1, out, s, e1, H, W, 1, 1, 0, batch, 1, 0, e1 + e3, &d1);
    if (rc != SQN_OK) return rc;
    rc = make_conv_desc(scratch, w_e3, b_e3, out, s, e3, H, W, 3, 1, 1, batch, 1, e1, e1 + e3, &d3);
    if (rc != SQN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const ConvDesc* seq[3] = {&dsq, &d1, &d3};
    dsq.f16 = d1.f16 = d3.f16 = dtype == SQN_F16 ? 1 : 0;
    if (is16(dtype))
        for (const ConvDesc* d : seq)
            if ((rc = conv_bf16_supported(*d)) != SQN_OK) return rc;
    for (const ConvDesc* d : seq) {
        rc = dtype == SQN_F32 ? launch_conv_f32(*d, st) : launch_conv_bf16_uncached(*d, st);
        if (rc != SQN_OK) return rc;
    }
    return SQN_OK;
}

// ---------------------------------------------------------------------------- pooling
extern "C" int maxpool3x3s2_forward(const void* in, void* out, int C, int H, int W, int batch, int dtype, void* stream)
{
    if (!in || !out || C <= 0 || H < 3 || W < 3 || batch <= 0) return SQN_ERR_BADARG;
    if (!valid_dtype(dtype)) return SQN_ERR_BADARG;
    if (!aligned16(in) || !aligned16(out)) return SQN_ERR_ALIGN;
    return launch_maxpool3x3s2(in, out, C, H, W, batch, dtype, static_cast<cudaStream_t>(stream));
}

extern "C" int avgpool_softmax_forward(const void* in, void* logits_f32, void* probs_f32, int C, int H, int W,
                                       int batch, int dtype, void* stream)
{
    if (!in || !logits_f32 || C <= 0 || H <= 0 || W <= 0 || batch <= 0) return SQN_ERR_BADARG;
    if (!valid_dtype(dtype)) return SQN_ERR_BADARG;
    if (C > 8192 || batch > 65535) return SQN_ERR_UNSUPPORTED;       // (the image index is the grid's y dimension)
    // the kernels read the map with 16-byte (bf16) or 8-byte (fp32) loads and the logits as floats
    if (!aligned16(in) || (reinterpret_cast<uintptr_t>(logits_f32) & 3u) || (reinterpret_cast<uintptr_t>(probs_f32) & 3u))
        return SQN_ERR_ALIGN;
    return launch_avgpool_softmax(in, static_cast<float*>(logits_f32), static_cast<float*>(probs_f32), C, H, W, batch,
                                  dtype, static_cast<cudaStream_t>(stream));
}

// ------------------------------------------------------------------ SqueezeNet v1.0
namespace {

struct FireSpec { const char* name; int cin, s, e, hw; bool pool_after; };
const FireSpec kFire[8] = {
    {"fire2", 96, 16, 64, 55, false},  {"fire3", 128, 16, 64, 55, false}, {"fire4", 128, 32, 128, 55, true},
    {"fire5", 256, 32, 128, 27, false}, {"fire6", 256, 48, 192, 27, false}, {"fire7", 384, 48, 192, 27, false},
    {"fire8", 384, 64, 256, 27, true},  {"fire9", 512, 64, 256, 13, false}};

struct Slot { std::string name; int C, H, W; size_t offset; };   // offset in bytes for batch 1 element counts below

}  // namespace

struct sqn_net {
    const void* w[26];
    const float* b[26];
    int dtype;
    int max_batch;
    std::vector<Slot> slots;   // per-image element counts; byte offsets are computed per batch
    // optional per-launch timing: a ring of event rows, one row per forward
    int prof_slots = 0;
    long long prof_forwards = 0;
    std::vector<std::string> prof_names;
    std::vector<std::vector<cudaEvent_t>> prof_events;
    // squeezenet_forward_host: the input copy of call k runs on a stream of its own into one of two staging
    // buffers, so that it overlaps the forward of call k-1
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t in_ready[2] = {nullptr, nullptr};   // copy into staging buffer b has finished
    cudaEvent_t in_free[2] = {nullptr, nullptr};    // the forward that read staging buffer b has finished
    int copy_device = -1;
    unsigned long long host_calls = 0;
    int stem_prepacked = 0;     // squeezenet_set_stem_prepacked
    int fused_head = 0;             // the last forward took conv10 and the average in one kernel (conv10's map was not stored)
    unsigned fused_fire_mask = 0;   // bit i: the last forward ran fire layer i as one kernel (its squeeze map was not stored)
};

namespace {

constexpr int IMG = 227;

void build_slots(sqn_net* net)
{
    auto add = [&](const std::string& n, int C, int H, int W) { net->slots.push_back({n, C, H, W, 0}); };
    add("conv1", 96, 111, 111);
    add("pool1", 96, 55, 55);
    for (const FireSpec& f : kFire) {
        add(std::string(f.name) + "_sq", f.s, f.hw, f.hw);
        add(f.name, 2 * f.e, f.hw, f.hw);
        if (f.pool_after) add(std::string("pool") + (f.name + 4), 2 * f.e, (f.hw - 3) / 2 + 1, (f.hw - 3) / 2 + 1);
    }
    add("conv10", 1000, 13, 13);
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Byte offset of every slot inside the workspace for a given batch; returns total bytes.
size_t layout(const sqn_net* net, int batch, std::vector<size_t>* offs, size_t* stem_off)
{
    size_t cur = 0;
    const size_t es = esize(net->dtype);
    if (offs) offs->clear();
    for (const Slot& s : net->slots) {
        if (offs) offs->push_back(cur);
        cur = align_up(cur + (size_t)batch * s.C * s.H * s.W * es, 1024);
    }
    if (stem_off) *stem_off = cur;
    if (is16(net->dtype)) cur = align_up(cur + stem_bf16_workspace_bytes(batch, IMG, IMG, 96), 1024);
    return cur;
}

// Bytes of one input batch in the layout the net reads.
size_t input_bytes(const sqn_net* net, int batch)
{
    if (net->stem_prepacked) return (size_t)batch * stem_packed_rows(IMG) * stem_packed_cols(IMG) * 4 * 2;
    return (size_t)batch * IMG * IMG * 3 * esize(net->dtype);
}

int find_slot(const sqn_net* net, const char* name)
{
    for (size_t i = 0; i < net->slots.size(); ++i)
        if (net->slots[i].name == name) return (int)i;
    return -1;
}

}  // namespace

namespace {
void free_profile(sqn_net* net);
void free_copy_pipeline(sqn_net* net)
{
    for (int b = 0; b < 2; ++b) {
        if (net->in_ready[b]) cudaEventDestroy(net->in_ready[b]);
        if (net->in_free[b]) cudaEventDestroy(net->in_free[b]);
        net->in_ready[b] = net->in_free[b] = nullptr;
    }
    if (net->copy_stream) cudaStreamDestroy(net->copy_stream);
    net->copy_stream = nullptr;
    net->copy_device = -1;
    net->host_calls = 0;
}
}

extern "C" int squeezenet_create(sqn_net** net, const void* const* weights26, const void* const* bias26, int dtype,
                                 int max_batch)
{
    if (!net || !weights26 || !bias26 || max_batch <= 0) return SQN_ERR_BADARG;
    if (!valid_dtype(dtype)) return SQN_ERR_BADARG;
    for (int i = 0; i < 26; ++i) {
        if (!weights26[i] || !bias26[i]) return SQN_ERR_BADARG;
        if (!aligned16(weights26[i]) || (reinterpret_cast<uintptr_t>(bias26[i]) & 3u)) return SQN_ERR_ALIGN;
    }
    sqn_net* n = new (std::nothrow) sqn_net();
    if (!n) return SQN_ERR_BADARG;
    for (int i = 0; i < 26; ++i) { n->w[i] = weights26[i]; n->b[i] = static_cast<const float*>(bias26[i]); }
    n->dtype = dtype;
    n->max_batch = max_batch;
    build_slots(n);
    *net = n;
    return SQN_OK;
}

extern "C" int squeezenet_destroy(sqn_net* net)
{
    if (net) {
        free_profile(net);
        free_copy_pipeline(net);
    }
    delete net;
    return SQN_OK;
}

extern "C" int squeezenet_set_stem_prepacked(sqn_net* net, int on)
{
    if (!net) return SQN_ERR_BADARG;
    if (net->dtype != SQN_BF16) return on ? SQN_ERR_UNSUPPORTED : SQN_OK;      // (the pack helpers write bf16)
    net->stem_prepacked = on ? 1 : 0;
    return SQN_OK;
}

extern "C" int squeezenet_workspace_bytes(const sqn_net* net, int batch, size_t* bytes)
{
    if (!net || !bytes || batch <= 0 || batch > net->max_batch) return SQN_ERR_BADARG;
    *bytes = layout(net, batch, nullptr, nullptr);
    return SQN_OK;
}

extern "C" int squeezenet_layer_output(const sqn_net* net, const char* name, void* workspace, int batch, void** ptr,
                                       int* C, int* H, int* W)
{
    if (!net || !name || !workspace || !ptr || batch <= 0 || batch > net->max_batch) return SQN_ERR_BADARG;
    const int i = find_slot(net, name);
    if (i < 0) return SQN_ERR_BADARG;
    if (is16(net->dtype) && batch >= 16 &&
        (std::strcmp(name, "conv1") == 0 || std::strcmp(name, "fire4") == 0 || std::strcmp(name, "fire8") == 0))
        return SQN_ERR_UNSUPPORTED;   // computed inside the kernels that write pool1 / pool4, never stored
    if (net->fused_head && std::strcmp(name, "conv10") == 0) return SQN_ERR_UNSUPPORTED;     // averaged inside the kernel
    for (int f = 0; f < 8; ++f)
        if ((net->fused_fire_mask >> f & 1u) && std::string(kFire[f].name) + "_sq" == name)
            return SQN_ERR_UNSUPPORTED;   // kept in shared memory by the fused fire kernel of the last forward
    std::vector<size_t> offs;
    layout(net, batch, &offs, nullptr);
    *ptr = static_cast<char*>(workspace) + offs[i];
    if (C) *C = net->slots[i].C;
    if (H) *H = net->slots[i].H;
    if (W) *W = net->slots[i].W;
    return SQN_OK;
}

namespace {

void free_profile(sqn_net* net)
{
    for (auto& row : net->prof_events)
        for (cudaEvent_t e : row) cudaEventDestroy(e);
    net->prof_events.clear();
    net->prof_names.clear();
    net->prof_slots = 0;
    net->prof_forwards = 0;
}

}  // namespace

extern "C" int squeezenet_forward(sqn_net* net, const void* in_nhwc, void* logits_f32, void* probs_f32,
                                  void* workspace, int batch, void* stream)
{
    if (!net || !in_nhwc || !logits_f32 || batch <= 0 || batch > net->max_batch) return SQN_ERR_BADARG;
    if (!workspace) return SQN_ERR_WORKSPACE;
    if (!aligned16(in_nhwc) || !aligned16(workspace)) return SQN_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int dt = net->dtype;
    std::vector<size_t> offs;
    size_t stem_off = 0;
    const size_t total = layout(net, batch, &offs, &stem_off);
    char* ws = static_cast<char*>(workspace);
    auto buf = [&](const std::string& name) -> void* { return ws + offs[find_slot(net, name.c_str())]; };

    // per-launch timing (off unless squeezenet_profile enabled it)
    const bool prof = net->prof_slots > 0;
    std::vector<cudaEvent_t>* row = prof ? &net->prof_events[net->prof_forwards % net->prof_slots] : nullptr;
    const bool first = prof && net->prof_names.empty();
    size_t mark_i = 0;
    auto mark = [&](const char* name) {
        if (!prof) return;
        if (first) net->prof_names.push_back(name);
        if (row->size() <= mark_i) {
            cudaEvent_t e;
            cudaEventCreate(&e);
            row->push_back(e);
        }
        cudaEventRecord((*row)[mark_i++], st);
    };
    mark("start");

    int rc;
    ConvDesc d;
    // conv1 7x7/2 + ReLU, then max-pool
    // The fused conv+pool kernels hand a whole strip of 16 output rows to one CTA: worth it once there are
    // enough strips to fill the GPU (8 per image for conv1, 4 for fire4), i.e. from a batch of 16 on.
    const bool fuse_pools = is16(dt) && batch >= 16;
    const int f16 = dt == SQN_F16 ? 1 : 0;
    // bf16 stem: on operands packed offline (squeezenet_set_stem_prepacked), else after a repack pass
    auto stem_bf16 = [&](ConvDesc& sd) -> int {
        sd.params_static = 1;
        sd.f16 = f16;
        if (net->stem_prepacked) {
            sd.stem_prepacked = 1;
            return launch_stem_conv_bf16_prepacked(sd, st);
        }
        const int prc = launch_stem_pack_bf16(sd, ws + stem_off, total - stem_off, st);
        if (prc != SQN_OK) return prc;
        mark("conv1_pack");
        return launch_stem_conv_bf16(sd, ws + stem_off, total - stem_off, st);
    };
    if (fuse_pools) {
        // stem and its max-pool in one kernel: the 96x111x111 map never goes to memory
        rc = make_conv_desc(in_nhwc, net->w[0], net->b[0], buf("pool1"), 3, 96, IMG, IMG, 7, 2, 0, batch, 1, 0, 0, &d);
        if (rc != SQN_OK) return rc;
        d.pool = 1;
        if ((rc = stem_bf16(d)) != SQN_OK) return rc;
        mark("conv1+pool1");
    } else {
        rc = make_conv_desc(in_nhwc, net->w[0], net->b[0], buf("conv1"), 3, 96, IMG, IMG, 7, 2, 0, batch, 1, 0, 0, &d);
        if (rc != SQN_OK) return rc;
        if (is16(dt)) {
            if ((rc = stem_bf16(d)) != SQN_OK) return rc;
        } else {
            if ((rc = launch_conv_f32(d, st)) != SQN_OK) return rc;
        }
        mark("conv1");
        if ((rc = launch_maxpool3x3s2(buf("conv1"), buf("pool1"), 96, 111, 111, batch, dt, st)) != SQN_OK) return rc;
        mark("pool1");
    }

    const void* cur = buf("pool1");
    net->fused_fire_mask = 0;
    for (int i = 0; i < 8; ++i) {
        const FireSpec& f = kFire[i];
        void* sq = buf(std::string(f.name) + "_sq");
        void* out = buf(f.name);
        ConvDesc dsq, d1, d3;
        rc = make_conv_desc(cur, net->w[1 + 3 * i], net->b[1 + 3 * i], sq, f.cin, f.s, f.hw, f.hw, 1, 1, 0, batch, 1, 0,
                            0, &dsq);
        if (rc != SQN_OK) return rc;
        rc = make_conv_desc(sq, net->w[2 + 3 * i], net->b[2 + 3 * i], out, f.s, f.e, f.hw, f.hw, 1, 1, 0, batch, 1, 0,
                            2 * f.e, &d1);
        if (rc != SQN_OK) return rc;
        rc = make_conv_desc(sq, net->w[3 + 3 * i], net->b[3 + 3 * i], out, f.s, f.e, f.hw, f.hw, 3, 1, 1, batch, 1, f.e,
                            2 * f.e, &d3);
        if (rc != SQN_OK) return rc;
        // the net's kernels and bias are not written by anything this forward enqueues
        dsq.params_static = d1.params_static = d3.params_static = 1;
        dsq.f16 = d1.f16 = d3.f16 = f16;
        const std::string nm(f.name);
        // bf16: squeeze and both expands as one kernel where it applies (no pool behind the layer)
        if (is16(dt) && fused_fire_enabled() && !(f.pool_after && fuse_pools)) {
            rc = launch_fire_fused_bf16(dsq, d1, d3, st);
            if (rc == SQN_OK) {
                net->fused_fire_mask |= 1u << i;
                mark((nm + "_fused").c_str());
                cur = out;
                if (f.pool_after) {
                    const std::string pn = std::string("pool") + (f.name + 4);
                    void* po = buf(pn);
                    if ((rc = launch_maxpool3x3s2(cur, po, 2 * f.e, f.hw, f.hw, batch, dt, st)) != SQN_OK) return rc;
                    mark(pn.c_str());
                    cur = po;
                }
                continue;
            }
            if (rc != SQN_ERR_UNSUPPORTED) return rc;
        }
        if ((rc = run_conv(dsq, dt, nullptr, 0, st)) != SQN_OK) return rc;
        mark((nm + "_sq").c_str());
        // bf16: where a max-pool follows and the expands' kernels fit in shared memory, both expands pool
        // in their epilogues and write their halves of the pooled map; the unpooled map is never stored
        bool fused_pool = false;
        if (f.pool_after && fuse_pools) {
            const std::string pn = std::string("pool") + (f.name + 4);
            ConvDesc p1 = d1, p3 = d3;
            p1.out = p3.out = buf(pn);
            p1.pool = p3.pool = 1;
            // the pooled kernels take up to 128 output layers: wider expands (fire8: 256) go out in slices of 128
            const int parts = f.e > 128 && f.e % 128 == 0 ? f.e / 128 : 1;
            ConvDesc q1[4], q3[4];
            bool fits = parts <= 4;
            for (int h = 0; h < parts && fits; ++h) {
                q1[h] = p1; q3[h] = p3;
                q1[h].Cout = q3[h].Cout = f.e / parts;
                q1[h].w = static_cast<const char*>(p1.w) + (size_t)h * (f.e / parts) * f.s * esize(dt);
                q3[h].w = static_cast<const char*>(p3.w) + (size_t)h * (f.e / parts) * 9 * f.s * esize(dt);
                q1[h].bias = p1.bias + h * (f.e / parts);
                q3[h].bias = p3.bias + h * (f.e / parts);
                q1[h].out_c_offset = p1.out_c_offset + h * (f.e / parts);
                q3[h].out_c_offset = p3.out_c_offset + h * (f.e / parts);
                fits = conv_bf16_pool_fits(q1[h]) && conv_bf16_pool_fits(q3[h]);
            }
            if (fits) {
                if (pair_launch_enabled()) {
                    // the 1x1 expand riding on the 3x3 expand's patches (per slice of 128 layers), all in one launch
                    bool done = false;
                    if (parts <= 2) {
                        rc = launch_conv_bf16_pool_riders(q3, q1, parts, st);
                        if (rc != SQN_OK && rc != SQN_ERR_UNSUPPORTED) return rc;
                        done = rc == SQN_OK;
                    }
                    if (!done && parts == 2) {  // both slices of both expands as one grid, the 3x3 slices first
                        const ConvDesc four[4] = {q3[0], q3[1], q1[0], q1[1]};
                        rc = launch_conv_bf16_pool4(four, st);
                        if (rc != SQN_OK && rc != SQN_ERR_UNSUPPORTED) return rc;
                        done = rc == SQN_OK;
                    }
                    for (int h = 0; h < parts && !done; ++h)
                        if ((rc = run_expands(q1[h], q3[h], dt, st, nullptr)) != SQN_OK) return rc;
                    mark((nm + "_e1+e3+pool").c_str());
                } else {
                    for (int h = 0; h < parts; ++h)
                        if ((rc = run_conv(q1[h], dt, nullptr, 0, st)) != SQN_OK) return rc;
                    mark((nm + "_e1+pool").c_str());
                    for (int h = 0; h < parts; ++h)
                        if ((rc = run_conv(q3[h], dt, nullptr, 0, st)) != SQN_OK) return rc;
                    mark((nm + "_e3+pool").c_str());
                }
                cur = buf(pn);
                fused_pool = true;
            }
        }
        if (!fused_pool) {
            if (is16(dt) && pair_launch_enabled()) {
                if ((rc = run_expands(d1, d3, dt, st, nullptr)) != SQN_OK) return rc;
                mark((nm + "_e1+e3").c_str());
            } else {
                if ((rc = run_conv(d1, dt, nullptr, 0, st)) != SQN_OK) return rc;
                mark((nm + "_e1").c_str());
                if ((rc = run_conv(d3, dt, nullptr, 0, st)) != SQN_OK) return rc;
                mark((nm + "_e3").c_str());
            }
            cur = out;
            if (f.pool_after) {
                const std::string pn = std::string("pool") + (f.name + 4);
                void* po = buf(pn);
                if ((rc = launch_maxpool3x3s2(cur, po, 2 * f.e, f.hw, f.hw, batch, dt, st)) != SQN_OK) return rc;
                mark(pn.c_str());
                cur = po;
            }
        }
    }
    // conv10 1x1 + ReLU, global average, softmax
    rc = make_conv_desc(cur, net->w[25], net->b[25], buf("conv10"), 512, 1000, 13, 13, 1, 1, 0, batch, 1, 0, 0, &d);
    if (rc != SQN_OK) return rc;
    d.params_static = 1;
    d.f16 = f16;
    net->fused_head = 0;
    if (is16(dt) && fused_head_enabled()) {
        // conv10, ReLU and the global average in one kernel: the 1000 x 13 x 13 map is never stored
        rc = launch_conv_avgpool_bf16(d, static_cast<float*>(logits_f32), st);
        if (rc == SQN_OK) {
            net->fused_head = 1;
            mark("conv10+avgpool");
            if (probs_f32) {
                if ((rc = launch_softmax(static_cast<const float*>(logits_f32), static_cast<float*>(probs_f32), 1000, batch, st)) != SQN_OK)
                    return rc;
                mark("softmax");
            }
            if (prof) net->prof_forwards++;
            return SQN_OK;
        }
        if (rc != SQN_ERR_UNSUPPORTED) return rc;
    }
    if ((rc = run_conv(d, dt, nullptr, 0, st)) != SQN_OK) return rc;
    mark("conv10");
    rc = launch_avgpool_softmax(buf("conv10"), static_cast<float*>(logits_f32), static_cast<float*>(probs_f32), 1000,
                                13, 13, batch, dt, st);
    if (rc != SQN_OK) return rc;
    mark("head");
    if (prof) net->prof_forwards++;
    return SQN_OK;
}

extern "C" int squeezenet_host_workspace_bytes(const sqn_net* net, int batch, size_t* bytes)
{
    if (!net || !bytes || batch <= 0 || batch > net->max_batch) return SQN_ERR_BADARG;
    const size_t in_bytes = align_up(input_bytes(net, batch), 1024);
    const size_t out_bytes = align_up((size_t)batch * 1000 * sizeof(float), 1024);
    *bytes = layout(net, batch, nullptr, nullptr) + 2 * in_bytes + 2 * out_bytes;
    return SQN_OK;
}

namespace {
// Stream and events of the input-copy pipeline, made on the first host-buffer forward on a device.
int ensure_copy_pipeline(sqn_net* net)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SQN_ERR_CUDA;
    if (net->copy_stream && net->copy_device == dev) return SQN_OK;
    free_copy_pipeline(net);
    if (cudaStreamCreateWithFlags(&net->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return SQN_ERR_CUDA;
    for (int b = 0; b < 2; ++b)
        if (cudaEventCreateWithFlags(&net->in_ready[b], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&net->in_free[b], cudaEventDisableTiming) != cudaSuccess) {
            free_copy_pipeline(net);
            return SQN_ERR_CUDA;
        }
    net->copy_device = dev;
    return SQN_OK;
}
}  // namespace

extern "C" int squeezenet_forward_host(sqn_net* net, const void* in_host, void* logits_host, void* probs_host,
                                       void* workspace, int batch, void* stream)
{
    if (!net || !in_host || !logits_host || batch <= 0 || batch > net->max_batch) return SQN_ERR_BADARG;
    if (!workspace) return SQN_ERR_WORKSPACE;
    if (!aligned16(workspace)) return SQN_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc = ensure_copy_pipeline(net);
    if (rc != SQN_OK) return rc;
    const size_t fwd_bytes = layout(net, batch, nullptr, nullptr);
    const size_t in_bytes = input_bytes(net, batch);
    const size_t out_bytes = (size_t)batch * 1000 * sizeof(float);
    char* ws = static_cast<char*>(workspace);
    const int b = (int)(net->host_calls & 1ull);
    char* d_in = ws + fwd_bytes + (size_t)b * align_up(in_bytes, 1024);
    char* d_logits = ws + fwd_bytes + 2 * align_up(in_bytes, 1024);
    char* d_probs = d_logits + align_up(out_bytes, 1024);
    // Input copy on the copy stream: it waits only for the forward of two calls ago (the last reader of this
    // staging buffer), not for the work queued on `stream`, and so runs beside the forward of the call before.
    if (net->host_calls >= 2 && cudaStreamWaitEvent(net->copy_stream, net->in_free[b], 0) != cudaSuccess) return SQN_ERR_CUDA;
    if (cudaMemcpyAsync(d_in, in_host, in_bytes, cudaMemcpyHostToDevice, net->copy_stream) != cudaSuccess) return SQN_ERR_CUDA;
    if (cudaEventRecord(net->in_ready[b], net->copy_stream) != cudaSuccess) return SQN_ERR_CUDA;
    if (cudaStreamWaitEvent(st, net->in_ready[b], 0) != cudaSuccess) return SQN_ERR_CUDA;
    net->host_calls++;
    rc = squeezenet_forward(net, d_in, d_logits, probs_host ? d_probs : nullptr, workspace, batch, stream);
    if (cudaEventRecord(net->in_free[b], st) != cudaSuccess) return SQN_ERR_CUDA;
    if (rc != SQN_OK) return rc;
    if (cudaMemcpyAsync(logits_host, d_logits, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return SQN_ERR_CUDA;
    if (probs_host && cudaMemcpyAsync(probs_host, d_probs, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return SQN_ERR_CUDA;
    return SQN_OK;
}

extern "C" int squeezenet_profile(sqn_net* net, int slots)
{
    if (!net || slots < 0 || slots > 4096) return SQN_ERR_BADARG;
    free_profile(net);
    net->prof_slots = slots;
    net->prof_events.resize((size_t)slots);
    return SQN_OK;
}

extern "C" int squeezenet_profile_read(sqn_net* net, float* ms_sum, int capacity, int* launches, int* forwards)
{
    if (!net || !launches || !forwards) return SQN_ERR_BADARG;
    const int n = net->prof_names.empty() ? 0 : (int)net->prof_names.size() - 1;
    *launches = n;
    const long long have = net->prof_forwards < net->prof_slots ? net->prof_forwards : net->prof_slots;
    *forwards = (int)have;
    if (!ms_sum) return SQN_OK;
    if (capacity < n) return SQN_ERR_BADARG;
    for (int i = 0; i < n; ++i) ms_sum[i] = 0.f;
    for (long long r = 0; r < have; ++r) {
        std::vector<cudaEvent_t>& row = net->prof_events[(size_t)r];
        if ((int)row.size() < n + 1) return SQN_ERR_CUDA;
        if (cudaEventSynchronize(row[n]) != cudaSuccess) return SQN_ERR_CUDA;
        for (int i = 0; i < n; ++i) {
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, row[i], row[i + 1]) != cudaSuccess) return SQN_ERR_CUDA;
            ms_sum[i] += ms;
        }
    }
    return SQN_OK;
}

extern "C" const char* squeezenet_profile_name(const sqn_net* net, int i)
{
    if (!net || i < 0 || i + 1 >= (int)net->prof_names.size()) return "";
    return net->prof_names[(size_t)i + 1].c_str();
}

// ---------------------------------------------------------------- host layout helpers
extern "C" int sqn_pack_weights_oihw_to_ohwi(const float* src, void* dst, int O, int I, int K, int dtype)
{
    if (!src || !dst || O <= 0 || I <= 0 || K <= 0) return SQN_ERR_BADARG;
    if (!valid_dtype(dtype)) return SQN_ERR_BADARG;
    for (int o = 0; o < O; ++o)
        for (int i = 0; i < I; ++i)
            for (int kh = 0; kh < K; ++kh)
                for (int kw = 0; kw < K; ++kw) {
                    const float v = src[(((size_t)o * I + i) * K + kh) * K + kw];
                    const size_t di = (((size_t)o * K + kh) * K + kw) * I + i;
                    if (dtype == SQN_F32) static_cast<float*>(dst)[di] = v;
                    else static_cast<uint16_t*>(dst)[di] = f32_to_16(v, dtype);
                }
    return SQN_OK;
}

extern "C" int sqn_pack_nchw_to_nhwc(const float* src, void* dst, int N, int C, int H, int W, int dtype)
{
    if (!src || !dst || N <= 0 || C <= 0 || H <= 0 || W <= 0) return SQN_ERR_BADARG;
    if (!valid_dtype(dtype)) return SQN_ERR_BADARG;
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w) {
                    const float v = src[(((size_t)n * C + c) * H + h) * W + w];
                    const size_t di = (((size_t)n * H + h) * W + w) * C + c;
                    if (dtype == SQN_F32) static_cast<float*>(dst)[di] = v;
                    else static_cast<uint16_t*>(dst)[di] = f32_to_16(v, dtype);
                }
    return SQN_OK;
}

extern "C" int sqn_unpack_nhwc_to_nchw(const void* src, float* dst, int N, int C, int H, int W, int dtype)
{
    if (!src || !dst || N <= 0 || C <= 0 || H <= 0 || W <= 0) return SQN_ERR_BADARG;
    if (!valid_dtype(dtype)) return SQN_ERR_BADARG;
    for (int n = 0; n < N; ++n)
        for (int h = 0; h < H; ++h)
            for (int w = 0; w < W; ++w)
                for (int c = 0; c < C; ++c) {
                    const size_t si = (((size_t)n * H + h) * W + w) * C + c;
                    const float v = dtype == SQN_F32 ? static_cast<const float*>(src)[si]
                                                     : f16bits_to_f32(static_cast<const uint16_t*>(src)[si], dtype);
                    dst[(((size_t)n * C + c) * H + h) * W + w] = v;
                }
    return SQN_OK;
}

// Stem operands in the layouts the bf16 stem kernel reads (what stem_pack produces on the device).
extern "C" int sqn_stem_packed_extent(int H, int W, int* Hp, int* Wp)
{
    if (H <= 0 || W <= 0 || !Hp || !Wp) return SQN_ERR_BADARG;
    *Hp = stem_packed_rows(H);
    *Wp = stem_packed_cols(W);
    return SQN_OK;
}

extern "C" int sqn_pack_stem_input(const float* src, void* dst, int N, int H, int W)
{
    if (!src || !dst || N <= 0 || H <= 0 || W <= 0) return SQN_ERR_BADARG;
    const int Hp = stem_packed_rows(H), Wp = stem_packed_cols(W);
    uint16_t* o = static_cast<uint16_t*>(dst);
    const uint16_t one = f32_to_bf16_rne(1.0f);
    for (int n = 0; n < N; ++n)
        for (int y = 0; y < Hp; ++y)
            for (int x = 0; x < Wp; ++x) {
                uint16_t* px = o + (((size_t)n * Hp + y) * Wp + x) * 4;
                const bool inside = y < H && x < W;
                for (int c = 0; c < 3; ++c)
                    px[c] = inside ? f32_to_bf16_rne(src[(((size_t)n * 3 + c) * H + y) * W + x]) : (uint16_t)0;
                px[3] = inside ? one : (uint16_t)0;        // meets the bias folded into the kernels
            }
    return SQN_OK;
}

extern "C" int sqn_pack_stem_weights(const float* src, const float* bias, void* dst, int O)
{
    if (!src || !bias || !dst || O <= 0) return SQN_ERR_BADARG;
    uint16_t* o = static_cast<uint16_t*>(dst);
    for (int m = 0; m < O; ++m)
        for (int kh = 0; kh < 7; ++kh)
            for (int px = 0; px < 8; ++px)
                for (int c = 0; c < 4; ++c) {
                    uint16_t v = 0;
                    if (px < 7 && c < 3) v = f32_to_bf16_rne(src[(((size_t)m * 3 + c) * 7 + kh) * 7 + px]);
                    if (c == 3 && kh == 0 && px < 2) {          // the bias as hi + lo, against the input's constant 1
                        const uint16_t hi = f32_to_bf16_rne(bias[m]);
                        v = px == 0 ? hi : f32_to_bf16_rne(bias[m] - bf16_to_f32(hi));
                    }
                    o[(((size_t)m * 7 + kh) * 8 + px) * 4 + c] = v;
                }
    return SQN_OK;
}

// ------------------------------------------------------------------------------ misc
extern "C" int sqn_check(void* stream)
{
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return SQN_ERR_CUDA;
    int* word = device_status_word();
    if (!word) return SQN_ERR_CUDA;
    int v = 0;
    if (cudaMemcpy(&v, word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return SQN_ERR_CUDA;
    if (v != 0) {
        const int zero = 0;
        if (cudaMemcpy(word, &zero, sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) return SQN_ERR_CUDA;
    }
    return v;
}

extern "C" int sqn_selftest_wait_timeout(long long limit_cycles, void* stream)
{
    if (limit_cycles < 1000 || limit_cycles > 2000000000LL) return SQN_ERR_BADARG;
    return launch_wait_timeout_selftest(limit_cycles, static_cast<cudaStream_t>(stream));
}

extern "C" int sqn_selftest_mma_rate(int n, int row_bytes, int issuers, int iters, void* out, int* sm_count_out, void* stream)
{
    if (n < 16 || n > 256 || n % 16 != 0 || (row_bytes != 32 && row_bytes != 64 && row_bytes != 128) || issuers < 1 || issuers > 2 ||
        iters < 1 || iters > 1000000 || !out)
        return SQN_ERR_BADARG;
    if (reinterpret_cast<uintptr_t>(out) & 7u) return SQN_ERR_ALIGN;
    if (sm_count_out) {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return SQN_ERR_CUDA;
        *sm_count_out = sms;
    }
    return launch_mma_rate_selftest(n, row_bytes, issuers, iters, static_cast<long long*>(out), static_cast<cudaStream_t>(stream));
}

extern "C" const char* sqn_status_string(int status)
{
    switch (status) {
        case SQN_OK: return "ok";
        case SQN_ERR_BADARG: return "bad argument";
        case SQN_ERR_UNSUPPORTED: return "unsupported shape for this dtype path";
        case SQN_ERR_ALIGN: return "alignment rule violated";
        case SQN_ERR_CUDA: return "CUDA call failed";
        case SQN_ERR_TIMEOUT: return "device-side wait timed out";
        case SQN_ERR_WORKSPACE: return "workspace missing or too small";
        case SQN_ERR_DEBUG: return "index check of the debug build failed";
        default: return "unknown status";
    }
}

extern "C" unsigned long long sqn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }
