/*
 * sqn.h -- C ABI of the forward-CNN library (SqueezeNet v1.0 hot path, sm_100a).
 *
 * Conventions that hold for every entry point unless its comment says otherwise
 * ---------------------------------------------------------------------------
 *  - Pointers named in/out/weights/bias/workspace/scratch/logits/probs are DEVICE
 *    pointers owned by the caller.  The library never allocates or frees device
 *    memory on the caller's behalf and never keeps a pointer past the call,
 *    except the weight/bias pointers stored inside an sqn_net the caller created.
 *  - Activations are NHWC: [batch][row][col][layer], layers contiguous.
 *    Kernels are OHWI: [outLayer][K][K][inLayer].  Bias is fp32 [outLayer].
 *    (The paper, Section III-B/C, reorders data so that values of consecutive
 *    layers at one pixel are adjacent and has every layer write its output in
 *    that order; NHWC/OHWI is the same idea carried to all layers of a pixel.)
 *  - dtype SQN_F32: activations and kernels fp32, fp32 FFMA accumulation.
 *    dtype SQN_BF16: activations and kernels bf16, fp32 accumulation on the
 *    tensor cores, bias/ReLU/pooling arithmetic in fp32, outputs rounded to
 *    bf16 (round to nearest even).  Logits and probabilities are always fp32.
 *    dtype SQN_F16: the same kernels on IEEE half precision (10 mantissa bits
 *    instead of bf16's 7, a narrower exponent): a third precision point between
 *    the exact path and bf16 (the paper, Section IV-B, trades precision for speed
 *    in two steps, "relaxed" and "imprecise", and accepts a step when the
 *    predictions do not change).  Wherever this header says SQN_BF16 about shapes
 *    and alignment, SQN_F16 is accepted under the same rules; values above 65504
 *    overflow to infinity as in any fp16 computation.
 *  - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is
 *    the legacy default stream).  No entry point synchronises except sqn_check.
 *  - Every argument is validated on the host before anything is launched.  On
 *    error nothing is launched and a negative sqn_status is returned.  There is
 *    no CPU fallback and no silent slow path: a shape the selected dtype path
 *    cannot run returns SQN_ERR_UNSUPPORTED.
 *  - in and out must not overlap.  All base pointers must be 16-byte aligned.
 */
#ifndef SQN_H
#define SQN_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SQN_OK = 0,
    SQN_ERR_BADARG = -1,       /* null pointer, non-positive size, window larger than padded input */
    SQN_ERR_UNSUPPORTED = -2,  /* valid request the selected dtype path does not implement */
    SQN_ERR_ALIGN = -3,        /* pointer or layer count breaks an alignment rule */
    SQN_ERR_CUDA = -4,         /* a CUDA runtime/driver call failed */
    SQN_ERR_TIMEOUT = -5,      /* a bounded device-side wait ran out (reported by sqn_check) */
    SQN_ERR_WORKSPACE = -6,    /* workspace missing or too small */
    SQN_ERR_DEBUG = -7         /* an index check of the debug build (-DSQN_DEBUG) failed; the access was skipped (sqn_check) */
} sqn_status;

typedef enum { SQN_F32 = 0, SQN_BF16 = 1, SQN_F16 = 2 } sqn_dtype;

/*
 * Convolution layer (paper Section II; Section III Fig. 2 prose; Eq. 1):
 *   out[n][h][w][m] = max(0, bias[m] + sum_{i,j<K, c<numInputLayers}
 *                              in[n][h*S+i-pad][w*S+j-pad][c] * weights[m][i][j][c])
 * with zero padding, output extent (H + 2*pad - K)/S + 1 in each direction
 * (integer division).  fp32, ReLU on, dense output (all numOutputLayers layers),
 * legacy default stream.
 *   in       [batch][H][W][numInputLayers]
 *   weights  [numOutputLayers][K][K][numInputLayers]
 *   bias     [numOutputLayers] fp32
 *   out      [batch][outH][outW][numOutputLayers]
 * Any K>=1, S>=1, pad>=0 and any layer counts are accepted.
 */
int conv_forward(const void* in, const void* weights, const void* bias, void* out,
                 int numInputLayers, int numOutputLayers, int H, int W, int K, int S, int pad, int batch);

/*
 * Options for conv_forward_ex.
 *   dtype          SQN_F32 or SQN_BF16
 *   relu           non-zero: max(0, .) after the bias; zero: identity
 *   out_c_offset,
 *   out_c_total    the layer writes layers [out_c_offset, out_c_offset+numOutputLayers) of an
 *                  output tensor that has out_c_total layers per pixel (a fire layer's two
 *                  expands write their halves of one tensor this way).  out_c_total = 0 means
 *                  dense: offset 0, total numOutputLayers.
 *   stream         cudaStream_t
 *   workspace,
 *   workspace_bytes  device scratch, needed only when conv_workspace_bytes reports > 0
 *   fuse_global_avgpool   the global average pooling that follows the layer (paper Section III-E) is taken inside the
 *                  kernel and the layer's own map is never stored: out is fp32 [batch][numOutputLayers], the mean over
 *                  all outH x outW pixels of max(0, .) of the layer (or of the layer itself when relu is zero).
 *                  SQN_BF16 only, K = 1, S = 1, pad = 0, numInputLayers a multiple of 64, at most 256 pixels per
 *                  image, out_c_total = 0, not together with fuse_maxpool; otherwise SQN_ERR_UNSUPPORTED / SQN_ERR_BADARG.
 *   fuse_maxpool   the 3x3 / stride 2 max-pool that follows the layer (paper Section III-E) is applied inside the
 *                  kernel and only the pooled map is written: out is [batch][(outH-3)/2+1][(outW-3)/2+1][out_c_total].
 *                  SQN_BF16 only, stride 1 (or the stem shape), numOutputLayers a multiple of 32 up to 128, kernels
 *                  small enough to stay in shared memory; otherwise SQN_ERR_UNSUPPORTED.
 */
typedef struct {
    int dtype;
    int relu;
    int out_c_offset;
    int out_c_total;
    void* stream;
    void* workspace;
    size_t workspace_bytes;
    int fuse_maxpool;   /* non-zero: out receives maxpool3x3/stride2 of the layer's output, extent ((outH-3)/2+1) */
    int fuse_global_avgpool;   /* non-zero: out receives the per-layer mean of the layer's output, fp32 [batch][numOutputLayers] */
} sqn_conv_opts;

/*
 * Same operation as conv_forward with every choice exposed.  opts may be NULL
 * (fp32, ReLU, dense, default stream).
 * SQN_BF16 accepts (else SQN_ERR_UNSUPPORTED / SQN_ERR_ALIGN):
 *   - S == 1, K <= 7 (pad == 0 when K == 1), numInputLayers a multiple of 16,
 *     numOutputLayers a multiple of 16 (of 8 when above 256), out_c_offset and out_c_total
 *     multiples of 8; or
 *   - the stem shape K=7, S=2, pad=0, numInputLayers=3 with numOutputLayers a multiple of 16
 *     up to 256, which needs a workspace (conv_workspace_bytes) for its repacked input and kernels.
 */
int conv_forward_ex(const void* in, const void* weights, const void* bias, void* out,
                    int numInputLayers, int numOutputLayers, int H, int W, int K, int S, int pad, int batch,
                    const sqn_conv_opts* opts);

/* Bytes of workspace conv_forward_ex needs for this shape and dtype (0 for most). */
int conv_workspace_bytes(int numInputLayers, int numOutputLayers, int H, int W, int K, int S, int pad, int batch,
                         int dtype, size_t* bytes);

/*
 * Fire layer (paper Section II: one squeeze layer feeding two expand layers):
 *   sq  = relu(conv1x1(in,  w_sq, b_sq))            [batch][H][W][s]     -> squeeze_scratch
 *   out[..., 0:e1]      = relu(conv1x1(sq, w_e1, b_e1))
 *   out[..., e1:e1+e3]  = relu(conv3x3 pad 1 (sq, w_e3, b_e3))
 * Both expands store straight into their slice of out [batch][H][W][e1+e3];
 * there is no concatenation pass.  squeeze_scratch must hold batch*H*W*s
 * elements of the chosen dtype and must not overlap in or out.
 * SQN_BF16: Cin, s multiples of 16; e1, e3 multiples of 16.
 */
int fire_forward(const void* in, const void* w_sq, const void* b_sq, const void* w_e1, const void* b_e1,
                 const void* w_e3, const void* b_e3, void* squeeze_scratch, void* out,
                 int Cin, int s, int e1, int e3, int H, int W, int batch, int dtype, void* stream);

/*
 * fire_forward for callers that must not allocate.  (The paper has no counterpart: this is a
 * convenience of this library, not a step of the method.)
 *
 * Who needs it: code that runs where device memory can no longer be obtained -- a worker inside a
 * serving process whose memory was handed out once at start-up and is owned by someone else, a
 * plug-in or callback that is forbidden to call cudaMalloc because that call may synchronise the
 * whole device under the host application's feet, or a process running under a fixed memory
 * budget that is already spent.  Such a caller has its input, its kernels and its output, but
 * nowhere to put the squeeze map that fire_forward wants in `squeeze_scratch`.
 *
 * This entry point computes exactly what fire_forward computes, with the squeeze map kept in a
 * buffer built into the library image.  It calls no cudaMalloc/cudaFree and no allocating library
 * routine, on the device or on the host (the bf16 path encodes its tensor maps on the stack on
 * every call instead of caching them).
 *
 *   - Limit: batch*H*W*s elements of `dtype` must fit in 8 MiB (8388608 bytes), e.g. fire4 in fp32
 *     up to batch 21.  Larger requests return SQN_ERR_WORKSPACE and launch nothing.
 *   - Every GPU that loads the library carries those 8 MiB until the process exits.
 *   - The first call on a device looks up the buffer's device address (cudaGetSymbolAddress, with
 *     that device current) and keeps it; make that first call before any stream capture begins.
 *   - All calls on a device share the one buffer, whatever their stream: two calls that overlap on
 *     the GPU race on it.  Order them (same stream, or events).  Nothing needs clearing between
 *     calls: every element the expands read is written by the squeeze of the same call.
 * Arguments, layouts and dtype rules are those of fire_forward minus `squeeze_scratch`.
 */
int fire_forward_static(const void* in, const void* w_sq, const void* b_sq, const void* w_e1, const void* b_e1,
                        const void* w_e3, const void* b_e3, void* out,
                        int Cin, int s, int e1, int e3, int H, int W, int batch, int dtype, void* stream);

/*
 * Max pooling 3x3, stride 2, no padding (paper Section III-E):
 *   out[n][h][w][c] = max_{i,j<3} in[n][2h+i][2w+j][c],  out extent (H-3)/2+1.
 */
int maxpool3x3s2_forward(const void* in, void* out, int C, int H, int W, int batch, int dtype, void* stream);

/*
 * Global average pooling followed by softmax (paper Section III-E):
 *   logits[n][c] = mean over H*W of in[n][.][.][c]        (fp32)
 *   probs[n][c]  = exp(logits[n][c] - max_c) / sum_c exp(logits[n][c] - max_c)
 * in has dtype `dtype`; logits and probs are fp32 [batch][C]; probs may be NULL.
 * C <= 8192 and batch <= 65535 (else SQN_ERR_UNSUPPORTED); in 16-byte aligned, logits and probs
 * 4-byte aligned (else SQN_ERR_ALIGN).
 */
int avgpool_softmax_forward(const void* in, void* logits_f32, void* probs_f32, int C, int H, int W, int batch,
                            int dtype, void* stream);

/*
 * SqueezeNet v1.0 forward (paper Section II: two convolutional layers, eight
 * fire layers, pooling, softmax, 1000 classes) on 227x227x3 images:
 *   conv1 96x7x7/2 -> maxpool -> fire2,3 (16,64,64) -> fire4 (32,128,128) -> maxpool
 *   -> fire5 (32,128,128) -> fire6,7 (48,192,192) -> fire8 (64,256,256) -> maxpool
 *   -> fire9 (64,256,256) -> conv10 1000x1x1 -> global average -> softmax,
 * ReLU after every convolution (conv10 included).
 *
 * squeezenet_create: weights26/bias26 are host arrays of 26 device pointers in
 *   network order (conv1; fireN squeeze, expand1x1, expand3x3 for N=2..9; conv10),
 *   kernels OHWI in `dtype`, bias fp32.  The net stores the pointers (the caller
 *   keeps the memory alive) and host-side launch plans; it holds no device memory.
 *   The kernels and bias must be complete before squeezenet_forward is called: the
 *   forward's launches may fetch them while earlier work on `stream` is still running
 *   (conv_forward_ex and fire_forward make no such assumption).
 * squeezenet_workspace_bytes: device scratch one forward of `batch` images needs.
 * squeezenet_forward: in_nhwc [batch][227][227][3] in the net's dtype;
 *   logits_f32, probs_f32 fp32 [batch][1000] (probs may be NULL);
 *   batch <= max_batch.  Returns after enqueuing all launches on `stream`.
 * squeezenet_layer_output: after a forward with the same workspace and batch,
 *   gives the device address, layer count and extent of a named intermediate
 *   ("conv1", "pool1", "fire2_sq", "fire2", ..., "pool8", "fire9", "conv10");
 *   the data is in the net's dtype, NHWC, valid until the next forward.  From a batch of 16 on a bf16 net
 *   computes conv1+pool1, fire4+pool4 and fire8+pool8 in fused kernels and never stores the maps of conv1, fire4
 *   and fire8: asking for one of those then returns SQN_ERR_UNSUPPORTED.  A bf16 net also runs the fire layers whose
 *   kernels fit in shared memory (fire2, fire3, fire5; fire4 too below a batch of 16) as one kernel each, without
 *   storing their squeeze maps, and takes conv10, its ReLU and the global average in one kernel without storing
 *   conv10's map: "fireN_sq" of those layers and "conv10" then return SQN_ERR_UNSUPPORTED as well.  With
 *   SQN_FUSED_FIRE=0 and SQN_FUSED_HEAD=0 in the environment (read at every call) these layers run as separate
 *   launches and their maps can be read.
 */
typedef struct sqn_net sqn_net;
int squeezenet_create(sqn_net** net, const void* const* weights26, const void* const* bias26, int dtype,
                      int max_batch);
int squeezenet_workspace_bytes(const sqn_net* net, int batch, size_t* bytes);
int squeezenet_forward(sqn_net* net, const void* in_nhwc, void* logits_f32, void* probs_f32, void* workspace,
                       int batch, void* stream);
int squeezenet_layer_output(const sqn_net* net, const char* name, void* workspace, int batch, void** ptr, int* C,
                            int* H, int* W);
int squeezenet_destroy(sqn_net* net);

/*
 * Stem operands reordered offline (the paper, Section III-C, reorders the model file once so that no
 * layer repacks data at run time; here the same is done for the one layer whose operands the tensor
 * cores cannot read as they are: conv1, 7x7 / stride 2 on 3 input layers, bf16).
 * squeezenet_set_stem_prepacked(net, 1) (SQN_BF16 nets only, else SQN_ERR_UNSUPPORTED) declares that
 *   - squeezenet_forward's input is [batch][Hp][Wp][4] bf16 as written by sqn_pack_stem_input
 *     (Hp, Wp from sqn_stem_packed_extent(227, 227): 228 x 228; the fourth layer of every image pixel
 *     holds 1.0, padding rows and columns are zero), and
 *   - the net's first kernel pointer (weights26[0]) is [96][7][8][4] bf16 as written by
 *     sqn_pack_stem_weights, which folds conv1's bias into two unused places; bias26[0] is then not read.
 * The forward then launches no repack kernel.  squeezenet_forward_host copies such an input as it is.
 * The three helpers take HOST pointers: src [N][3][H][W] fp32 (the oracle's order), kernels [O][3][7][7]
 * fp32, bias [O] fp32; dst must hold N*Hp*Wp*4, respectively O*224, 16-bit words.
 */
int squeezenet_set_stem_prepacked(sqn_net* net, int on);
int sqn_stem_packed_extent(int H, int W, int* Hp, int* Wp);
int sqn_pack_stem_input(const float* src, void* dst, int N, int H, int W);
int sqn_pack_stem_weights(const float* src, const float* bias, void* dst, int O);

/*
 * The same forward with HOST input and output buffers (the call a user with data in host
 * memory makes): copy of in_host [batch][227][227][3] (net dtype) to the device, the forward,
 * copies of logits (and probs, unless NULL) [batch][1000] fp32 back to the host.  The copies
 * are asynchronous when the host buffers are pinned.  workspace is DEVICE memory of
 * squeezenet_host_workspace_bytes(net, batch) bytes (the forward's scratch, two staging
 * buffers for the input and staging for the two outputs).
 * Ordering: the forward and the copies back are enqueued on `stream`.  The input copy runs on
 * a stream the net owns (made on the first call on a device) and alternates between the two
 * staging buffers, so the copy of one call overlaps the forward of the call before it; it is
 * NOT ordered after work queued earlier on `stream`: in_host must hold the images when the
 * call is made.  All host buffers must stay valid, and in_host unchanged, until `stream` has
 * passed the call.  Calls on one net must come from one thread at a time.
 */
int squeezenet_host_workspace_bytes(const sqn_net* net, int batch, size_t* bytes);
int squeezenet_forward_host(sqn_net* net, const void* in_host, void* logits_host, void* probs_host,
                            void* workspace, int batch, void* stream);

/*
 * Per-launch timing of squeezenet_forward with CUDA events on the caller's stream (the
 * paper reports per-layer times, Section IV, Table 4).
 * squeezenet_profile(net, slots): slots > 0 records an event after every launch of each
 *   following forward, keeping the most recent `slots` forwards; 0 turns it off.
 * squeezenet_profile_read: waits for the recorded forwards, then writes into ms_sum[i] the
 *   time of launch group i summed over *forwards recorded forwards; *launches = number of
 *   groups per forward.  ms_sum may be NULL to query the counts only.
 * squeezenet_profile_name(net, i): name of group i ("conv1_pack", "conv1", "pool1",
 *   "fire2_sq", "fire2_e1", "fire2_e3", ..., "conv10", "head"; launches that cover several
 *   steps carry all of them: "conv1+pool1", "fire2_e1+e3", "fire4_e1+e3+pool"); "" if out
 *   of range.
 */
int squeezenet_profile(sqn_net* net, int slots);
int squeezenet_profile_read(sqn_net* net, float* ms_sum, int capacity, int* launches, int* forwards);
const char* squeezenet_profile_name(const sqn_net* net, int i);

/*
 * Host-side layout helpers (the paper's offline reordering of the model file,
 * Section III-C).  src and dst are HOST pointers.  dtype selects the element
 * type of the reordered side (fp32, or bf16 rounded to nearest even).
 */
int sqn_pack_weights_oihw_to_ohwi(const float* src, void* dst, int O, int I, int K, int dtype);
int sqn_pack_nchw_to_nhwc(const float* src, void* dst, int N, int C, int H, int W, int dtype);
int sqn_unpack_nhwc_to_nchw(const void* src, float* dst, int N, int C, int H, int W, int dtype);

/*
 * Synchronises `stream` and returns SQN_OK, SQN_ERR_CUDA, or the error a kernel
 * recorded (SQN_ERR_TIMEOUT when a bounded device-side wait ran out).  The
 * recorded error is cleared by the call.
 */
int sqn_check(void* stream);

/*
 * Self-test of the failure path every kernel of the library shares.  All device-side waits are bounded: when one
 * runs out the CTA records SQN_ERR_TIMEOUT, lets its outstanding copies land, frees its tensor memory and returns,
 * so the context stays usable and the next sqn_check reports the error.  This call launches one small CTA that
 * waits, for at most limit_cycles SM clocks (1e3 .. 2e9), on a barrier nothing arrives on.  After it, sqn_check
 * returns SQN_ERR_TIMEOUT once, then SQN_OK, and every other entry point works as before.  (Diagnostic: the paper
 * has no counterpart.)
 */
int sqn_selftest_wait_timeout(long long limit_cycles, void* stream);

/*
 * Measurement behind the kernels' role layout: on every SM `issuers` (1 or 2) warps each issue `iters` tensor-core
 * MMAs of 128 x n x 16 (bf16 operands in shared memory, rows of row_bytes = 32 / 64 / 128 in the matching swizzle)
 * back to back.  out is DEVICE memory for 6 64-bit integers per SM (the SM count is returned in *sm_count_out, a host
 * pointer, may be NULL): per issuer {clocks until the last MMA was issued, clocks until all had completed, 1 if the
 * bounded wait for them ended in time}.  n a multiple of 16 in 16 .. 256.  (Diagnostic: the paper has no counterpart.)
 */
int sqn_selftest_mma_rate(int n, int row_bytes, int issuers, int iters, void* out, int* sm_count_out, void* stream);

/* Static, human-readable name of a status code. */
const char* sqn_status_string(int status);

/* Number of kernel launches the library has enqueued since it was loaded (host counter). */
unsigned long long sqn_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SQN_H */
