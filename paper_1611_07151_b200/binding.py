"""ctypes binding of libsqn.so (declared in include/sqn.h).

Argument marshalling only: every function here has the name and argument order
of the C entry point it calls; tensors are passed as device addresses and
PyTorch is used for nothing but device memory and the current CUDA stream.
There is no fallback: if the library has not been built, loading it raises.
"""
import ctypes
import os

import numpy as np

SQN_F32 = 0
SQN_BF16 = 1
SQN_F16 = 2

SQN_OK = 0
SQN_ERR_BADARG = -1
SQN_ERR_UNSUPPORTED = -2
SQN_ERR_ALIGN = -3
SQN_ERR_CUDA = -4
SQN_ERR_TIMEOUT = -5
SQN_ERR_WORKSPACE = -6
SQN_ERR_DEBUG = -7

# SQN_LIBRARY in the environment names another build of the same library (the bounds-checked libsqn_debug.so)
LIB_PATH = os.environ.get("SQN_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsqn.so")

_c_int = ctypes.c_int
_c_vp = ctypes.c_void_p
_c_sz = ctypes.c_size_t


class sqn_conv_opts(ctypes.Structure):
    _fields_ = [("dtype", _c_int), ("relu", _c_int), ("out_c_offset", _c_int), ("out_c_total", _c_int),
                ("stream", _c_vp), ("workspace", _c_vp), ("workspace_bytes", _c_sz), ("fuse_maxpool", _c_int),
                ("fuse_global_avgpool", _c_int)]


# name -> (restype, argtypes); the same list is checked against include/sqn.h by the tests
SIGNATURES = {
    "conv_forward": (_c_int, [_c_vp] * 4 + [_c_int] * 8),
    "conv_forward_ex": (_c_int, [_c_vp] * 4 + [_c_int] * 8 + [ctypes.POINTER(sqn_conv_opts)]),
    "conv_workspace_bytes": (_c_int, [_c_int] * 9 + [ctypes.POINTER(_c_sz)]),
    "fire_forward": (_c_int, [_c_vp] * 9 + [_c_int] * 8 + [_c_vp]),
    "fire_forward_static": (_c_int, [_c_vp] * 8 + [_c_int] * 8 + [_c_vp]),
    "maxpool3x3s2_forward": (_c_int, [_c_vp, _c_vp] + [_c_int] * 5 + [_c_vp]),
    "avgpool_softmax_forward": (_c_int, [_c_vp] * 3 + [_c_int] * 5 + [_c_vp]),
    "squeezenet_create": (_c_int, [ctypes.POINTER(_c_vp), ctypes.POINTER(_c_vp), ctypes.POINTER(_c_vp), _c_int, _c_int]),
    "squeezenet_workspace_bytes": (_c_int, [_c_vp, _c_int, ctypes.POINTER(_c_sz)]),
    "squeezenet_forward": (_c_int, [_c_vp] * 5 + [_c_int, _c_vp]),
    "squeezenet_layer_output": (_c_int, [_c_vp, ctypes.c_char_p, _c_vp, _c_int, ctypes.POINTER(_c_vp),
                                         ctypes.POINTER(_c_int), ctypes.POINTER(_c_int), ctypes.POINTER(_c_int)]),
    "squeezenet_destroy": (_c_int, [_c_vp]),
    "squeezenet_set_stem_prepacked": (_c_int, [_c_vp, _c_int]),
    "sqn_stem_packed_extent": (_c_int, [_c_int, _c_int, ctypes.POINTER(_c_int), ctypes.POINTER(_c_int)]),
    "sqn_pack_stem_input": (_c_int, [_c_vp, _c_vp, _c_int, _c_int, _c_int]),
    "sqn_pack_stem_weights": (_c_int, [_c_vp, _c_vp, _c_vp, _c_int]),
    "squeezenet_host_workspace_bytes": (_c_int, [_c_vp, _c_int, ctypes.POINTER(_c_sz)]),
    "squeezenet_forward_host": (_c_int, [_c_vp] * 5 + [_c_int, _c_vp]),
    "squeezenet_profile": (_c_int, [_c_vp, _c_int]),
    "squeezenet_profile_read": (_c_int, [_c_vp, ctypes.POINTER(ctypes.c_float), _c_int, ctypes.POINTER(_c_int),
                                         ctypes.POINTER(_c_int)]),
    "squeezenet_profile_name": (ctypes.c_char_p, [_c_vp, _c_int]),
    "sqn_pack_weights_oihw_to_ohwi": (_c_int, [_c_vp, _c_vp, _c_int, _c_int, _c_int, _c_int]),
    "sqn_pack_nchw_to_nhwc": (_c_int, [_c_vp, _c_vp] + [_c_int] * 5),
    "sqn_unpack_nhwc_to_nchw": (_c_int, [_c_vp, _c_vp] + [_c_int] * 5),
    "sqn_check": (_c_int, [_c_vp]),
    "sqn_selftest_wait_timeout": (_c_int, [ctypes.c_longlong, _c_vp]),
    "sqn_selftest_mma_rate": (_c_int, [_c_int, _c_int, _c_int, _c_int, _c_vp, ctypes.POINTER(_c_int), _c_vp]),
    "sqn_status_string": (ctypes.c_char_p, [_c_int]),
    "sqn_launch_count": (ctypes.c_ulonglong, []),
}

_lib = None


class SqnError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        msg = lib().sqn_status_string(status).decode()
        super().__init__("%s: %s (%d)" % (where, msg, status))


def lib():
    """Load libsqn.so (once).  Raises if it has not been built: there is no other path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libsqn.so is missing (%s): build it with "
                               "`python -m paper_1611_07151_b200.build`; there is no CPU fallback" % LIB_PATH)
        l = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype = res
            fn.argtypes = args
        _lib = l
    return _lib


def _check(rc, where):
    if rc != SQN_OK:
        raise SqnError(rc, where)


def _p(t):
    """Device (or host) address of a tensor / array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def current_stream():
    import torch
    return torch.cuda.current_stream().cuda_stream


# ------------------------------------------------------------------ entry points

def conv_forward(inp, weights, bias, out, numInputLayers, numOutputLayers, H, W, K, S, pad, batch):
    """fp32, ReLU, dense output, legacy default stream (see include/sqn.h)."""
    _check(lib().conv_forward(_p(inp), _p(weights), _p(bias), _p(out), numInputLayers, numOutputLayers, H, W, K, S,
                              pad, batch), "conv_forward")


def conv_forward_ex(inp, weights, bias, out, numInputLayers, numOutputLayers, H, W, K, S, pad, batch, dtype=SQN_F32,
                    relu=True, out_c_offset=0, out_c_total=0, stream=None, workspace=None, workspace_bytes=0,
                    fuse_maxpool=False, fuse_global_avgpool=False):
    opts = sqn_conv_opts(dtype, 1 if relu else 0, out_c_offset, out_c_total,
                         current_stream() if stream is None else stream, _p(workspace), workspace_bytes,
                         1 if fuse_maxpool else 0, 1 if fuse_global_avgpool else 0)
    _check(lib().conv_forward_ex(_p(inp), _p(weights), _p(bias), _p(out), numInputLayers, numOutputLayers, H, W, K, S,
                                 pad, batch, ctypes.byref(opts)), "conv_forward_ex")


def conv_workspace_bytes(numInputLayers, numOutputLayers, H, W, K, S, pad, batch, dtype):
    n = _c_sz(0)
    _check(lib().conv_workspace_bytes(numInputLayers, numOutputLayers, H, W, K, S, pad, batch, dtype,
                                      ctypes.byref(n)), "conv_workspace_bytes")
    return n.value


def fire_forward(inp, w_sq, b_sq, w_e1, b_e1, w_e3, b_e3, squeeze_scratch, out, Cin, s, e1, e3, H, W, batch, dtype,
                 stream=None):
    _check(lib().fire_forward(_p(inp), _p(w_sq), _p(b_sq), _p(w_e1), _p(b_e1), _p(w_e3), _p(b_e3),
                              _p(squeeze_scratch), _p(out), Cin, s, e1, e3, H, W, batch, dtype,
                              current_stream() if stream is None else stream), "fire_forward")


def fire_forward_static(inp, w_sq, b_sq, w_e1, b_e1, w_e3, b_e3, out, Cin, s, e1, e3, H, W, batch, dtype, stream=None):
    """fire_forward without a scratch argument: the squeeze map lives in an 8 MiB buffer inside the
    library, so nothing is allocated.  For callers that cannot obtain device memory (see include/sqn.h)."""
    _check(lib().fire_forward_static(_p(inp), _p(w_sq), _p(b_sq), _p(w_e1), _p(b_e1), _p(w_e3), _p(b_e3), _p(out),
                                     Cin, s, e1, e3, H, W, batch, dtype,
                                     current_stream() if stream is None else stream), "fire_forward_static")


def maxpool3x3s2_forward(inp, out, C, H, W, batch, dtype, stream=None):
    _check(lib().maxpool3x3s2_forward(_p(inp), _p(out), C, H, W, batch, dtype,
                                      current_stream() if stream is None else stream), "maxpool3x3s2_forward")


def avgpool_softmax_forward(inp, logits_f32, probs_f32, C, H, W, batch, dtype, stream=None):
    _check(lib().avgpool_softmax_forward(_p(inp), _p(logits_f32), _p(probs_f32), C, H, W, batch, dtype,
                                         current_stream() if stream is None else stream), "avgpool_softmax_forward")


def squeezenet_create(weights26, bias26, dtype, max_batch):
    """weights26 / bias26: sequences of 26 device tensors (kept alive by the caller). Returns a handle."""
    if len(weights26) != 26 or len(bias26) != 26:
        raise ValueError("need 26 kernels and 26 biases")
    wa = (_c_vp * 26)(*[_p(w) for w in weights26])
    ba = (_c_vp * 26)(*[_p(b) for b in bias26])
    h = _c_vp(0)
    _check(lib().squeezenet_create(ctypes.byref(h), wa, ba, dtype, max_batch), "squeezenet_create")
    return h


def squeezenet_workspace_bytes(net, batch):
    n = _c_sz(0)
    _check(lib().squeezenet_workspace_bytes(net, batch, ctypes.byref(n)), "squeezenet_workspace_bytes")
    return n.value


def squeezenet_forward(net, in_nhwc, logits_f32, probs_f32, workspace, batch, stream=None):
    _check(lib().squeezenet_forward(net, _p(in_nhwc), _p(logits_f32), _p(probs_f32), _p(workspace), batch,
                                    current_stream() if stream is None else stream), "squeezenet_forward")


def squeezenet_layer_output(net, name, workspace, batch):
    """(device address, C, H, W) of a named intermediate of the last forward."""
    ptr, C, H, W = _c_vp(0), _c_int(0), _c_int(0), _c_int(0)
    _check(lib().squeezenet_layer_output(net, name.encode(), _p(workspace), batch, ctypes.byref(ptr), ctypes.byref(C),
                                         ctypes.byref(H), ctypes.byref(W)), "squeezenet_layer_output")
    return ptr.value, C.value, H.value, W.value


def squeezenet_destroy(net):
    _check(lib().squeezenet_destroy(net), "squeezenet_destroy")


def squeezenet_set_stem_prepacked(net, on=True):
    _check(lib().squeezenet_set_stem_prepacked(net, 1 if on else 0), "squeezenet_set_stem_prepacked")


def sqn_stem_packed_extent(H, W):
    hp, wp = _c_int(0), _c_int(0)
    _check(lib().sqn_stem_packed_extent(H, W, ctypes.byref(hp), ctypes.byref(wp)), "sqn_stem_packed_extent")
    return hp.value, wp.value


def sqn_pack_stem_input(src):
    """[N][3][H][W] float32 -> [N][Hp][Wp][4] bf16 words (the layout the bf16 stem kernel reads)."""
    src = np.ascontiguousarray(src, dtype=np.float32)
    N, C, H, W = src.shape
    assert C == 3
    hp, wp = sqn_stem_packed_extent(H, W)
    dst = np.empty((N, hp, wp, 4), dtype=np.uint16)
    _check(lib().sqn_pack_stem_input(src.ctypes.data, dst.ctypes.data, N, H, W), "sqn_pack_stem_input")
    return dst


def sqn_pack_stem_weights(src, bias):
    """[O][3][7][7] float32 kernels and [O] bias -> [O][7][8][4] bf16 words with the bias folded in."""
    src = np.ascontiguousarray(src, dtype=np.float32)
    bias = np.ascontiguousarray(bias, dtype=np.float32)
    O = src.shape[0]
    assert src.shape == (O, 3, 7, 7) and bias.shape == (O,)
    dst = np.empty((O, 7, 8, 4), dtype=np.uint16)
    _check(lib().sqn_pack_stem_weights(src.ctypes.data, bias.ctypes.data, dst.ctypes.data, O), "sqn_pack_stem_weights")
    return dst


def squeezenet_host_workspace_bytes(net, batch):
    n = _c_sz(0)
    _check(lib().squeezenet_host_workspace_bytes(net, batch, ctypes.byref(n)), "squeezenet_host_workspace_bytes")
    return n.value


def squeezenet_forward_host(net, in_host, logits_host, probs_host, workspace, batch, stream=None):
    """in_host / logits_host / probs_host: host tensors or arrays (pinned for asynchronous copies)."""
    _check(lib().squeezenet_forward_host(net, _p(in_host), _p(logits_host), _p(probs_host), _p(workspace), batch,
                                         current_stream() if stream is None else stream), "squeezenet_forward_host")


def squeezenet_profile(net, slots):
    _check(lib().squeezenet_profile(net, slots), "squeezenet_profile")


def squeezenet_profile_read(net):
    """-> (names, ms summed over the recorded forwards, number of forwards recorded)."""
    n, f = _c_int(0), _c_int(0)
    _check(lib().squeezenet_profile_read(net, None, 0, ctypes.byref(n), ctypes.byref(f)), "squeezenet_profile_read")
    ms = (ctypes.c_float * max(n.value, 1))()
    _check(lib().squeezenet_profile_read(net, ms, n.value, ctypes.byref(n), ctypes.byref(f)), "squeezenet_profile_read")
    names = [lib().squeezenet_profile_name(net, i).decode() for i in range(n.value)]
    return names, [float(ms[i]) for i in range(n.value)], f.value


def sqn_check(stream=None):
    return lib().sqn_check(current_stream() if stream is None else stream)


def sqn_selftest_wait_timeout(limit_cycles, stream=None):
    _check(lib().sqn_selftest_wait_timeout(limit_cycles, current_stream() if stream is None else stream),
           "sqn_selftest_wait_timeout")


def sqn_selftest_mma_rate(n, row_bytes=128, issuers=1, iters=2000):
    """Clocks per tcgen05.mma of 128 x n x 16 (mean over the SMs): (issue loop, until complete) per issuer."""
    import torch
    out = torch.zeros(6 * 256, dtype=torch.int64, device="cuda")
    sms = _c_int(0)
    _check(lib().sqn_selftest_mma_rate(n, row_bytes, issuers, iters, _p(out), ctypes.byref(sms), current_stream()),
           "sqn_selftest_mma_rate")
    torch.cuda.synchronize()
    o = out[:6 * sms.value].view(sms.value, 2, 3).cpu().numpy()
    assert (o[:, :issuers, 2] == 1).all()
    return [(float(o[:, w, 0].mean()) / iters, float(o[:, w, 1].mean()) / iters) for w in range(issuers)]


def sqn_status_string(status):
    return lib().sqn_status_string(status).decode()


def sqn_launch_count():
    return int(lib().sqn_launch_count())


# ------------------------------------------------- host layout helpers (numpy in/out)

def _np_dtype(dtype):
    return np.float32 if dtype == SQN_F32 else np.uint16     # bf16 / fp16 travel as raw 16-bit words


def sqn_pack_weights_oihw_to_ohwi(src, dtype=SQN_F32):
    src = np.ascontiguousarray(src, dtype=np.float32)
    O, I, K, K2 = src.shape
    assert K == K2
    dst = np.empty((O, K, K, I), dtype=_np_dtype(dtype))
    _check(lib().sqn_pack_weights_oihw_to_ohwi(src.ctypes.data, dst.ctypes.data, O, I, K, dtype), "pack_weights")
    return dst


def sqn_pack_nchw_to_nhwc(src, dtype=SQN_F32):
    src = np.ascontiguousarray(src, dtype=np.float32)
    N, C, H, W = src.shape
    dst = np.empty((N, H, W, C), dtype=_np_dtype(dtype))
    _check(lib().sqn_pack_nchw_to_nhwc(src.ctypes.data, dst.ctypes.data, N, C, H, W, dtype), "pack_nchw_to_nhwc")
    return dst


def sqn_unpack_nhwc_to_nchw(src, dtype=SQN_F32):
    src = np.ascontiguousarray(src, dtype=_np_dtype(dtype))
    N, H, W, C = src.shape
    dst = np.empty((N, C, H, W), dtype=np.float32)
    _check(lib().sqn_unpack_nhwc_to_nchw(src.ctypes.data, dst.ctypes.data, N, C, H, W, dtype), "unpack_nhwc_to_nchw")
    return dst


# ------------------------------------------------------ device memory (torch plumbing)

def to_device(a, dtype=SQN_F32):
    """Host array produced by a pack helper -> CUDA tensor (bf16 words are reinterpreted, not converted)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype == SQN_BF16:
        t = t.view(torch.int16).view(torch.bfloat16)
    elif dtype == SQN_F16:
        t = t.view(torch.int16).view(torch.float16)
    return t.cuda()


def to_host(t, dtype=SQN_F32):
    """CUDA tensor -> host array in the form the unpack helper takes."""
    import torch
    if dtype in (SQN_BF16, SQN_F16):
        return t.detach().cpu().view(torch.int16).numpy().view(np.uint16)
    return t.detach().cpu().numpy()


def empty_device(shape, dtype=SQN_F32):
    import torch
    return torch.empty(shape, dtype={SQN_F32: torch.float32, SQN_BF16: torch.bfloat16, SQN_F16: torch.float16}[dtype], device="cuda")
