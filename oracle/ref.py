"""CPU oracle: Python face of oracle/conv_ref.c plus the layer compositions.

TEST INFRASTRUCTURE ONLY.  Everything here works on NumPy float32 arrays in the
paper's default row-major order (Eq. 5): activations [batch, layer, row, col],
kernels [outLayer, inLayer, K, K].  Accumulation is in double (in the C code).

What each function follows:
  conv2d           Section II (output pixel = sum over input layers of KxK
                   kernel . window, slid by stride S); Section III, Fig. 2 prose.
  maxpool,
  global_avgpool,
  softmax          Section III-E.
  fire             Section II (a fire layer = one squeeze convolution feeding
                   two expand convolutions whose outputs are stacked by layer).
  squeezenet       Section II (two plain convolutional layers, eight fire
                   layers, pooling, softmax, 1000 classes); layer sizes are the
                   SqueezeNet v1.0 ones.

Parity pins live in tests/test_oracle_pins.py.  The end-to-end network value is
"parity unpinned" beyond its per-layer pins, its shape chain and its parameter
count: the paper prints no activations or logits.
"""
import ctypes

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        fp = ctypes.POINTER(ctypes.c_float)
        i = ctypes.c_int
        lib.oracle_conv2d.argtypes = [fp, fp, fp, fp, i, i, i, i, i, i, i, i, i]
        lib.oracle_conv2d.restype = None
        lib.oracle_maxpool.argtypes = [fp, fp, i, i, i, i, i, i]
        lib.oracle_maxpool.restype = None
        lib.oracle_global_avgpool.argtypes = [fp, fp, i, i, i, i]
        lib.oracle_global_avgpool.restype = None
        lib.oracle_softmax.argtypes = [fp, fp, i, i]
        lib.oracle_softmax.restype = None
        lib.oracle_out_extent.argtypes = [i, i, i, i]
        lib.oracle_out_extent.restype = i
        lib.oracle_max_threads.restype = i
        lib.oracle_set_threads.argtypes = [i]
        _lib = lib
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def set_threads(n: int) -> None:
    _load().oracle_set_threads(int(n))


def out_extent(H: int, K: int, S: int, pad: int) -> int:
    """(H + 2*pad - K) / S + 1 with integer division."""
    return int(_load().oracle_out_extent(H, K, S, pad))


def conv2d(x, ker, bias=None, S=1, pad=0, relu=True):
    """Convolution layer; x [N,C,H,W], ker [M,C,K,K], bias [M] or None."""
    x = _f32(x)
    ker = _f32(ker)
    N, C, H, W = x.shape
    M, C2, K, K2 = ker.shape
    if C != C2 or K != K2:
        raise ValueError("kernel shape %r does not match input %r" % (ker.shape, x.shape))
    if H + 2 * pad < K or W + 2 * pad < K:
        raise ValueError("window larger than padded input")
    oh, ow = out_extent(H, K, S, pad), out_extent(W, K, S, pad)
    out = np.empty((N, M, oh, ow), dtype=np.float32)
    if bias is not None:
        bias = _f32(bias)
        if bias.shape != (M,):
            raise ValueError("bias shape")
    _load().oracle_conv2d(_ptr(x), _ptr(ker), _ptr(bias) if bias is not None else None,
                          _ptr(out), N, C, H, W, M, K, S, pad, 1 if relu else 0)
    return out


def maxpool(x, K=3, S=2):
    x = _f32(x)
    N, C, H, W = x.shape
    out = np.empty((N, C, out_extent(H, K, S, 0), out_extent(W, K, S, 0)), dtype=np.float32)
    _load().oracle_maxpool(_ptr(x), _ptr(out), N, C, H, W, K, S)
    return out


def global_avgpool(x):
    x = _f32(x)
    N, C, H, W = x.shape
    out = np.empty((N, C), dtype=np.float32)
    _load().oracle_global_avgpool(_ptr(x), _ptr(out), N, C, H, W)
    return out


def softmax(z):
    z = _f32(z)
    N, K = z.shape
    out = np.empty((N, K), dtype=np.float32)
    _load().oracle_softmax(_ptr(z), _ptr(out), N, K)
    return out


def fire(x, w_sq, b_sq, w_e1, b_e1, w_e3, b_e3, return_squeeze=False):
    """Fire layer: squeeze 1x1 -> {expand 1x1, expand 3x3 pad 1}, stacked by layer."""
    s = conv2d(x, w_sq, b_sq, S=1, pad=0, relu=True)
    e1 = conv2d(s, w_e1, b_e1, S=1, pad=0, relu=True)
    e3 = conv2d(s, w_e3, b_e3, S=1, pad=1, relu=True)
    out = np.concatenate([e1, e3], axis=1)
    return (out, s) if return_squeeze else out


# SqueezeNet v1.0: (name, squeeze, expand1x1, expand3x3) for fire2..fire9 and
# the places where a 3x3/stride-2 max-pool follows.
_FIRE = [("fire2", 16, 64, 64), ("fire3", 16, 64, 64), ("fire4", 32, 128, 128),
         ("fire5", 32, 128, 128), ("fire6", 48, 192, 192), ("fire7", 48, 192, 192),
         ("fire8", 64, 256, 256), ("fire9", 64, 256, 256)]
_POOL_AFTER = ("conv1", "fire4", "fire8")


def squeezenet(x, params, conv10_relu=True, trace=None):
    """SqueezeNet v1.0 forward.

    x       [N,3,227,227]
    params  dict name -> (kernel, bias) with names conv1, fire{2..9}_{sq,e1,e3}, conv10
    trace   optional dict; receives every intermediate activation by name
    returns (logits [N,1000] = global average of conv10's map, probs [N,1000])
    """
    def keep(name, a):
        if trace is not None:
            trace[name] = a
        return a

    a = keep("conv1", conv2d(x, *params["conv1"], S=2, pad=0, relu=True))
    a = keep("pool1", maxpool(a, 3, 2))
    for name, _s, _e1, _e3 in _FIRE:
        out, s = fire(a, *params[name + "_sq"], *params[name + "_e1"], *params[name + "_e3"],
                      return_squeeze=True)
        keep(name + "_sq", s)
        a = keep(name, out)
        if name in _POOL_AFTER:
            a = keep("pool" + name[-1], maxpool(a, 3, 2))
    a = keep("conv10", conv2d(a, *params["conv10"], S=1, pad=0, relu=conv10_relu))
    logits = keep("logits", global_avgpool(a))
    probs = keep("probs", softmax(logits))
    return logits, probs
