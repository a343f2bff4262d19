"""Helpers for the GPU parity tests: move oracle-layout arrays through the library's
pack helpers, call the C ABI via the binding, and bring results back as NCHW float32."""
import numpy as np

from paper_1611_07151_b200 import binding as B

TOL = {B.SQN_F32: 1e-4, B.SQN_BF16: 2e-2, B.SQN_F16: 3e-3}     # max|delta| / max|ref| per layer


def rel_err(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    scale = np.abs(ref).max()
    return float(np.abs(np.asarray(got, dtype=np.float64) - ref).max() / (scale if scale > 0 else 1.0))


def dev_act(x_nchw, dtype):
    return B.to_device(B.sqn_pack_nchw_to_nhwc(x_nchw, dtype), dtype)


def dev_w(w_oihw, dtype):
    return B.to_device(B.sqn_pack_weights_oihw_to_ohwi(w_oihw, dtype), dtype)


def dev_b(b):
    return B.to_device(np.ascontiguousarray(b, dtype=np.float32), B.SQN_F32)


def host_act(t, dtype):
    return B.sqn_unpack_nhwc_to_nchw(B.to_host(t, dtype), dtype)


def out_extent(H, K, S, pad):
    return (H + 2 * pad - K) // S + 1


def gpu_conv(x, w, b, S, pad, relu=True, dtype=B.SQN_F32, c_offset=0, c_total=0, fill=None, fuse_maxpool=False):
    """Run one convolution through conv_forward_ex; returns the full output tensor as NCHW."""
    import torch
    N, C, H, W = x.shape
    M, _, K, _ = w.shape
    oh, ow = out_extent(H, K, S, pad), out_extent(W, K, S, pad)
    if fuse_maxpool:
        oh, ow = (oh - 3) // 2 + 1, (ow - 3) // 2 + 1
    ct = c_total if c_total else M
    out = B.empty_device((N, oh, ow, ct), dtype)
    out.fill_(float("nan") if fill is None else fill)
    ws_bytes = B.conv_workspace_bytes(C, M, H, W, K, S, pad, N, dtype)
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")
    xd, wd, bd = dev_act(x, dtype), dev_w(w, dtype), dev_b(b)
    B.conv_forward_ex(xd, wd, bd, out, C, M, H, W, K, S, pad, N, dtype=dtype, relu=relu, out_c_offset=c_offset,
                      out_c_total=c_total, workspace=ws, workspace_bytes=ws_bytes, fuse_maxpool=fuse_maxpool)
    assert B.sqn_check() == B.SQN_OK
    return host_act(out, dtype)
