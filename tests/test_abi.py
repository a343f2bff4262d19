"""CPU-side checks of the boundary: the library loads, exports what include/sqn.h declares,
validates arguments before touching the GPU, and its host layout helpers are exact."""
import os
import re

import numpy as np
import pytest
import torch

from paper_1611_07151_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sqn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b([a-z_0-9]+)\s*\(", text)) - {"defined"})


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert "conv_forward" in names and "fire_forward" in names and "squeezenet_forward" in names
    l = B.lib()
    for n in names:
        assert hasattr(l, n), "libsqn.so does not export " + n
    assert sorted(B.SIGNATURES) == names, "binding and header disagree on the entry points"


def test_status_strings():
    assert B.sqn_status_string(0) == "ok"
    for s in range(-6, 0):
        assert B.sqn_status_string(s) not in ("ok", "unknown status")
    assert B.sqn_status_string(-99) == "unknown status"


def test_bad_arguments_are_rejected_before_any_launch():
    l = B.lib()
    n0 = B.sqn_launch_count()
    p = 0x1000      # never dereferenced: validation fails first
    assert l.conv_forward(None, p, p, p, 3, 4, 8, 8, 3, 1, 1, 1) == B.SQN_ERR_BADARG
    assert l.conv_forward(p, p, p, p, 0, 4, 8, 8, 3, 1, 1, 1) == B.SQN_ERR_BADARG
    assert l.conv_forward(p, p, p, p, 3, 4, 8, 8, 0, 1, 1, 1) == B.SQN_ERR_BADARG
    assert l.conv_forward(p, p, p, p, 3, 4, 8, 8, 3, 0, 1, 1) == B.SQN_ERR_BADARG
    assert l.conv_forward(p, p, p, p, 3, 4, 8, 8, 3, 1, -1, 1) == B.SQN_ERR_BADARG
    assert l.conv_forward(p, p, p, p, 3, 4, 2, 2, 5, 1, 1, 1) == B.SQN_ERR_BADARG      # window > padded input
    assert l.conv_forward(p + 4, p, p, p, 3, 4, 8, 8, 3, 1, 1, 1) == B.SQN_ERR_ALIGN
    opts = B.sqn_conv_opts(7, 1, 0, 0, None, None, 0)
    assert l.conv_forward_ex(p, p, p, p, 3, 4, 8, 8, 3, 1, 1, 1, opts) == B.SQN_ERR_BADARG   # unknown dtype
    opts = B.sqn_conv_opts(B.SQN_F32, 1, 4, 6, None, None, 0)
    assert l.conv_forward_ex(p, p, p, p, 3, 4, 8, 8, 3, 1, 1, 1, opts) == B.SQN_ERR_BADARG   # slice overruns
    assert l.maxpool3x3s2_forward(p, p, 8, 2, 8, 1, 0, None) == B.SQN_ERR_BADARG
    assert l.avgpool_softmax_forward(p, p, p, 10000, 2, 2, 1, 0, None) == B.SQN_ERR_UNSUPPORTED
    assert l.avgpool_softmax_forward(p, p, p, 1000, 13, 13, 70000, 1, None) == B.SQN_ERR_UNSUPPORTED   # batch > 65535
    assert l.avgpool_softmax_forward(p + 4, p, p, 1000, 13, 13, 1, 0, None) == B.SQN_ERR_ALIGN    # fp32 map, 4-byte aligned
    assert l.avgpool_softmax_forward(p + 2, p, p, 1000, 13, 13, 1, 1, None) == B.SQN_ERR_ALIGN    # bf16 map, 2-byte aligned
    assert l.avgpool_softmax_forward(p, p + 2, p, 1000, 13, 13, 1, 0, None) == B.SQN_ERR_ALIGN    # logits
    assert l.avgpool_softmax_forward(p, p, p + 1, 1000, 13, 13, 1, 0, None) == B.SQN_ERR_ALIGN    # probs
    # fire_forward_static: a squeeze map whose byte count wraps 64 bits is refused like any other that is too large
    assert l.fire_forward_static(p, p, p, p, p, p, p, p, 16, 65536, 16, 16, 65536, 65536, 65536, 0, None) == B.SQN_ERR_WORKSPACE
    assert l.fire_forward(p, p, p, p, p, p, p, None, p, 8, 4, 8, 8, 5, 5, 1, 0, None) == B.SQN_ERR_BADARG
    assert B.sqn_launch_count() == n0


def test_bf16_path_refuses_shapes_outside_its_family():
    l = B.lib()
    p = 0x1000
    n0 = B.sqn_launch_count()
    for (cin, cout, k, s, pad) in [(12, 16, 1, 1, 0), (16, 20, 1, 1, 0), (16, 16, 3, 2, 1), (16, 16, 9, 1, 4), (16, 16, 1, 1, 1)]:
        opts = B.sqn_conv_opts(B.SQN_BF16, 1, 0, 0, None, None, 0)
        rc = l.conv_forward_ex(p, p, p, p, cin, cout, 9, 9, k, s, pad, 1, opts)
        assert rc in (B.SQN_ERR_UNSUPPORTED, B.SQN_ERR_ALIGN), (cin, cout, k, s, pad, rc)
    assert B.sqn_launch_count() == n0


def test_pack_helpers_are_exact_transposes():
    rng = np.random.default_rng(0)
    w = rng.standard_normal((5, 3, 7, 7)).astype(np.float32)
    np.testing.assert_array_equal(B.sqn_pack_weights_oihw_to_ohwi(w), w.transpose(0, 2, 3, 1))
    x = rng.standard_normal((2, 6, 4, 5)).astype(np.float32)
    nhwc = B.sqn_pack_nchw_to_nhwc(x)
    np.testing.assert_array_equal(nhwc, x.transpose(0, 2, 3, 1))
    np.testing.assert_array_equal(B.sqn_unpack_nhwc_to_nchw(nhwc), x)


def test_bf16_rounding_is_nearest_even():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(4096).astype(np.float32) * 10,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40, np.inf], np.float32)])
    x = x.reshape(1, -1, 1, 1)
    got = B.sqn_pack_nchw_to_nhwc(x, B.SQN_BF16).ravel()
    exp = torch.from_numpy(x.ravel()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(got, exp)
    back = B.sqn_unpack_nhwc_to_nchw(got.reshape(1, 1, 1, -1), B.SQN_BF16).ravel()
    np.testing.assert_array_equal(back, torch.from_numpy(x.ravel()).to(torch.bfloat16).float().numpy())


def test_squeezenet_handle_and_workspace_without_gpu():
    l = B.lib()
    p = 0x1000
    h = B.squeezenet_create([p] * 26, [p] * 26, B.SQN_F32, 4)
    b1 = B.squeezenet_workspace_bytes(h, 1)
    b4 = B.squeezenet_workspace_bytes(h, 4)
    per_image = 4 * (1182816 + 290400 + 2 * (48400 + 387200) + 96800 + 774400 + 186624 + 23328 + 186624
                     + 2 * (34992 + 279936) + 46656 + 373248 + 86528 + 10816 + 86528 + 169000)
    assert per_image <= b1 <= per_image + 32 * 1024
    assert 4 * per_image <= b4 <= 4 * per_image + 32 * 1024
    with pytest.raises(B.SqnError):
        B.squeezenet_workspace_bytes(h, 5)            # beyond max_batch
    ptr, C, H, W = B.squeezenet_layer_output(h, "fire4", 0x100000, 1)
    assert (C, H, W) == (256, 55, 55) and ptr > 0x100000
    with pytest.raises(B.SqnError):
        B.squeezenet_layer_output(h, "fire99", 0x100000, 1)
    B.squeezenet_destroy(h)


def test_stem_pack_helpers_give_the_layout_the_stem_kernel_reads():
    """[N][3][H][W] -> [N][Hp][Wp][4] with 1.0 in the fourth layer of image pixels and zero padding; kernels
    [O][3][7][7] -> [O][7][8][4] with bias hi + lo in the fourth layer of the first two pixels of the first row."""
    rng = np.random.default_rng(5)
    x = rng.random((2, 3, 9, 11), dtype=np.float32)
    assert B.sqn_stem_packed_extent(9, 11) == (10, 12) and B.sqn_stem_packed_extent(227, 227) == (228, 228)
    got = B.sqn_pack_stem_input(x)
    bf = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    exp = np.zeros((2, 10, 12, 4), dtype=np.uint16)
    exp[:, :9, :11, :3] = bf(x.transpose(0, 2, 3, 1))
    exp[:, :9, :11, 3] = 0x3f80
    np.testing.assert_array_equal(got, exp)
    w = rng.standard_normal((5, 3, 7, 7)).astype(np.float32)
    b = rng.standard_normal(5).astype(np.float32)
    gw = B.sqn_pack_stem_weights(w, b)
    ew = np.zeros((5, 7, 8, 4), dtype=np.uint16)
    ew[:, :, :7, :3] = bf(w.transpose(0, 2, 3, 1))
    hi = torch.from_numpy(b).to(torch.bfloat16)
    lo = (torch.from_numpy(b) - hi.float()).to(torch.bfloat16)
    ew[:, 0, 0, 3] = hi.view(torch.int16).numpy().view(np.uint16)
    ew[:, 0, 1, 3] = lo.view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(gw, ew)
    h = B.squeezenet_create([0x1000] * 26, [0x1000] * 26, B.SQN_F32, 1)
    with pytest.raises(B.SqnError):
        B.squeezenet_set_stem_prepacked(h, True)          # bf16 nets only
    B.squeezenet_destroy(h)


def test_fp16_rounding_is_nearest_even():
    rng = np.random.default_rng(2)
    x = np.concatenate([rng.standard_normal(4096).astype(np.float32) * 10,
                        np.array([0.0, -0.0, 1.0, 1.00048828125, 1.0009765625, 65504.0, 65520.0, 1e-8, 6e-8, np.inf], np.float32)])
    x = x.reshape(1, -1, 1, 1)
    got = B.sqn_pack_nchw_to_nhwc(x, B.SQN_F16).ravel()
    exp = torch.from_numpy(x.ravel()).to(torch.float16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(got, exp)
    back = B.sqn_unpack_nhwc_to_nchw(got.reshape(1, 1, 1, -1), B.SQN_F16).ravel()
    np.testing.assert_array_equal(back, torch.from_numpy(x.ravel()).to(torch.float16).float().numpy())
