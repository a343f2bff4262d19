"""Third precision point: fp16 activations and kernels (fp32 accumulation on the tensor cores) through the same kernels
as bf16, against the fp32 oracle.  Bar: max|delta| / max|ref| <= 3e-3 per layer (operands carry 2^-11 relative
rounding each, the stored output once more), top-1 unchanged on a seeded batch -- the acceptance test of the paper's
Section IV-B for its relaxed / imprecise modes."""
import numpy as np
import pytest

from oracle import ref
from paper_1611_07151_b200 import binding as B
from paper_1611_07151_b200 import synth
import gpu_util as G
from test_gpu_f32 import run_net

pytestmark = pytest.mark.gpu
F16 = B.SQN_F16
TOL = G.TOL[F16]


# (N, Cin, Cout, H, W, K, S, pad, pooled)
CONVS = [
    (3, 96, 16, 55, 55, 1, 1, 0, False),        # flat 1x1
    (2, 16, 64, 55, 55, 3, 1, 1, False),        # patch mode
    (2, 64, 256, 13, 13, 3, 1, 1, False),       # streamed kernels
    (1, 512, 1000, 13, 13, 1, 1, 0, False),     # conv10
    (2, 3, 96, 227, 227, 7, 2, 0, False),       # stem (repack on the device)
    (2, 3, 96, 227, 227, 7, 2, 0, True),        # stem + pool1
    (2, 32, 128, 55, 55, 3, 1, 1, True),        # fire4 expand-3x3 + pool4
]


@pytest.mark.parametrize("shape", CONVS, ids=lambda s: "x".join(map(str, s)))
def test_conv_shapes_f16(shape):
    N, C, M, H, W, K, S, pad, pooled = shape
    rng = np.random.default_rng(sum(shape[:8]))
    x = synth.draw_input(rng, (N, C, H, W))
    w, b = synth.draw_conv_params(rng, C, M, K)
    b = b + np.float32(0.2) * rng.standard_normal(M).astype(np.float32)
    exp = ref.conv2d(x, w, b, S=S, pad=pad, relu=True)
    if pooled:
        exp = ref.maxpool(exp, 3, 2)
    got = G.gpu_conv(x, w, b, S, pad, True, F16, fuse_maxpool=pooled)
    assert got.shape == exp.shape
    assert not np.isnan(got).any()
    assert G.rel_err(got, exp) <= TOL


def test_fused_global_average_f16():
    import torch
    N, C, M, H = 3, 512, 1000, 13
    rng = np.random.default_rng(5)
    x = synth.draw_input(rng, (N, C, H, H))
    w, b = synth.draw_conv_params(rng, C, M, 1)
    exp = ref.global_avgpool(ref.conv2d(x, w, b, S=1, pad=0, relu=True))
    out = torch.full((N, M), float("nan"), device="cuda")
    B.conv_forward_ex(G.dev_act(x, F16), G.dev_w(w, F16), G.dev_b(b), out, C, M, H, H, 1, 1, 0, N, dtype=F16,
                      fuse_global_avgpool=True)
    assert B.sqn_check() == B.SQN_OK
    assert G.rel_err(out.cpu().numpy(), exp) <= TOL


# (batch, Cin, s, e, H): one-kernel fire layers and the flat-patch expands
FIRES = [(2, 96, 16, 64, 55), (2, 256, 32, 128, 27), (2, 256, 48, 192, 27), (3, 512, 64, 256, 13)]


@pytest.mark.parametrize("shape", FIRES, ids=lambda s: "x".join(map(str, s)))
def test_fire_layers_f16(shape):
    N, cin, s, e, H = shape
    x, sq, x1, x3 = synth.fire_case(sum(shape), N, cin, s, e, e, H)
    exp = ref.fire(x, *sq, *x1, *x3)
    scratch = B.empty_device((N, H, H, s), F16)
    out = B.empty_device((N, H, H, 2 * e), F16)
    out.fill_(float("nan"))
    B.fire_forward(G.dev_act(x, F16), G.dev_w(sq[0], F16), G.dev_b(sq[1]), G.dev_w(x1[0], F16), G.dev_b(x1[1]),
                   G.dev_w(x3[0], F16), G.dev_b(x3[1]), scratch, out, cin, s, e, e, H, H, N, F16)
    assert B.sqn_check() == B.SQN_OK
    got = G.host_act(out, F16)
    assert not np.isnan(got).any()
    assert G.rel_err(got[:, :e], exp[:, :e]) <= TOL
    assert G.rel_err(got[:, e:], exp[:, e:]) <= TOL


def test_maxpool_and_head_f16():
    import torch
    rng = np.random.default_rng(33)
    half = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).half().float().numpy()
    for (N, C, H, W) in [(2, 96, 111, 111), (2, 6, 9, 8)]:
        x = half(rng.standard_normal((N, C, H, W)).astype(np.float32) - 1.0)
        out = B.empty_device((N, (H - 3) // 2 + 1, (W - 3) // 2 + 1, C), F16)
        B.maxpool3x3s2_forward(G.dev_act(x, F16), out, C, H, W, N, F16)
        np.testing.assert_array_equal(G.host_act(out, F16), ref.maxpool(x, 3, 2))       # exact: max of fp16 values
    for C in (1000, 10):
        x = half((rng.standard_normal((3, C, 13, 13)) * 3).astype(np.float32))
        logits = torch.empty((3, C), device="cuda")
        probs = torch.empty((3, C), device="cuda")
        B.avgpool_softmax_forward(G.dev_act(x, F16), logits, probs, C, 13, 13, 3, F16)
        z = ref.global_avgpool(x)
        assert G.rel_err(logits.cpu().numpy(), z) <= 1e-5
        np.testing.assert_allclose(probs.cpu().numpy(), ref.softmax(z), rtol=0, atol=1e-5)


@pytest.mark.parametrize("batch", [2, 32])
def test_full_forward_f16(batch):
    """Whole network in fp16 (batch 2: separate pools; batch 32: fused pools): every stored map within 1e-2 of the
    oracle's chain, logits within 3e-3, every image classified as the oracle classifies it."""
    x, params = synth.squeezenet_case(3, batch)
    trace = {}
    z, p = ref.squeezenet(x, params, trace=trace)
    logits, probs, layers = run_net(x, params, F16, batch)
    worst = max(G.rel_err(got, trace[name]) for name, got in layers.items())
    assert worst <= 1e-2, worst
    assert G.rel_err(logits, z) <= TOL
    assert (logits.argmax(1) == z.argmax(1)).all()
    np.testing.assert_allclose(probs.astype(np.float64).sum(1), 1.0, rtol=0, atol=1e-5)
    # the three precision points in order: fp16 sits between the exact path and bf16
    logits_bf16 = run_net(x, params, B.SQN_BF16, batch)[0]
    assert G.rel_err(logits, z) < G.rel_err(logits_bf16, z)
