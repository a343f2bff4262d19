"""fp32 path vs the CPU oracle, element by element, through the C ABI.
Bar: max|delta| / max|ref| <= 1e-4 per layer."""
import numpy as np
import pytest

from oracle import ref
from paper_1611_07151_b200 import binding as B
from paper_1611_07151_b200 import synth
import gpu_util as G

pytestmark = pytest.mark.gpu
F32 = B.SQN_F32
TOL = G.TOL[F32]


def test_config0_fire2_expand3x3():
    """Single conv layer: 1x16x55x55 ~U[0,1), 64x16x3x3 He-normal, bias N(0,.01), K=3,S=1,pad=1, ReLU; seed 0."""
    x, w, b = synth.conv_layer_case(0, 1, 16, 64, 55, 3)
    exp = ref.conv2d(x, w, b, S=1, pad=1, relu=True)
    got = G.gpu_conv(x, w, b, 1, 1, True, F32)
    assert got.shape == (1, 64, 55, 55)
    assert G.rel_err(got, exp) <= TOL


def test_plain_conv_forward_entry_point():
    import torch
    x, w, b = synth.conv_layer_case(7, 2, 8, 24, 9, 3)
    exp = ref.conv2d(x, w, b, S=1, pad=1, relu=True)
    xd, wd, bd = G.dev_act(x, F32), G.dev_w(w, F32), G.dev_b(b)
    out = B.empty_device((2, 9, 9, 24), F32)
    torch.cuda.synchronize()
    B.conv_forward(xd, wd, bd, out, 8, 24, 9, 9, 3, 1, 1, 2)       # legacy default stream
    torch.cuda.synchronize()
    assert G.rel_err(G.host_act(out, F32), exp) <= TOL


# (N, Cin, Cout, H, K, S, pad): tiles with ragged tails, layer counts off the vector widths,
# every output-tile configuration, strides and paddings beyond SqueezeNet's
AWKWARD = [
    (1, 3, 96, 37, 7, 2, 0),      # stem shape, small map
    (3, 3, 5, 11, 3, 1, 1),       # scalar path, tiny layer count
    (2, 5, 7, 9, 2, 1, 0),        # even kernel, odd everything
    (2, 4, 16, 13, 3, 2, 1),      # vector path, Kdim = 36 (not a multiple of the k tile)
    (1, 12, 33, 10, 1, 1, 0),     # Cout one past a tile
    (3, 16, 48, 14, 3, 1, 1),     # 48-wide tile
    (2, 32, 192, 9, 1, 1, 0),     # 96-wide tiles
    (1, 64, 256, 13, 3, 1, 1),    # 128-wide tiles, Kdim 576
    (1, 48, 130, 7, 3, 1, 2),     # pad larger than SqueezeNet's, ragged Cout
    (5, 20, 17, 6, 5, 3, 2),      # stride 3, 5x5
    (1, 8, 8, 1, 1, 1, 0),        # 1x1 map
    (1, 7, 9, 5, 5, 1, 0),        # window == input: single output pixel
    (2, 515, 10, 4, 3, 1, 1),     # long scalar reduction (table does not fit)
]


@pytest.mark.parametrize("shape", AWKWARD, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("relu", [True, False])
def test_awkward_shapes(shape, relu):
    N, C, M, H, K, S, pad = shape
    rng = np.random.default_rng(sum(shape))
    x = rng.standard_normal((N, C, H, H + 1)).astype(np.float32)      # non-square map
    w, b = synth.draw_conv_params(rng, C, M, K)
    exp = ref.conv2d(x, w, b, S=S, pad=pad, relu=relu)
    got = G.gpu_conv(x, w, b, S, pad, relu, F32)
    assert got.shape == exp.shape
    assert not np.isnan(got).any()
    assert G.rel_err(got, exp) <= TOL


def test_output_slice_leaves_other_layers_untouched():
    x, w, b = synth.conv_layer_case(8, 2, 16, 24, 7, 3)
    exp = ref.conv2d(x, w, b, S=1, pad=1, relu=True)
    got = G.gpu_conv(x, w, b, 1, 1, True, F32, c_offset=8, c_total=40, fill=-7.0)
    assert G.rel_err(got[:, 8:32], exp) <= TOL
    assert (got[:, :8] == -7.0).all() and (got[:, 32:] == -7.0).all()


def test_per_layer_sweep_batch1_and_3():
    """Every distinct SqueezeNet conv shape, isolated, seed 4."""
    seen = set()
    for name, cin, cout, k, s, pad, hw in synth.SQUEEZENET_CONVS:
        key = (cin, cout, k, s, pad, hw)
        if key in seen:
            continue
        seen.add(key)
        for batch in (1, 3):
            if hw > 100 and batch > 1:
                continue
            x, w, b = synth.conv_layer_case(4, batch, cin, cout, hw, k)
            exp = ref.conv2d(x, w, b, S=s, pad=pad, relu=True)
            got = G.gpu_conv(x, w, b, s, pad, True, F32)
            assert G.rel_err(got, exp) <= TOL, (name, batch)


def test_maxpool_and_head():
    import torch
    rng = np.random.default_rng(30)
    for (N, C, H, W) in [(2, 96, 111, 111), (1, 256, 55, 55), (3, 512, 27, 27), (2, 6, 9, 8), (1, 3, 3, 3)]:
        x = rng.standard_normal((N, C, H, W)).astype(np.float32) - 1.0
        out = B.empty_device((N, (H - 3) // 2 + 1, (W - 3) // 2 + 1, C), F32)
        B.maxpool3x3s2_forward(G.dev_act(x, F32), out, C, H, W, N, F32)
        np.testing.assert_array_equal(G.host_act(out, F32), ref.maxpool(x, 3, 2))
    for (N, C, H, W) in [(3, 1000, 13, 13), (2, 10, 4, 5), (1, 8192, 2, 2)]:
        x = (rng.standard_normal((N, C, H, W)) * 3).astype(np.float32)
        logits = torch.empty((N, C), device="cuda")
        probs = torch.empty((N, C), device="cuda")
        B.avgpool_softmax_forward(G.dev_act(x, F32), logits, probs, C, H, W, N, F32)
        z = ref.global_avgpool(x)
        assert G.rel_err(logits.cpu().numpy(), z) <= 1e-5
        p = probs.cpu().numpy()
        np.testing.assert_allclose(p, ref.softmax(z), rtol=0, atol=1e-5)
        np.testing.assert_allclose(p.astype(np.float64).sum(1), 1.0, rtol=0, atol=1e-5)


def test_config1_fire4():
    """Full fire module (fire4), batch 1: 1x128x55x55 ~|N(0,1)|, squeeze 32, expands 128+128; seed 1."""
    x, sq, e1, e3 = synth.fire_case(1, 1, 128, 32, 128, 128, 55)
    exp, s_exp = ref.fire(x, *sq, *e1, *e3, return_squeeze=True)
    xd = G.dev_act(x, F32)
    scratch = B.empty_device((1, 55, 55, 32), F32)
    out = B.empty_device((1, 55, 55, 256), F32)
    out.fill_(float("nan"))
    B.fire_forward(xd, G.dev_w(sq[0], F32), G.dev_b(sq[1]), G.dev_w(e1[0], F32), G.dev_b(e1[1]),
                   G.dev_w(e3[0], F32), G.dev_b(e3[1]), scratch, out, 128, 32, 128, 128, 55, 55, 1, F32)
    assert B.sqn_check() == B.SQN_OK
    got = G.host_act(out, F32)
    assert G.rel_err(G.host_act(scratch, F32), s_exp) <= TOL
    assert G.rel_err(got[:, :128], exp[:, :128]) <= TOL
    assert G.rel_err(got[:, 128:], exp[:, 128:]) <= TOL


LAYER_NAMES = ["conv1", "pool1"] + ["fire%d%s" % (i, s) for i in range(2, 10) for s in ("_sq", "")] + \
    ["pool4", "pool8", "conv10"]


def run_net_device(x, params, dtype, batch):
    """One forward through squeezenet_forward.  Returns (logits, probs, {layer name: device view [batch][H][W][C]});
    the views alias the forward's workspace (kept alive by them)."""
    import torch
    names = [n for n, *_ in synth.SQUEEZENET_CONVS]
    ws = [G.dev_w(params[n][0], dtype) for n in names]
    bs = [G.dev_b(params[n][1]) for n in names]
    net = B.squeezenet_create(ws, bs, dtype, batch)
    nbytes = B.squeezenet_workspace_bytes(net, batch)
    work = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    logits = torch.empty((batch, 1000), device="cuda")
    probs = torch.empty((batch, 1000), device="cuda")
    B.squeezenet_forward(net, G.dev_act(x, dtype), logits, probs, work, batch)
    assert B.sqn_check() == B.SQN_OK
    views = {}
    for name in LAYER_NAMES:
        try:
            ptr, C, H, W = B.squeezenet_layer_output(net, name, work, batch)
        except B.SqnError as e:          # a layer the net fused away (bf16: conv1 lives inside conv1+pool1)
            assert e.status == B.SQN_ERR_UNSUPPORTED
            continue
        off = ptr - work.data_ptr()
        es = 4 if dtype == F32 else 2
        raw = work[off:off + batch * C * H * W * es]
        views[name] = raw.view({F32: torch.float32, B.SQN_BF16: torch.bfloat16, B.SQN_F16: torch.float16}[dtype]).view(batch, H, W, C)
    B.squeezenet_destroy(net)
    return logits.cpu().numpy(), probs.cpu().numpy(), views


def run_net(x, params, dtype, batch):
    logits, probs, views = run_net_device(x, params, dtype, batch)
    return logits, probs, {name: G.host_act(t, dtype) for name, t in views.items()}


def test_config2_full_forward_batch1():
    """SqueezeNet v1.0 full forward, fp32, batch 1, input 3x227x227 ~U[0,1); seed 2."""
    x, params = synth.squeezenet_case(2, 1)
    trace = {}
    z, p = ref.squeezenet(x, params, trace=trace)
    logits, probs, layers = run_net(x, params, F32, 1)
    for name, got in layers.items():                      # chained: each layer fed the GPU's own previous output
        assert G.rel_err(got, trace[name]) <= TOL, name
    assert G.rel_err(logits, z) <= TOL
    assert int(logits[0].argmax()) == int(z[0].argmax())
    np.testing.assert_allclose(probs, p, rtol=0, atol=1e-5)
    assert abs(float(probs.astype(np.float64).sum()) - 1.0) <= 1e-5


def test_full_forward_batch3_images_independent():
    x, params = synth.squeezenet_case(9, 3)
    z, _ = ref.squeezenet(x, params)
    logits, probs, _ = run_net(x, params, F32, 3)
    assert G.rel_err(logits, z) <= TOL
    assert (logits.argmax(1) == z.argmax(1)).all()
