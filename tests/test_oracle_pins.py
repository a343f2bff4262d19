"""Pins for the CPU oracle: hand-worked fixtures, closed forms, invariants,
library routines and brute force.  None of these values comes from the CUDA path.

The pins are collected in `conv_pins(conv)` so that the last tests can plant
mistakes in the oracle (on the CPU) and show that each one trips a pin.
"""
import numpy as np
import pytest
import scipy.signal
import torch

from oracle import ref
from paper_1611_07151_b200 import synth
from golden_io import read_blocks, read_shapes


def _as4(a):
    return np.asarray(a, dtype=np.float32)[None, None]


# ----------------------------------------------------------------- conv pins

def pin_hand_2x2(conv):
    g = read_blocks("conv_2x2_on_3x3.txt")
    out = conv(_as4(g["input"]), _as4(g["kernel"]), g["bias"].ravel().astype(np.float32), 1, 0, False)
    np.testing.assert_array_equal(out[0, 0], g["expected"])


def pin_hand_stride_pad(conv):
    g = read_blocks("conv_3x3_stride2_pad1.txt")
    out = conv(_as4(g["input"]), _as4(g["kernel"]), g["bias"].ravel().astype(np.float32), 2, 1, False)
    assert out.shape == (1, 1, 2, 2)
    np.testing.assert_array_equal(out[0, 0], g["expected"])


def pin_hand_asymmetric(conv):
    g = read_blocks("conv_asymmetric_kernel.txt")
    k3 = np.zeros((3, 3))
    k3[:2, :] = g["kernel"]                      # third kernel row is zero
    x = np.vstack([g["input"], np.zeros((1, 4))])  # one extra zero row so a 3x3 window fits twice
    out = conv(_as4(x), _as4(k3), None, 1, 0, False)
    np.testing.assert_array_equal(out[0, 0, :2, :2], g["expected"])


def pin_bias_and_relu(conv):
    x = _as4([[1.0, -2.0], [3.0, -4.0]])
    k = _as4([[1.0]])
    out = conv(x, k, np.array([0.5], np.float32), 1, 0, True)
    np.testing.assert_array_equal(out[0, 0], [[1.5, 0.0], [3.5, 0.0]])
    out = conv(x, k, np.array([0.5], np.float32), 1, 0, False)
    np.testing.assert_array_equal(out[0, 0], [[1.5, -1.5], [3.5, -3.5]])


def pin_identity_1x1(conv):
    rng = np.random.default_rng(10)
    x = rng.random((2, 5, 6, 7), dtype=np.float32)
    k = np.eye(5, dtype=np.float32).reshape(5, 5, 1, 1)
    np.testing.assert_array_equal(conv(x, k, None, 1, 0, True), x)


def pin_impulse_gives_flipped_kernel(conv):
    """A unit impulse at (y0,x0) of layer c yields ker[m][c][y0+pad-h*S][x0+pad-w*S]:
    the kernel appears spatially reversed in the output (dot product, no flip)."""
    rng = np.random.default_rng(11)
    M, C, K, H, W = 3, 2, 3, 7, 8
    ker = rng.standard_normal((M, C, K, K)).astype(np.float32)
    for (S, pad) in [(1, 1), (1, 0), (2, 1)]:
        for (c, y0, x0) in [(0, 3, 4), (1, 2, 2), (1, 0, 0)]:
            x = np.zeros((1, C, H, W), np.float32)
            x[0, c, y0, x0] = 1.0
            out = conv(x, ker, None, S, pad, False)
            exp = np.zeros_like(out)
            for h in range(out.shape[2]):
                for w in range(out.shape[3]):
                    i, j = y0 + pad - h * S, x0 + pad - w * S
                    if 0 <= i < K and 0 <= j < K:
                        exp[0, :, h, w] = ker[:, c, i, j]
            np.testing.assert_array_equal(out, exp)


def pin_all_ones(conv):
    C, K = 6, 3
    x = np.ones((1, C, 9, 9), np.float32)
    k = np.ones((4, C, K, K), np.float32)
    b = np.array([0.0, 1.0, -2.0, 0.25], np.float32)
    out = conv(x, k, b, 2, 0, False)
    assert out.shape == (1, 4, 4, 4)
    for m in range(4):
        np.testing.assert_array_equal(out[0, m], np.full((4, 4), C * K * K + b[m]))


def pin_linearity_and_layer_sum(conv):
    rng = np.random.default_rng(12)
    x = rng.standard_normal((1, 3, 8, 8)).astype(np.float32)
    y = rng.standard_normal((1, 3, 8, 8)).astype(np.float32)
    k = rng.standard_normal((4, 3, 3, 3)).astype(np.float32)
    lhs = conv((2.0 * x + y).astype(np.float32), k, None, 1, 1, False)
    rhs = 2.0 * conv(x, k, None, 1, 1, False) + conv(y, k, None, 1, 1, False)
    np.testing.assert_allclose(lhs, rhs, rtol=0, atol=2e-5)
    # the sum over input layers: a 3-layer result is the sum of three 1-layer results
    parts = sum(conv(x[:, c:c + 1], k[:, c:c + 1], None, 1, 1, False).astype(np.float64) for c in range(3))
    np.testing.assert_allclose(conv(x, k, None, 1, 1, False), parts, rtol=0, atol=2e-6)


def pin_centre_tap_is_1x1(conv):
    rng = np.random.default_rng(13)
    x = rng.random((2, 4, 6, 5), dtype=np.float32)
    k1 = rng.standard_normal((3, 4, 1, 1)).astype(np.float32)
    k3 = np.zeros((3, 4, 3, 3), np.float32)
    k3[:, :, 1, 1] = k1[:, :, 0, 0]
    b = rng.standard_normal(3).astype(np.float32)
    np.testing.assert_array_equal(conv(x, k3, b, 1, 1, True), conv(x, k1, b, 1, 0, True))


def pin_matmul_1x1(conv):
    """A 1x1/s1 layer is the matrix product [pixels, Cin] . [Cin, Cout]."""
    rng = np.random.default_rng(14)
    x = rng.random((2, 24, 5, 7), dtype=np.float32)
    k = rng.standard_normal((10, 24, 1, 1)).astype(np.float32)
    b = rng.standard_normal(10).astype(np.float32)
    A = x.transpose(0, 2, 3, 1).reshape(-1, 24).astype(np.float64)
    exp = (A @ k.reshape(10, 24).astype(np.float64).T + b).reshape(2, 5, 7, 10).transpose(0, 3, 1, 2)
    np.testing.assert_allclose(conv(x, k, b, 1, 0, False), exp, rtol=0, atol=1e-6)


def pin_scipy_correlate(conv):
    """Stride-1 layers against scipy.signal.correlate2d summed over input layers;
    strided layers are the stride-1 result sub-sampled."""
    rng = np.random.default_rng(15)
    for (C, M, H, W, K, S, pad) in [(3, 2, 9, 8, 3, 1, 1), (2, 3, 11, 11, 7, 2, 0), (4, 2, 6, 7, 2, 1, 0),
                                    (1, 1, 5, 5, 5, 1, 2), (2, 2, 10, 9, 3, 3, 1)]:
        x = rng.standard_normal((1, C, H, W)).astype(np.float32)
        k = rng.standard_normal((M, C, K, K)).astype(np.float32)
        b = rng.standard_normal(M).astype(np.float32)
        xp = np.pad(x.astype(np.float64), ((0, 0), (0, 0), (pad, pad), (pad, pad)))
        exp = np.stack([sum(scipy.signal.correlate2d(xp[0, c], k[m, c].astype(np.float64), mode="valid")
                            for c in range(C)) + b[m] for m in range(M)])[:, ::S, ::S]
        out = conv(x, k, b, S, pad, False)
        assert out.shape[1:] == exp.shape
        np.testing.assert_allclose(out[0], exp, rtol=0, atol=1e-5)


def pin_torch_conv2d(conv):
    rng = np.random.default_rng(16)
    for (N, C, M, H, W, K, S, pad) in [(2, 16, 8, 9, 9, 3, 1, 1), (1, 3, 6, 23, 23, 7, 2, 0), (3, 8, 5, 4, 6, 1, 1, 0),
                                       (1, 5, 4, 12, 10, 3, 2, 1)]:
        x = rng.random((N, C, H, W), dtype=np.float32)
        k = rng.standard_normal((M, C, K, K)).astype(np.float32)
        b = rng.standard_normal(M).astype(np.float32)
        exp = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(k).double(),
                                         torch.from_numpy(b).double(), stride=S, padding=pad).relu().numpy()
        np.testing.assert_allclose(conv(x, k, b, S, pad, True), exp, rtol=0, atol=1e-5)


def pin_scatter_form(conv):
    """Brute force in a different formulation: loop over input pixels and add each
    one's contribution into the outputs it touches (pure Python, tiny case)."""
    rng = np.random.default_rng(17)
    C, M, H, W, K, S, pad = 2, 2, 5, 6, 3, 2, 1
    x = rng.standard_normal((1, C, H, W)).astype(np.float32)
    k = rng.standard_normal((M, C, K, K)).astype(np.float32)
    oh, ow = (H + 2 * pad - K) // S + 1, (W + 2 * pad - K) // S + 1
    exp = np.zeros((1, M, oh, ow))
    for c in range(C):
        for y in range(H):
            for xx in range(W):
                for m in range(M):
                    for i in range(K):
                        for j in range(K):
                            hn, wn = y + pad - i, xx + pad - j
                            if hn % S or wn % S:
                                continue
                            h, w = hn // S, wn // S
                            if 0 <= h < oh and 0 <= w < ow:
                                exp[0, m, h, w] += float(x[0, c, y, xx]) * float(k[m, c, i, j])
    np.testing.assert_allclose(conv(x, k, None, S, pad, False), exp, rtol=0, atol=1e-6)


def pin_batch_independence(conv):
    rng = np.random.default_rng(18)
    x = rng.random((3, 4, 6, 6), dtype=np.float32)
    k = rng.standard_normal((5, 4, 3, 3)).astype(np.float32)
    b = rng.standard_normal(5).astype(np.float32)
    full = conv(x, k, b, 1, 1, True)
    for n in range(3):
        np.testing.assert_array_equal(full[n:n + 1], conv(x[n:n + 1], k, b, 1, 1, True))


CONV_PINS = [pin_hand_2x2, pin_hand_stride_pad, pin_hand_asymmetric, pin_bias_and_relu, pin_identity_1x1,
             pin_impulse_gives_flipped_kernel, pin_all_ones, pin_linearity_and_layer_sum, pin_centre_tap_is_1x1,
             pin_matmul_1x1, pin_scipy_correlate, pin_torch_conv2d, pin_scatter_form, pin_batch_independence]


def oracle_conv(x, k, b, S, pad, relu):
    return ref.conv2d(x, k, b, S=S, pad=pad, relu=relu)


@pytest.mark.parametrize("pin", CONV_PINS, ids=lambda f: f.__name__)
def test_conv_pin(pin):
    pin(oracle_conv)


# ------------------------------------------------- planted mistakes trip the pins

def _mutants():
    def flipped(x, k, b, S, pad, relu):
        return ref.conv2d(x, k[:, :, ::-1, ::-1], b, S=S, pad=pad, relu=relu)

    def transposed(x, k, b, S, pad, relu):
        return ref.conv2d(x, np.swapaxes(k, 2, 3), b, S=S, pad=pad, relu=relu)

    def no_bias(x, k, b, S, pad, relu):
        return ref.conv2d(x, k, None, S=S, pad=pad, relu=relu)

    def bias_after_relu(x, k, b, S, pad, relu):
        out = ref.conv2d(x, k, None, S=S, pad=pad, relu=relu)
        return out if b is None else out + np.asarray(b, np.float32)[None, :, None, None]

    def relu_always(x, k, b, S, pad, relu):
        return ref.conv2d(x, k, b, S=S, pad=pad, relu=True)

    def relu_never(x, k, b, S, pad, relu):
        return ref.conv2d(x, k, b, S=S, pad=pad, relu=False)

    def swapped_layers(x, k, b, S, pad, relu):
        return ref.conv2d(x, k[:, ::-1], b, S=S, pad=pad, relu=relu)

    def dropped_last_layer(x, k, b, S, pad, relu):
        k = np.array(k, np.float32)
        if k.shape[1] > 1:
            k[:, -1] = 0
        return ref.conv2d(x, k, b, S=S, pad=pad, relu=relu)

    def shifted_window(x, k, b, S, pad, relu):
        # a window that starts one pixel late: same as shifting the input left/up
        xs = np.zeros_like(x)
        xs[:, :, :-1, :-1] = x[:, :, 1:, 1:]
        return ref.conv2d(xs, k, b, S=S, pad=pad, relu=relu)

    def edge_replicated(x, k, b, S, pad, relu):
        if pad == 0:
            return ref.conv2d(x, k, b, S=S, pad=0, relu=relu)
        xp = np.pad(x, ((0, 0), (0, 0), (pad, pad), (pad, pad)), mode="edge")
        return ref.conv2d(xp, k, b, S=S, pad=0, relu=relu)

    def stride_one(x, k, b, S, pad, relu):
        return ref.conv2d(x, k, b, S=1, pad=pad, relu=relu)[:, :, ::1, ::1]

    return [flipped, transposed, no_bias, bias_after_relu, relu_always, relu_never, swapped_layers,
            dropped_last_layer, shifted_window, edge_replicated, stride_one]


@pytest.mark.parametrize("mutant", _mutants(), ids=lambda f: f.__name__)
def test_planted_mistake_trips_a_pin(mutant):
    tripped = []
    for pin in CONV_PINS:
        try:
            pin(mutant)
        except (AssertionError, ValueError):
            tripped.append(pin.__name__)
    assert tripped, "no pin noticed the planted mistake %s" % mutant.__name__


# ------------------------------------------------------------ pooling, softmax

def test_maxpool_hand_case():
    g = read_blocks("maxpool_3x3_s2_ramp5.txt")
    np.testing.assert_array_equal(ref.maxpool(_as4(g["input"]), 3, 2)[0, 0], g["expected"])


def test_maxpool_matches_torch_and_handles_negatives():
    rng = np.random.default_rng(20)
    x = rng.standard_normal((2, 5, 13, 11)).astype(np.float32) - 3.0   # mostly negative: a max seeded with 0 fails
    exp = torch.nn.functional.max_pool2d(torch.from_numpy(x), 3, 2).numpy()
    np.testing.assert_array_equal(ref.maxpool(x, 3, 2), exp)
    assert ref.maxpool(x, 3, 2).shape == (2, 5, 6, 5)


def test_global_avgpool_closed_form_and_torch():
    ramp = np.arange(169, dtype=np.float32).reshape(1, 1, 13, 13)
    assert ref.global_avgpool(ramp)[0, 0] == 84.0               # mean of 0..168
    rng = np.random.default_rng(21)
    x = rng.random((3, 7, 13, 13), dtype=np.float32)
    np.testing.assert_allclose(ref.global_avgpool(x), x.astype(np.float64).mean(axis=(2, 3)), rtol=0, atol=1e-7)


def test_softmax_hand_case_and_invariants():
    g = read_blocks("softmax_logs.txt")
    np.testing.assert_allclose(ref.softmax(g["input"].astype(np.float32)), g["expected"], rtol=0, atol=1e-7)
    rng = np.random.default_rng(22)
    z = (rng.standard_normal((4, 1000)) * 5).astype(np.float32)
    p = ref.softmax(z)
    np.testing.assert_allclose(p.astype(np.float64).sum(axis=1), 1.0, rtol=0, atol=1e-6)
    np.testing.assert_allclose(ref.softmax(z + np.float32(3.0)), p, rtol=0, atol=1e-7)   # shift invariance
    np.testing.assert_allclose(p, torch.softmax(torch.from_numpy(z).double(), dim=1).numpy(), rtol=0, atol=1e-7)
    big = np.array([[1000.0, 1001.0]], np.float32)                                      # no overflow
    np.testing.assert_allclose(ref.softmax(big), [[1 / (1 + np.e), np.e / (1 + np.e)]], rtol=0, atol=1e-7)


# ------------------------------------------------------------- fire, whole net

def test_out_extent_formula():
    assert ref.out_extent(227, 7, 2, 0) == 111
    assert ref.out_extent(111, 3, 2, 0) == 55
    assert ref.out_extent(55, 3, 2, 0) == 27
    assert ref.out_extent(27, 3, 2, 0) == 13
    assert ref.out_extent(55, 3, 1, 1) == 55
    assert ref.out_extent(224, 7, 2, 0) == 109        # the paper's 224 input: integer division


def test_fire_is_three_convolutions_stacked_by_layer():
    x, sq, e1, e3 = synth.fire_case(1, 2, 12, 4, 8, 6, 9)
    out, s = ref.fire(x, *sq, *e1, *e3, return_squeeze=True)
    assert out.shape == (2, 14, 9, 9)
    np.testing.assert_array_equal(s, ref.conv2d(x, *sq, S=1, pad=0, relu=True))
    np.testing.assert_array_equal(out[:, :8], ref.conv2d(s, *e1, S=1, pad=0, relu=True))
    np.testing.assert_array_equal(out[:, 8:], ref.conv2d(s, *e3, S=1, pad=1, relu=True))
    # against torch, double precision, composed independently
    t = lambda a: torch.from_numpy(np.asarray(a)).double()
    F = torch.nn.functional
    ts = F.conv2d(t(x), t(sq[0]), t(sq[1])).relu().float().double()     # squeeze map stored as float
    exp = torch.cat([F.conv2d(ts, t(e1[0]), t(e1[1])).relu(), F.conv2d(ts, t(e3[0]), t(e3[1]), padding=1).relu()], 1)
    np.testing.assert_allclose(out, exp.numpy(), rtol=0, atol=1e-5)


def test_squeezenet_shapes_parameters_and_softmax():
    shapes, nparams = read_shapes("squeezenet_v1_0_shapes.txt")
    x, params = synth.squeezenet_case(2, 1)
    assert sum(w.size + b.size for w, b in params.values()) == nparams
    trace = {}
    logits, probs = ref.squeezenet(x, params, trace=trace)
    for name, c, h, w in shapes:
        assert trace[name].shape == (1, c, h, w), name
    assert logits.shape == (1, 1000) and probs.shape == (1, 1000)
    assert abs(float(probs.astype(np.float64).sum()) - 1.0) <= 1e-6
    assert (trace["fire4"] >= 0).all()                      # post-ReLU maps
    # the generator's shape list and the oracle's own table describe the same network
    assert [n for n, *_ in synth.SQUEEZENET_CONVS] == [k for k in params]
    for name, cin, cout, k, s, pad, hw in synth.SQUEEZENET_CONVS:
        assert params[name][0].shape == (cout, cin, k, k)


def test_squeezenet_chain_matches_torch_double():
    """The whole chain against torch CPU ops composed independently (double)."""
    x, params = synth.squeezenet_case(5, 1)
    logits, probs = ref.squeezenet(x, params)
    t = lambda a: torch.from_numpy(np.asarray(a)).double()
    F = torch.nn.functional
    cv = lambda a, n, **kw: F.conv2d(a, t(params[n][0]), t(params[n][1]), **kw).relu()
    a = F.max_pool2d(cv(t(x), "conv1", stride=2), 3, 2)
    for i in range(2, 10):
        s = cv(a, "fire%d_sq" % i)
        a = torch.cat([cv(s, "fire%d_e1" % i), cv(s, "fire%d_e3" % i, padding=1)], 1)
        if i in (4, 8):
            a = F.max_pool2d(a, 3, 2)
    z = cv(a, "conv10").mean(dim=(2, 3))
    scale = float(z.abs().max())
    np.testing.assert_allclose(logits, z.numpy(), rtol=0, atol=1e-4 * scale)
    assert int(np.argmax(logits[0])) == int(torch.argmax(z[0]))
    np.testing.assert_allclose(probs, torch.softmax(z, 1).numpy(), rtol=0, atol=1e-6)


def test_batch_images_are_independent():
    x, params = synth.squeezenet_case(6, 2)
    l2, _ = ref.squeezenet(x, params)
    l0, _ = ref.squeezenet(x[1:2], params)
    np.testing.assert_array_equal(l2[1:2], l0)
