"""Seeded synthetic inputs for tests and benchmarks.

This module only draws random numbers and lists workload shapes; it contains
none of the layer arithmetic.  Generator: NumPy default_rng(seed) (PCG64), with
a fixed draw order -- the input tensor first, then for every convolution in
network order its kernels and then its bias.

Distributions (stand-ins for natural images and trained weights, keeping the
shapes and the post-ReLU, non-negative activation statistics):
  inputs   U[0,1)  or |N(0,1)|            float32, [batch, layer, row, col]
  kernels  N(0, 2/fan_in), fan_in = Cin*K*K (He-normal)   [Cout, Cin, K, K]
  bias     N(0, sigma = 0.01)                             [Cout]
"""
import numpy as np

# (name, Cin, Cout, K, S, pad, input H=W) for the 26 convolutions of
# SqueezeNet v1.0 on a 227x227 image, in network order.
SQUEEZENET_CONVS = [("conv1", 3, 96, 7, 2, 0, 227)]
for _name, _cin, _s, _e, _hw in [("fire2", 96, 16, 64, 55), ("fire3", 128, 16, 64, 55),
                                 ("fire4", 128, 32, 128, 55), ("fire5", 256, 32, 128, 27),
                                 ("fire6", 256, 48, 192, 27), ("fire7", 384, 48, 192, 27),
                                 ("fire8", 384, 64, 256, 27), ("fire9", 512, 64, 256, 13)]:
    SQUEEZENET_CONVS += [(_name + "_sq", _cin, _s, 1, 1, 0, _hw),
                         (_name + "_e1", _s, _e, 1, 1, 0, _hw),
                         (_name + "_e3", _s, _e, 3, 1, 1, _hw)]
SQUEEZENET_CONVS.append(("conv10", 512, 1000, 1, 1, 0, 13))


# A second workload for the single-layer entry points: the distinct 1x1 / 3x3 stride-1 convolution shapes of a
# bottleneck residual network on a 224x224 image (name, Cin, Cout, K, S, pad, input H=W).
BOTTLENECK_CONVS = [
    ("stage2_reduce", 256, 64, 1, 1, 0, 56), ("stage2_3x3", 64, 64, 3, 1, 1, 56), ("stage2_expand", 64, 256, 1, 1, 0, 56),
    ("stage3_reduce", 512, 128, 1, 1, 0, 28), ("stage3_3x3", 128, 128, 3, 1, 1, 28), ("stage3_expand", 128, 512, 1, 1, 0, 28),
    ("stage4_reduce", 1024, 256, 1, 1, 0, 14), ("stage4_3x3", 256, 256, 3, 1, 1, 14), ("stage4_expand", 256, 1024, 1, 1, 0, 14),
    ("stage5_reduce", 2048, 512, 1, 1, 0, 7), ("stage5_3x3", 512, 512, 3, 1, 1, 7), ("stage5_expand", 512, 2048, 1, 1, 0, 7),
]


def draw_input(rng, shape, dist="uniform"):
    if dist == "uniform":
        return rng.random(shape, dtype=np.float32)
    if dist == "absnormal":
        return np.abs(rng.standard_normal(shape, dtype=np.float32))
    raise ValueError(dist)


def draw_conv_params(rng, cin, cout, k):
    """He-normal kernels [cout,cin,k,k] and N(0, 0.01) bias [cout], float32."""
    std = np.float32(np.sqrt(2.0 / (cin * k * k)))
    w = rng.standard_normal((cout, cin, k, k), dtype=np.float32) * std
    b = rng.standard_normal((cout,), dtype=np.float32) * np.float32(0.01)
    return w, b


def conv_layer_case(seed, batch, cin, cout, hw, k, dist="uniform"):
    """One convolution layer: (input [batch,cin,hw,hw], kernels, bias)."""
    rng = np.random.default_rng(seed)
    x = draw_input(rng, (batch, cin, hw, hw), dist)
    w, b = draw_conv_params(rng, cin, cout, k)
    return x, w, b


def fire_case(seed, batch, cin, s, e1, e3, hw, dist="absnormal"):
    """One fire layer: input plus (kernel, bias) for squeeze, expand 1x1, expand 3x3."""
    rng = np.random.default_rng(seed)
    x = draw_input(rng, (batch, cin, hw, hw), dist)
    sq = draw_conv_params(rng, cin, s, 1)
    x1 = draw_conv_params(rng, s, e1, 1)
    x3 = draw_conv_params(rng, s, e3, 3)
    return x, sq, x1, x3


def squeezenet_params(rng):
    """dict name -> (kernels, bias) for the 26 convolutions, drawn in network order."""
    return {name: draw_conv_params(rng, cin, cout, k)
            for name, cin, cout, k, _s, _p, _hw in SQUEEZENET_CONVS}


def squeezenet_case(seed, batch):
    """Full network: (image batch [batch,3,227,227] ~ U[0,1), params dict)."""
    rng = np.random.default_rng(seed)
    x = draw_input(rng, (batch, 3, 227, 227), "uniform")
    return x, squeezenet_params(rng)
