"""A second workload through the single-layer entry point: the 1x1 / 3x3 convolution shapes of a bottleneck residual
network (up to 2048 layers, maps down to 7x7), in the three precisions, against the oracle."""
import numpy as np
import pytest

from oracle import ref
from paper_1611_07151_b200 import binding as B
from paper_1611_07151_b200 import synth
import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("layer", synth.BOTTLENECK_CONVS, ids=lambda l: l[0])
@pytest.mark.parametrize("dtype", [B.SQN_F32, B.SQN_BF16, B.SQN_F16], ids=["f32", "bf16", "f16"])
def test_bottleneck_shapes(layer, dtype):
    name, cin, cout, k, s, pad, hw = layer
    batch = 2 if hw >= 28 else 5
    rng = np.random.default_rng(cin + cout + hw)
    x = synth.draw_input(rng, (batch, cin, hw, hw))
    w, b = synth.draw_conv_params(rng, cin, cout, k)
    exp = ref.conv2d(x, w, b, S=s, pad=pad, relu=True)
    got = G.gpu_conv(x, w, b, s, pad, True, dtype)
    assert got.shape == exp.shape
    assert not np.isnan(got).any()
    assert G.rel_err(got, exp) <= G.TOL[dtype], name
