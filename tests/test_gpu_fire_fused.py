"""The fire layer as one kernel (squeeze map kept in shared memory), bf16, against the fp32 oracle through
fire_forward.  Bar: max|delta| / max|ref| <= 2e-2 for each expand on its own scale."""
import os

import numpy as np
import pytest

from oracle import ref
from paper_1611_07151_b200 import binding as B
from paper_1611_07151_b200 import synth
import gpu_util as G

pytestmark = pytest.mark.gpu
BF16 = B.SQN_BF16
TOL = G.TOL[BF16]


def _fire_case(seed, batch, cin, s, e1, e3, H, W):
    rng = np.random.default_rng(seed)
    x = synth.draw_input(rng, (batch, cin, H, W), "absnormal")
    sq = synth.draw_conv_params(rng, cin, s, 1)
    x1 = synth.draw_conv_params(rng, s, e1, 1)
    x3 = synth.draw_conv_params(rng, s, e3, 3)
    # biases large enough to matter, some squeeze layers mostly negative (ReLU clips them)
    sq = (sq[0], sq[1] + np.float32(0.3) * rng.standard_normal(s).astype(np.float32))
    x1 = (x1[0], x1[1] + np.float32(0.3) * rng.standard_normal(e1).astype(np.float32))
    x3 = (x3[0], x3[1] + np.float32(0.3) * rng.standard_normal(e3).astype(np.float32))
    return x, sq, x1, x3


def _run(x, sq, x1, x3, fused=True, band=None):
    N, cin, H, W = x.shape
    s, e1, e3 = sq[0].shape[0], x1[0].shape[0], x3[0].shape[0]
    scratch = B.empty_device((N, H, W, s), BF16)
    scratch.fill_(float("nan"))
    out = B.empty_device((N, H, W, e1 + e3), BF16)
    out.fill_(float("nan"))
    old = {k: os.environ.get(k) for k in ("SQN_FUSED_FIRE", "SQN_FIRE_BAND")}
    try:
        os.environ["SQN_FUSED_FIRE"] = "1" if fused else "0"
        if band is not None:
            os.environ["SQN_FIRE_BAND"] = str(band)
        else:
            os.environ.pop("SQN_FIRE_BAND", None)
        n0 = B.sqn_launch_count()
        B.fire_forward(G.dev_act(x, BF16), G.dev_w(sq[0], BF16), G.dev_b(sq[1]), G.dev_w(x1[0], BF16), G.dev_b(x1[1]),
                       G.dev_w(x3[0], BF16), G.dev_b(x3[1]), scratch, out, cin, s, e1, e3, H, W, N, BF16)
        assert B.sqn_check() == B.SQN_OK
        launches = B.sqn_launch_count() - n0
    finally:
        for k, v in old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v
    return G.host_act(out, BF16), launches, scratch


def _check(got, exp, e1):
    assert got.shape == exp.shape
    assert not np.isnan(got).any()
    assert G.rel_err(got[:, :e1], exp[:, :e1]) <= TOL
    assert G.rel_err(got[:, e1:], exp[:, e1:]) <= TOL
    for n in range(got.shape[0]):          # per image: a band written to the wrong place must not hide
        assert G.rel_err(got[n], exp[n]) <= TOL, n


# (batch, Cin, s, e1, e3, H, W)
SHAPES = [
    (2, 96, 16, 64, 64, 55, 55),        # fire2: four bands per image, three 32-layer reduction chunks
    (3, 128, 16, 64, 64, 55, 55),       # fire3
    (2, 128, 32, 128, 128, 55, 55),     # fire4 (without its pool): both accumulators fill the TMEM
    (3, 256, 32, 128, 128, 27, 27),     # fire5: two bands of 16 and 11 rows
    (5, 256, 64, 64, 64, 13, 13),       # 128-byte patch rows, whole image per band, four reduction chunks
    (2, 64, 16, 64, 64, 9, 20),         # small non-square map
    (1, 32, 32, 64, 192, 31, 17),       # e1 != e3, odd extents
    (3, 64, 16, 64, 64, 3, 3),          # smaller than one tile
    (1, 32, 16, 64, 64, 1, 126),        # one row, widest supported map
    (2, 32, 16, 32, 32, 10, 9),         # 32-layer store chunks
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_fused_fire_matches_the_oracle(shape):
    N, cin, s, e1, e3, H, W = shape
    x, sq, x1, x3 = _fire_case(sum(shape), N, cin, s, e1, e3, H, W)
    exp = ref.fire(x, *sq, *x1, *x3)
    got, launches, scratch = _run(x, sq, x1, x3)
    assert launches == 1                                   # one kernel for the whole layer
    assert bool(scratch.isnan().all())                     # the squeeze map was not stored
    _check(got, exp, e1)
    # the three-launch path on the same operands agrees to output rounding (the accumulation order differs)
    sep, launches, _ = _run(x, sq, x1, x3, fused=False)
    assert launches >= 2
    assert G.rel_err(got, sep) <= 1e-2


@pytest.mark.parametrize("band", [2, 6, 28, 56])
def test_fused_fire_band_heights(band):
    """Any band height gives the same layer: bands of one tile, of many, and the whole image (where it fits)."""
    N, cin, s, e, H = 2, 96, 16, 64, 55
    x, sq, x1, x3 = _fire_case(100 + band, N, cin, s, e, e, H, H)
    exp = ref.fire(x, *sq, *x1, *x3)
    got, launches, _ = _run(x, sq, x1, x3, band=band)
    assert launches == 1
    _check(got, exp, e)


def test_fused_fire_many_items_per_cta():
    """More bands than CTAs: every CTA walks several bands (top, middle and bottom ones of different images), the
    patch is reused and its border rows are cleared in between."""
    N, cin, s, e, H = 160, 96, 16, 64, 55                    # 640 bands on at most 148 CTAs
    x, sq, x1, x3 = _fire_case(7, N, cin, s, e, e, H, H)
    exp = ref.fire(x, *sq, *x1, *x3)
    got, launches, _ = _run(x, sq, x1, x3)
    assert launches == 1
    _check(got, exp, e)
    N, cin, s, e, H = 200, 256, 32, 128, 27                  # fire5 shape: 400 bands of 16 and 11 rows
    x, sq, x1, x3 = _fire_case(8, N, cin, s, e, e, H, H)
    exp = ref.fire(x, *sq, *x1, *x3)
    got, launches, _ = _run(x, sq, x1, x3)
    assert launches == 1
    _check(got, exp, e)


# (batch, Cin, s, e1, e3, H, W): layers whose kernels do not fit one CTA beside a squeeze pipeline
SPLIT_SHAPES = [
    (2, 256, 48, 192, 192, 27, 27),     # fire6: three 16-layer chunks per tap, output layers split over two CTAs
    (2, 384, 48, 192, 192, 27, 27),     # fire7
    (3, 512, 64, 256, 256, 13, 13),     # fire9: output layers split over four CTAs
    (2, 384, 64, 256, 256, 27, 27),     # fire8 (without its pool)
    (1, 64, 96, 64, 128, 21, 30),       # three 32-layer chunks, e1 != e3, non-square
]


@pytest.mark.parametrize("shape", SPLIT_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_expands_on_a_stored_squeeze_map(shape):
    """Where the one-kernel path does not apply (s = 48, or kernels too large for one CTA), fire_forward runs the squeeze
    as its own launch and both expands as one launch of the flat-patch kernel (patch loaded by TMA, output layers
    split over up to four CTAs)."""
    N, cin, s, e1, e3, H, W = shape
    x, sq, x1, x3 = _fire_case(sum(shape), N, cin, s, e1, e3, H, W)
    exp = ref.fire(x, *sq, *x1, *x3)
    got, launches, scratch = _run(x, sq, x1, x3)
    assert launches == 2 and not bool(scratch.isnan().any())
    _check(got, exp, e1)
    # the tap-by-tap kernels on the same operands agree to output rounding
    sep, launches, _ = _run(x, sq, x1, x3, fused=False)
    assert launches >= 2
    assert G.rel_err(got, sep) <= 1e-2


def test_expands_many_bands_per_cta():
    N, cin, s, e, H = 100, 256, 48, 192, 27                  # 400 bands on 73 groups of two CTAs
    x, sq, x1, x3 = _fire_case(9, N, cin, s, e, e, H, H)
    exp = ref.fire(x, *sq, *x1, *x3)
    got, launches, _ = _run(x, sq, x1, x3)
    assert launches == 2
    _check(got, exp, e)
    N, cin, s, e, H = 150, 512, 64, 256, 13                  # 150 images on 37 groups of four CTAs
    x, sq, x1, x3 = _fire_case(10, N, cin, s, e, e, H, H)
    exp = ref.fire(x, *sq, *x1, *x3)
    got, launches, _ = _run(x, sq, x1, x3)
    assert launches == 2
    _check(got, exp, e)


def test_tuning_knobs_of_the_flat_expands_give_the_same_values():
    """SQN_FIRE_PATCHES (patches in shared memory), SQN_FIRE_CS (split of the output layers over CTAs) and
    SQN_FIRE_ESLOTS (expand accumulators) only change how the flat expand kernel is scheduled: every number of patches
    and accumulators that fits must give exactly the values of the library's own choice, every split the same values up
    to the rounding of the output (more bands than CTAs, so that patches are reused)."""
    x, sq, x1, x3 = _fire_case(61, 70, 384, 48, 192, 192, 27, 27)
    knobs = ("SQN_FIRE_PATCHES", "SQN_FIRE_CS", "SQN_FIRE_ESLOTS")
    old = {k: os.environ.get(k) for k in knobs}
    ran = 0
    try:
        for k in knobs:
            os.environ.pop(k, None)
        want, launches, _ = _run(x, sq, x1, x3)
        assert launches == 2
        for knob, values in (("SQN_FIRE_PATCHES", (2, 3, 4)), ("SQN_FIRE_CS", (2, 3, 4)), ("SQN_FIRE_ESLOTS", (2, 3))):
            for v in values:
                os.environ[knob] = str(v)
                try:
                    got, launches, _ = _run(x, sq, x1, x3)
                finally:
                    os.environ.pop(knob, None)
                if launches != 2:           # (the setting does not fit: the layer ran on other kernels)
                    continue
                if knob == "SQN_FIRE_CS":
                    # another split adds the taps' products in another order (the 1x1 expand rides on the centre tap
                    # or is a job of its own): equal up to the rounding of the stored value
                    assert G.rel_err(got, want) <= 1e-2, (knob, v)
                else:
                    np.testing.assert_array_equal(got, want, err_msg="%s=%d" % (knob, v))
                ran += 1
    finally:
        for k, v in old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v
    assert ran >= 5
