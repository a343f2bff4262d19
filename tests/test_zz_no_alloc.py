"""fire_forward_static: the fire layer for callers that cannot allocate device memory (a worker in a
serving process whose memory was handed out at start-up, a callback that must not call cudaMalloc).
It keeps the squeeze map in a buffer inside the library.  Checked against fire_forward, which takes
the scratch from the caller, on two calls in a row: the second call reuses the same built-in buffer
with different data, so anything left over from the first call would show.

This file is collected last on purpose: if it fails, a run that stops at the first failure has
already run every other test."""
import numpy as np
import pytest

from oracle import ref
from paper_1611_07151_b200 import binding as B
from paper_1611_07151_b200 import synth
import gpu_util as G

pytestmark = pytest.mark.gpu


def _run_both(seed, batch, cin, s, e, hw, dtype):
    x, sq, e1, e3 = synth.fire_case(seed, batch, cin, s, e, e, hw)
    dev = [G.dev_act(x, dtype), G.dev_w(sq[0], dtype), G.dev_b(sq[1]), G.dev_w(e1[0], dtype), G.dev_b(e1[1]),
           G.dev_w(e3[0], dtype), G.dev_b(e3[1])]
    scratch = B.empty_device((batch, hw, hw, s), dtype)
    ref_out = B.empty_device((batch, hw, hw, 2 * e), dtype)
    new_out = B.empty_device((batch, hw, hw, 2 * e), dtype)
    ref_out.fill_(float("nan"))
    new_out.fill_(float("nan"))
    B.fire_forward(*dev, scratch, ref_out, cin, s, e, e, hw, hw, batch, dtype)
    B.fire_forward_static(*dev, new_out, cin, s, e, e, hw, hw, batch, dtype)
    assert B.sqn_check() == B.SQN_OK
    a, b = G.host_act(ref_out, dtype), G.host_act(new_out, dtype)
    assert not np.isnan(b).any()
    assert G.rel_err(b, a) <= G.TOL[dtype]
    exp = ref.fire(x, *sq, *e1, *e3)                        # and against the oracle, each expand on its own scale
    assert G.rel_err(b[:, :e], exp[:, :e]) <= G.TOL[dtype]
    assert G.rel_err(b[:, e:], exp[:, e:]) <= G.TOL[dtype]
    return b


@pytest.mark.parametrize("dtype", [B.SQN_F32, B.SQN_BF16], ids=["f32", "bf16"])
def test_static_scratch_matches_caller_scratch_twice_in_a_row(dtype):
    first = _run_both(11, 2, 128, 32, 128, 27, dtype)      # fire5-like
    second = _run_both(12, 3, 96, 16, 64, 19, dtype)       # smaller map, other data, same built-in buffer
    assert first.shape == (2, 256, 27, 27) and second.shape == (3, 128, 19, 19)


def test_request_beyond_the_built_in_buffer_is_refused():
    import torch
    n0 = B.sqn_launch_count()
    p = torch.empty(64, device="cuda")       # never read: the size check comes first
    with pytest.raises(B.SqnError) as e:
        B.fire_forward_static(p, p, p, p, p, p, p, p, 128, 32, 128, 128, 55, 55, 64, B.SQN_F32)   # 24.8 MB squeeze map
    assert e.value.status == B.SQN_ERR_WORKSPACE
    assert B.sqn_launch_count() == n0


def test_calls_leave_the_free_device_memory_unchanged():
    """The point of the entry point: after a first call on the device (which looks up the built-in buffer's address)
    further calls, in either dtype, take no device memory."""
    import torch
    cases = []
    for dtype in (B.SQN_F32, B.SQN_BF16):
        x, sq, e1, e3 = synth.fire_case(5, 2, 64, 16, 64, 64, 13)
        dev = [G.dev_act(x, dtype), G.dev_w(sq[0], dtype), G.dev_b(sq[1]), G.dev_w(e1[0], dtype), G.dev_b(e1[1]),
               G.dev_w(e3[0], dtype), G.dev_b(e3[1])]
        cases.append((dev, B.empty_device((2, 13, 13, 128), dtype), dtype))
    for dev, out, dtype in cases:                          # first calls: address look-up, kernel images loaded
        B.fire_forward_static(*dev, out, 64, 16, 64, 64, 13, 13, 2, dtype)
    assert B.sqn_check() == B.SQN_OK
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        for dev, out, dtype in cases:
            B.fire_forward_static(*dev, out, 64, 16, 64, 64, 13, 13, 2, dtype)
    assert B.sqn_check() == B.SQN_OK
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
