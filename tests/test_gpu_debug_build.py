"""The bounds-checked build of the library (the same sources compiled with -DSQN_DEBUG): index checks in the kernels'
staging, patch and store addressing record SQN_ERR_DEBUG in the status word and skip the access.  The small-shape
parity tests run against that build in a child process (the library is chosen when the binding loads it), and must
pass with the status word clean -- every one of those tests reads it with sqn_check."""
import os
import subprocess
import sys

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)

SMALL_SHAPE_TESTS = [
    "tests/test_gpu_fire_fused.py",
    "tests/test_gpu_f16.py",
    "tests/test_gpu_second_workload.py",
    "tests/test_gpu_bf16.py::test_conv_shapes",
    "tests/test_gpu_bf16.py::test_stem_7x7_stride2",
    "tests/test_gpu_bf16.py::test_conv_with_fused_maxpool",
    "tests/test_gpu_bf16.py::test_conv_with_fused_global_average",
    "tests/test_gpu_bf16.py::test_full_forward_bf16_small_batch_keeps_every_map",
    "tests/test_gpu_f32.py::test_awkward_shapes",
    "tests/test_gpu_f32.py::test_config2_full_forward_batch1",
]


@pytest.mark.gpu
def test_small_shapes_under_debug_build():
    from paper_1611_07151_b200 import build as lib_build
    lib = lib_build.build(debug=True)
    assert os.path.exists(lib)
    env = dict(os.environ, SQN_LIBRARY=lib)
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider"] + SMALL_SHAPE_TESTS,
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = (r.stdout or "")[-3000:] + (r.stderr or "")[-1000:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "failed" not in r.stdout, tail


def test_debug_library_exports_the_same_symbols():
    """Host-only: the debug flavour builds and exports every entry point the header declares."""
    import ctypes
    from paper_1611_07151_b200 import binding as B, build as lib_build
    lib = ctypes.CDLL(lib_build.build(debug=True))
    for name in B.SIGNATURES:
        assert hasattr(lib, name), name
