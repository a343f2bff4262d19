"""Build the C-ABI library (libsqn.so) in-tree with nvcc for sm_100a.

Usage: python -m paper_1611_07151_b200.build [--force] [--verbose]
"""
import glob
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libsqn.so")
LIB_DEBUG = os.path.join(PKG, "libsqn_debug.so")      # the same sources with -DSQN_DEBUG: index checks in the kernels
OBJ_DIR = os.path.join(PKG, "_build")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return _sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(ROOT, "include", "*.h"))


def up_to_date(lib=LIB):
    if not os.path.exists(lib):
        return False
    t = os.path.getmtime(lib)
    return all(os.path.getmtime(f) <= t for f in _deps())


def build(force=False, verbose=False, debug=False):
    """Compile every .cu under csrc/ and link them into libsqn.so (debug=True: libsqn_debug.so, with -DSQN_DEBUG)."""
    lib = LIB_DEBUG if debug else LIB
    if not force and up_to_date(lib):
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    obj_dir = OBJ_DIR + ("_debug" if debug else "")
    os.makedirs(obj_dir, exist_ok=True)
    extra = (["-Xptxas", "-v"] if verbose else []) + (["-DSQN_DEBUG"] if debug else [])
    hdr_t = max(os.path.getmtime(f) for f in _deps() if not f.endswith(".cu"))
    objs, procs = [], []
    for src in _sources():
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if (not force and os.path.exists(obj)
                and os.path.getmtime(obj) >= max(os.path.getmtime(src), hdr_t)):
            continue
        procs.append((src, subprocess.Popen([nvcc] + NVCC_FLAGS + extra + ["-c", src, "-o", obj])))
    for src, p in procs:
        if p.wait() != 0:
            raise RuntimeError("nvcc failed on " + src)
    tmp = lib + ".tmp.%d" % os.getpid()
    subprocess.run([nvcc, "-shared", "-o", tmp] + objs + ["-lcudart"], check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
