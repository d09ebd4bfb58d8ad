"""Build liblordba.so (sm_100a only) in-tree with nvcc.

``python -m paper_2605_24058_b200.build`` or ``build_library()``.  Objects go
to ``paper_2605_24058_b200/_build``; the shared object sits next to this file so
that it travels with a snapshot of the tree.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
BUILD = os.path.join(PKG, "_build")
LIB = os.path.join(PKG, "liblordba.so")
TESTHOOKS_LIB = os.path.join(PKG, "liblordba_testhooks.so")
SOURCES = ("api.cu", "pack.cu", "fit.cu", "forward_fma.cu", "forward_tc.cu", "forward_mma.cu")
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Wno-deprecated-gpu-targets",
              "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; liblordba.so cannot be built")


def _newest_header() -> float:
    paths = [os.path.join(ROOT, "include", "lordba.h")]
    paths += [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    return max(os.path.getmtime(p) for p in paths)


def build_library(force: bool = False, verbose: bool = False, test_hooks: bool = False) -> str:
    """Build the library.  test_hooks=True builds a second library, liblordba_testhooks.so, from
    the same sources with -DLORDBA_TEST_HOOKS (bounded device-side waits give up after about a
    millisecond, and lordba_test_skip_item makes one copy request go missing): only the test of
    the timeout path loads it; the product library never has the hooks."""
    build_dir = BUILD + ("_testhooks" if test_hooks else "")
    lib_path = TESTHOOKS_LIB if test_hooks else LIB
    extra = ["-DLORDBA_TEST_HOOKS"] if test_hooks else []
    os.makedirs(build_dir, exist_ok=True)
    nvcc = _nvcc()
    hdr = _newest_header()
    jobs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(build_dir, src + ".o")
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), hdr):
            cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            jobs.append(cmd)

    def run(cmd):
        p = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or p.returncode != 0:
            sys.stderr.write(p.stdout + p.stderr)
        if p.returncode != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))

    with ThreadPoolExecutor(max_workers=4) as ex:
        list(ex.map(run, jobs))
    objs = [os.path.join(build_dir, s + ".o") for s in SOURCES]
    if jobs or not os.path.exists(lib_path):
        tmp = lib_path + ".tmp.%d" % os.getpid()
        run([nvcc, "-shared", "-o", tmp] + objs + ["-Xlinker", "--exclude-libs=ALL"])
        os.replace(tmp, lib_path)
    return lib_path


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv,
                        test_hooks="--test-hooks" in sys.argv))
