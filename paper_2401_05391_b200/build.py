"""Build the segkv C-ABI shared library in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libsegkv.so")
# the same library with per-CTA time stamps compiled in (read by paper_2401_05391_b200/timeline.py);
# never loaded by the binding, the tests or the benchmark
LIB_TIMELINE = os.path.join(PKG, "libsegkv_timeline.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")

FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--use_fast_math",
    "-I", os.path.join(ROOT, "include"), "-I", CSRC,
] + os.environ.get("SEGKV_NVCC_FLAGS", "").split()


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False, timeline: bool = False) -> str:
    """Compile every .cu under csrc/ into libsegkv.so (no-op when up to date).  `timeline` builds
    the instrumented copy libsegkv_timeline.so instead."""
    lib = LIB_TIMELINE if timeline else LIB
    if not (force or _stale(lib)):
        return lib
    objs = []
    procs = []
    for src in sources():
        obj = os.path.splitext(src)[0] + (".tl.o" if timeline else ".o")
        cmd = [NVCC, *FLAGS, *(["-DSEGKV_TIMELINE", "-DSEGKV_TC5_TIMELINE=1"] if timeline else []), "-c", src, "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode:
            sys.stderr.write(f"--- {os.path.basename(src)}\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = lib + f".{os.getpid()}.tmp"
    subprocess.check_call([NVCC, "-shared", "-gencode", "arch=compute_100a,code=sm_100a",
                           "-cudart", "static", "-o", tmp, *objs])
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, timeline="--timeline" in sys.argv))
