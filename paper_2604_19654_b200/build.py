"""Builds libfeplb.so (C ABI + sm_100a kernels) in-tree with nvcc.

``python -m paper_2604_19654_b200.build [--force] [-v] [--nvcc-flag=FLAG ...]`` or ``build()``;
nvcc cross-compiles without a GPU.  ``-v`` prints ptxas resource usage; ``--nvcc-flag`` appends one
extra compiler flag per occurrence (kernel experiments only; the product build takes none and
reads no environment variable besides NVCC, the compiler's path).
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libfeplb.so")
SOURCES = ["feplb_plan.cpp", "feplb_api.cu", "feplb_route.cu", "feplb_combine.cu", "feplb_gemm.cu",
           "feplb_noalloc.cu", "feplb_gemm_bwd.cu", "feplb_gemm_wm.cu"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: libfeplb cannot be built (there is no CPU fallback)")


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "feplb.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False, extra_flags=()) -> str:
    if not force and not needs_build():
        return LIB
    # Several processes may get here at once (one per GPU under torchrun): one builds, to a
    # temporary name that is renamed into place, the others wait on the lock and find it done.
    import fcntl
    with open(LIB + ".lock", "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        try:
            if not force and not needs_build():
                return LIB
            tmp = f"{LIB}.{os.getpid()}.tmp"
            cmd = [_nvcc(), "-shared", "-O3", "-std=c++17", "-lineinfo",
                   "-gencode", "arch=compute_100a,code=sm_100a",
                   "-Xcompiler", "-fPIC,-pthread",
                   "-I", os.path.join(ROOT, "include"), "-I", CSRC,
                   "-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
            cmd[1:1] = list(extra_flags)
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            r = subprocess.run(cmd, capture_output=True, text=True)
            if verbose or r.returncode:
                sys.stderr.write(r.stdout + r.stderr)
            if r.returncode:
                if os.path.exists(tmp):
                    os.remove(tmp)
                raise RuntimeError("nvcc failed building libfeplb.so")
            os.replace(tmp, LIB)
            return LIB
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv,
                extra_flags=[a.split("=", 1)[1] for a in sys.argv if a.startswith("--nvcc-flag=")]))
