"""Builds the CUDA library in-tree: csrc/*.cu -> libppo_b200.so (sm_100a only)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
INCLUDE = os.path.join(_ROOT, "include")
LIB_PATH = os.path.join(_HERE, "libppo_b200.so")

ARCH_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a"]
NVCC_FLAGS = ARCH_FLAGS + ["-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    env = os.environ.get("NVCC")
    if env:
        return env
    return "/usr/local/cuda/bin/nvcc" if os.path.exists("/usr/local/cuda/bin/nvcc") else "nvcc"


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every kernel for sm_100a into one shared library (cross-compiles without a GPU)."""
    if not force and not needs_build():
        return LIB_PATH
    obj_dir = os.path.join(_HERE, "_build")
    os.makedirs(obj_dir, exist_ok=True)
    procs, objs = [], []
    for src in sources():
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        extra = os.environ.get("PPO_NVCC_EXTRA", "").split()      # e.g. -DNAME for a tuning experiment
        cmd = [_nvcc(), *NVCC_FLAGS, *extra, *(["-Xptxas", "-v"] if verbose else []), "-I", INCLUDE, "-I", CSRC,
               "-c", src, "-o", obj]
        procs.append(subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
        objs.append(obj)
    failed = False
    for p in procs:
        out, _ = p.communicate()
        if out.strip():
            sys.stderr.write(out)
        failed = failed or p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    subprocess.check_call([_nvcc(), "-shared", "-o", LIB_PATH, *objs, "-cudart", "static", *ARCH_FLAGS,
                           "-Xcompiler", "-fPIC"])
    return LIB_PATH


def build_variant(out_path: str, defines, only=None) -> str:
    """A second copy of the library compiled with extra -D macros (tests of the bounded waits use one in which the
    hand-over flags are withheld). `only`: basenames of the sources to compile; objects go next to `out_path`."""
    obj_dir = out_path + ".obj"
    os.makedirs(obj_dir, exist_ok=True)
    srcs = [s for s in sources() if only is None or os.path.basename(s) in only]
    procs, objs = [], []
    for src in srcs:
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        cmd = [_nvcc(), *NVCC_FLAGS, *["-D" + d for d in defines], "-I", INCLUDE, "-I", CSRC, "-c", src, "-o", obj]
        procs.append(subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
        objs.append(obj)
    for p in procs:
        out, _ = p.communicate()
        if p.returncode != 0:
            sys.stderr.write(out)
            raise RuntimeError("nvcc failed")
    subprocess.check_call([_nvcc(), "-shared", "-o", out_path, *objs, "-cudart", "static", *ARCH_FLAGS,
                           "-Xcompiler", "-fPIC"])
    return out_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
