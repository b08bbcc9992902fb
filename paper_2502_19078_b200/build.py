"""Build ``libclada.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(_HERE), "include")
LIB = os.path.join(_HERE, "libclada.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "-Xcompiler", "-fPIC"]
OBJ_DIR = os.path.join(_HERE, "_build")

# Opt-in builds of the same sources, each into its own library beside the release one (select it at run time with
# the CLADA_LIB environment variable):
#   bounds  every neuron index is range-checked on its way into a row address or a list slot; a bad one is
#           recorded as CLADA_STATUS_BAD_INDEX in the call's status word and made harmless, nothing traps
#   nvtx    NVTX ranges around the C entry points
VARIANTS = {"bounds": ["-DCLADA_DEBUG_BOUNDS"], "nvtx": ["-DCLADA_NVTX"]}


def lib_path(variant: str | None = None) -> str:
    return LIB if not variant else os.path.join(_HERE, f"libclada_{variant}.so")


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    return "nvcc"


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def needs_build(variant: str | None = None) -> bool:
    lib = lib_path(variant)
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def _headers():
    return glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))


def build(force: bool = False, verbose: bool = False, variant: str | None = None) -> str:
    """Compile every csrc/*.cu to an object (in parallel, only those older than their source or any header)
    and link them into libclada.so (libclada_<variant>.so for one of VARIANTS).  The kernels of different files
    share no device code, so no relocatable device code is needed."""
    lib = lib_path(variant)
    if not force and not needs_build(variant):
        return lib
    from concurrent.futures import ThreadPoolExecutor
    obj_dir = OBJ_DIR if not variant else os.path.join(OBJ_DIR, variant)
    os.makedirs(obj_dir, exist_ok=True)
    newest_header = max(os.path.getmtime(h) for h in _headers())
    # CLADA_NVCC_FLAGS: extra compiler flags for an opt-in build, e.g. -DCLADA_NVTX (NVTX ranges around the C
    # entry points) or -DCLADA_STACK_TRACE / -DCLADA_BD_TRACE (in-kernel time stamps); rebuild with --force
    base = [_nvcc()] + NVCC_FLAGS + os.environ.get("CLADA_NVCC_FLAGS", "").split() + \
        (VARIANTS[variant] if variant else []) + ["-I", INCLUDE, "-I", CSRC]
    if verbose:
        base += ["-Xptxas", "-v"]
    jobs, objs = [], []
    for src in sources():
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), newest_header):
            jobs.append(base + ["-c", src, "-o", obj])
    with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4) or 1) as pool:
        for done in pool.map(lambda c: subprocess.run(c, check=False), jobs):
            if done.returncode != 0:
                raise subprocess.CalledProcessError(done.returncode, done.args)
    subprocess.run([_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a"] + objs + ["-o", lib], check=True)
    return lib


if __name__ == "__main__":
    _variant = sys.argv[sys.argv.index("--variant") + 1] if "--variant" in sys.argv else None
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, variant=_variant))
