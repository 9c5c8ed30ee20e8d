"""Builds libhbf.so (the CUDA library behind the C ABI) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
SO = os.path.join(HERE, "libhbf.so")
SOURCES = ["hbf_api.cu", "submit_kernels.cu", "inorder_kernels.cu", "paged_kernels.cu", "energy_bins.cu", "rom_kernels.cu", "retention_kernels.cu", "thermal_kernels.cu", "noalloc_thermal.cu"]
HEADERS = ["hbf_dev.cuh", "device_utils.cuh", os.path.join("..", "..", "include", "hbf.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]
# One translation unit launches kernels from the device (the sort path's fall-back chain): it alone is compiled as
# relocatable device code and device-linked with the device runtime; the others keep whole-program compilation
# (measured: relocatable code costs the in-order serve kernel about 1.3 %).
RDC_SOURCES = {"submit_kernels.cu"}
OBJ_DIR = os.path.join(HERE, "build")


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def is_stale() -> bool:
    if not os.path.exists(SO):
        return True
    t = os.path.getmtime(SO)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, extra_flags=(), out: str | None = None) -> str:
    """Compiles the library.  extra_flags (e.g. -D switches of an experiment) and out (another file name for the result)
    serve measurement builds; the package itself loads the default file."""
    so = out or SO
    if not force and not extra_flags and out is None and not is_stale():
        return SO
    from concurrent.futures import ThreadPoolExecutor
    os.makedirs(OBJ_DIR, exist_ok=True)
    nvcc = _nvcc()
    extra = (["-Xptxas", "-v"] if verbose else []) + list(extra_flags)
    tag = ".tmp%d" % os.getpid()

    def compile_one(src):
        obj = os.path.join(OBJ_DIR, src.replace(".cu", tag + ".o"))
        mode = ["-dc"] if src in RDC_SOURCES else ["-c"]
        subprocess.check_call([nvcc] + NVCC_FLAGS + extra + mode + [os.path.join(CSRC, src), "-o", obj])
        return obj

    with ThreadPoolExecutor(max(1, min(len(SOURCES), os.cpu_count() or 1))) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    try:
        rdc_objs = [o for o, src in zip(objs, SOURCES) if src in RDC_SOURCES]
        dlink = os.path.join(OBJ_DIR, "device_link" + tag + ".o")
        subprocess.check_call([nvcc] + NVCC_FLAGS + ["-dlink"] + rdc_objs + ["-lcudadevrt", "-o", dlink])
        tmp = so + tag
        subprocess.check_call([nvcc] + NVCC_FLAGS + ["--shared", "-cudart", "shared"] + objs + [dlink, "-lcudadevrt", "-o", tmp])
        os.replace(tmp, so)
    finally:
        for o in objs + [os.path.join(OBJ_DIR, "device_link" + tag + ".o")]:
            if os.path.exists(o):
                os.remove(o)
    return so


if __name__ == "__main__":
    flags = [a for a in sys.argv[1:] if a.startswith("-D")]
    outs = [a[len("--out="):] for a in sys.argv[1:] if a.startswith("--out=")]
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, extra_flags=flags, out=outs[0] if outs else None))
