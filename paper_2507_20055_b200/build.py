"""Builds the CUDA library in-tree with nvcc for sm_100a (no GPU needed).

Every .cu file is compiled to an object of its own (in parallel, and only when it or a header changed)
and the objects are linked into libcert_b200.so next to this file."""
from __future__ import annotations

import glob
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libcert_b200.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def headers():
    return glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(HERE, "..", "include", "*.h"))


def _obj(src: str, tag: str) -> str:
    return os.path.join(OBJ, tag + os.path.basename(src)[:-3] + ".o")


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in sources() + headers())


CHECKED_LIB = os.path.join(HERE, "libcert_b200_checked.so")


def build_checked(force: bool = False) -> str:
    """The checking build (-DCERT_BOUNDS: every plain global store of the non-TMA kernels is looked up in a table
    of the call's writable buffers first), as a library of its own beside the ordinary one."""
    return build(force=force, defines=("CERT_BOUNDS",), lib=CHECKED_LIB)


def build(force: bool = False, verbose: bool = False, defines=(), lib: str = LIB) -> str:
    """defines: extra -D macros (a checking build goes to a library of its own, see `lib`)."""
    if not force and os.path.exists(lib):
        t = os.path.getmtime(lib)
        if not any(os.path.getmtime(d) > t for d in sources() + headers()):
            return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)
    tag = "".join(sorted(d.replace("=", "_") + "." for d in defines))
    hdr_time = max(os.path.getmtime(h) for h in headers())
    flags = NVCC_FLAGS + ["-D" + d for d in defines] + (["-Xptxas", "-v"] if verbose else [])

    def compile_one(src):
        obj = _obj(src, tag)
        if (not force and os.path.exists(obj)
                and os.path.getmtime(obj) > max(os.path.getmtime(src), hdr_time)):
            return
        subprocess.check_call([nvcc] + flags + ["-c", "-o", obj, src])

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        list(pool.map(compile_one, sources()))
    subprocess.check_call([nvcc] + NVCC_FLAGS + ["-shared", "-o", lib] + [_obj(s, tag) for s in sources()])
    return lib


if __name__ == "__main__":
    import sys
    if "--checked" in sys.argv:
        print(build_checked(force="--force" in sys.argv))
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
