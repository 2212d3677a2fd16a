"""Builds libsquat.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

`build(checked=True)` (or `python -m paper_2503_24358_b200.build --checked`) builds libsquat_checked.so from the same
sources with -DSQUAT_CHECKED: the key and value kernels then test every address they form against the extent of the
buffer or on-chip region it belongs to and report through SQUAT_FLAG_BOUNDS instead of accessing.  Select it with the
environment variable SQUAT_LIBRARY=<path> before the package is first used."""
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(_HERE), "include")
OBJ_DIR = os.path.join(_HERE, "build")
LIB = os.path.join(_HERE, "libsquat.so")
OBJ_DIR_CHECKED = os.path.join(_HERE, "build_checked")
LIB_CHECKED = os.path.join(_HERE, "libsquat_checked.so")
SOURCES = ["api.cu", "values.cu", "keys.cu", "subspace.cu", "power.cu", "attention.cu", "peak.cu", "keys_lowrank.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", INCLUDE]


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def _deps_mtime():
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "squat.h")]
    return max(os.path.getmtime(p) for p in paths)


def _compile(src, verbose, obj_dir=OBJ_DIR, extra=()):
    obj = os.path.join(obj_dir, src.replace(".cu", ".o"))
    hdr_time = max(os.path.getmtime(os.path.join(CSRC, "squat_internal.cuh")),
                   os.path.getmtime(os.path.join(INCLUDE, "squat.h")))
    src_path = os.path.join(CSRC, src)
    if os.path.exists(obj) and os.path.getmtime(obj) >= max(os.path.getmtime(src_path), hdr_time):
        return obj
    cmd = [_nvcc()] + NVCC_FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + ["-c", src_path, "-o", obj]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode != 0:
        print(r.stdout + r.stderr)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed on {src}")
    return obj


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    obj_dir, lib = (OBJ_DIR_CHECKED, LIB_CHECKED) if checked else (OBJ_DIR, LIB)
    extra = ("-DSQUAT_CHECKED",) if checked else ()
    os.makedirs(obj_dir, exist_ok=True)
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= _deps_mtime():
        return lib
    if force:
        for f in os.listdir(obj_dir):
            if f.endswith(".o"):
                os.remove(os.path.join(obj_dir, f))
    with ThreadPoolExecutor(max_workers=len(SOURCES)) as ex:
        objs = list(ex.map(lambda s: _compile(s, verbose, obj_dir, extra), SOURCES))
    cmd = [_nvcc(), "-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib] + objs
    subprocess.run(cmd, check=True)
    return lib


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
