"""Builds ``liblaq.so`` in-tree with nvcc for sm_100a (one object per .cu, then a shared link).

Run ``python -m paper_2505_20334_b200.build`` or call :func:`build_liblaq`. The CUDA runtime is
linked statically and the driver API is resolved at run time, so the library loads (but cannot
launch) on a machine without a GPU.
"""
from __future__ import annotations

import concurrent.futures
import glob
import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "liblaq.so")
OBJ_DIR = os.path.join(PKG_DIR, "_build")

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
    "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps_mtime():
    files = _sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(ROOT, "include", "laq.h")]
    return max(os.path.getmtime(f) for f in files)


def build_liblaq(force: bool = False, verbose: bool = False, defines=(), variant: str = "") -> str:
    """Compiles liblaq.so if it is missing or older than its sources. `defines` are extra
    ``-DNAME=VALUE`` strings for tuning builds (they force a rebuild). A non-empty `variant` builds
    ``_build/<variant>/liblaq_<variant>.so`` from the same sources with those defines and leaves
    liblaq.so alone (the tests use it for a copy of the library with test hooks compiled in)."""
    lib_path, obj_dir = LIB_PATH, OBJ_DIR
    if variant:
        obj_dir = os.path.join(OBJ_DIR, variant)
        lib_path = os.path.join(obj_dir, f"liblaq_{variant}.so")
    else:
        force = force or bool(defines)
    if not force and os.path.exists(lib_path) and os.path.getmtime(lib_path) >= _deps_mtime():
        return lib_path
    os.makedirs(obj_dir, exist_ok=True)
    nvcc = os.environ.get("NVCC", "nvcc")
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(src):
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        cmd = [nvcc, *NVCC_FLAGS, *extra, *defines, "-c", src, "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        return obj, r

    objs = []
    with concurrent.futures.ThreadPoolExecutor(max_workers=8) as ex:
        for obj, r in ex.map(compile_one, _sources()):
            if verbose or r.returncode != 0:
                sys.stderr.write(r.stdout + r.stderr)
            if r.returncode != 0:
                raise RuntimeError(f"nvcc failed for {obj}")
            objs.append(obj)
    link = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib_path, *objs]
    r = subprocess.run(link, capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("link of liblaq.so failed")
    return lib_path


if __name__ == "__main__":
    print(build_liblaq(force="--force" in sys.argv, verbose="-v" in sys.argv,
                       defines=[a for a in sys.argv[1:] if a.startswith("-D")]))
