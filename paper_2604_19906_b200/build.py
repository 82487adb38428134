"""Builds the CUDA libraries of this package in-tree with nvcc for sm_100a.

``lib/libekl_tpo.so``    the product: C-ABI operators (``include/ekl_tpo.h``)
``lib/libekl_inputs.so`` device twin of the seeded input stream (``inputs.py``)
``lib/libekl_probe.so``  measurement helpers (``include/ekl_probe.h``), not on the product path

Objects go to ``_build/`` (not tracked).  Only sources newer than their object are
recompiled; any header change recompiles everything.
"""
from __future__ import annotations

import concurrent.futures as cf
import glob
import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIBDIR = os.path.join(PKG, "lib")
OBJDIR = os.path.join(ROOT, "_build")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include")]

LIBS = {
    "libekl_inputs.so": ["inputs_fill.cu"],
    "libekl_probe.so": ["peak_probe.cu"],
    # every other .cu under csrc/ belongs to the product library
}


def _nvcc() -> str:
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        raise RuntimeError("nvcc not found")
    return nvcc


def _newest_header() -> float:
    hs = glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(ROOT, "include", "*.h"))
    return max(os.path.getmtime(h) for h in hs) if hs else 0.0


def _compile(src: str, verbose: bool) -> str:
    obj = os.path.join(OBJDIR, os.path.basename(src)[:-3] + ".o")
    stamp = max(os.path.getmtime(src), _newest_header(), os.path.getmtime(__file__))
    if os.path.exists(obj) and os.path.getmtime(obj) >= stamp:
        return obj
    cmd = [_nvcc(), *NVCC_FLAGS, "-c", src, "-o", obj]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode:
        raise RuntimeError(f"nvcc failed on {src}")
    return obj


def build(verbose: bool = False) -> dict:
    """Compile everything that is stale; returns {library name: path}."""
    os.makedirs(LIBDIR, exist_ok=True)
    os.makedirs(OBJDIR, exist_ok=True)
    all_src = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    aux = {s for v in LIBS.values() for s in v}
    groups = dict(LIBS)
    groups["libekl_tpo.so"] = [os.path.basename(s) for s in all_src
                               if os.path.basename(s) not in aux]
    with cf.ThreadPoolExecutor(max_workers=os.cpu_count() or 4) as pool:
        objs = dict(zip(all_src, pool.map(lambda s: _compile(s, verbose), all_src)))
    out = {}
    for lib, names in groups.items():
        path = os.path.join(LIBDIR, lib)
        deps = [objs[os.path.join(CSRC, n)] for n in names]
        if not os.path.exists(path) or any(os.path.getmtime(o) > os.path.getmtime(path) for o in deps):
            tmp = path + f".tmp{os.getpid()}"
            subprocess.run([_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a",
                            "-o", tmp, *deps], check=True)
            os.replace(tmp, path)
        out[lib] = path
    return out


if __name__ == "__main__":
    for k, v in build(verbose="-v" in sys.argv).items():
        print(k, "->", v)
