"""Runs the measurement helpers of ``lib/libekl_probe.so`` (``include/ekl_probe.h``) and
reports their rates in TFLOP/s.  Not on the product path.

    python -m paper_2604_19906_b200.probes [--only NAME] [--repeats R]

prints one JSON object.  ``bench.py`` calls :func:`run_probes` after its timed region so that
the FP64 figures the roofline fractions refer to are measured in the same run.
"""
from __future__ import annotations

import ctypes
import json
import os
import sys

_LIBPATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib", "libekl_probe.so")
_lib = None

SM_COUNT = 148


def library() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(_LIBPATH):
            raise RuntimeError(f"{_LIBPATH} is missing: run `python -m paper_2604_19906_b200.build`")
        lib = ctypes.CDLL(_LIBPATH)
        vp, i = ctypes.c_void_p, ctypes.c_int
        dp = ctypes.POINTER(ctypes.c_double)
        lib.ekl_probe_fp64_fma_chain.argtypes = [vp, i, i, dp, vp]
        lib.ekl_probe_fp64_fma_contraction.argtypes = [vp, i, i, dp, vp]
        lib.ekl_probe_fp64_dmma.argtypes = [vp, i, i, i, dp, vp]
        lib.ekl_probe_fp64_dmma_plus_fma.argtypes = [vp, i, i, dp, vp]
        lib.ekl_probe_stage_loop_n14.argtypes = [vp, i, i, dp, dp, vp]
        lib.ekl_probe_stage_loop_n14_fma.argtypes = [vp, i, i, dp, vp]
        _lib = lib
    return _lib


def _time(torch, stream, launch, repeats):
    """Best CUDA-event time in seconds of `launch()` over `repeats` runs after one warm-up."""
    best = None
    for it in range(repeats + 1):
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record(stream)
        rc = launch()
        e.record(stream)
        stream.synchronize()
        if rc:
            raise RuntimeError(f"probe launch failed with code {rc}")
        if it:
            ms = s.elapsed_time(e)
            best = ms if best is None else min(best, ms)
    return best * 1e-3


def run_probes(device=None, stream=None, only: str | None = None, repeats: int = 3) -> dict:
    """{name: TFLOP/s}.  Names: fma_chain, fma_contraction, dmma_1chain, dmma_2chains,
    dmma_4chains, dmma_plus_fma, stage_loop_n14_dmma (useful rate; ``..._padded`` the rate the
    tensor pipe executes), stage_loop_n14_fma."""
    import torch
    lib = library()
    dev = torch.device(device if device is not None else "cuda:0")
    stream = stream or torch.cuda.current_stream(dev)
    sp = ctypes.c_void_p(stream.cuda_stream)
    blocks = SM_COUNT * 8
    sink = torch.empty(blocks * 256, dtype=torch.float64, device=dev)
    ptr = ctypes.c_void_p(sink.data_ptr())
    f, g = ctypes.c_double(0.0), ctypes.c_double(0.0)
    out = {}

    def want(name):
        return only is None or only == name

    with torch.cuda.device(dev), torch.cuda.stream(stream):
        if want("fma_chain"):
            t = _time(torch, stream, lambda: lib.ekl_probe_fp64_fma_chain(
                ptr, blocks, 20000, ctypes.byref(f), sp), repeats)
            out["fma_chain"] = f.value / t / 1e12
        if want("fma_contraction"):
            t = _time(torch, stream, lambda: lib.ekl_probe_fp64_fma_contraction(
                ptr, blocks, 12000, ctypes.byref(f), sp), repeats)
            out["fma_contraction"] = f.value / t / 1e12
        for chains in (1, 2, 4):
            name = f"dmma_{chains}chain" + ("s" if chains > 1 else "")
            if want(name):
                t = _time(torch, stream, lambda c=chains: lib.ekl_probe_fp64_dmma(
                    ptr, SM_COUNT * 2, 20000, c, ctypes.byref(f), sp), repeats)
                out[name] = f.value / t / 1e12
        if want("dmma_plus_fma"):
            t = _time(torch, stream, lambda: lib.ekl_probe_fp64_dmma_plus_fma(
                ptr, SM_COUNT * 2, 20000, ctypes.byref(f), sp), repeats)
            out["dmma_plus_fma"] = f.value / t / 1e12
        if want("stage_loop_n14_dmma"):
            t = _time(torch, stream, lambda: lib.ekl_probe_stage_loop_n14(
                ptr, SM_COUNT * 2, 1200, ctypes.byref(f), ctypes.byref(g), sp), repeats)
            out["stage_loop_n14_dmma"] = f.value / t / 1e12
            out["stage_loop_n14_dmma_padded"] = g.value / t / 1e12
        if want("stage_loop_n14_fma"):
            t = _time(torch, stream, lambda: lib.ekl_probe_stage_loop_n14_fma(
                ptr, SM_COUNT * 2, 1200, ctypes.byref(f), sp), repeats)
            out["stage_loop_n14_fma"] = f.value / t / 1e12
    return out


def main(argv=None):
    import argparse
    ap = argparse.ArgumentParser()
    ap.add_argument("--only", default=None)
    ap.add_argument("--repeats", type=int, default=3)
    args = ap.parse_args(argv)
    from . import build
    build.build()
    print(json.dumps({k: round(v, 3) for k, v in run_probes(only=args.only,
                                                            repeats=args.repeats).items()}))


if __name__ == "__main__":
    sys.exit(main())
