"""The C-ABI library loads, exports what include/*.h declares, and rejects bad
arguments on the host before anything touches a device (no GPU needed: every call
below returns from validation)."""
import ctypes
import glob
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2604_19906_b200 import build, ops
    build.build()
    return ops.library()


def declared_symbols():
    names = set()
    for h in glob.glob(os.path.join(ROOT, "include", "*.h")):
        text = re.sub(r"/\*.*?\*/", "", open(h).read(), flags=re.S)
        names |= set(re.findall(r"\b(ekl_tpo_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"ekl_tpo_inv_helmholtz", "ekl_tpo_apply", "ekl_tpo_inv_helmholtz_f32",
            "ekl_tpo_apply_f32", "ekl_tpo_status_string", "ekl_tpo_version",
            "ekl_tpo_last_cuda_error"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"


def test_version_and_status_strings(lib):
    assert lib.ekl_tpo_version() >= 100
    seen = {lib.ekl_tpo_status_string(s) for s in range(7)}
    assert len(seen) == 7 and all(seen)
    assert lib.ekl_tpo_status_string(99)


P = 0x7F0000001000          # a made-up, suitably aligned "device" address: never dereferenced


@pytest.mark.parametrize("fn,w", [("ekl_tpo_inv_helmholtz", 8), ("ekl_tpo_inv_helmholtz_f32", 4)])
def test_inv_helmholtz_validation(lib, fn, w):
    f = getattr(lib, fn)
    OK, NULL, SHAPE, UNSUP, ALIGN, OVERLAP = 0, 1, 2, 3, 4, 5
    n, E = 4, 10
    field = E * n ** 3 * w
    S, D, u, v = P, P + 0x1000, P + 0x1000 + field, P + 0x1000 + 2 * field
    assert f(S, D, u, v, 0, E, None) == SHAPE
    assert f(S, D, u, v, -3, E, None) == SHAPE
    assert f(S, D, u, v, n, -1, None) == SHAPE
    assert f(None, None, None, None, n, 0, None) == OK          # E == 0 is a no-op
    assert f(None, D, u, v, n, E, None) == NULL
    assert f(S, D, u, None, n, E, None) == NULL
    assert f(S, D, u, v, 1000, E, None) == UNSUP
    assert f(S, D, u, v, 25 if w == 8 else 31, E, None) == UNSUP
    assert f(S, D, u + w // 2, v, n, E, None) == ALIGN
    assert f(S, D, u, v + 1, n, E, None) == ALIGN
    assert f(S, D, u, D, n, E, None) == OVERLAP                  # v aliases D
    assert f(S, D, u, u + w, n, E, None) == OVERLAP              # v partially overlaps u
    assert f(S, D, u, S, n, E, None) == OVERLAP
    assert f(S, D, u, D + field - w, n, E, None) == OVERLAP      # tail of D


@pytest.mark.parametrize("fn,w", [("ekl_tpo_apply", 8), ("ekl_tpo_apply_f32", 4)])
def test_apply_validation(lib, fn, w):
    f = getattr(lib, fn)
    OK, NULL, SHAPE, UNSUP, ALIGN, OVERLAP = 0, 1, 2, 3, 4, 5
    E = 6
    A, B, C = P, P + 0x400, P + 0x800
    u = P + 0x1000
    v = u + E * 8 ** 3 * w
    dims = (8, 8, 8, 12, 12, 12)
    assert f(A, B, C, u, v, 8, 8, 0, 12, 12, 12, E, None) == SHAPE
    assert f(A, B, C, u, v, 8, 8, 8, 12, -1, 12, E, None) == SHAPE
    assert f(A, B, C, u, v, *dims, -2, None) == SHAPE
    assert f(None, None, None, None, None, *dims, 0, None) == OK
    assert f(A, None, C, u, v, *dims, E, None) == NULL
    assert f(A, B, C, u, v, 64, 64, 64, 64, 64, 64, E, None) == UNSUP
    assert f(A, B, C, u, v, 40000, 40000, 40000, 40000, 40000, 40000, E, None) == UNSUP
    assert f(A, B, C + 2, u, v, *dims, E, None) == ALIGN
    assert f(A, B, C, u, u, *dims, E, None) == OVERLAP           # no in-place for apply
    assert f(A, B, C, u, v - w, *dims, E, None) == OVERLAP
    assert f(A, B, C, u, A, *dims, E, None) == OVERLAP


def test_convection_and_host_variants_validation(lib):
    OK, NULL, SHAPE, UNSUP, ALIGN, OVERLAP = 0, 1, 2, 3, 4, 5
    vp, i, ll, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong, ctypes.c_size_t
    f = lib.ekl_tpo_convection
    f.argtypes = [vp] * 5 + [i, i, ll, vp]
    f.restype = i
    nq, nv, E = 12, 8, 4
    D, I = P, P + 0x1000
    M = P + 0x2000
    Pf = M + E * nq ** 3 * 8
    F = Pf + 0x40000000
    assert f(D, I, M, Pf, F, nq, nv, 0, None) == OK
    assert f(D, I, M, Pf, F, 0, nv, E, None) == SHAPE
    assert f(D, I, M, Pf, F, nq, nv, -1, None) == SHAPE
    assert f(D, None, M, Pf, F, nq, nv, E, None) == NULL
    assert f(D, I, M, Pf, F, 100, 8, E, None) == UNSUP           # beyond 64
    assert f(D, I, M, Pf, F, 40, 40, E, None) == UNSUP           # does not fit in shared memory
    assert f(D, I, M + 4, Pf, F, nq, nv, E, None) == ALIGN
    assert f(D, I, M, Pf, F + 4, nq, nv, E, None) == ALIGN
    assert f(D, I, M, Pf, Pf, nq, nv, E, None) == OVERLAP
    assert f(D, I, M, Pf, M, nq, nv, E, None) == OVERLAP
    g = lib.ekl_tpo_inv_helmholtz_host
    g.argtypes = [vp, vp, vp, vp, i, ll, vp, sz, vp]
    g.restype = i
    n = 4
    S, Dh, u, v = P, P + 0x1000, P + 0x2000, P + 0x3000
    ws = 0x7F1000000000
    assert g(S, Dh, u, v, n, 0, None, 0, None) == OK
    assert g(S, Dh, u, v, 0, 3, ws, 1 << 20, None) == SHAPE
    assert g(S, Dh, u, v, n, 3, None, 1 << 20, None) == NULL
    assert g(S, Dh, u, v, 99, 3, ws, 1 << 20, None) == UNSUP
    assert g(S, Dh, u + 1, v, n, 3, ws, 1 << 20, None) == ALIGN
    assert g(S, Dh, u, Dh, n, 3, ws, 1 << 20, None) == OVERLAP
    assert g(S, Dh, u, v, n, 3, ws + 8, 1 << 20, None) == ALIGN   # workspace must be 256-byte aligned
    assert g(S, Dh, u, v, n, 3, ws, 64, None) == UNSUP            # workspace too small
    h = lib.ekl_tpo_inv_helmholtz_host_static
    h.argtypes = [vp, vp, vp, vp, i, ll, vp]
    h.restype = i
    assert h(S, Dh, u, v, n, 0, None) == OK
    assert h(S, Dh, u, v, 14, 510, None) == UNSUP                 # beyond the fixed staging area
    assert h(S, Dh, None, v, n, 3, None) == NULL
    w = lib.ekl_tpo_host_workspace_bytes
    w.argtypes = [ll, i, ll, ll, ll, i]
    w.restype = sz
    assert w(64, 2, 64, 16, 10, 8) >= 3 * 10 * 3 * 64 * 8 and w(64, 2, 64, 16, 0, 8) == 0


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_2604_19906_b200 import ops
    monkeypatch.setattr(ops, "_lib", None)
    monkeypatch.setattr(ops, "_LIBPATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        ops.library()


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2604_19906_b200")
    for path in glob.glob(os.path.join(pkg, "**", "*"), recursive=True):
        if path.endswith((".py", ".cu", ".cuh", ".h")):
            text = open(path).read()
            assert "import oracle" not in text and "from oracle" not in text, path
            assert "tpo_oracle" not in text, path
    for path in glob.glob(os.path.join(ROOT, "oracle", "*")):
        if path.endswith((".py", ".c", ".h")):
            assert "paper_2604_19906_b200" not in open(path).read(), path


def test_header_compiles_as_c_and_validation_answers_from_a_c_program(lib, tmp_path):
    """gcc (a C compiler, not nvcc) sees include/ekl_tpo.h and links the library."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    cuda_inc = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "include")
    if not gcc or not os.path.exists(os.path.join(cuda_inc, "cuda_runtime_api.h")):
        pytest.skip("gcc or the CUDA headers are not available")
    libdir = os.path.join(ROOT, "paper_2604_19906_b200", "lib")
    exe = str(tmp_path / "abi_check")
    subprocess.run([gcc, "-std=c11", "-Wall", "-Wextra", "-Werror",
                    "-I", os.path.join(ROOT, "include"), "-I", cuda_inc,
                    os.path.join(ROOT, "tests", "c_abi", "abi_check.c"), "-o", exe,
                    "-L", libdir, "-lekl_tpo", f"-Wl,-rpath,{libdir}"], check=True)
    r = subprocess.run([exe], capture_output=True, text=True)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "abi_check: ok" in r.stdout


def test_probe_library_exports_what_its_header_declares():
    """The measurement helpers live in a library of their own, not in the product library."""
    from paper_2604_19906_b200 import build, ops, probes
    build.build()
    text = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "ekl_probe.h")).read(),
                  flags=re.S)
    names = sorted(set(re.findall(r"\b(ekl_probe_[a-z0-9_]+)\s*\(", text)))
    assert len(names) >= 6
    plib = probes.library()
    for n in names:
        assert hasattr(plib, n), n
        assert not hasattr(ops.library(), n), f"{n} must not be exported by the product library"
    # argument checks answer without a GPU
    f = ctypes.c_double(0.0)
    assert plib.ekl_probe_fp64_fma_chain(None, 1, 1, ctypes.byref(f), None) == 1
    assert plib.ekl_probe_fp64_dmma(ctypes.c_void_p(P), 1, 1, 3, ctypes.byref(f), None) == 2
