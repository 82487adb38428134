"""CPU oracle for the batched sum-factorised tensor-product operators.

TEST INFRASTRUCTURE ONLY.  This package is the definition of "correct" that the
CUDA library is compared against, and the host baseline that gets timed next to
it.  Only the test-suite, the smoke check and the benchmark's CPU-baseline leg
may import it; the product package never does, and this package never imports
the product package.  It is plain, slow and obviously correct on purpose.

The arithmetic lives in ``tpo_oracle.c`` (plain C loops, fp64, built with
``-ffp-contract=off`` and without fast-math); this module only compiles that
file with gcc and marshals numpy arrays into it.

Operators (row-major arrays, element index slowest, see ``tpo_oracle.c``):

* ``inv_helmholtz(S, D, u)``: ``v_e = (S⊗S⊗S)·(D_e ∘ ((Sᵀ⊗Sᵀ⊗Sᵀ)·u_e))`` with the
  lifted (sum-factorised) reductions of Section 5.2 of the paper.
* ``inv_helmholtz3(S0, S1, S2, D, u)``: the same with one operator and one extent per
  direction, ``v_e = (S0⊗S1⊗S2)·(D_e ∘ ((S0ᵀ⊗S1ᵀ⊗S2ᵀ)·u_e))`` (per-direction matrices as in Eq. 1).
* ``tpo_apply(A, B, C, u)``: ``v_e = (A⊗B⊗C)·u_e``, rectangular factors, the
  operator family of Eq. 1.
* ``convection(Dvq, Ivq, M, P)``: the volume integral of the convective flux, Eq. 1.
* ``*_bruteforce``: the same operators through the explicit Kronecker matrix (or, for
  ``convection``, the three explicit Kronecker matrices of Eq. 1).
* ``*_ld``: the same operators with every intermediate in ``long double``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tpo_oracle.c")
_LIB = os.path.join(_HERE, "libtpo_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile ``tpo_oracle.c`` into ``libtpo_oracle.so`` next to it (gcc, -O2, no FMA
    contraction, no fast-math, OpenMP for the loop over independent elements)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp",
           "-ffp-contract=off", "-fno-fast-math", "-Wall", "-Wextra",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        i, ll = ctypes.c_int, ctypes.c_longlong
        lib.oracle_threads.argtypes = [i]
        lib.oracle_threads.restype = i
        lib.oracle_inv_helmholtz_f64.argtypes = [dp, dp, dp, dp, i, ll, i]
        lib.oracle_inv_helmholtz_bruteforce_f64.argtypes = [dp, dp, dp, dp, i, ll]
        lib.oracle_inv_helmholtz_ld.argtypes = [dp, dp, dp, dp, i, ll]
        lib.oracle_tpo_apply_f64.argtypes = [dp, dp, dp, dp, dp, i, i, i, i, i, i, ll, i]
        lib.oracle_tpo_apply_bruteforce_f64.argtypes = [dp, dp, dp, dp, dp, i, i, i, i, i, i, ll]
        lib.oracle_tpo_apply_ld.argtypes = [dp, dp, dp, dp, dp, i, i, i, i, i, i, ll]
        lib.oracle_convection_f64.argtypes = [dp, dp, dp, dp, dp, i, i, ll, i]
        lib.oracle_convection_bruteforce_f64.argtypes = [dp, dp, dp, dp, dp, i, i, ll]
        lib.oracle_inv_helmholtz3_f64.argtypes = [dp, dp, dp, dp, dp, dp, i, i, i, ll, i]
        lib.oracle_inv_helmholtz3_bruteforce_f64.argtypes = [dp, dp, dp, dp, dp, dp, i, i, i, ll]
        lib.oracle_inv_helmholtz3_f64.restype = i
        lib.oracle_inv_helmholtz3_bruteforce_f64.restype = i
        lib.oracle_convection_f64.restype = i
        lib.oracle_convection_bruteforce_f64.restype = i
        for f in (lib.oracle_inv_helmholtz_f64, lib.oracle_inv_helmholtz_bruteforce_f64,
                  lib.oracle_inv_helmholtz_ld, lib.oracle_tpo_apply_f64,
                  lib.oracle_tpo_apply_bruteforce_f64, lib.oracle_tpo_apply_ld):
            f.restype = i
        _lib = lib
    return _lib


def _f64(a) -> np.ndarray:
    """C-contiguous float64 copy/view (fp32 inputs are widened exactly)."""
    return np.ascontiguousarray(np.asarray(a), dtype=np.float64)


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def threads_used(threads: int = 0) -> int:
    """How many threads a call with this ``threads`` argument runs on."""
    return int(_load().oracle_threads(int(threads)))


def _check_ih(S, D, u):
    S, D, u = _f64(S), _f64(D), _f64(u)
    if S.ndim != 2 or S.shape[0] != S.shape[1]:
        raise ValueError("S must be [n,n]")
    n = S.shape[0]
    if u.ndim != 4 or u.shape[1:] != (n, n, n) or D.shape != u.shape:
        raise ValueError("D and u must be [E,n,n,n]")
    return S, D, u, n, u.shape[0]


def inv_helmholtz(S, D, u, threads: int = 0) -> np.ndarray:
    """Sum-factorised inverse Helmholtz, fp64, all elements.  ``threads<=0``: all cores."""
    S, D, u, n, E = _check_ih(S, D, u)
    v = np.empty_like(u)
    if E and _load().oracle_inv_helmholtz_f64(_ptr(S), _ptr(D), _ptr(u), _ptr(v), n, E,
                                              int(threads)):
        raise MemoryError("oracle scratch allocation failed")
    return v


def lambda_factor(lam, c) -> np.ndarray:
    """``D[e,i,j,k] = 1/(((lam[i]+lam[j])+lam[k])+c[e])``, the sums taken in this order."""
    lam, c = _f64(lam), _f64(c)
    s = (lam[:, None, None] + lam[None, :, None]) + lam[None, None, :]
    return 1.0 / (s[None, :, :, :] + c[:, None, None, None])


def inv_helmholtz_lambda(S, lam, c, u, threads: int = 0) -> np.ndarray:
    """Inverse Helmholtz whose pointwise factor is given by its eigenvalue sums: the factor is
    written out with :func:`lambda_factor` and handed to :func:`inv_helmholtz`."""
    return inv_helmholtz(S, lambda_factor(lam, c), u, threads)


def _check_ih3(S0, S1, S2, D, u):
    S0, S1, S2, D, u = _f64(S0), _f64(S1), _f64(S2), _f64(D), _f64(u)
    for S in (S0, S1, S2):
        if S.ndim != 2 or S.shape[0] != S.shape[1]:
            raise ValueError("S0, S1, S2 must be square matrices")
    nn = (S0.shape[0], S1.shape[0], S2.shape[0])
    if u.ndim != 4 or u.shape[1:] != nn or D.shape != u.shape:
        raise ValueError("D and u must be [E,n0,n1,n2] with n_d the order of S_d")
    return S0, S1, S2, D, u, nn, u.shape[0]


def inv_helmholtz3(S0, S1, S2, D, u, threads: int = 0) -> np.ndarray:
    """Inverse Helmholtz with one operator and one extent per direction:
    ``v_e = (S0⊗S1⊗S2)·(D_e ∘ ((S0ᵀ⊗S1ᵀ⊗S2ᵀ)·u_e))``, S0 on the slowest in-element axis."""
    S0, S1, S2, D, u, nn, E = _check_ih3(S0, S1, S2, D, u)
    v = np.empty_like(u)
    if E and _load().oracle_inv_helmholtz3_f64(_ptr(S0), _ptr(S1), _ptr(S2), _ptr(D), _ptr(u),
                                               _ptr(v), *nn, E, int(threads)):
        raise MemoryError("oracle scratch allocation failed")
    return v


def inv_helmholtz3_bruteforce(S0, S1, S2, D, u) -> np.ndarray:
    """The same operator through the explicit Kronecker matrices (tiny extents only)."""
    S0, S1, S2, D, u, nn, E = _check_ih3(S0, S1, S2, D, u)
    if np.prod(nn) > 256:
        raise ValueError("brute force is meant for tiny shapes")
    v = np.empty_like(u)
    if E and _load().oracle_inv_helmholtz3_bruteforce_f64(_ptr(S0), _ptr(S1), _ptr(S2), _ptr(D),
                                                          _ptr(u), _ptr(v), *nn, E):
        raise MemoryError("oracle scratch allocation failed")
    return v


def inv_helmholtz_bruteforce(S, D, u) -> np.ndarray:
    """Same operator through the explicit n³×n³ Kronecker matrices (tiny n only)."""
    S, D, u, n, E = _check_ih(S, D, u)
    if n > 6:
        raise ValueError("brute force is meant for n <= 6")
    v = np.empty_like(u)
    if E and _load().oracle_inv_helmholtz_bruteforce_f64(_ptr(S), _ptr(D), _ptr(u), _ptr(v),
                                                         n, E):
        raise MemoryError("oracle scratch allocation failed")
    return v


def inv_helmholtz_ld(S, D, u) -> np.ndarray:
    """Same operator, intermediates in long double, rounded to fp64 once."""
    S, D, u, n, E = _check_ih(S, D, u)
    v = np.empty_like(u)
    if E and _load().oracle_inv_helmholtz_ld(_ptr(S), _ptr(D), _ptr(u), _ptr(v), n, E):
        raise MemoryError("oracle scratch allocation failed")
    return v


def _check_apply(A, B, C, u):
    A, B, C, u = _f64(A), _f64(B), _f64(C), _f64(u)
    if A.ndim != 2 or B.ndim != 2 or C.ndim != 2 or u.ndim != 4:
        raise ValueError("A,B,C must be matrices and u [E,n0,n1,n2]")
    (m0, n0), (m1, n1), (m2, n2) = A.shape, B.shape, C.shape
    if u.shape[1:] != (n0, n1, n2):
        raise ValueError("u must be [E,n0,n1,n2] with n_d = columns of A,B,C")
    return A, B, C, u, (n0, n1, n2), (m0, m1, m2), u.shape[0]


def tpo_apply(A, B, C, u, threads: int = 0) -> np.ndarray:
    """Sum-factorised ``(A⊗B⊗C)·u_e``, contraction order C, then B, then A."""
    A, B, C, u, nn, mm, E = _check_apply(A, B, C, u)
    v = np.empty((E,) + mm, dtype=np.float64)
    if E and _load().oracle_tpo_apply_f64(_ptr(A), _ptr(B), _ptr(C), _ptr(u), _ptr(v),
                                          *nn, *mm, E, int(threads)):
        raise MemoryError("oracle scratch allocation failed")
    return v


def tpo_apply_bruteforce(A, B, C, u) -> np.ndarray:
    """``kron(A,B,C) @ vec(u_e)`` with the explicit matrix (tiny sizes only)."""
    A, B, C, u, nn, mm, E = _check_apply(A, B, C, u)
    if np.prod(nn) * np.prod(mm) > 1 << 22:
        raise ValueError("brute force is meant for tiny shapes")
    v = np.empty((E,) + mm, dtype=np.float64)
    if E and _load().oracle_tpo_apply_bruteforce_f64(_ptr(A), _ptr(B), _ptr(C), _ptr(u),
                                                     _ptr(v), *nn, *mm, E):
        raise MemoryError("oracle scratch allocation failed")
    return v


def tpo_apply_ld(A, B, C, u) -> np.ndarray:
    """Same operator, intermediates in long double, rounded to fp64 once."""
    A, B, C, u, nn, mm, E = _check_apply(A, B, C, u)
    v = np.empty((E,) + mm, dtype=np.float64)
    if E and _load().oracle_tpo_apply_ld(_ptr(A), _ptr(B), _ptr(C), _ptr(u), _ptr(v),
                                         *nn, *mm, E):
        raise MemoryError("oracle scratch allocation failed")
    return v


def _check_convection(Dvq, Ivq, M, P):
    Dvq, Ivq, M, P = _f64(Dvq), _f64(Ivq), _f64(M), _f64(P)
    if Dvq.ndim != 2 or Dvq.shape != Ivq.shape:
        raise ValueError("Dvq and Ivq must both be [nv,nq]")
    nv, nq = Dvq.shape
    if M.ndim != 4 or M.shape[1:] != (nq, nq, nq):
        raise ValueError("M must be [E,nq,nq,nq]")
    E = M.shape[0]
    if P.shape != (3, 3, E, nq, nq, nq):
        raise ValueError("P must be [3,3,E,nq,nq,nq]")
    return Dvq, Ivq, M, P, nq, nv, E


def convection(Dvq, Ivq, M, P, threads: int = 0) -> np.ndarray:
    """Volume integral of the convective flux (Eq. 1): for each component c and element e,
    ``(I⊗I⊗D)(M∘P[c,0]) + (I⊗D⊗I)(M∘P[c,1]) + (D⊗I⊗I)(M∘P[c,2])``; returns F [3,E,nv,nv,nv]."""
    Dvq, Ivq, M, P, nq, nv, E = _check_convection(Dvq, Ivq, M, P)
    F = np.empty((3, E, nv, nv, nv), dtype=np.float64)
    if E and _load().oracle_convection_f64(_ptr(Dvq), _ptr(Ivq), _ptr(M), _ptr(P), _ptr(F),
                                           nq, nv, E, int(threads)):
        raise MemoryError("oracle scratch allocation failed")
    return F


def convection_bruteforce(Dvq, Ivq, M, P) -> np.ndarray:
    """The same operator through the three explicit Kronecker matrices of Eq. 1, I⊗I⊗D, I⊗D⊗I
    and D⊗I⊗I (tiny sizes only)."""
    Dvq, Ivq, M, P, nq, nv, E = _check_convection(Dvq, Ivq, M, P)
    if nq > 6 or nv > 6:
        raise ValueError("brute force is meant for tiny shapes")
    F = np.empty((3, E, nv, nv, nv), dtype=np.float64)
    if E and _load().oracle_convection_bruteforce_f64(_ptr(Dvq), _ptr(Ivq), _ptr(M), _ptr(P),
                                                      _ptr(F), nq, nv, E):
        raise MemoryError("oracle scratch allocation failed")
    return F


def rel_err_per_element(v, v_ref) -> np.ndarray:
    """Normwise relative error per element: ‖v_e − v̂_e‖₂ / ‖v̂_e‖₂ (2-norm over the
    element's outputs, v̂ = oracle).  A zero reference norm is guarded by 1e-300; any
    NaN/Inf in ``v`` yields inf for that element."""
    v = np.asarray(v, dtype=np.float64)
    r = np.asarray(v_ref, dtype=np.float64)
    E = r.shape[0]
    d = (v - r).reshape(E, -1)
    num = np.sqrt(np.sum(d * d, axis=1))
    den = np.sqrt(np.sum(r.reshape(E, -1) ** 2, axis=1))
    err = num / np.maximum(den, 1e-300)
    bad = ~np.isfinite(v.reshape(E, -1)).all(axis=1)
    err[bad] = np.inf
    return err
