"""Seeded synthetic inputs for the tensor-product-operator workloads.

This module only *makes inputs*: it contains none of the operator's arithmetic and
is the one module both the CUDA path's callers and the CPU oracle's callers use.

Small arrays (S, A, B, C, λ) come from a seeded NumPy ``PCG64`` stream on the host.
Large arrays (u, and D through the per-element shift c_e) come from a counter-based
generator so that any slice can be regenerated anywhere, bit for bit:

    h      = splitmix64_finaliser(key + (index + 1)·0x9E3779B97F4A7C15)   (mod 2^64)
    r      = (h >> 11) · 2^-53                     in [0, 1), exact in fp64
    value  = lo + scale·r                          (one multiply, one add, both RN)

(the finaliser is the published SplitMix64 output function).  The same definition is
implemented once here with NumPy ``uint64`` arithmetic and once as a device fill
kernel (``csrc/inputs_fill.cu``); integer arithmetic makes both bit-identical, so
multi-gigabyte fields never have to cross PCIe and the oracle can be fed any chunk.

Workload recipe (the five configurations of the benchmark):

* inverse Helmholtz, fp64: S = Q of the QR factorisation of an n×n N(0,1) matrix,
  u ~ U(-1,1) of shape [E,n,n,n], D[e,i,j,k] = 1/(((λ_i+λ_j)+λ_k)+c_e) with one
  shared λ ~ U(0.1,2)^n and c_e ~ U(0.5,1.5); (n,E) = (4,64), (8,4096), (12,65536),
  (14,131072).
* forward rectangular operator, fp64: A, B, C of shape 12×8 ~ N(0, variance 1/8),
  u ~ U(-1,1) of shape [E,8,8,8], E = 131072.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np

BASE_SEED = 260419906

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

# array ids mixed into the key so that u, c_e, ... are independent streams
ARRAY_U = 1
ARRAY_C = 2
ARRAY_M = 3
ARRAY_P = 4


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration."""
    index: int
    op: str                      # "inv_helmholtz" | "apply"
    n: tuple                     # input extents per direction
    m: tuple                     # output extents per direction
    E: int
    dtype: str = "f64"

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    @property
    def name(self) -> str:
        if self.op == "inv_helmholtz":
            return f"cfg{self.index}:inv_helmholtz_{self.dtype}_n{self.n[0]}_E{self.E}"
        if self.op == "convection":
            return f"cfg{self.index}:convection_{self.dtype}_nq{self.n[0]}_nv{self.m[0]}_E{self.E}"
        return (f"cfg{self.index}:apply_{self.dtype}_{self.n[0]}x{self.n[1]}x{self.n[2]}"
                f"_to_{self.m[0]}x{self.m[1]}x{self.m[2]}_E{self.E}")

    @property
    def flops_per_element(self) -> int:
        """Algorithmic flops: 12n⁴+n³ (inverse Helmholtz); contraction order C→B→A,
        2·(n0·n1·m2·n2 + n0·m1·m2·n1 + m0·m1·m2·n0) (forward operator); for the convective
        flux nine such forward operators (3 components × 3 directions) plus the 9 nq³
        products with M and the 6 nv³ additions."""
        n0, n1, n2 = self.n
        m0, m1, m2 = self.m
        if self.op == "inv_helmholtz":
            return 12 * n0 ** 4 + n0 ** 3
        tpo = 2 * (n0 * n1 * m2 * n2 + n0 * m1 * m2 * n1 + m0 * m1 * m2 * n0)
        if self.op == "convection":
            return 9 * tpo + 9 * n0 * n1 * n2 + 6 * m0 * m1 * m2
        return tpo

    @property
    def bytes_per_element(self) -> int:
        """Algorithmic HBM bytes: read u (and D), write v; operator matrices not counted."""
        w = 8 if self.dtype == "f64" else 4
        nin = self.n[0] * self.n[1] * self.n[2]
        nout = self.m[0] * self.m[1] * self.m[2]
        if self.op == "inv_helmholtz":
            return 3 * w * nin
        if self.op == "convection":
            return w * (10 * nin + 3 * nout)          # M, nine P fields in; three F fields out
        return w * (nin + nout)


CONFIGS = (
    Workload(0, "inv_helmholtz", (4, 4, 4), (4, 4, 4), 64),
    Workload(1, "inv_helmholtz", (8, 8, 8), (8, 8, 8), 4096),
    Workload(2, "inv_helmholtz", (12, 12, 12), (12, 12, 12), 65536),
    Workload(3, "inv_helmholtz", (14, 14, 14), (14, 14, 14), 131072),
    Workload(4, "apply", (8, 8, 8), (12, 12, 12), 131072),
    # not one of the five stated configurations: the convective-flux integral of Eq. 1 on the
    # paper's batch size (8192 elements per call), 12 quadrature -> 8 volume points
    Workload(5, "convection", (12, 12, 12), (8, 8, 8), 8192),
    # the largest inverse-Helmholtz configuration with single-precision fields (tolerance 1e-5):
    # the same streams, rounded to fp32
    Workload(6, "inv_helmholtz", (14, 14, 14), (14, 14, 14), 131072, "f32"),
)


# ---------------------------------------------------------------- counter-based stream

def _finalise(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def stream_key(seed: int, array_id: int) -> int:
    """64-bit key of one (seed, array) stream."""
    with np.errstate(over="ignore"):
        z = np.array([np.uint64(seed & 0xFFFFFFFFFFFFFFFF)], dtype=np.uint64)
        z = _finalise(z * _GOLDEN + np.uint64(array_id))
    return int(z[0])


def counter_u01(key: int, start: int, count: int) -> np.ndarray:
    """``count`` doubles in [0,1) of stream ``key`` at indices start … start+count-1."""
    with np.errstate(over="ignore"):
        idx = np.arange(start + 1, start + 1 + count, dtype=np.uint64)
        h = _finalise(np.uint64(key) + idx * _GOLDEN)
    return (h >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)


def counter_uniform(key: int, start: int, count: int, lo: float, hi: float) -> np.ndarray:
    """``lo + (hi-lo)·r`` for the same stream."""
    r = counter_u01(key, start, count)
    return lo + (hi - lo) * r


# ---------------------------------------------------------------- small host arrays

def orthogonal_S(n: int, seed: int) -> np.ndarray:
    """Q factor of the QR factorisation of a seeded n×n N(0,1) matrix (orthogonal)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    q, _ = np.linalg.qr(rng.standard_normal((n, n)))
    return np.ascontiguousarray(q)


def eigen_lambda(n: int, seed: int) -> np.ndarray:
    """The shared λ ~ U(0.1,2) vector of length n."""
    rng = np.random.Generator(np.random.PCG64(seed + 7919))
    return rng.uniform(0.1, 2.0, size=n)


def gaussian_factor(m: int, n: int, seed: int, which: int) -> np.ndarray:
    """An m×n matrix ~ N(0, variance 1/n) (σ = n^-½), independent per ``which``."""
    rng = np.random.Generator(np.random.PCG64(seed + 104729 * (which + 1)))
    return np.ascontiguousarray(rng.standard_normal((m, n)) / np.sqrt(float(n)))


# ---------------------------------------------------------------- host fields (any slice)

def host_u(wl: Workload, e0: int, e1: int) -> np.ndarray:
    """u[e0:e1] ~ U(-1,1), shape [e1-e0, n0, n1, n2], fp64."""
    per = wl.n[0] * wl.n[1] * wl.n[2]
    key = stream_key(wl.seed, ARRAY_U)
    x = counter_uniform(key, e0 * per, (e1 - e0) * per, -1.0, 1.0)
    return x.reshape((e1 - e0,) + tuple(wl.n))


def host_c(wl: Workload, e0: int, e1: int) -> np.ndarray:
    """c_e ~ U(0.5,1.5) for e0 ≤ e < e1."""
    return counter_uniform(stream_key(wl.seed, ARRAY_C), e0, e1 - e0, 0.5, 1.5)


def host_D(wl: Workload, lam: np.ndarray, e0: int, e1: int) -> np.ndarray:
    """D[e,i,j,k] = 1/(((λ_i+λ_j)+λ_k)+c_e), shape [e1-e0, n, n, n], fp64."""
    c = host_c(wl, e0, e1)
    s = (lam[:, None, None] + lam[None, :, None]) + lam[None, None, :]
    return 1.0 / (s[None, :, :, :] + c[:, None, None, None])


def host_M(wl: Workload, e0: int, e1: int) -> np.ndarray:
    """M[e0:e1] ~ U(0.5,1.5), shape [e1-e0, nq, nq, nq]."""
    per = wl.n[0] * wl.n[1] * wl.n[2]
    x = counter_uniform(stream_key(wl.seed, ARRAY_M), e0 * per, (e1 - e0) * per, 0.5, 1.5)
    return x.reshape((e1 - e0,) + tuple(wl.n))


def host_P(wl: Workload, e0: int, e1: int) -> np.ndarray:
    """P[:, :, e0:e1] ~ U(-1,1), shape [3,3,e1-e0,nq,nq,nq]; the stream index is that of the
    full [3,3,E,...] array."""
    per = wl.n[0] * wl.n[1] * wl.n[2]
    key = stream_key(wl.seed, ARRAY_P)
    out = np.empty((3, 3, e1 - e0) + tuple(wl.n))
    for c in range(3):
        for d in range(3):
            start = ((c * 3 + d) * wl.E + e0) * per
            out[c, d] = counter_uniform(key, start, (e1 - e0) * per, -1.0, 1.0).reshape(
                (e1 - e0,) + tuple(wl.n))
    return out


def host_case(wl: Workload, e0: int = 0, e1: int | None = None) -> dict:
    """All inputs of ``wl`` for elements [e0,e1) as NumPy arrays (fp64; rounded to fp32 for a
    single-precision workload)."""
    e1 = wl.E if e1 is None else e1
    if wl.dtype == "f32":
        wide = host_case(Workload(wl.index, wl.op, wl.n, wl.m, wl.E, "f64"), e0, e1)
        return {k: (v if k == "lam" else v.astype(np.float32)) for k, v in wide.items()}
    if wl.op == "convection":
        return {"Dvq": gaussian_factor(wl.m[0], wl.n[0], wl.seed, 0),
                "Ivq": gaussian_factor(wl.m[0], wl.n[0], wl.seed, 1),
                "M": host_M(wl, e0, e1), "P": host_P(wl, e0, e1)}
    if wl.op == "inv_helmholtz":
        n = wl.n[0]
        lam = eigen_lambda(n, wl.seed)
        return {"S": orthogonal_S(n, wl.seed), "lam": lam,
                "D": host_D(wl, lam, e0, e1), "u": host_u(wl, e0, e1)}
    return {"A": gaussian_factor(wl.m[0], wl.n[0], wl.seed, 0),
            "B": gaussian_factor(wl.m[1], wl.n[1], wl.seed, 1),
            "C": gaussian_factor(wl.m[2], wl.n[2], wl.seed, 2),
            "u": host_u(wl, e0, e1)}


# ---------------------------------------------------------------- device fields

_LIBNAME = os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib", "libekl_inputs.so")
_fill = None


def _fill_lib():
    global _fill
    if _fill is None:
        if not os.path.exists(_LIBNAME):
            raise RuntimeError(f"{_LIBNAME} is missing: run build() first")
        lib = ctypes.CDLL(_LIBNAME)
        vp, ll, u64, d = ctypes.c_void_p, ctypes.c_longlong, ctypes.c_uint64, ctypes.c_double
        lib.ekl_inputs_fill_uniform_f64.argtypes = [vp, ll, ll, u64, d, d, vp]
        lib.ekl_inputs_fill_uniform_f64.restype = ctypes.c_int
        lib.ekl_inputs_fill_D_f64.argtypes = [vp, vp, ctypes.c_int, ll, ll, u64, vp]
        lib.ekl_inputs_fill_D_f64.restype = ctypes.c_int
        _fill = lib
    return _fill


def device_case(wl: Workload, device="cuda:0", e0: int = 0, e1: int | None = None) -> dict:
    """Inputs of ``wl`` for elements [e0,e1) as torch tensors on ``device``; the big
    fields are generated in place by the device fill kernels (bit-identical to
    ``host_case``)."""
    import torch

    e1 = wl.E if e1 is None else e1
    if wl.dtype == "f32":
        # generated in fp64 by the same kernels, then rounded field by field
        wide = Workload(wl.index, wl.op, wl.n, wl.m, wl.E, "f64")
        out = {}
        for k, t in device_case(wide, device, e0, e1).items():
            out[k] = t if k == "lam" else t.float()
            del t
        return out
    E = e1 - e0
    dev = torch.device(device)
    lib = _fill_lib()
    per = wl.n[0] * wl.n[1] * wl.n[2]
    out = {}
    if wl.op == "convection":
        with torch.cuda.device(dev):
            st = torch.cuda.current_stream(dev).cuda_stream
            M = torch.empty((E,) + tuple(wl.n), dtype=torch.float64, device=dev)
            P = torch.empty((3, 3, E) + tuple(wl.n), dtype=torch.float64, device=dev)
            rc = lib.ekl_inputs_fill_uniform_f64(M.data_ptr(), e0 * per, E * per,
                                                 stream_key(wl.seed, ARRAY_M), 0.5, 1.0, st) if E else 0
            for c in range(3):
                for d in range(3):
                    if E and not rc:
                        rc = lib.ekl_inputs_fill_uniform_f64(
                            P[c, d].data_ptr(), ((c * 3 + d) * wl.E + e0) * per, E * per,
                            stream_key(wl.seed, ARRAY_P), -1.0, 2.0, st)
            if rc:
                raise RuntimeError(f"fill_uniform failed with CUDA error {rc}")
            out = {"M": M, "P": P,
                   "Dvq": torch.from_numpy(gaussian_factor(wl.m[0], wl.n[0], wl.seed, 0)).to(dev),
                   "Ivq": torch.from_numpy(gaussian_factor(wl.m[0], wl.n[0], wl.seed, 1)).to(dev)}
            torch.cuda.synchronize(dev)
        return out
    with torch.cuda.device(dev):
        st = torch.cuda.current_stream(dev).cuda_stream
        u = torch.empty((E,) + tuple(wl.n), dtype=torch.float64, device=dev)
        if E:
            rc = lib.ekl_inputs_fill_uniform_f64(u.data_ptr(), e0 * per, E * per,
                                                 stream_key(wl.seed, ARRAY_U), -1.0, 2.0, st)
            if rc:
                raise RuntimeError(f"fill_uniform failed with CUDA error {rc}")
        out["u"] = u
        if wl.op == "inv_helmholtz":
            n = wl.n[0]
            lam = eigen_lambda(n, wl.seed)
            out["S"] = torch.from_numpy(orthogonal_S(n, wl.seed)).to(dev)
            out["lam"] = lam
            lam_d = torch.from_numpy(lam).to(dev)
            D = torch.empty_like(u)
            if E:
                rc = lib.ekl_inputs_fill_D_f64(D.data_ptr(), lam_d.data_ptr(), n, e0, E,
                                               stream_key(wl.seed, ARRAY_C), st)
                if rc:
                    raise RuntimeError(f"fill_D failed with CUDA error {rc}")
            out["D"] = D
        else:
            for w, nm in enumerate("ABC"):
                out[nm] = torch.from_numpy(
                    gaussian_factor(wl.m[w], wl.n[w], wl.seed, w)).to(dev)
        torch.cuda.synchronize(dev)
    return out
