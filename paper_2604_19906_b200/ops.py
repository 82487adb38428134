"""Thin Python binding of the C-ABI library (``include/ekl_tpo.h``).

Argument marshalling only: every function here takes CUDA tensors, checks dtype /
device / contiguity, and passes raw device pointers, extents and the current CUDA
stream to the entry point of the same name in ``lib/libekl_tpo.so``.  All arithmetic
runs in the library's kernels; there is no fallback -- if the library is missing or a
call is rejected, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

# EKL_TPO_LIBRARY selects another build of the same library (A/B measurements)
_LIBPATH = os.environ.get("EKL_TPO_LIBRARY") or os.path.join(
    os.path.dirname(os.path.abspath(__file__)), "lib", "libekl_tpo.so")
_lib = None

STATUS_NAMES = {0: "EKL_TPO_OK", 1: "EKL_TPO_ERR_NULL", 2: "EKL_TPO_ERR_SHAPE",
                3: "EKL_TPO_ERR_UNSUPPORTED", 4: "EKL_TPO_ERR_ALIGN", 5: "EKL_TPO_ERR_OVERLAP",
                6: "EKL_TPO_ERR_CUDA"}


class EklTpoError(RuntimeError):
    """A library call returned a status other than EKL_TPO_OK."""

    def __init__(self, status: int, where: str):
        self.status = status
        lib = library()
        msg = lib.ekl_tpo_status_string(status).decode()
        extra = f", cudaError {lib.ekl_tpo_last_cuda_error()}" if status == 6 else ""
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({msg}{extra})")


def library() -> ctypes.CDLL:
    """The loaded C-ABI library with argument types declared (raises if it is not built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIBPATH):
            raise RuntimeError(
                f"{_LIBPATH} is missing: build it with `python -m paper_2604_19906_b200.build` "
                "(there is no fallback implementation)")
        lib = ctypes.CDLL(_LIBPATH)
        vp, i, ll = ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong
        for name in ("ekl_tpo_inv_helmholtz", "ekl_tpo_inv_helmholtz_f32"):
            f = getattr(lib, name)
            f.argtypes = [vp, vp, vp, vp, i, ll, vp]
            f.restype = i
        for name in ("ekl_tpo_apply", "ekl_tpo_apply_f32"):
            f = getattr(lib, name)
            f.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, ll, vp]
            f.restype = i
        lib.ekl_tpo_status_string.argtypes = [i]
        lib.ekl_tpo_status_string.restype = ctypes.c_char_p
        lib.ekl_tpo_version.restype = i
        lib.ekl_tpo_last_cuda_error.restype = i
        _lib = lib
    return _lib


def _dev_ptr(t: torch.Tensor, name: str, dtype: torch.dtype, device: torch.device) -> int:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if t.device != device:
        raise ValueError(f"{name} is on {t.device}, expected {device}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous (row-major)")
    return t.data_ptr()


def _stream(device: torch.device) -> int:
    return torch.cuda.current_stream(device).cuda_stream


def _inv_helmholtz(fn_name, dtype, S, D, u, out):
    if u.dim() != 4 or S.dim() != 2:
        raise ValueError("S must be [n,n] and u [E,n,n,n]")
    E, n = u.shape[0], S.shape[0]
    if tuple(S.shape) != (n, n) or tuple(u.shape[1:]) != (n, n, n) or D.shape != u.shape:
        raise ValueError("expected S [n,n] and D,u [E,n,n,n]")
    dev = u.device
    if out is None:
        out = torch.empty_like(u)
    elif out.shape != u.shape:
        raise ValueError("out must have the shape of u")
    ptrs = [_dev_ptr(t, nm, dtype, dev) for t, nm in ((S, "S"), (D, "D"), (u, "u"), (out, "out"))]
    with torch.cuda.device(dev):
        st = getattr(library(), fn_name)(*ptrs, n, E, _stream(dev))
    if st:
        raise EklTpoError(st, fn_name)
    return out


def ekl_tpo_inv_helmholtz(S, D, u, out=None):
    """``v[e] = (S⊗S⊗S)·(D[e] ∘ ((Sᵀ⊗Sᵀ⊗Sᵀ)·u[e]))`` in fp64 on the current stream.
    ``out`` may be ``u`` itself (in place)."""
    return _inv_helmholtz("ekl_tpo_inv_helmholtz", torch.float64, S, D, u, out)


def ekl_tpo_inv_helmholtz_f32(S, D, u, out=None):
    """Single-precision twin of :func:`ekl_tpo_inv_helmholtz`."""
    return _inv_helmholtz("ekl_tpo_inv_helmholtz_f32", torch.float32, S, D, u, out)


def _apply(fn_name, dtype, A, B, C, u, out):
    if u.dim() != 4 or A.dim() != 2 or B.dim() != 2 or C.dim() != 2:
        raise ValueError("A,B,C must be matrices and u [E,n0,n1,n2]")
    (m0, n0), (m1, n1), (m2, n2) = A.shape, B.shape, C.shape
    E = u.shape[0]
    if tuple(u.shape[1:]) != (n0, n1, n2):
        raise ValueError("u must be [E,n0,n1,n2] with n_d the column counts of A,B,C")
    dev = u.device
    if out is None:
        out = torch.empty((E, m0, m1, m2), dtype=dtype, device=dev)
    elif tuple(out.shape) != (E, m0, m1, m2):
        raise ValueError("out must be [E,m0,m1,m2]")
    ptrs = [_dev_ptr(t, nm, dtype, dev)
            for t, nm in ((A, "A"), (B, "B"), (C, "C"), (u, "u"), (out, "out"))]
    with torch.cuda.device(dev):
        st = getattr(library(), fn_name)(*ptrs, n0, n1, n2, m0, m1, m2, E, _stream(dev))
    if st:
        raise EklTpoError(st, fn_name)
    return out


def ekl_tpo_apply(A, B, C, u, out=None):
    """``v[e] = (A⊗B⊗C)·u[e]`` in fp64 on the current stream."""
    return _apply("ekl_tpo_apply", torch.float64, A, B, C, u, out)


def ekl_tpo_apply_f32(A, B, C, u, out=None):
    """Single-precision twin of :func:`ekl_tpo_apply`."""
    return _apply("ekl_tpo_apply_f32", torch.float32, A, B, C, u, out)


def ekl_tpo_inv_helmholtz3(S0, S1, S2, D, u, out=None):
    """``v[e] = (S0⊗S1⊗S2)·(D[e] ∘ ((S0ᵀ⊗S1ᵀ⊗S2ᵀ)·u[e]))``: one operator and one extent per
    direction, fp64, on the current stream.  ``out`` may be ``u`` itself (in place)."""
    lib = library()
    fn = lib.ekl_tpo_inv_helmholtz3
    fn.argtypes = [ctypes.c_void_p] * 6 + [ctypes.c_int] * 3 + [ctypes.c_longlong, ctypes.c_void_p]
    fn.restype = ctypes.c_int
    if u.dim() != 4 or any(S.dim() != 2 or S.shape[0] != S.shape[1] for S in (S0, S1, S2)):
        raise ValueError("S0, S1, S2 must be square matrices and u [E,n0,n1,n2]")
    nn = (S0.shape[0], S1.shape[0], S2.shape[0])
    if tuple(u.shape[1:]) != nn or D.shape != u.shape:
        raise ValueError("D and u must be [E,n0,n1,n2] with n_d the order of S_d")
    dev = u.device
    if out is None:
        out = torch.empty_like(u)
    elif out.shape != u.shape:
        raise ValueError("out must have the shape of u")
    ptrs = [_dev_ptr(t, nm, torch.float64, dev)
            for t, nm in ((S0, "S0"), (S1, "S1"), (S2, "S2"), (D, "D"), (u, "u"), (out, "out"))]
    with torch.cuda.device(dev):
        st = fn(*ptrs, *nn, u.shape[0], _stream(dev))
    if st:
        raise EklTpoError(st, "ekl_tpo_inv_helmholtz3")
    return out


def ekl_tpo_inv_helmholtz_lambda(S, lam, c, u, out=None):
    """Inverse Helmholtz with ``D[e,i,j,k] = 1/(((lam[i]+lam[j])+lam[k])+c[e])`` formed on the
    fly (fp64, 4 <= n <= 20); bit-identical to :func:`ekl_tpo_inv_helmholtz` on that D."""
    lib = library()
    fn = lib.ekl_tpo_inv_helmholtz_lambda
    fn.argtypes = [ctypes.c_void_p] * 5 + [ctypes.c_int, ctypes.c_longlong, ctypes.c_void_p]
    fn.restype = ctypes.c_int
    E, n = u.shape[0], S.shape[0]
    if tuple(S.shape) != (n, n) or tuple(u.shape[1:]) != (n, n, n) or tuple(lam.shape) != (n,) \
            or tuple(c.shape) != (E,):
        raise ValueError("expected S [n,n], lam [n], c [E], u [E,n,n,n]")
    dev = u.device
    if out is None:
        out = torch.empty_like(u)
    ptrs = [_dev_ptr(t, nm, torch.float64, dev)
            for t, nm in ((S, "S"), (lam, "lam"), (c, "c"), (u, "u"), (out, "out"))]
    with torch.cuda.device(dev):
        st = fn(*ptrs, n, E, _stream(dev))
    if st:
        raise EklTpoError(st, "ekl_tpo_inv_helmholtz_lambda")
    return out


def ekl_tpo_convection(Dvq, Ivq, M, P, out=None):
    """Volume integral of the convective flux: ``F[c,e] = (I⊗I⊗D)(M∘P[c,0]) + (I⊗D⊗I)(M∘P[c,1])
    + (D⊗I⊗I)(M∘P[c,2])`` in fp64 on the current stream; P is [3,3,E,nq,nq,nq], F [3,E,nv,nv,nv]."""
    lib = library()
    fn = lib.ekl_tpo_convection
    fn.argtypes = [ctypes.c_void_p] * 5 + [ctypes.c_int, ctypes.c_int, ctypes.c_longlong,
                                           ctypes.c_void_p]
    fn.restype = ctypes.c_int
    if Dvq.dim() != 2 or Dvq.shape != Ivq.shape or M.dim() != 4 or P.dim() != 6:
        raise ValueError("expected Dvq,Ivq [nv,nq], M [E,nq,nq,nq], P [3,3,E,nq,nq,nq]")
    nv, nq = Dvq.shape
    E = M.shape[0]
    if tuple(M.shape[1:]) != (nq, nq, nq) or tuple(P.shape) != (3, 3, E, nq, nq, nq):
        raise ValueError("expected M [E,nq,nq,nq] and P [3,3,E,nq,nq,nq]")
    dev = M.device
    if out is None:
        out = torch.empty((3, E, nv, nv, nv), dtype=torch.float64, device=dev)
    elif tuple(out.shape) != (3, E, nv, nv, nv):
        raise ValueError("out must be [3,E,nv,nv,nv]")
    ptrs = [_dev_ptr(t, nm, torch.float64, dev)
            for t, nm in ((Dvq, "Dvq"), (Ivq, "Ivq"), (M, "M"), (P, "P"), (out, "out"))]
    with torch.cuda.device(dev):
        st = fn(*ptrs, nq, nv, E, _stream(dev))
    if st:
        raise EklTpoError(st, "ekl_tpo_convection")
    return out


def ekl_tpo_version() -> int:
    return int(library().ekl_tpo_version())


# ----------------------------------------------------------------------------- host buffers

_workspaces: dict = {}


def _declare_host(lib):
    if getattr(lib, "_host_declared", False):
        return
    vp, i, ll, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong, ctypes.c_size_t
    lib.ekl_tpo_inv_helmholtz_host.argtypes = [vp, vp, vp, vp, i, ll, vp, sz, vp]
    lib.ekl_tpo_inv_helmholtz_host.restype = i
    lib.ekl_tpo_apply_host.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, ll, vp, sz, vp]
    lib.ekl_tpo_apply_host.restype = i
    lib.ekl_tpo_inv_helmholtz_host_f32.argtypes = lib.ekl_tpo_inv_helmholtz_host.argtypes
    lib.ekl_tpo_inv_helmholtz_host_f32.restype = i
    lib.ekl_tpo_apply_host_f32.argtypes = lib.ekl_tpo_apply_host.argtypes
    lib.ekl_tpo_apply_host_f32.restype = i
    lib.ekl_tpo_host_workspace_bytes.argtypes = [ll, i, ll, ll, ll, i]
    lib.ekl_tpo_host_workspace_bytes.restype = sz
    lib._host_declared = True


def host_workspace(device, nbytes: int) -> torch.Tensor:
    """A cached device scratch buffer of at least ``nbytes`` bytes for host-buffer calls on the
    current stream of ``device`` (device memory comes from torch; the library itself allocates
    none).  One buffer per (device, stream): calls that share a workspace must be ordered on
    one stream.  The library also works on the buffer from two helper streams that torch's
    allocator does not know of, so before a buffer is replaced by a larger one the stream it
    served is synchronised -- the last call's copies have then left it."""
    dev = torch.device(device)
    stream = torch.cuda.current_stream(dev)
    key = (dev.type, dev.index, stream.cuda_stream)
    ws = _workspaces.get(key)
    if ws is None or ws.numel() < nbytes:
        if ws is not None:
            stream.synchronize()
        ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        _workspaces[key] = ws
    return ws


def _host_ptr(t: torch.Tensor, name: str, dtype: torch.dtype = torch.float64) -> int:
    if not isinstance(t, torch.Tensor) or t.is_cuda:
        raise TypeError(f"{name} must be a CPU tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous (row-major)")
    return t.data_ptr()


def ekl_tpo_inv_helmholtz_host(S, D, u, out, device="cuda:0", chunk: int = 2048,
                               workspace: torch.Tensor | None = None):
    """Inverse Helmholtz with HOST tensors in and out (pinned memory lets copies and
    kernels overlap), float64 or float32 (the dtype of ``u`` decides).  Enqueues on the current
    stream of ``device`` and returns; the result is complete once that stream has been
    synchronised."""
    lib = library()
    _declare_host(lib)
    dtype = u.dtype
    if dtype not in (torch.float64, torch.float32):
        raise TypeError("u must be float64 or float32")
    w = 8 if dtype == torch.float64 else 4
    fn = lib.ekl_tpo_inv_helmholtz_host if w == 8 else lib.ekl_tpo_inv_helmholtz_host_f32
    E, n = u.shape[0], S.shape[0]
    if tuple(S.shape) != (n, n) or tuple(u.shape[1:]) != (n, n, n) or D.shape != u.shape \
            or out.shape != u.shape:
        raise ValueError("expected S [n,n] and D,u,out [E,n,n,n]")
    dev = torch.device(device)
    if workspace is None:
        need = lib.ekl_tpo_host_workspace_bytes(n ** 3, 2, n ** 3, n * n, max(1, min(chunk, E)), w)
        workspace = host_workspace(dev, need)
    ptrs = [_host_ptr(t, nm, dtype) for t, nm in ((S, "S"), (D, "D"), (u, "u"), (out, "out"))]
    with torch.cuda.device(dev):
        st = fn(*ptrs, n, E, workspace.data_ptr(), workspace.numel(), _stream(dev))
    if st:
        raise EklTpoError(st, "ekl_tpo_inv_helmholtz_host")
    return out


def ekl_tpo_apply_host(A, B, C, u, out, device="cuda:0", chunk: int = 4096,
                       workspace: torch.Tensor | None = None):
    """Forward operator with HOST tensors in and out; see
    :func:`ekl_tpo_inv_helmholtz_host`."""
    lib = library()
    _declare_host(lib)
    dtype = u.dtype
    if dtype not in (torch.float64, torch.float32):
        raise TypeError("u must be float64 or float32")
    w = 8 if dtype == torch.float64 else 4
    fn = lib.ekl_tpo_apply_host if w == 8 else lib.ekl_tpo_apply_host_f32
    (m0, n0), (m1, n1), (m2, n2) = A.shape, B.shape, C.shape
    E = u.shape[0]
    if tuple(u.shape[1:]) != (n0, n1, n2) or tuple(out.shape) != (E, m0, m1, m2):
        raise ValueError("expected u [E,n0,n1,n2] and out [E,m0,m1,m2]")
    dev = torch.device(device)
    if workspace is None:
        need = lib.ekl_tpo_host_workspace_bytes(n0 * n1 * n2, 1, m0 * m1 * m2,
                                                m0 * n0 + m1 * n1 + m2 * n2,
                                                max(1, min(chunk, E)), w)
        workspace = host_workspace(dev, need)
    ptrs = [_host_ptr(t, nm, dtype)
            for t, nm in ((A, "A"), (B, "B"), (C, "C"), (u, "u"), (out, "out"))]
    with torch.cuda.device(dev):
        st = fn(*ptrs, n0, n1, n2, m0, m1, m2, E, workspace.data_ptr(), workspace.numel(),
                _stream(dev))
    if st:
        raise EklTpoError(st, "ekl_tpo_apply_host")
    return out


# ----------------------------------------------------------------------------- no allocation

STATIC_SCRATCH_BYTES = 32 * 1024 * 1024


def static_scratch_need(n: int, E: int) -> int:
    """Bytes of the library's fixed staging area a call with these sizes occupies."""
    r = lambda x: (x + 255) // 256 * 256
    return r(8 * n * n) + 3 * r(8 * E * n ** 3)


def ekl_tpo_inv_helmholtz_host_static(S, D, u, out, device="cuda:0"):
    """Inverse Helmholtz with HOST tensors in and out, for callers that cannot allocate
    device memory: the call is staged in a fixed array inside the library, so neither
    this wrapper nor the library allocates anything on the GPU.  The whole batch must
    fit in that array (``static_scratch_need(n, E) <= STATIC_SCRATCH_BYTES``); larger
    batches raise.  Calls share the array, so keep them on one stream."""
    lib = library()
    fn = lib.ekl_tpo_inv_helmholtz_host_static
    fn.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int, ctypes.c_longlong, ctypes.c_void_p]
    fn.restype = ctypes.c_int
    E, n = u.shape[0], S.shape[0]
    if tuple(S.shape) != (n, n) or tuple(u.shape[1:]) != (n, n, n) or D.shape != u.shape \
            or out.shape != u.shape:
        raise ValueError("expected S [n,n] and D,u,out [E,n,n,n]")
    dev = torch.device(device)
    ptrs = [_host_ptr(t, nm) for t, nm in ((S, "S"), (D, "D"), (u, "u"), (out, "out"))]
    with torch.cuda.device(dev):
        st = fn(*ptrs, n, E, _stream(dev))
    if st == 3 and static_scratch_need(n, E) > STATIC_SCRATCH_BYTES:
        raise EklTpoError(st, "ekl_tpo_inv_helmholtz_host_static: the batch needs "
                              f"{static_scratch_need(n, E)} bytes of staging, the fixed area "
                              f"holds {STATIC_SCRATCH_BYTES}")
    if st:
        raise EklTpoError(st, "ekl_tpo_inv_helmholtz_host_static")
    return out
