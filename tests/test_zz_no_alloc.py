"""The allocation-free entry point, collected last on purpose.

``ekl_tpo_inv_helmholtz_host_static`` serves callers that cannot allocate device
memory (fixed memory budgets, plug-ins that do not own the GPU heap, latency-critical
paths): it stages the call in a fixed array inside the library.  Checked here, through
the C ABI: it gives the same result as ``ekl_tpo_inv_helmholtz_host`` on two calls in
a row with different data (so nothing stale survives in the shared array), it performs
no device allocation, and it refuses batches beyond its stated maximum.
"""
import ctypes

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL64 = 1e-12


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2604_19906_b200 import build, ops
    build.build()
    assert torch.cuda.is_available()
    return {"torch": torch, "ops": ops, "dev": torch.device("cuda:0")}


def make_case(torch, n, E, seed):
    g = np.random.Generator(np.random.PCG64(seed))
    S, _ = np.linalg.qr(g.standard_normal((n, n)))
    D = g.uniform(0.1, 1.3, (E, n, n, n))
    u = g.uniform(-1, 1, (E, n, n, n))
    return [torch.from_numpy(np.ascontiguousarray(x)).pin_memory() for x in (S, D, u)]


def rel_err(torch, got, want):
    E = want.shape[0]
    num = torch.linalg.vector_norm((got - want).view(E, -1), dim=1)
    den = torch.linalg.vector_norm(want.view(E, -1), dim=1)
    return float((num / den).max())


def test_static_variant_matches_workspace_variant_twice_in_a_row(env):
    torch, ops, dev = env["torch"], env["ops"], env["dev"]
    # second call: other sizes and other data, sharing the same staging area
    for n, E, seed in ((14, 300, 1), (8, 77, 2)):
        S, D, u = make_case(torch, n, E, seed)
        want = torch.empty_like(u).pin_memory()
        ops.ekl_tpo_inv_helmholtz_host(S, D, u, want, device=dev, chunk=64)
        torch.cuda.synchronize()
        got = torch.full(u.shape, float("nan"), dtype=torch.float64).pin_memory()
        before = torch.cuda.memory_allocated(dev)
        free_before, _ = torch.cuda.mem_get_info(dev)
        ops.ekl_tpo_inv_helmholtz_host_static(S, D, u, got, device=dev)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info(dev)
        assert torch.cuda.memory_allocated(dev) == before        # nothing through torch
        if (n, E) != (14, 300):                                  # first call may load the context's lazy state
            assert free_before - free_after < (2 << 20)          # nothing through the driver either
        assert bool(torch.isfinite(got).all())
        assert rel_err(torch, got, want) <= TOL64


def test_static_variant_rejects_batches_beyond_its_maximum(env):
    torch, ops, dev = env["torch"], env["ops"], env["dev"]
    n = 14
    E_ok = 509
    assert ops.static_scratch_need(n, E_ok) <= ops.STATIC_SCRATCH_BYTES
    assert ops.static_scratch_need(n, E_ok + 1) > ops.STATIC_SCRATCH_BYTES
    S, D, u = make_case(torch, n, E_ok + 1, 3)
    out = torch.zeros_like(u)
    with pytest.raises(ops.EklTpoError, match="UNSUPPORTED"):
        ops.ekl_tpo_inv_helmholtz_host_static(S, D, u, out, device=dev)
    assert bool((out == 0).all())                                # rejected before any work
    # the largest batch that fits goes through, straight through the C symbol
    lib = ops.library()
    fn = lib.ekl_tpo_inv_helmholtz_host_static
    fn.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int, ctypes.c_longlong, ctypes.c_void_p]
    fn.restype = ctypes.c_int
    S, D, u = (t[:E_ok] if t.dim() == 4 else t for t in (S, D, u))
    D, u = D.contiguous(), u.contiguous()
    got = torch.empty_like(u)
    with torch.cuda.device(dev):
        st = fn(S.data_ptr(), D.data_ptr(), u.data_ptr(), got.data_ptr(), n, E_ok,
                torch.cuda.current_stream(dev).cuda_stream)
    torch.cuda.synchronize()
    assert st == 0
    want = torch.empty_like(u)
    ops.ekl_tpo_inv_helmholtz_host(S, D, u, want, device=dev, chunk=128)
    torch.cuda.synchronize()
    assert rel_err(torch, got, want) <= TOL64
    # E == 0 and bad extents behave like the other entry points
    with torch.cuda.device(dev):
        assert fn(None, None, None, None, n, 0, None) == 0
        assert fn(S.data_ptr(), D.data_ptr(), u.data_ptr(), got.data_ptr(), 0, 5, None) == 2


def test_static_variant_against_the_oracle_odd_and_large_extents_in_place_and_queued(env):
    """Directly against the CPU oracle (not only against the workspace variant): an odd extent,
    an extent that takes the general kernel, v == u on pinned memory, and two calls of
    different sizes queued on one stream with a single synchronise, which is the documented
    way to share the staging area."""
    import oracle
    torch, ops, dev = env["torch"], env["ops"], env["dev"]
    cases = []
    for n, E, seed in ((5, 41, 11), (22, 9, 12), (14, 65, 13), (3, 7, 14)):
        S, D, u = make_case(torch, n, E, seed)
        want = oracle.inv_helmholtz(S.numpy(), D.numpy(), u.numpy())
        cases.append((S, D, u, want))
    # queued back to back, one synchronise at the end
    outs = [torch.full(c[2].shape, float("nan"), dtype=torch.float64).pin_memory() for c in cases]
    for (S, D, u, _), out in zip(cases, outs):
        ops.ekl_tpo_inv_helmholtz_host_static(S, D, u, out, device=dev)
    torch.cuda.synchronize()
    for (S, D, u, want), out in zip(cases, outs):
        assert oracle.rel_err_per_element(out.numpy(), want).max() <= TOL64
    # in place: v == u
    S, D, u, want = cases[0]
    inplace = u.clone().pin_memory()
    ops.ekl_tpo_inv_helmholtz_host_static(S, D, inplace, inplace, device=dev)
    torch.cuda.synchronize()
    assert np.array_equal(inplace.numpy(), outs[0].numpy())
    # the status code cannot see a device-side wait that gave up; the flags can
    assert ops.library().ekl_tpo_device_error_flags() == 0
