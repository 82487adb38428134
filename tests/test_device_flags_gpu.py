"""The only failure the device code can meet is a bulk copy that never completes; every wait
on one has a time budget, after which the kernel raises a flag and returns.  This test makes a
wait run out (a barrier armed for bytes that nothing sends) and reads the flag."""
import ctypes
import time

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_expired_wait_sets_the_flag_once_and_leaves_the_context_usable():
    import torch
    import oracle
    from paper_2604_19906_b200 import build, ops
    build.build()
    lib = ops.library()
    lib.ekl_tpo_selftest_expired_wait.argtypes = [ctypes.c_void_p]
    lib.ekl_tpo_selftest_expired_wait.restype = ctypes.c_int
    lib.ekl_tpo_device_error_flags.restype = ctypes.c_int
    dev = torch.device("cuda:0")
    torch.cuda.synchronize(dev)
    assert lib.ekl_tpo_device_error_flags() == 0
    t0 = time.perf_counter()
    assert lib.ekl_tpo_selftest_expired_wait(None) == 0
    assert lib.ekl_tpo_device_error_flags() == 1          # synchronises: the wait has run out
    dt = time.perf_counter() - t0
    assert 1.0 < dt < 10.0, dt                             # a short limit, not minutes
    assert lib.ekl_tpo_device_error_flags() == 0          # read once, then clear
    # the context still works
    g = np.random.Generator(np.random.PCG64(3))
    n, E = 6, 11
    S = np.linalg.qr(g.standard_normal((n, n)))[0]
    D = g.uniform(0.2, 1.2, (E, n, n, n))
    u = g.uniform(-1, 1, (E, n, n, n))
    got = ops.ekl_tpo_inv_helmholtz(*[torch.from_numpy(np.ascontiguousarray(x)).to(dev)
                                      for x in (S, D, u)])
    assert oracle.rel_err_per_element(got.cpu().numpy(), oracle.inv_helmholtz(S, D, u)).max() <= 1e-12
    assert lib.ekl_tpo_device_error_flags() == 0
