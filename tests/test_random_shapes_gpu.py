"""Seeded random shapes through both operators: every accepted extent combination must agree
with the oracle, whichever kernel the library picks for it."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    import oracle
    from paper_2604_19906_b200 import build, ops
    build.build()
    return {"torch": torch, "oracle": oracle, "ops": ops, "dev": torch.device("cuda:0")}


def dev_of(env, a):
    return env["torch"].from_numpy(np.ascontiguousarray(a)).to(env["dev"])


def test_forward_operator_random_rectangular_shapes(env):
    g = np.random.Generator(np.random.PCG64(20260419))
    for trial in range(60):
        nn = tuple(int(x) for x in g.integers(1, 17, size=3))
        mm = tuple(int(x) for x in g.integers(1, 17, size=3))
        if trial % 5 == 0:                       # cubic even shapes take the tensor path
            n, m = int(g.choice([4, 6, 8, 10, 12, 14, 16])), int(g.choice([4, 6, 8, 10, 12, 14, 16]))
            nn, mm = (n, n, n), (m, m, m)
        E = int(g.integers(1, 70))
        A, B, C = (g.standard_normal((mm[d], nn[d])) / np.sqrt(nn[d]) for d in range(3))
        u = g.uniform(-1, 1, (E,) + nn)
        want = env["oracle"].tpo_apply(A, B, C, u)
        got = env["ops"].ekl_tpo_apply(*(dev_of(env, x) for x in (A, B, C, u)))
        err = env["oracle"].rel_err_per_element(got.cpu().numpy(), want)
        assert err.max() <= 1e-12, (nn, mm, E, err.max())


def test_inverse_helmholtz_random_sizes_and_dtypes(env):
    torch = env["torch"]
    g = np.random.Generator(np.random.PCG64(19906))
    for trial in range(40):
        n = int(g.integers(1, 21))
        E = int(g.integers(1, 400))
        S = g.standard_normal((n, n)) / np.sqrt(n)          # not orthogonal, not symmetric
        D = g.uniform(0.1, 1.3, (E, n, n, n))
        u = g.uniform(-1, 1, (E, n, n, n))
        if trial % 2:
            S32, D32, u32 = (x.astype(np.float32) for x in (S, D, u))
            want = env["oracle"].inv_helmholtz(S32, D32, u32)
            got = env["ops"].ekl_tpo_inv_helmholtz_f32(dev_of(env, S32), dev_of(env, D32),
                                                       dev_of(env, u32))
            err = env["oracle"].rel_err_per_element(got.cpu().numpy().astype(np.float64), want)
            assert err.max() <= 1e-5, (n, E, "f32", err.max())
        else:
            want = env["oracle"].inv_helmholtz(S, D, u)
            got = env["ops"].ekl_tpo_inv_helmholtz(dev_of(env, S), dev_of(env, D), dev_of(env, u))
            err = env["oracle"].rel_err_per_element(got.cpu().numpy(), want)
            assert err.max() <= 1e-12, (n, E, "f64", err.max())
    torch.cuda.synchronize()
