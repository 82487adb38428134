"""Inverse Helmholtz with one operator and one extent per direction: the CUDA library through
its C ABI against the oracle (``oracle.inv_helmholtz3``), bar 1e-12 per element."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL64 = 1e-12
# shapes with a tensor-path instance, then shapes that take the general kernel
TENSOR_SHAPES = [(4, 4, 4), (6, 6, 6), (8, 8, 8), (10, 10, 10), (12, 12, 12), (14, 14, 14),
                 (16, 16, 16), (8, 10, 12), (12, 10, 8), (14, 12, 8), (8, 8, 16), (16, 8, 8),
                 # with an odd extent: u comes in by 8-byte copies where a plane is odd
                 (5, 5, 5), (7, 7, 7), (9, 9, 9), (11, 11, 11), (13, 13, 13), (15, 15, 15),
                 (5, 7, 9), (9, 7, 5), (6, 7, 8), (7, 8, 9)]
GENERAL_SHAPES = [(1, 1, 1), (2, 3, 4), (5, 4, 3), (7, 7, 5), (6, 8, 10), (9, 2, 11),
                  (13, 14, 15), (18, 4, 4), (1, 16, 3)]


@pytest.fixture(scope="module")
def env():
    import torch
    import oracle
    from paper_2604_19906_b200 import build, ops
    build.build()
    return {"torch": torch, "oracle": oracle, "ops": ops, "dev": torch.device("cuda:0")}


def synth(nn, E, seed, orthogonal=True):
    g = np.random.Generator(np.random.PCG64(seed))
    if orthogonal:
        S = [np.linalg.qr(g.standard_normal((n, n)))[0] for n in nn]
    else:
        S = [g.standard_normal((n, n)) / np.sqrt(n) for n in nn]
    D = g.uniform(0.13, 1.25, (E,) + tuple(nn))
    u = g.uniform(-1, 1, (E,) + tuple(nn))
    return [np.ascontiguousarray(x) for x in S], D, u


def dev(env, a):
    return env["torch"].from_numpy(np.ascontiguousarray(a)).to(env["dev"])


@pytest.mark.parametrize("nn", TENSOR_SHAPES + GENERAL_SHAPES)
@pytest.mark.parametrize("E", [1, 2, 3, 37, 603])
def test_matches_oracle(env, nn, E):
    if E == 603 and np.prod(nn) > 3000:
        E = 301
    S, D, u = synth(nn, E, 7000 + 100 * nn[0] + 10 * nn[1] + nn[2] + E, orthogonal=(E != 37))
    want = env["oracle"].inv_helmholtz3(*S, D, u)
    v = env["torch"].full(u.shape, float("nan"), dtype=env["torch"].float64, device=env["dev"])
    got = env["ops"].ekl_tpo_inv_helmholtz3(*[dev(env, s) for s in S], dev(env, D), dev(env, u), out=v)
    env["torch"].cuda.synchronize()
    err = env["oracle"].rel_err_per_element(got.cpu().numpy(), want)
    assert err.max() <= TOL64, (nn, E, err.max())


@pytest.mark.parametrize("nn", [(14, 14, 14), (8, 10, 12), (16, 8, 8), (5, 4, 3), (9, 9, 9), (5, 7, 9),
                                (6, 7, 8)])
def test_many_batches_per_cta_in_place_and_repeatable(env, nn):
    """Enough elements that every CTA draws several batches; in place; bitwise repeatable."""
    torch = env["torch"]
    E = 5003
    S, D, u = synth(nn, E, 99 + sum(nn))
    want = env["oracle"].inv_helmholtz3(*S, D, u)
    Sd = [dev(env, s) for s in S]
    Dd, ud = dev(env, D), dev(env, u)
    a = env["ops"].ekl_tpo_inv_helmholtz3(*Sd, Dd, ud)
    b = env["ops"].ekl_tpo_inv_helmholtz3(*Sd, Dd, ud)
    inplace = ud.clone()
    env["ops"].ekl_tpo_inv_helmholtz3(*Sd, Dd, inplace, out=inplace)
    torch.cuda.synchronize()
    assert env["oracle"].rel_err_per_element(a.cpu().numpy(), want).max() <= TOL64
    assert torch.equal(a, b) and torch.equal(a, inplace)
    if (nn[1] * nn[2]) % 2 == 1:
        # odd planes: u may start 8 bytes off a 16-byte boundary and still take the same kernel
        buf = torch.zeros(ud.numel() + 1, dtype=torch.float64, device=env["dev"])
        shifted = buf[1:].view(ud.shape)
        shifted.copy_(ud)
        c = env["ops"].ekl_tpo_inv_helmholtz3(*Sd, Dd, shifted)
        assert torch.equal(a, c)
    assert env["ops"].library().ekl_tpo_device_error_flags() == 0


@pytest.mark.parametrize("nn", [(12, 12, 12), (14, 12, 8), (6, 8, 10)])
def test_exact_special_cases(env, nn):
    torch = env["torch"]
    E = 41
    _, D, u = synth(nn, E, 5)
    eyes = [dev(env, np.eye(n)) for n in nn]
    got = env["ops"].ekl_tpo_inv_helmholtz3(*eyes, dev(env, D), dev(env, u))
    assert torch.equal(got, dev(env, D * u))                    # identities: bit for bit
    # one shared operator: the single-operator entry point, to rounding
    if nn[0] == nn[1] == nn[2]:
        S, D, u = synth(nn, E, 6, orthogonal=False)
        a = env["ops"].ekl_tpo_inv_helmholtz3(dev(env, S[0]), dev(env, S[0]), dev(env, S[0]),
                                              dev(env, D), dev(env, u))
        want = env["oracle"].inv_helmholtz(S[0], D, u)
        assert env["oracle"].rel_err_per_element(a.cpu().numpy(), want).max() <= TOL64


def test_argument_validation(env):
    torch, ops = env["torch"], env["ops"]
    lib = ops.library()
    import ctypes
    fn = lib.ekl_tpo_inv_helmholtz3
    fn.argtypes = [ctypes.c_void_p] * 6 + [ctypes.c_int] * 3 + [ctypes.c_longlong, ctypes.c_void_p]
    fn.restype = ctypes.c_int
    n = 4
    S = torch.eye(n, dtype=torch.float64, device=env["dev"])
    f = torch.ones(2 * n ** 3 + 1, dtype=torch.float64, device=env["dev"])
    o = torch.empty(2 * n ** 3 + 1, dtype=torch.float64, device=env["dev"])
    p = lambda t: t.data_ptr()
    assert fn(p(S), p(S), p(S), p(f), p(f), p(o), n, n, n, 0, None) == 0          # E = 0
    assert fn(p(S), p(S), p(S), p(f), p(f), p(o), n, 0, n, 2, None) == 2          # extent < 1
    assert fn(p(S), p(S), p(S), p(f), p(f), p(o), n, n, n, -1, None) == 2         # E < 0
    assert fn(p(S), None, p(S), p(f), p(f), p(o), n, n, n, 2, None) == 1          # null
    assert fn(p(S), p(S), p(S), p(f), p(f), p(o), 40, 40, 40, 2, None) == 3       # too large
    assert fn(p(S), p(S), p(S), p(f), p(f), p(o) + 4, n, n, n, 2, None) == 4      # misaligned
    assert fn(p(S), p(S), p(S), p(f), p(f), p(f) + 8, n, n, n, 2, None) == 5      # partial overlap
    assert fn(p(S), p(S), p(S), p(f), p(o), p(f), n, n, n, 2, None) == 5          # v on D
    torch.cuda.synchronize()
