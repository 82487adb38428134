"""Fields with more than 2^31 values: the kernels' index arithmetic has to be 64-bit.

Elements at both ends and on both sides of the 2^31-value mark are recomputed by the oracle
(the fields are generated on the device; only the sampled elements travel to the host)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL64 = 1e-12
TOL32 = 1e-5


@pytest.fixture(scope="module")
def env():
    import torch
    import oracle
    from paper_2604_19906_b200 import build, ops
    build.build()
    dev = torch.device("cuda:0")
    free, _ = torch.cuda.mem_get_info(dev)
    if free < 80 * 2 ** 30:
        pytest.skip("needs about 60 GB of device memory")
    return {"torch": torch, "oracle": oracle, "ops": ops, "dev": dev}


def sample_ranges(E, per_element):
    """Element index ranges: the first and last elements and those around value 2^31."""
    mark = 2 ** 31 // per_element
    assert 8 < mark < E - 8
    return [(0, 5), (mark - 3, mark + 4), (E - 5, E)]


@pytest.mark.parametrize("n", [8, 3, 5])
def test_inverse_helmholtz_beyond_2_to_31_values(env, n):
    """n = 8: tensor path with bulk copies; n = 5: tensor path with 8-byte copies; n = 3: the
    general kernel."""
    torch, dev = env["torch"], env["dev"]
    E = (2 ** 31 + 2 ** 27) // n ** 3
    g = torch.Generator(device=dev)
    g.manual_seed(1234 + n)
    S = torch.linalg.qr(torch.randn(n, n, dtype=torch.float64))[0].contiguous().to(dev)
    u = torch.rand(E, n, n, n, dtype=torch.float64, device=dev, generator=g) * 2 - 1
    D = torch.rand(E, n, n, n, dtype=torch.float64, device=dev, generator=g) + 0.13
    assert u.numel() > 2 ** 31
    v = env["ops"].ekl_tpo_inv_helmholtz(S, D, u)
    torch.cuda.synchronize()
    for a, b in sample_ranges(E, n ** 3):
        want = env["oracle"].inv_helmholtz(S.cpu().numpy(), D[a:b].cpu().numpy(), u[a:b].cpu().numpy())
        err = env["oracle"].rel_err_per_element(v[a:b].cpu().numpy(), want)
        assert err.max() <= TOL64, (n, a, b, err.max())
    # nothing is left unwritten anywhere in between
    assert bool(torch.isfinite(v).all())
    assert env["ops"].library().ekl_tpo_device_error_flags() == 0
    del u, D, v
    torch.cuda.empty_cache()


def test_forward_f32_beyond_2_to_31_values(env):
    """4^3 -> 6^3 with fp32 fields: the output field passes 2^31 values."""
    torch, dev = env["torch"], env["dev"]
    n, m = 4, 6
    E = (2 ** 31 + 2 ** 27) // m ** 3
    g = torch.Generator(device=dev)
    g.manual_seed(77)
    A, B, C = (torch.randn(m, n, dtype=torch.float32, device=dev, generator=g) / 2 for _ in range(3))
    u = torch.rand(E, n, n, n, dtype=torch.float32, device=dev, generator=g) * 2 - 1
    v = env["ops"].ekl_tpo_apply_f32(A, B, C, u)
    torch.cuda.synchronize()
    assert v.numel() > 2 ** 31
    for a, b in sample_ranges(E, m ** 3):
        want = env["oracle"].tpo_apply(A.cpu().numpy(), B.cpu().numpy(), C.cpu().numpy(),
                                       u[a:b].cpu().numpy())
        err = env["oracle"].rel_err_per_element(v[a:b].cpu().numpy().astype(np.float64), want)
        assert err.max() <= TOL32, (a, b, err.max())
    assert bool(torch.isfinite(v).all())
    del u, v
    torch.cuda.empty_cache()


def test_convection_beyond_2_to_31_values(env):
    """nq = 6 -> nv = 4: the flux array P[3,3,E,nq^3] passes 2^31 values."""
    torch, dev = env["torch"], env["dev"]
    nq, nv = 6, 4
    E = (2 ** 31 + 2 ** 27) // (9 * nq ** 3)
    g = torch.Generator(device=dev)
    g.manual_seed(5)
    Dvq, Ivq = (torch.randn(nv, nq, dtype=torch.float64, device=dev, generator=g) / 2 for _ in range(2))
    M = torch.rand(E, nq, nq, nq, dtype=torch.float64, device=dev, generator=g) + 0.5
    P = torch.rand(3, 3, E, nq, nq, nq, dtype=torch.float64, device=dev, generator=g) * 2 - 1
    assert P.numel() > 2 ** 31
    F = env["ops"].ekl_tpo_convection(Dvq, Ivq, M, P)
    torch.cuda.synchronize()
    for a, b in [(0, 4), (E // 2 - 2, E // 2 + 2), (E - 4, E)]:
        want = env["oracle"].convection(Dvq.cpu().numpy(), Ivq.cpu().numpy(), M[a:b].cpu().numpy(),
                                        np.ascontiguousarray(P[:, :, a:b].cpu().numpy()))
        got = F[:, a:b].cpu().numpy()
        err = env["oracle"].rel_err_per_element(got.reshape(-1, nv, nv, nv),
                                                want.reshape(-1, nv, nv, nv))
        assert err.max() <= TOL64, (a, b, err.max())
    assert bool(torch.isfinite(F).all())
    del M, P, F
    torch.cuda.empty_cache()
