"""Inverse Helmholtz with the factor formed on the fly from lam[n] and c[E]."""
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


@pytest.mark.parametrize("n", list(range(4, 21)))
@pytest.mark.parametrize("E", [1, 3, 130, 1501])
def test_lambda_variant_matches_oracle_and_field_variant(env, n, E):
    if n > 16 and E > 130:
        E = 301
    torch, ops = env["torch"], env["ops"]
    g = np.random.Generator(np.random.PCG64(31 * n + E))
    S, _ = np.linalg.qr(g.standard_normal((n, n)))
    lam = g.uniform(0.1, 2.0, n)
    c = g.uniform(0.5, 1.5, E)
    u = g.uniform(-1, 1, (E, n, n, n))
    want = env["oracle"].inv_helmholtz_lambda(S, lam, c, u)
    d = [torch.from_numpy(np.ascontiguousarray(x)).to(env["dev"]) for x in (S, lam, c, u)]
    got = ops.ekl_tpo_inv_helmholtz_lambda(*d)
    torch.cuda.synchronize()
    assert env["oracle"].rel_err_per_element(got.cpu().numpy(), want).max() <= 1e-12
    # same arithmetic as the stored-factor entry point on the materialised factor
    Dd = torch.from_numpy(env["oracle"].lambda_factor(lam, c)).to(env["dev"])
    ref = ops.ekl_tpo_inv_helmholtz(d[0], Dd, d[3])
    assert torch.equal(got, ref)
    inplace = d[3].clone()
    ops.ekl_tpo_inv_helmholtz_lambda(d[0], d[1], d[2], inplace, out=inplace)
    assert torch.equal(inplace, got)


def test_lambda_variant_refuses_what_it_cannot_do(env):
    torch, ops = env["torch"], env["ops"]
    dev = env["dev"]
    for n in (3, 21):
        S = torch.eye(n, dtype=torch.float64, device=dev)
        lam = torch.ones(n, dtype=torch.float64, device=dev)
        c = torch.ones(2, dtype=torch.float64, device=dev)
        u = torch.ones(2, n, n, n, dtype=torch.float64, device=dev)
        with pytest.raises(ops.EklTpoError, match="UNSUPPORTED"):
            ops.ekl_tpo_inv_helmholtz_lambda(S, lam, c, u)
    n = 8
    buf = torch.zeros(2 * n ** 3 + 1, dtype=torch.float64, device=dev)
    with pytest.raises(ops.EklTpoError, match="ALIGN"):
        ops.ekl_tpo_inv_helmholtz_lambda(torch.eye(n, dtype=torch.float64, device=dev),
                                         torch.ones(n, dtype=torch.float64, device=dev),
                                         torch.ones(2, dtype=torch.float64, device=dev),
                                         buf[1:].view(2, n, n, n))
