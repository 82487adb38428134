"""Host-buffer entry points (chunked copy-in | compute | copy-out pipeline) against the
device-pointer entry points and the oracle."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    import oracle
    from paper_2604_19906_b200 import build, inputs, ops
    build.build()
    return {"torch": torch, "oracle": oracle, "inputs": inputs, "ops": ops,
            "dev": torch.device("cuda:0")}


@pytest.mark.parametrize("n,E,chunk,pinned", [(4, 64, 7, True), (8, 1000, 128, True),
                                              (14, 333, 50, True), (14, 97, 1000, False),
                                              (5, 31, 1, True)])
def test_inv_helmholtz_host_matches_oracle_and_device_path(env, n, E, chunk, pinned):
    torch, ops, oracle = env["torch"], env["ops"], env["oracle"]
    g = np.random.Generator(np.random.PCG64(n * 100 + E))
    S, _ = np.linalg.qr(g.standard_normal((n, n)))
    D = g.uniform(0.1, 1.3, (E, n, n, n))
    u = g.uniform(-1, 1, (E, n, n, n))
    want = oracle.inv_helmholtz(S, D, u)

    def host(a):
        t = torch.from_numpy(np.ascontiguousarray(a))
        return t.pin_memory() if pinned else t

    hS, hD, hu = host(S), host(D), host(u)
    out = torch.full((E, n, n, n), float("nan"), dtype=torch.float64)
    out = out.pin_memory() if pinned else out
    for _ in range(2):                                  # second call reuses the workspace
        ops.ekl_tpo_inv_helmholtz_host(hS, hD, hu, out, device=env["dev"], chunk=chunk)
        torch.cuda.synchronize()
        assert oracle.rel_err_per_element(out.numpy(), want).max() <= 1e-12
    dev_out = ops.ekl_tpo_inv_helmholtz(hS.to(env["dev"]), hD.to(env["dev"]), hu.to(env["dev"]))
    assert np.array_equal(dev_out.cpu().numpy(), out.numpy())
    # in place on the host: v == u
    inplace = hu.clone()
    inplace = inplace.pin_memory() if pinned else inplace
    ops.ekl_tpo_inv_helmholtz_host(hS, hD, inplace, inplace, device=env["dev"], chunk=chunk)
    torch.cuda.synchronize()
    assert np.array_equal(inplace.numpy(), out.numpy())


def test_apply_host_matches_oracle(env):
    torch, ops, oracle = env["torch"], env["ops"], env["oracle"]
    g = np.random.Generator(np.random.PCG64(5))
    nn, mm, E = (8, 8, 8), (12, 12, 12), 301
    A, B, C = (g.standard_normal((mm[d], nn[d])) / np.sqrt(8.0) for d in range(3))
    u = g.uniform(-1, 1, (E,) + nn)
    want = oracle.tpo_apply(A, B, C, u)
    h = [torch.from_numpy(np.ascontiguousarray(x)).pin_memory() for x in (A, B, C, u)]
    out = torch.full((E,) + mm, float("nan"), dtype=torch.float64).pin_memory()
    ops.ekl_tpo_apply_host(*h, out, device=env["dev"], chunk=64)
    torch.cuda.synchronize()
    assert oracle.rel_err_per_element(out.numpy(), want).max() <= 1e-12


@pytest.mark.parametrize("n,E,chunk", [(14, 203, 40), (7, 100, 13), (22, 5, 2)])
def test_host_variants_in_single_precision(env, n, E, chunk):
    torch, ops, oracle = env["torch"], env["ops"], env["oracle"]
    g = np.random.Generator(np.random.PCG64(900 + n))
    S = np.linalg.qr(g.standard_normal((n, n)))[0].astype(np.float32)
    D = g.uniform(0.1, 1.3, (E, n, n, n)).astype(np.float32)
    u = g.uniform(-1, 1, (E, n, n, n)).astype(np.float32)
    want = oracle.inv_helmholtz(S, D, u)                  # the oracle widens and works in fp64
    h = [torch.from_numpy(np.ascontiguousarray(x)).pin_memory() for x in (S, D, u)]
    out = torch.full((E, n, n, n), float("nan"), dtype=torch.float32).pin_memory()
    ops.ekl_tpo_inv_helmholtz_host(*h, out, device=env["dev"], chunk=chunk)
    torch.cuda.synchronize()
    assert oracle.rel_err_per_element(out.numpy(), want).max() <= 1e-5
    nn, mm = (8, 8, 8), (12, 12, 12)
    A, B, C = (g.standard_normal((mm[d], nn[d])).astype(np.float32) / np.float32(np.sqrt(8.0))
               for d in range(3))
    ua = g.uniform(-1, 1, (E,) + nn).astype(np.float32)
    wanta = oracle.tpo_apply(A, B, C, ua)
    ha = [torch.from_numpy(np.ascontiguousarray(x)).pin_memory() for x in (A, B, C, ua)]
    outa = torch.full((E,) + mm, float("nan"), dtype=torch.float32).pin_memory()
    ops.ekl_tpo_apply_host(*ha, outa, device=env["dev"], chunk=chunk)
    torch.cuda.synchronize()
    assert oracle.rel_err_per_element(outa.numpy(), wanta).max() <= 1e-5


def test_host_workspace_rules(env):
    torch, ops = env["torch"], env["ops"]
    lib = ops.library()
    ops._declare_host(lib)
    n, E = 6, 10
    need1 = lib.ekl_tpo_host_workspace_bytes(n ** 3, 2, n ** 3, n * n, 1, 8)
    assert need1 > 0 and lib.ekl_tpo_host_workspace_bytes(0, 2, 1, 1, 1, 8) == 0
    S = torch.eye(n, dtype=torch.float64)
    x = torch.ones(E, n, n, n, dtype=torch.float64)
    out = torch.empty_like(x)
    tiny = torch.empty(1024, dtype=torch.uint8, device=env["dev"])
    with pytest.raises(ops.EklTpoError, match="UNSUPPORTED"):
        ops.ekl_tpo_inv_helmholtz_host(S, x, x.clone(), out, device=env["dev"], workspace=tiny)
    ws = torch.empty(need1 + 256, dtype=torch.uint8, device=env["dev"])
    with pytest.raises(ops.EklTpoError, match="ALIGN"):
        ops.ekl_tpo_inv_helmholtz_host(S, x, x.clone(), out, device=env["dev"], workspace=ws[8:])
    ops.ekl_tpo_inv_helmholtz_host(S, x, x.clone(), out, device=env["dev"], workspace=ws[:need1])
    torch.cuda.synchronize()
    assert bool((out == 1.0).all())                      # S = I, D = 1, u = 1
