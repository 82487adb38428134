"""Convective-flux volume integral (Eq. 1) on the GPU against the oracle."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL64 = 1e-12
PAIRS = [(4, 4), (6, 4), (6, 6), (8, 4), (8, 6), (8, 8), (10, 8), (10, 10), (12, 8), (12, 10),
         (12, 12), (14, 12)]
# tensor-path instances with an odd extent (odd nq: no bulk copies; odd nv: unpaired stores)
ODD_PAIRS = [(5, 5), (7, 5), (7, 7), (8, 5), (9, 6), (9, 7), (9, 9), (11, 7), (14, 9), (15, 10)]


@pytest.fixture(scope="module")
def env():
    import torch
    import oracle
    from paper_2604_19906_b200 import build, ops
    build.build()
    return {"torch": torch, "oracle": oracle, "ops": ops, "dev": torch.device("cuda:0")}


def case(nq, nv, E, seed):
    g = np.random.Generator(np.random.PCG64(seed))
    Dvq = g.standard_normal((nv, nq)) / np.sqrt(nq)
    Ivq = g.standard_normal((nv, nq)) / np.sqrt(nq)
    M = g.uniform(0.5, 1.5, (E, nq, nq, nq))
    P = g.uniform(-1, 1, (3, 3, E, nq, nq, nq))
    return Dvq, Ivq, M, P


@pytest.mark.parametrize("nq,nv", ODD_PAIRS)
@pytest.mark.parametrize("E", [1, 2, 5, 311, 1301])
def test_convection_odd_extents_match_oracle(env, nq, nv, E):
    """E = 1301 gives every CTA more than four elements (the dynamic deal); for an odd nq the
    fields M and P also start 8 bytes off a 16-byte boundary."""
    torch = env["torch"]
    Dvq, Ivq, M, P = case(nq, nv, E, 100 * nq + nv + E)
    want = env["oracle"].convection(Dvq, Ivq, M, P)
    dev = [torch.from_numpy(np.ascontiguousarray(x)).to(env["dev"]) for x in (Dvq, Ivq, M, P)]
    if nq % 2 == 1:
        for i in (2, 3):
            buf = torch.zeros(dev[i].numel() + 1, dtype=torch.float64, device=env["dev"])
            shifted = buf[1:].view(dev[i].shape)
            shifted.copy_(dev[i])
            dev[i] = shifted
    got = env["ops"].ekl_tpo_convection(*dev)
    torch.cuda.synchronize()
    err = env["oracle"].rel_err_per_element(got.cpu().numpy().reshape(3 * E, nv, nv, nv),
                                            want.reshape(3 * E, nv, nv, nv))
    assert err.max() <= TOL64, (nq, nv, E, err.max())
    assert env["ops"].library().ekl_tpo_device_error_flags() == 0


@pytest.mark.parametrize("nq,nv", PAIRS)
@pytest.mark.parametrize("E", [1, 2, 5, 311])
def test_convection_matches_oracle(env, nq, nv, E):
    torch = env["torch"]
    Dvq, Ivq, M, P = case(nq, nv, E, 100 * nq + nv + E)
    want = env["oracle"].convection(Dvq, Ivq, M, P)
    dev = [torch.from_numpy(np.ascontiguousarray(x)).to(env["dev"]) for x in (Dvq, Ivq, M, P)]
    got = env["ops"].ekl_tpo_convection(*dev)
    torch.cuda.synchronize()
    err = env["oracle"].rel_err_per_element(got.cpu().numpy().reshape(3 * E, nv, nv, nv),
                                            want.reshape(3 * E, nv, nv, nv))
    assert err.max() <= TOL64, (nq, nv, E, err.max())


def test_convection_repeatable_guards_and_errors(env):
    torch, ops = env["torch"], env["ops"]
    nq, nv, E = 12, 8, 700
    Dvq, Ivq, M, P = case(nq, nv, E, 5)
    dev = [torch.from_numpy(np.ascontiguousarray(x)).to(env["dev"]) for x in (Dvq, Ivq, M, P)]
    pad = 256
    big = torch.full((3 * E * nv ** 3 + 2 * pad,), float("nan"), dtype=torch.float64,
                     device=env["dev"])
    big[:pad] = 7.0
    big[-pad:] = 9.0
    out = big[pad:-pad].view(3, E, nv, nv, nv)
    ops.ekl_tpo_convection(*dev, out=out)
    first = out.clone()
    out.fill_(float("nan"))
    ops.ekl_tpo_convection(*dev, out=out)
    assert torch.equal(first, out) and not bool(torch.isnan(out).any())
    assert bool((big[:pad] == 7.0).all()) and bool((big[-pad:] == 9.0).all())
    want = env["oracle"].convection(Dvq, Ivq, M, P)
    err = env["oracle"].rel_err_per_element(out.cpu().numpy().reshape(3 * E, nv, nv, nv),
                                            want.reshape(3 * E, nv, nv, nv))
    assert err.max() <= TOL64
    # extents beyond shared memory are refused before anything runs
    D5 = torch.zeros(40, 40, dtype=torch.float64, device=env["dev"])
    M7 = torch.zeros(1, 40, 40, 40, dtype=torch.float64, device=env["dev"])
    P7 = torch.zeros(3, 3, 1, 40, 40, 40, dtype=torch.float64, device=env["dev"])
    with pytest.raises(ops.EklTpoError, match="UNSUPPORTED"):
        ops.ekl_tpo_convection(D5, D5.clone(), M7, P7)
    # M only 8-byte aligned: the general kernel takes over, same result
    buf = torch.zeros(E * nq ** 3 + 1, dtype=torch.float64, device=env["dev"])
    M8 = buf[1:].view(E, nq, nq, nq)
    M8.copy_(dev[2])
    got8 = ops.ekl_tpo_convection(dev[0], dev[1], M8, dev[3])
    err = env["oracle"].rel_err_per_element(got8.cpu().numpy().reshape(3 * E, nv, nv, nv),
                                            want.reshape(3 * E, nv, nv, nv))
    assert err.max() <= TOL64
    lib = ops.library()
    assert lib.ekl_tpo_device_error_flags() == 0


@pytest.mark.parametrize("nq,nv", [(3, 2), (5, 7), (6, 5), (11, 11), (13, 8), (16, 12), (2, 1), (1, 1)])
@pytest.mark.parametrize("E", [1, 4, 97])
def test_convection_general_kernel_shapes(env, nq, nv, E):
    """Extents without a tensor-path instance run on the run-time-sized kernel."""
    torch = env["torch"]
    Dvq, Ivq, M, P = case(nq, nv, E, 7 * nq + nv + E)
    want = env["oracle"].convection(Dvq, Ivq, M, P)
    dev = [torch.from_numpy(np.ascontiguousarray(x)).to(env["dev"]) for x in (Dvq, Ivq, M, P)]
    got = env["ops"].ekl_tpo_convection(*dev)
    torch.cuda.synchronize()
    err = env["oracle"].rel_err_per_element(got.cpu().numpy().reshape(3 * E, nv, nv, nv),
                                            want.reshape(3 * E, nv, nv, nv))
    assert err.max() <= TOL64, (nq, nv, E, err.max())


def test_convection_workload_full_size_sampled(env):
    """The benchmark's convection workload (nq = 12, nv = 8, E = 8192) generated on the
    device, every element computed, the oracle recomputing runs at both ends and the middle."""
    torch = env["torch"]
    from paper_2604_19906_b200 import inputs
    wl = inputs.CONFIGS[5]
    case_d = inputs.device_case(wl, env["dev"])
    got = env["ops"].ekl_tpo_convection(case_d["Dvq"], case_d["Ivq"], case_d["M"], case_d["P"])
    torch.cuda.synchronize()
    assert bool(torch.isfinite(got).all())
    E, nv = wl.E, wl.m[0]
    for e0, e1 in ((0, 64), (E // 2 - 30, E // 2 + 41), (E - 50, E)):
        h = inputs.host_case(wl, e0, e1)
        want = env["oracle"].convection(h["Dvq"], h["Ivq"], h["M"], h["P"])
        g = got[:, e0:e1].cpu().numpy()
        err = env["oracle"].rel_err_per_element(g.reshape(-1, nv, nv, nv), want.reshape(-1, nv, nv, nv))
        assert err.max() <= TOL64, (e0, err.max())
