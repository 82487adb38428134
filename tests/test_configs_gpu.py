"""The five benchmark configurations at full size, in the launch configuration the
benchmark times, against the oracle.

Configurations 0 and 1 are compared element by element.  Configurations 2-4 hold
gigabytes: their inputs are generated on the device, the operator runs over all E
elements, and the oracle recomputes a sample -- the first and last elements, a
contiguous run across several CTA batches, and seeded random picks -- from inputs
regenerated on the host (bit-identical by construction of the counter stream).
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL64 = 1e-12


@pytest.fixture(scope="module")
def env():
    import torch
    import oracle
    from paper_2604_19906_b200 import build, inputs, ops
    build.build()
    return {"torch": torch, "oracle": oracle, "inputs": inputs, "ops": ops,
            "dev": torch.device("cuda:0")}


def run_config(env, wl, case):
    ops = env["ops"]
    if wl.op == "inv_helmholtz":
        return ops.ekl_tpo_inv_helmholtz(case["S"], case["D"], case["u"])
    return ops.ekl_tpo_apply(case["A"], case["B"], case["C"], case["u"])


def oracle_config(env, wl, host):
    if wl.op == "inv_helmholtz":
        return env["oracle"].inv_helmholtz(host["S"], host["D"], host["u"])
    return env["oracle"].tpo_apply(host["A"], host["B"], host["C"], host["u"])


@pytest.mark.parametrize("idx", [0, 1])
def test_small_configs_every_element(env, idx):
    wl = env["inputs"].CONFIGS[idx]
    case = env["inputs"].device_case(wl, env["dev"])
    got = run_config(env, wl, case).cpu().numpy()
    want = oracle_config(env, wl, env["inputs"].host_case(wl))
    err = env["oracle"].rel_err_per_element(got, want)
    assert err.max() <= TOL64, err.max()


@pytest.mark.parametrize("idx", [2, 3, 4])
def test_large_configs_sampled(env, idx):
    torch = env["torch"]
    wl = env["inputs"].CONFIGS[idx]
    case = env["inputs"].device_case(wl, env["dev"])
    got = run_config(env, wl, case)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(got).all())
    E = wl.E
    # contiguous runs: start, an interior stretch spanning many CTA batches, the ragged end
    runs = [(0, 96), (E // 2 - 40, E // 2 + 88), (E - 77, E)]
    for e0, e1 in runs:
        host = env["inputs"].host_case(wl, e0, e1)
        want = oracle_config(env, wl, host)
        err = env["oracle"].rel_err_per_element(got[e0:e1].cpu().numpy(), want)
        assert err.max() <= TOL64, (idx, e0, err.max())
    # seeded random single elements
    g = np.random.Generator(np.random.PCG64(900 + idx))
    for e in sorted(g.integers(0, E, size=160).tolist()):
        host = env["inputs"].host_case(wl, e, e + 1)
        want = oracle_config(env, wl, host)
        err = env["oracle"].rel_err_per_element(got[e:e + 1].cpu().numpy(), want)
        assert err.max() <= TOL64, (idx, e, err.max())
    # a property that holds at any size: for the orthogonal-S inverse Helmholtz,
    # ‖v_e‖ ≤ max|D_e|·‖u_e‖ for every element (both stages are isometries)
    if wl.op == "inv_helmholtz":
        nu = torch.linalg.vector_norm(case["u"].view(E, -1), dim=1)
        nv = torch.linalg.vector_norm(got.view(E, -1), dim=1)
        dmax = case["D"].view(E, -1).abs().amax(dim=1)
        dmin = case["D"].view(E, -1).abs().amin(dim=1)
        assert bool((nv <= dmax * nu * (1 + 1e-12)).all())
        assert bool((nv >= dmin * nu * (1 - 1e-12)).all())


def test_largest_config_in_single_precision_sampled(env):
    """The largest inverse-Helmholtz configuration with fp32 fields (the TF32 tensor path with
    split operands), at full size in the launch shape the benchmark times, sampled against the
    oracle on the same rounded inputs: bar 1e-5 per element."""
    torch = env["torch"]
    wl = env["inputs"].CONFIGS[6]
    assert wl.dtype == "f32" and wl.n == (14, 14, 14) and wl.E == 131072
    case = env["inputs"].device_case(wl, env["dev"])
    assert case["u"].dtype == torch.float32
    got = env["ops"].ekl_tpo_inv_helmholtz_f32(case["S"], case["D"], case["u"])
    torch.cuda.synchronize()
    assert bool(torch.isfinite(got).all())
    E = wl.E
    for e0, e1 in [(0, 96), (E // 2 - 40, E // 2 + 88), (E - 77, E)]:
        host = env["inputs"].host_case(wl, e0, e1)
        want = env["oracle"].inv_helmholtz(host["S"], host["D"], host["u"])
        err = env["oracle"].rel_err_per_element(got[e0:e1].cpu().numpy().astype(np.float64), want)
        assert err.max() <= 1e-5, (e0, err.max())
    g = np.random.Generator(np.random.PCG64(906))
    for e in sorted(g.integers(0, E, size=120).tolist()):
        host = env["inputs"].host_case(wl, e, e + 1)
        want = env["oracle"].inv_helmholtz(host["S"], host["D"], host["u"])
        err = env["oracle"].rel_err_per_element(got[e:e + 1].cpu().numpy().astype(np.float64), want)
        assert err.max() <= 1e-5, (e, err.max())
    # both transforms are isometries for the orthogonal S: min|D| ‖u‖ <= ‖v‖ <= max|D| ‖u‖
    nu = torch.linalg.vector_norm(case["u"].double().view(E, -1), dim=1)
    nv = torch.linalg.vector_norm(got.double().view(E, -1), dim=1)
    dmax = case["D"].double().view(E, -1).abs().amax(dim=1)
    dmin = case["D"].double().view(E, -1).abs().amin(dim=1)
    assert bool((nv <= dmax * nu * (1 + 1e-5)).all())
    assert bool((nv >= dmin * nu * (1 - 1e-5)).all())
