"""The fp32 inverse Helmholtz on the asynchronous tensor path (tcgen05.mma, accumulator in
tensor memory), selected with EKL_TPO_F32_PATH=tcgen05.  The library reads the switch once,
so each case runs in a child process; the child compares against the CPU oracle (1e-5 per
element) and against the default path of the same library call made without the switch."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import json, sys
import numpy as np, torch
sys.path.insert(0, %(root)r)
import oracle
from paper_2604_19906_b200 import ops
n, E = %(n)d, %(E)d
g = np.random.Generator(np.random.PCG64(4100 + n))
S = (g.standard_normal((n, n)) / np.sqrt(n)).astype(np.float32)
D = g.uniform(0.13, 1.25, (E, n, n, n)).astype(np.float32)
u = g.uniform(-1, 1, (E, n, n, n)).astype(np.float32)
dev = torch.device("cuda:0")
dS, dD, du = (torch.from_numpy(x).to(dev) for x in (S, D, u))
got = ops.ekl_tpo_inv_helmholtz_f32(dS, dD, du)
again = ops.ekl_tpo_inv_helmholtz_f32(dS, dD, du, out=du)        # in place, same bits
torch.cuda.synchronize()
want = oracle.inv_helmholtz(S, D, u)
err = float(oracle.rel_err_per_element(got.cpu().numpy().astype(np.float64), want).max())
print(json.dumps({"err": err, "same": bool(torch.equal(got, again)),
                  "flags": int(ops.library().ekl_tpo_device_error_flags()),
                  "sum": float(got.double().abs().sum().item())}))
"""


def run_child(n, E, tcgen05):
    env = dict(os.environ)
    env.pop("EKL_TPO_F32_PATH", None)
    if tcgen05:
        env["EKL_TPO_F32_PATH"] = "tcgen05"
    out = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT, "n": n, "E": E}],
                         env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    return json.loads(out.stdout.strip().splitlines()[-1])


@pytest.mark.gpu
@pytest.mark.parametrize("n,E", [(8, 333), (10, 70), (12, 1001), (14, 1), (14, 2500), (16, 129)])
def test_tcgen05_path_matches_the_oracle(n, E):
    r = run_child(n, E, True)
    assert r["flags"] == 0
    assert r["same"]
    assert r["err"] <= 1e-5, (n, E, r["err"])


@pytest.mark.gpu
def test_tcgen05_path_is_really_another_kernel():
    """The two paths round differently, so their outputs differ in the last bits while both
    meet the bar; identical sums would mean the switch did nothing."""
    a = run_child(14, 600, True)
    b = run_child(14, 600, False)
    assert a["err"] <= 1e-5 and b["err"] <= 1e-5
    assert a["sum"] != b["sum"]
