"""Pins for the CPU oracle (no GPU needed).

The paper prints no worked numeric example for a tensor-product operator, so the
oracle is pinned against what the mathematics fixes: the un-lifted definition through
library routines (numpy.kron, numpy.einsum), exact integer arithmetic on tiny inputs
(fixtures under tests/golden/), closed forms and invariants.  Each pin is chosen so
that a plausible slip -- a transposed factor, swapped axes, a dropped D, the wrong
stage order -- fails at least one of them; ``test_pins_catch_planted_mistakes`` shows
that for the usual suspects.
"""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def kron3(A, B, C):
    return np.kron(np.kron(A, B), C)


def ref_apply_kron(A, B, C, u):
    E = u.shape[0]
    K = kron3(A, B, C)
    v = (K @ u.reshape(E, -1).T).T
    return v.reshape(E, A.shape[0], B.shape[0], C.shape[0])


def ref_inv_helmholtz_kron(S, D, u):
    E, n = u.shape[0], S.shape[0]
    K1 = kron3(S.T, S.T, S.T)
    K2 = kron3(S, S, S)
    t = (K1 @ u.reshape(E, -1).T).T * D.reshape(E, -1)
    return (K2 @ t.T).T.reshape(E, n, n, n)


def relmax(a, b):
    return float(oracle.rel_err_per_element(a, b).max())


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            out[key] = np.array([float(v) for v in vals])
    return out


# ------------------------------------------------------------------ definition pins

@pytest.mark.parametrize("nn,mm", [((2, 3, 4), (5, 2, 3)), ((3, 2, 2), (2, 4, 3)),
                                   ((1, 1, 1), (1, 1, 1)), ((4, 1, 3), (1, 5, 2)),
                                   ((3, 3, 3), (3, 3, 3))])
def test_apply_matches_numpy_kron_and_einsum(nn, mm):
    g = rng(11)
    A, B, C = (g.standard_normal((mm[d], nn[d])) for d in range(3))
    u = g.uniform(-1, 1, (5,) + nn)
    v = oracle.tpo_apply(A, B, C, u)
    assert v.shape == (5,) + mm
    assert relmax(v, ref_apply_kron(A, B, C, u)) < 1e-14
    assert relmax(v, np.einsum("il,jm,kn,elmn->eijk", A, B, C, u)) < 1e-14
    assert relmax(oracle.tpo_apply_bruteforce(A, B, C, u), ref_apply_kron(A, B, C, u)) < 1e-14


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5])
def test_inv_helmholtz_matches_numpy_kron(n):
    g = rng(100 + n)
    S = g.standard_normal((n, n))            # deliberately NOT orthogonal, not symmetric
    D = g.uniform(0.1, 1.3, (3, n, n, n))
    u = g.uniform(-1, 1, (3, n, n, n))
    ref = ref_inv_helmholtz_kron(S, D, u)
    assert relmax(oracle.inv_helmholtz(S, D, u), ref) < 1e-13
    assert relmax(oracle.inv_helmholtz_bruteforce(S, D, u), ref) < 1e-13
    ein = np.einsum("il,jm,kn,elmn->eijk", S, S, S,
                    D * np.einsum("li,mj,nk,elmn->eijk", S, S, S, u))
    assert relmax(oracle.inv_helmholtz(S, D, u), ein) < 1e-13


def test_golden_integer_fixtures_are_reproduced_exactly():
    for name in ("inv_helmholtz_n2_int.txt", "inv_helmholtz_n3_int.txt"):
        g = read_golden(name)
        n = int(g["n"][0])
        S = g["S"].reshape(n, n)
        D = g["D"].reshape(1, n, n, n)
        u = g["u"].reshape(1, n, n, n)
        want = g["v"].reshape(1, n, n, n)
        assert np.array_equal(oracle.inv_helmholtz(S, D, u), want)
        assert np.array_equal(oracle.inv_helmholtz_bruteforce(S, D, u), want)
        assert np.array_equal(oracle.inv_helmholtz_ld(S, D, u), want)
    g = read_golden("apply_2x3x4_to_3x2x5_int.txt")
    nn = tuple(int(x) for x in g["nn"])
    mm = tuple(int(x) for x in g["mm"])
    A, B, C = (g[k].reshape(mm[d], nn[d]) for d, k in enumerate("ABC"))
    u = g["u"].reshape((1,) + nn)
    want = g["v"].reshape((1,) + mm)
    assert np.array_equal(oracle.tpo_apply(A, B, C, u), want)
    assert np.array_equal(oracle.tpo_apply_bruteforce(A, B, C, u), want)
    assert np.array_equal(oracle.tpo_apply_ld(A, B, C, u), want)


# ------------------------------------------------------------------ invariants / closed forms

@pytest.mark.parametrize("n", [2, 4, 7, 8, 12, 14])
def test_identity_invariant_orthogonal_S_unit_D(n):
    g = rng(200 + n)
    S, _ = np.linalg.qr(g.standard_normal((n, n)))
    u = g.uniform(-1, 1, (4, n, n, n))
    v = oracle.inv_helmholtz(S, np.ones_like(u), u)
    assert relmax(v, u) < 50 * n * np.finfo(float).eps
    v = oracle.inv_helmholtz(S, np.full_like(u, -0.375), u)
    assert relmax(v, -0.375 * u) < 50 * n * np.finfo(float).eps


def test_identity_S_is_bitwise_pointwise_product():
    g = rng(3)
    n = 6
    D = g.uniform(0.1, 1.3, (3, n, n, n))
    u = g.uniform(-1, 1, (3, n, n, n))
    assert np.array_equal(oracle.inv_helmholtz(np.eye(n), D, u), D * u)


def test_permutation_S_is_exact_permuted_copy():
    g = rng(4)
    n = 5
    perm = g.permutation(n)
    S = np.zeros((n, n))
    S[np.arange(n), perm] = 1.0               # (S x)[i] = x[perm[i]]
    D = g.uniform(0.1, 1.3, (2, n, n, n))
    u = g.uniform(-1, 1, (2, n, n, n))
    # forward stage applies S^T on every axis: t[i,j,k] = u[inv[i],inv[j],inv[k]]
    inv = np.argsort(perm)
    t = u[:, inv][:, :, inv][:, :, :, inv]
    r = D * t
    want = r[:, perm][:, :, perm][:, :, :, perm]
    assert np.array_equal(oracle.inv_helmholtz(S, D, u), want)


def test_selection_matrices_gather_exactly():
    g = rng(5)
    nn, mm = (4, 5, 6), (2, 3, 4)
    rows = [g.choice(nn[d], size=mm[d], replace=False) for d in range(3)]
    A, B, C = (np.eye(nn[d])[rows[d]] for d in range(3))
    u = g.uniform(-1, 1, (3,) + nn)
    want = u[:, rows[0]][:, :, rows[1]][:, :, :, rows[2]]
    assert np.array_equal(oracle.tpo_apply(A, B, C, u), want)


def test_separable_input_closed_form():
    g = rng(6)
    nn, mm = (3, 4, 5), (6, 2, 4)
    A, B, C = (g.standard_normal((mm[d], nn[d])) for d in range(3))
    a, b, c = (g.standard_normal(nn[d]) for d in range(3))
    u = np.einsum("l,m,n->lmn", a, b, c)[None]
    want = np.einsum("i,j,k->ijk", A @ a, B @ b, C @ c)[None]
    assert relmax(oracle.tpo_apply(A, B, C, u), want) < 1e-14


def test_linearity_and_element_independence():
    g = rng(7)
    n, E = 5, 6
    S = g.standard_normal((n, n))
    D = g.uniform(0.1, 1.3, (E, n, n, n))
    u1, u2 = g.uniform(-1, 1, (2, E, n, n, n))
    lhs = oracle.inv_helmholtz(S, D, 0.5 * u1 - 2.0 * u2)
    rhs = 0.5 * oracle.inv_helmholtz(S, D, u1) - 2.0 * oracle.inv_helmholtz(S, D, u2)
    assert relmax(lhs, rhs) < 1e-13
    # permuting elements permutes outputs bit for bit; a single element equals its batch row
    p = g.permutation(E)
    full = oracle.inv_helmholtz(S, D, u1)
    assert np.array_equal(oracle.inv_helmholtz(S, D[p], u1[p]), full[p])
    assert np.array_equal(oracle.inv_helmholtz(S, D[3:4], u1[3:4]), full[3:4])
    # thread count does not change any bit
    assert np.array_equal(oracle.inv_helmholtz(S, D, u1, threads=1), full)


def test_empty_batch():
    S = np.eye(3)
    z = np.zeros((0, 3, 3, 3))
    assert oracle.inv_helmholtz(S, z, z).shape == (0, 3, 3, 3)
    assert oracle.tpo_apply(np.ones((2, 3)), np.ones((4, 3)), np.ones((1, 3)), z).shape == (0, 2, 4, 1)


# ------------------------------------------------------------------ accuracy level

@pytest.mark.parametrize("n", [4, 8, 14])
def test_double_oracle_is_far_inside_the_parity_tolerance(n):
    g = rng(300 + n)
    S, _ = np.linalg.qr(g.standard_normal((n, n)))
    lam = g.uniform(0.1, 2.0, n)
    c = g.uniform(0.5, 1.5, 8)
    D = 1.0 / (lam[:, None, None] + lam[None, :, None] + lam[None, None, :] + c[:, None, None, None])
    u = g.uniform(-1, 1, (8, n, n, n))
    err = relmax(oracle.inv_helmholtz(S, D, u), oracle.inv_helmholtz_ld(S, D, u))
    assert err < 6 * n * np.finfo(float).eps      # a-priori bound: six length-n dot products
    assert err < 1e-14
    A, B, C = (g.standard_normal((n + 2, n)) / np.sqrt(n) for _ in range(3))
    err = relmax(oracle.tpo_apply(A, B, C, u), oracle.tpo_apply_ld(A, B, C, u))
    assert err < 1e-14


# ------------------------------------------------------------------ the pins have teeth

def test_pins_catch_planted_mistakes():
    """Plant the usual slips *into the call of the oracle* and check that the library
    reference notices; this guards against pins that would pass a wrong oracle."""
    g = rng(8)
    n = 4
    S = g.standard_normal((n, n))
    D = g.uniform(0.1, 1.3, (2, n, n, n))
    u = g.uniform(-1, 1, (2, n, n, n))
    ref = ref_inv_helmholtz_kron(S, D, u)
    assert relmax(oracle.inv_helmholtz(S.T, D, u), ref) > 1e-3                    # transposed S
    assert relmax(oracle.inv_helmholtz(S, np.ones_like(D), u), ref) > 1e-3        # dropped D
    assert relmax(oracle.inv_helmholtz(S, D.transpose(0, 3, 2, 1), u), ref) > 1e-3  # D axes
    A, B, C = (g.standard_normal((n, n)) for _ in range(3))
    refa = ref_apply_kron(A, B, C, u)
    assert relmax(oracle.tpo_apply(C, B, A, u), refa) > 1e-3                      # factor order
    assert relmax(oracle.tpo_apply(A.T, B.T, C.T, u), refa) > 1e-3                # transposes
    # the identity invariant alone cannot see a joint transpose -- the kron pin above can
    Q, _ = np.linalg.qr(g.standard_normal((n, n)))
    assert relmax(oracle.inv_helmholtz(Q.T, np.ones_like(u), u), u) < 1e-13


def test_flop_accounting_matches_the_lifting_claim():
    """Section 5.2: lifting cuts the naive cost by a factor of order p² -- dense 2n⁶
    per stage against 6n⁴ for the three lifted sums."""
    from paper_2604_19906_b200.inputs import CONFIGS
    for wl in CONFIGS[:4]:
        n = wl.n[0]
        assert wl.flops_per_element == 12 * n ** 4 + n ** 3
        assert (2 * 2 * n ** 6) / (12 * n ** 4) == pytest.approx(n * n / 3)
    assert CONFIGS[4].flops_per_element == 58368
    assert CONFIGS[4].bytes_per_element == 17920
    assert CONFIGS[3].bytes_per_element == 65856


# ------------------------------------------------------------------ convective flux (Eq. 1)

def ref_convection_einsum(Dvq, Ivq, M, P):
    """The paper's one-statement form, index names as printed: F[c,e,k,j,i] with (l,m,n)
    summed, D on the (i,l) pair for direction 0, on (j,m) for 1, on (k,n) for 2."""
    out = []
    for c in range(3):
        t = (np.einsum("il,jm,kn,enml,enml->ekji", Dvq, Ivq, Ivq, M, P[c, 0])
             + np.einsum("il,jm,kn,enml,enml->ekji", Ivq, Dvq, Ivq, M, P[c, 1])
             + np.einsum("il,jm,kn,enml,enml->ekji", Ivq, Ivq, Dvq, M, P[c, 2]))
        out.append(t)
    return np.stack(out)


@pytest.mark.parametrize("nq,nv", [(3, 2), (4, 4), (5, 3), (2, 5), (12, 8)])
def test_convection_matches_the_printed_statement(nq, nv):
    g = rng(400 + nq * 10 + nv)
    E = 3
    Dvq, Ivq = g.standard_normal((2, nv, nq))
    M = g.uniform(0.5, 1.5, (E, nq, nq, nq))
    P = g.uniform(-1, 1, (3, 3, E, nq, nq, nq))
    F = oracle.convection(Dvq, Ivq, M, P)
    ref = ref_convection_einsum(Dvq, Ivq, M, P)
    assert F.shape == (3, E, nv, nv, nv)
    assert relmax(F.reshape(3 * E, nv, nv, nv), ref.reshape(3 * E, nv, nv, nv)) < 1e-13
    if nq <= 6 and nv <= 6:
        bf = oracle.convection_bruteforce(Dvq, Ivq, M, P)
        assert relmax(bf.reshape(3 * E, nv, nv, nv), ref.reshape(3 * E, nv, nv, nv)) < 1e-13


def test_convection_special_cases_and_planted_mistakes():
    g = rng(17)
    nq, nv, E = 4, 3, 2
    Dvq, Ivq = g.standard_normal((2, nv, nq))
    M = g.uniform(0.5, 1.5, (E, nq, nq, nq))
    P = g.uniform(-1, 1, (3, 3, E, nq, nq, nq))
    ref = ref_convection_einsum(Dvq, Ivq, M, P).reshape(3 * E, nv, nv, nv)
    flat = lambda F: F.reshape(3 * E, nv, nv, nv)
    # each direction alone is one forward operator with D on its own axis (M = 1)
    ones = np.ones_like(M)
    for d, (A, B, C) in enumerate([(Ivq, Ivq, Dvq), (Ivq, Dvq, Ivq), (Dvq, Ivq, Ivq)]):
        Pd = np.zeros_like(P)
        Pd[:, d] = P[:, d]
        want = np.stack([oracle.tpo_apply(A, B, C, P[c, d]) for c in range(3)])
        assert relmax(flat(oracle.convection(Dvq, Ivq, ones, Pd)), flat(want)) < 1e-13
    # D = 0 kills everything; M scales linearly
    assert np.all(oracle.convection(np.zeros_like(Dvq), Ivq, M, P) == 0.0)
    assert relmax(flat(oracle.convection(Dvq, Ivq, 2.0 * M, P)), 2.0 * ref) < 1e-13
    # planted slips are seen by the reference
    assert relmax(flat(oracle.convection(Ivq, Dvq, M, P)), ref) > 1e-3          # D and I swapped
    assert relmax(flat(oracle.convection(Dvq, Ivq, M, P[:, ::-1].copy())), ref) > 1e-3  # directions
    assert relmax(flat(oracle.convection(Dvq, Ivq, ones, P)), ref) > 1e-3       # dropped M


def test_lambda_factor_matches_its_definition_entry_by_entry():
    g = rng(77)
    n, E = 5, 4
    lam = g.uniform(0.1, 2.0, n)
    c = g.uniform(0.5, 1.5, E)
    D = oracle.lambda_factor(lam, c)
    for e in range(E):
        for i in range(n):
            for j in range(n):
                for k in range(n):
                    assert D[e, i, j, k] == 1.0 / (((lam[i] + lam[j]) + lam[k]) + c[e])
    S = g.standard_normal((n, n))
    u = g.uniform(-1, 1, (E, n, n, n))
    assert np.array_equal(oracle.inv_helmholtz_lambda(S, lam, c, u), oracle.inv_helmholtz(S, D, u))
    assert relmax(oracle.inv_helmholtz_lambda(S, lam, c, u), ref_inv_helmholtz_kron(S, D, u)) < 1e-13


# ------------------------------------------------------------------ one operator per direction

def ref_inv_helmholtz3_kron(S0, S1, S2, D, u):
    """numpy.kron (library routine): K2 diag(D) K1 with K1 = S0ᵀ⊗S1ᵀ⊗S2ᵀ, K2 = S0⊗S1⊗S2."""
    E = u.shape[0]
    K1 = np.kron(np.kron(S0.T, S1.T), S2.T)
    K2 = np.kron(np.kron(S0, S1), S2)
    t = (K1 @ u.reshape(E, -1).T).T * D.reshape(E, -1)
    return (K2 @ t.T).T.reshape(u.shape)


@pytest.mark.parametrize("nn", [(2, 3, 4), (4, 2, 3), (1, 5, 2), (3, 3, 3), (5, 1, 1)])
def test_inv_helmholtz3_matches_numpy_kron_and_einsum(nn):
    g = rng(500 + 100 * nn[0] + 10 * nn[1] + nn[2])
    S0, S1, S2 = (g.standard_normal((n, n)) for n in nn)      # three different, non-symmetric
    D = g.uniform(0.1, 1.3, (3,) + nn)
    u = g.uniform(-1, 1, (3,) + nn)
    ref = ref_inv_helmholtz3_kron(S0, S1, S2, D, u)
    got = oracle.inv_helmholtz3(S0, S1, S2, D, u)
    assert relmax(got, ref) < 1e-13
    assert relmax(oracle.inv_helmholtz3_bruteforce(S0, S1, S2, D, u), ref) < 1e-13
    ein = np.einsum("il,jm,kn,elmn->eijk", S0, S1, S2,
                    D * np.einsum("li,mj,nk,elmn->eijk", S0, S1, S2, u))
    assert relmax(got, ein) < 1e-13


def test_inv_helmholtz3_golden_integer_fixture_is_reproduced_exactly():
    g = read_golden("inv_helmholtz3_2x3x4_int.txt")
    nn = tuple(int(x) for x in g["nn"])
    S0, S1, S2 = (g[f"S{d}"].reshape(nn[d], nn[d]) for d in range(3))
    D = g["D"].reshape((1,) + nn)
    u = g["u"].reshape((1,) + nn)
    want = g["v"].reshape((1,) + nn)
    assert np.array_equal(oracle.inv_helmholtz3(S0, S1, S2, D, u), want)
    assert np.array_equal(oracle.inv_helmholtz3_bruteforce(S0, S1, S2, D, u), want)


def test_inv_helmholtz3_special_cases_and_planted_mistakes():
    g = rng(77)
    nn = (3, 4, 2)
    S0, S1, S2 = (g.standard_normal((n, n)) for n in nn)
    D = g.uniform(0.1, 1.3, (2,) + nn)
    u = g.uniform(-1, 1, (2,) + nn)
    ref = ref_inv_helmholtz3_kron(S0, S1, S2, D, u)
    # one shared matrix: the single-operator routine, bit for bit (same loops, same order)
    n = 4
    S = g.standard_normal((n, n))
    Dc = g.uniform(0.1, 1.3, (2, n, n, n))
    uc = g.uniform(-1, 1, (2, n, n, n))
    assert np.array_equal(oracle.inv_helmholtz3(S, S, S, Dc, uc), oracle.inv_helmholtz(S, Dc, uc))
    # identities on every axis: the pointwise product, bit for bit
    I0, I1, I2 = (np.eye(k) for k in nn)
    assert np.array_equal(oracle.inv_helmholtz3(I0, I1, I2, D, u), D * u)
    # orthogonal operators, unit factor: the identity
    Q0, Q1, Q2 = (np.linalg.qr(g.standard_normal((k, k)))[0] for k in nn)
    assert relmax(oracle.inv_helmholtz3(Q0, Q1, Q2, np.ones_like(u), u), u) < 1e-13
    # an identity on two axes leaves a one-axis operator: closed form with einsum
    one = np.einsum("il,eljk->eijk", S0, D * np.einsum("li,eljk->eijk", S0, u))
    assert relmax(oracle.inv_helmholtz3(S0, I1, I2, D, u), one) < 1e-13
    # planted slips in the call must be seen by the library reference
    assert relmax(oracle.inv_helmholtz3(S0.T, S1.T, S2.T, D, u), ref) > 1e-3      # transposes
    assert relmax(oracle.inv_helmholtz3(S0, S1, S2, np.ones_like(D), u), ref) > 1e-3  # dropped D
    nc = (3, 3, 3)
    T0, T1, T2 = (g.standard_normal((3, 3)) for _ in range(3))
    Dd = g.uniform(0.1, 1.3, (2,) + nc)
    ud = g.uniform(-1, 1, (2,) + nc)
    refc = ref_inv_helmholtz3_kron(T0, T1, T2, Dd, ud)
    assert relmax(oracle.inv_helmholtz3(T2, T1, T0, Dd, ud), refc) > 1e-3         # direction order
    assert relmax(oracle.inv_helmholtz3(T0, T2, T1, Dd, ud), refc) > 1e-3


def test_rel_err_per_element_edge_cases():
    ref = np.array([[1.0, 2.0, 2.0], [0.0, 0.0, 0.0], [3.0, 4.0, 0.0]])
    v = ref.copy()
    v[0, 0] = 1.0 + 3e-6
    v[1, 0] = 1e-3                         # zero reference norm: guarded denominator
    v[2, 1] = np.nan                       # any NaN in an element: infinite error
    err = oracle.rel_err_per_element(v, ref)
    assert abs(err[0] - 1e-6) < 1e-12
    assert np.isfinite(err[1]) and err[1] > 1e290      # compared absolutely, against 1e-300
    assert err[2] == np.inf
    v[2, 1] = np.inf
    assert oracle.rel_err_per_element(v, ref)[2] == np.inf
    assert np.array_equal(oracle.rel_err_per_element(ref, ref), np.zeros(3))


def test_scaling_by_a_power_of_two_is_exact_in_every_oracle_routine():
    """Each routine is linear in its field arguments, and a power of two changes no rounding:
    scaling u (or D, M, P) by 2^k scales the result by 2^k bit for bit.  A routine that took a
    square root, normalised, or mixed its arguments non-linearly would fail."""
    g = np.random.Generator(np.random.PCG64(2024))
    f = 2.0 ** 37
    n, E = 5, 3
    S = g.standard_normal((n, n))
    D = g.uniform(0.1, 1.0, (E, n, n, n))
    u = g.standard_normal((E, n, n, n))
    base = oracle.inv_helmholtz(S, D, u)
    assert np.array_equal(oracle.inv_helmholtz(S, D, u * f), base * f)
    assert np.array_equal(oracle.inv_helmholtz(S, D * f, u), base * f)
    nn = (3, 4, 5)
    S3 = [g.standard_normal((k, k)) for k in nn]
    D3 = g.uniform(0.1, 1.0, (E,) + nn)
    u3 = g.standard_normal((E,) + nn)
    base3 = oracle.inv_helmholtz3(*S3, D3, u3)
    assert np.array_equal(oracle.inv_helmholtz3(*S3, D3 / f, u3), base3 / f)
    assert np.array_equal(oracle.inv_helmholtz3(*S3, D3, u3 * f), base3 * f)
    A, B, C = g.standard_normal((4, 3)), g.standard_normal((2, 4)), g.standard_normal((6, 5))
    ua = g.standard_normal((E, 3, 4, 5))
    assert np.array_equal(oracle.tpo_apply(A, B, C, ua * f), oracle.tpo_apply(A, B, C, ua) * f)
    nq, nv = 4, 3
    Dvq, Ivq = g.standard_normal((nv, nq)), g.standard_normal((nv, nq))
    M = g.uniform(0.5, 1.5, (E, nq, nq, nq))
    P = g.standard_normal((3, 3, E, nq, nq, nq))
    basec = oracle.convection(Dvq, Ivq, M, P)
    assert np.array_equal(oracle.convection(Dvq, Ivq, M * f, P), basec * f)
    assert np.array_equal(oracle.convection(Dvq, Ivq, M, P / f), basec / f)
