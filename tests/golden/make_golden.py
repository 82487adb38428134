"""Writes the integer golden fixtures in this folder.

The expected values are computed here from the *definition* with exact Python integer
arithmetic -- the un-lifted triple sum of Section 5.2 of the paper for the forward
stage, a pointwise product with D, and the same triple sum with S in place of S^T for
the backward stage; Eq. 1's Kronecker ordering (last factor <-> fastest index) for the
rectangular operator.  Nothing here calls the CUDA path (or even the oracle): the
inputs are small integers, so every intermediate is exactly representable in fp64 and
any correct implementation must reproduce the expected values bit for bit.

Run:  python tests/golden/make_golden.py
"""
import itertools
import os

HERE = os.path.dirname(os.path.abspath(__file__))


def inv_helmholtz_int(S, D, u, n):
    rng = range(n)
    t = {}
    for i, j, k in itertools.product(rng, rng, rng):
        t[i, j, k] = sum(S[l][i] * S[m][j] * S[q][k] * u[l][m][q]
                         for l, m, q in itertools.product(rng, rng, rng))
    r = {x: D[x[0]][x[1]][x[2]] * t[x] for x in t}
    v = {}
    for i, j, k in itertools.product(rng, rng, rng):
        v[i, j, k] = sum(S[i][l] * S[j][m] * S[k][q] * r[l, m, q]
                         for l, m, q in itertools.product(rng, rng, rng))
    return [[[v[i, j, k] for k in rng] for j in rng] for i in rng]


def inv_helmholtz3_int(S0, S1, S2, D, u, nn):
    """One operator per direction: forward stage S0^T, S1^T, S2^T, backward stage S0, S1, S2."""
    idx = list(itertools.product(range(nn[0]), range(nn[1]), range(nn[2])))
    t = {(i, j, k): sum(S0[l][i] * S1[m][j] * S2[q][k] * u[l][m][q] for l, m, q in idx)
         for i, j, k in idx}
    r = {x: D[x[0]][x[1]][x[2]] * t[x] for x in idx}
    v = {(i, j, k): sum(S0[i][l] * S1[j][m] * S2[k][q] * r[l, m, q] for l, m, q in idx)
         for i, j, k in idx}
    return [[[v[i, j, k] for k in range(nn[2])] for j in range(nn[1])] for i in range(nn[0])]


def apply_int(A, B, C, u, nn, mm):
    return [[[sum(A[i][l] * B[j][m] * C[k][q] * u[l][m][q]
                  for l in range(nn[0]) for m in range(nn[1]) for q in range(nn[2]))
              for k in range(mm[2])] for j in range(mm[1])] for i in range(mm[0])]


def flat(x):
    if isinstance(x, list):
        return [z for y in x for z in flat(y)]
    return [x]


def write(name, header, rows):
    with open(os.path.join(HERE, name), "w") as f:
        f.write(header)
        for key, vals in rows:
            f.write(key + " " + " ".join(str(v) for v in vals) + "\n")


def main():
    # inverse Helmholtz, n = 2, one element, non-symmetric integer S
    n = 2
    S = [[1, 2], [-3, 4]]
    D = [[[1, 2], [3, -1]], [[2, 1], [-2, 3]]]
    u = [[[1, -1], [2, 3]], [[0, 4], [-2, 1]]]
    v = inv_helmholtz_int(S, D, u, n)
    write("inv_helmholtz_n2_int.txt",
          "# v = (S(x)S(x)S)(D o ((S^T(x)S^T(x)S^T) u)), exact integers; forward stage is the\n"
          "# un-lifted triple sum of Section 5.2 (t_ijk = sum_lmn S^T_li S^T_mj S^T_nk u_lmn).\n"
          "# rows: name then row-major values\n",
          [("n", [n]), ("S", flat(S)), ("D", flat(D)), ("u", flat(u)), ("v", flat(v))])

    # inverse Helmholtz, n = 3
    n = 3
    S = [[2, -1, 0], [1, 3, -2], [0, 1, 1]]
    D = [[[((3 * i + 5 * j + 7 * k) % 5) - 2 for k in range(n)] for j in range(n)]
         for i in range(n)]
    u = [[[((i * 9 + j * 3 + k) * 7 % 11) - 5 for k in range(n)] for j in range(n)]
         for i in range(n)]
    v = inv_helmholtz_int(S, D, u, n)
    write("inv_helmholtz_n3_int.txt",
          "# same operator as inv_helmholtz_n2_int.txt, n = 3\n",
          [("n", [n]), ("S", flat(S)), ("D", flat(D)), ("u", flat(u)), ("v", flat(v))])

    # rectangular forward operator, all six extents distinct where it matters
    nn, mm = (2, 3, 4), (3, 2, 5)
    A = [[((i * 2 + l) * 3 % 7) - 3 for l in range(nn[0])] for i in range(mm[0])]
    B = [[((j * 3 + m) * 5 % 9) - 4 for m in range(nn[1])] for j in range(mm[1])]
    C = [[((k * 4 + q) * 2 % 5) - 2 for q in range(nn[2])] for k in range(mm[2])]
    u = [[[((l * 12 + m * 4 + q) * 5 % 13) - 6 for q in range(nn[2])] for m in range(nn[1])]
         for l in range(nn[0])]
    v = apply_int(A, B, C, u, nn, mm)
    write("apply_2x3x4_to_3x2x5_int.txt",
          "# v = (A(x)B(x)C) u, Kronecker ordering of Eq. 1: A <-> slowest in-element axis,\n"
          "# C <-> contiguous axis; exact integers\n",
          [("nn", nn), ("mm", mm), ("A", flat(A)), ("B", flat(B)), ("C", flat(C)),
           ("u", flat(u)), ("v", flat(v))])

    # inverse Helmholtz with one operator and one extent per direction (per-direction
    # matrices as in Eq. 1): three different non-symmetric matrices, extents 2, 3, 4
    nn = (2, 3, 4)
    S0 = [[2, -1], [3, 1]]
    S1 = [[1, 0, -2], [2, 1, 1], [-1, 3, 0]]
    S2 = [[((a * 4 + b) * 3 % 7) - 3 for b in range(4)] for a in range(4)]
    D = [[[((2 * i + 3 * j + 5 * k) % 7) - 3 for k in range(nn[2])] for j in range(nn[1])]
         for i in range(nn[0])]
    u = [[[((i * 12 + j * 4 + k) * 5 % 9) - 4 for k in range(nn[2])] for j in range(nn[1])]
         for i in range(nn[0])]
    v = inv_helmholtz3_int(S0, S1, S2, D, u, nn)
    write("inv_helmholtz3_2x3x4_int.txt",
          "# v = (S0(x)S1(x)S2)(D o ((S0^T(x)S1^T(x)S2^T) u)), S0 <-> slowest in-element axis,\n"
          "# S2 <-> contiguous axis; exact integers\n",
          [("nn", nn), ("S0", flat(S0)), ("S1", flat(S1)), ("S2", flat(S2)), ("D", flat(D)),
           ("u", flat(u)), ("v", flat(v))])


if __name__ == "__main__":
    main()
