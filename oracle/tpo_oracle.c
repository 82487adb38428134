/*
 * CPU oracle for the batched, sum-factorised tensor-product operators.
 *
 * THIS IS TEST INFRASTRUCTURE.  It defines what "correct" means for the CUDA
 * library and is timed as the host baseline; it is never part of the product
 * path, shares no code with it, and is deliberately plain and slow.
 *
 * Conventions (all arrays dense, row-major, last index fastest, the element
 * index e slowest):
 *
 *   ((A (x) B (x) C) x)[i,j,k] = sum_l sum_m sum_n A[i,l] B[j,m] C[k,n] x[l,m,n]
 *
 *   A is [m0,n0] and acts on the slowest in-element axis, C is [m2,n2] and
 *   acts on the contiguous one (ordering of the factors as in Eq. 1 of the
 *   paper: last factor <-> fastest index).
 *
 * Two families of routines:
 *
 *  - "factored": the lifted reductions of Section 5.2 (reduction lifting),
 *        t_ijk = sum_l S^T_li sum_m S^T_mj sum_n S^T_nk u_lmn,
 *    taken inside-out, one axis at a time, with plain left-to-right sums and
 *    separate multiply and add (build with -ffp-contract=off).
 *  - "bruteforce": the un-lifted definition, i.e. the explicit Kronecker
 *    matrix of size (m0 m1 m2) x (n0 n1 n2) built entry by entry and applied
 *    as one dense matrix-vector product (the first line of the same equation).
 *
 * Parity pins: every factored routine is pinned in tests/test_oracle_pins.py
 * against numpy.kron / numpy.einsum, exact rational arithmetic on tiny inputs,
 * closed forms (separable inputs, identity and permutation matrices) and the
 * orthogonal-S identity invariant.  Nothing here is "parity unpinned".
 */
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- one element of the forward operator  v = (A (x) B (x) C) u ---------- */
/* p:[n0,n1,m2]  q:[n0,m1,m2] are caller-provided scratch.                    */
static void apply_one(const double *A, const double *B, const double *C,
                      const double *u, double *v, double *p, double *q,
                      int n0, int n1, int n2, int m0, int m1, int m2)
{
    /* innermost sum of the lifted form: contract the contiguous axis with C */
    for (int l = 0; l < n0; ++l)
        for (int m = 0; m < n1; ++m)
            for (int k = 0; k < m2; ++k) {
                double s = 0.0;
                for (int n = 0; n < n2; ++n)
                    s = s + C[k * n2 + n] * u[(l * n1 + m) * n2 + n];
                p[(l * n1 + m) * m2 + k] = s;
            }
    /* middle sum: contract the middle axis with B */
    for (int l = 0; l < n0; ++l)
        for (int j = 0; j < m1; ++j)
            for (int k = 0; k < m2; ++k) {
                double s = 0.0;
                for (int m = 0; m < n1; ++m)
                    s = s + B[j * n1 + m] * p[(l * n1 + m) * m2 + k];
                q[(l * m1 + j) * m2 + k] = s;
            }
    /* outer sum: contract the slowest axis with A */
    for (int i = 0; i < m0; ++i)
        for (int j = 0; j < m1; ++j)
            for (int k = 0; k < m2; ++k) {
                double s = 0.0;
                for (int l = 0; l < n0; ++l)
                    s = s + A[i * n0 + l] * q[(l * m1 + j) * m2 + k];
                v[(i * m1 + j) * m2 + k] = s;
            }
}

static int pick_threads(int threads)
{
#ifdef _OPENMP
    if (threads <= 0) threads = omp_get_max_threads();
    return threads;
#else
    (void)threads;
    return 1;
#endif
}

/* Number of threads a call with this `threads` argument will use. */
int oracle_threads(int threads) { return pick_threads(threads); }

/*
 * Forward rectangular operator, all E elements:
 *   v[e] = (A (x) B (x) C) u[e],  u:[E,n0,n1,n2]  v:[E,m0,m1,m2].
 * threads <= 0: all cores OpenMP offers.  Returns 0, or -1 on allocation failure.
 */
int oracle_tpo_apply_f64(const double *A, const double *B, const double *C,
                         const double *u, double *v,
                         int n0, int n1, int n2, int m0, int m1, int m2,
                         long long E, int threads)
{
    const size_t np = (size_t)n0 * n1 * m2, nq = (size_t)n0 * m1 * m2;
    const size_t nin = (size_t)n0 * n1 * n2, nout = (size_t)m0 * m1 * m2;
    int fail = 0;
    threads = pick_threads(threads);
#pragma omp parallel num_threads(threads)
    {
        double *p = (double *)malloc((np + nq + 1) * sizeof(double));
        if (!p) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
            double *q = p + np;
#pragma omp for schedule(static)
            for (long long e = 0; e < E; ++e)
                apply_one(A, B, C, u + (size_t)e * nin, v + (size_t)e * nout, p, q,
                          n0, n1, n2, m0, m1, m2);
        }
        free(p);
    }
    return fail ? -1 : 0;
}

/*
 * Inverse Helmholtz, all E elements:
 *   v[e] = (S (x) S (x) S) ( D[e] o ( (S^T (x) S^T (x) S^T) u[e] ) ).
 * S:[n,n]   D,u,v:[E,n,n,n].
 * The forward stage applies S^T on every axis, i.e. uses S[l,i] where the
 * backward stage uses S[i,l]; St below is that transpose written out once.
 */
int oracle_inv_helmholtz_f64(const double *S, const double *D, const double *u,
                             double *v, int n, long long E, int threads)
{
    const size_t n3 = (size_t)n * n * n;
    int fail = 0;
    double *St = (double *)malloc((size_t)n * n * sizeof(double) + 8);
    if (!St) return -1;
    for (int a = 0; a < n; ++a)
        for (int b = 0; b < n; ++b)
            St[a * n + b] = S[b * n + a];
    threads = pick_threads(threads);
#pragma omp parallel num_threads(threads)
    {
        double *p = (double *)malloc((3 * n3 + 1) * sizeof(double));
        if (!p) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
            double *q = p + n3, *t = q + n3;
#pragma omp for schedule(static)
            for (long long e = 0; e < E; ++e) {
                const double *ue = u + (size_t)e * n3, *De = D + (size_t)e * n3;
                apply_one(St, St, St, ue, t, p, q, n, n, n, n, n, n);
                for (size_t x = 0; x < n3; ++x) t[x] = De[x] * t[x];
                apply_one(S, S, S, t, v + (size_t)e * n3, p, q, n, n, n, n, n, n);
            }
        }
        free(p);
    }
    free(St);
    return fail ? -1 : 0;
}

/*
 * Inverse Helmholtz with one operator per direction and its own extent per direction
 * (the per-direction matrices of Eq. 1 and of the convective-flux listing, where every
 * axis has its own small matrix), all E elements:
 *   v[e] = (S0 (x) S1 (x) S2) ( D[e] o ( (S0^T (x) S1^T (x) S2^T) u[e] ) ).
 * S0:[n0,n0] acts on the slowest in-element axis, S2:[n2,n2] on the contiguous one;
 * D,u,v:[E,n0,n1,n2].
 */
static double *transposed(const double *S, int n)
{
    double *St = (double *)malloc((size_t)n * n * sizeof(double) + 8);
    if (!St) return NULL;
    for (int a = 0; a < n; ++a)
        for (int b = 0; b < n; ++b)
            St[a * n + b] = S[b * n + a];
    return St;
}

int oracle_inv_helmholtz3_f64(const double *S0, const double *S1, const double *S2,
                              const double *D, const double *u, double *v,
                              int n0, int n1, int n2, long long E, int threads)
{
    const size_t n3 = (size_t)n0 * n1 * n2;
    int fail = 0;
    double *St0 = transposed(S0, n0), *St1 = transposed(S1, n1), *St2 = transposed(S2, n2);
    if (!St0 || !St1 || !St2) { free(St0); free(St1); free(St2); return -1; }
    threads = pick_threads(threads);
#pragma omp parallel num_threads(threads)
    {
        double *p = (double *)malloc((3 * n3 + 1) * sizeof(double));
        if (!p) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
            double *q = p + n3, *t = q + n3;
#pragma omp for schedule(static)
            for (long long e = 0; e < E; ++e) {
                const double *ue = u + (size_t)e * n3, *De = D + (size_t)e * n3;
                apply_one(St0, St1, St2, ue, t, p, q, n0, n1, n2, n0, n1, n2);
                for (size_t x = 0; x < n3; ++x) t[x] = De[x] * t[x];
                apply_one(S0, S1, S2, t, v + (size_t)e * n3, p, q, n0, n1, n2, n0, n1, n2);
            }
        }
        free(p);
    }
    free(St0); free(St1); free(St2);
    return fail ? -1 : 0;
}

/*
 * Volume integral of the convective flux (Eq. 1 of the paper and its one-statement
 * listing), sum-factorised term by term:
 *
 *   F[c,e] = (I (x) I (x) D) (M[e] o P[c,0,e]) + (I (x) D (x) I) (M[e] o P[c,1,e])
 *          + (D (x) I (x) I) (M[e] o P[c,2,e]),          c = 0,1,2
 *
 * with the first Kronecker factor on the slowest in-element axis (k/n in the listing's
 * index names) and the last on the fastest (i/l).  Dvq, Ivq: [nv,nq];  M: [E,nq,nq,nq];
 * P: [3,3,E,nq,nq,nq];  F: [3,E,nv,nv,nv].
 */
int oracle_convection_f64(const double *Dvq, const double *Ivq, const double *M, const double *P,
                          double *F, int nq, int nv, long long E, int threads)
{
    const size_t q3 = (size_t)nq * nq * nq, v3 = (size_t)nv * nv * nv;
    int fail = 0;
    threads = pick_threads(threads);
#pragma omp parallel num_threads(threads)
    {
        const size_t np = (size_t)nq * nq * nv, nqq = (size_t)nq * nv * nv;
        double *w = (double *)malloc((q3 + np + nqq + v3 + 1) * sizeof(double));
        if (!w) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
            double *x = w, *p = x + q3, *q = p + np, *t = q + nqq;
#pragma omp for schedule(static) collapse(2)
            for (int c = 0; c < 3; ++c)
                for (long long e = 0; e < E; ++e) {
                    double *Fe = F + ((size_t)c * E + e) * v3;
                    for (size_t y = 0; y < v3; ++y) Fe[y] = 0.0;
                    for (int d = 0; d < 3; ++d) {
                        const double *Pd = P + (((size_t)c * 3 + d) * E + e) * q3;
                        for (size_t y = 0; y < q3; ++y) x[y] = M[(size_t)e * q3 + y] * Pd[y];
                        /* the derivative matrix sits on the fastest axis for d = 0, the
                         * middle one for d = 1, the slowest for d = 2 */
                        const double *A = (d == 2) ? Dvq : Ivq;
                        const double *B = (d == 1) ? Dvq : Ivq;
                        const double *C = (d == 0) ? Dvq : Ivq;
                        apply_one(A, B, C, x, t, p, q, nq, nq, nq, nv, nv, nv);
                        for (size_t y = 0; y < v3; ++y) Fe[y] = Fe[y] + t[y];
                    }
                }
        }
        free(w);
    }
    return fail ? -1 : 0;
}

/* ---- the un-lifted definition ------------------------------------------- */

/* K[(i m1 + j) m2 + k , (l n1 + m) n2 + n] = A[i,l] B[j,m] C[k,n]           */
static double *kron3(const double *A, const double *B, const double *C,
                     int n0, int n1, int n2, int m0, int m1, int m2)
{
    const size_t rows = (size_t)m0 * m1 * m2, cols = (size_t)n0 * n1 * n2;
    double *K = (double *)malloc(rows * cols * sizeof(double) + 8);
    if (!K) return NULL;
    for (int i = 0; i < m0; ++i)
        for (int j = 0; j < m1; ++j)
            for (int k = 0; k < m2; ++k)
                for (int l = 0; l < n0; ++l)
                    for (int m = 0; m < n1; ++m)
                        for (int n = 0; n < n2; ++n)
                            K[(((size_t)i * m1 + j) * m2 + k) * cols +
                              ((size_t)l * n1 + m) * n2 + n] =
                                A[i * n0 + l] * B[j * n1 + m] * C[k * n2 + n];
    return K;
}

static void matvec(const double *K, const double *x, double *y, size_t rows, size_t cols)
{
    for (size_t r = 0; r < rows; ++r) {
        double s = 0.0;
        for (size_t c = 0; c < cols; ++c) s = s + K[r * cols + c] * x[c];
        y[r] = s;
    }
}

/*
 * The convective-flux integral without lifting, from the Kronecker form of Eq. 1: the three
 * explicit matrices K0 = I (x) I (x) D, K1 = I (x) D (x) I, K2 = D (x) I (x) I (each nv^3 x nq^3)
 * are built entry by entry and applied to vec(M[e] o P[c,d,e]); tiny sizes only.
 */
int oracle_convection_bruteforce_f64(const double *Dvq, const double *Ivq, const double *M,
                                     const double *P, double *F, int nq, int nv, long long E)
{
    const size_t q3 = (size_t)nq * nq * nq, v3 = (size_t)nv * nv * nv;
    double *K[3];
    K[0] = kron3(Ivq, Ivq, Dvq, nq, nq, nq, nv, nv, nv);
    K[1] = kron3(Ivq, Dvq, Ivq, nq, nq, nq, nv, nv, nv);
    K[2] = kron3(Dvq, Ivq, Ivq, nq, nq, nq, nv, nv, nv);
    double *x = (double *)malloc(q3 * sizeof(double) + 8);
    double *t = (double *)malloc(v3 * sizeof(double) + 8);
    int rc = -1;
    if (K[0] && K[1] && K[2] && x && t) {
        for (int c = 0; c < 3; ++c)
            for (long long e = 0; e < E; ++e) {
                double *Fe = F + ((size_t)c * E + e) * v3;
                for (size_t y = 0; y < v3; ++y) Fe[y] = 0.0;
                for (int d = 0; d < 3; ++d) {
                    const double *Pd = P + (((size_t)c * 3 + d) * E + e) * q3;
                    for (size_t y = 0; y < q3; ++y) x[y] = M[(size_t)e * q3 + y] * Pd[y];
                    matvec(K[d], x, t, v3, q3);
                    for (size_t y = 0; y < v3; ++y) Fe[y] = Fe[y] + t[y];
                }
            }
        rc = 0;
    }
    free(K[0]); free(K[1]); free(K[2]); free(x); free(t);
    return rc;
}

/* v[e] = kron(A,B,C) vec(u[e]) with the explicit matrix; tiny sizes only.   */
int oracle_tpo_apply_bruteforce_f64(const double *A, const double *B, const double *C,
                                    const double *u, double *v,
                                    int n0, int n1, int n2, int m0, int m1, int m2,
                                    long long E)
{
    const size_t rows = (size_t)m0 * m1 * m2, cols = (size_t)n0 * n1 * n2;
    double *K = kron3(A, B, C, n0, n1, n2, m0, m1, m2);
    if (!K) return -1;
    for (long long e = 0; e < E; ++e)
        matvec(K, u + (size_t)e * cols, v + (size_t)e * rows, rows, cols);
    free(K);
    return 0;
}

/* v[e] = K2 diag(vec D[e]) K1 vec(u[e]),  K1 = kron(S^T,S^T,S^T), K2 = kron(S,S,S). */
int oracle_inv_helmholtz_bruteforce_f64(const double *S, const double *D, const double *u,
                                        double *v, int n, long long E)
{
    const size_t n3 = (size_t)n * n * n;
    double *St = (double *)malloc((size_t)n * n * sizeof(double) + 8);
    double *t = (double *)malloc(n3 * sizeof(double) + 8);
    if (!St || !t) { free(St); free(t); return -1; }
    for (int a = 0; a < n; ++a)
        for (int b = 0; b < n; ++b)
            St[a * n + b] = S[b * n + a];
    double *K1 = kron3(St, St, St, n, n, n, n, n, n);
    double *K2 = kron3(S, S, S, n, n, n, n, n, n);
    if (!K1 || !K2) { free(K1); free(K2); free(St); free(t); return -1; }
    for (long long e = 0; e < E; ++e) {
        matvec(K1, u + (size_t)e * n3, t, n3, n3);
        for (size_t x = 0; x < n3; ++x) t[x] = D[(size_t)e * n3 + x] * t[x];
        matvec(K2, t, v + (size_t)e * n3, n3, n3);
    }
    free(K1); free(K2); free(St); free(t);
    return 0;
}

/* v[e] = K2 diag(vec D[e]) K1 vec(u[e]),  K1 = kron(S0^T,S1^T,S2^T), K2 = kron(S0,S1,S2). */
int oracle_inv_helmholtz3_bruteforce_f64(const double *S0, const double *S1, const double *S2,
                                         const double *D, const double *u, double *v,
                                         int n0, int n1, int n2, long long E)
{
    const size_t n3 = (size_t)n0 * n1 * n2;
    double *St0 = transposed(S0, n0), *St1 = transposed(S1, n1), *St2 = transposed(S2, n2);
    double *t = (double *)malloc(n3 * sizeof(double) + 8);
    double *K1 = NULL, *K2 = NULL;
    int rc = -1;
    if (St0 && St1 && St2 && t) {
        K1 = kron3(St0, St1, St2, n0, n1, n2, n0, n1, n2);
        K2 = kron3(S0, S1, S2, n0, n1, n2, n0, n1, n2);
    }
    if (K1 && K2) {
        for (long long e = 0; e < E; ++e) {
            matvec(K1, u + (size_t)e * n3, t, n3, n3);
            for (size_t x = 0; x < n3; ++x) t[x] = D[(size_t)e * n3 + x] * t[x];
            matvec(K2, t, v + (size_t)e * n3, n3, n3);
        }
        rc = 0;
    }
    free(K1); free(K2); free(St0); free(St1); free(St2); free(t);
    return rc;
}

/* ---- extended-precision re-evaluation (accuracy level of the oracle) ----- */

static void apply_one_ld(const long double *A, const long double *B, const long double *C,
                         const long double *u, long double *v, long double *p, long double *q,
                         int n0, int n1, int n2, int m0, int m1, int m2)
{
    for (int l = 0; l < n0; ++l)
        for (int m = 0; m < n1; ++m)
            for (int k = 0; k < m2; ++k) {
                long double s = 0.0L;
                for (int n = 0; n < n2; ++n) s += C[k * n2 + n] * u[(l * n1 + m) * n2 + n];
                p[(l * n1 + m) * m2 + k] = s;
            }
    for (int l = 0; l < n0; ++l)
        for (int j = 0; j < m1; ++j)
            for (int k = 0; k < m2; ++k) {
                long double s = 0.0L;
                for (int m = 0; m < n1; ++m) s += B[j * n1 + m] * p[(l * n1 + m) * m2 + k];
                q[(l * m1 + j) * m2 + k] = s;
            }
    for (int i = 0; i < m0; ++i)
        for (int j = 0; j < m1; ++j)
            for (int k = 0; k < m2; ++k) {
                long double s = 0.0L;
                for (int l = 0; l < n0; ++l) s += A[i * n0 + l] * q[(l * m1 + j) * m2 + k];
                v[(i * m1 + j) * m2 + k] = s;
            }
}

/* Same operator as oracle_inv_helmholtz_f64, every intermediate in long double
 * (x87 80-bit on this platform); output rounded to double once at the end. */
int oracle_inv_helmholtz_ld(const double *S, const double *D, const double *u,
                            double *v, int n, long long E)
{
    const size_t n3 = (size_t)n * n * n, n2 = (size_t)n * n;
    long double *w = (long double *)malloc((2 * n2 + 5 * n3 + 1) * sizeof(long double));
    if (!w) return -1;
    long double *Sl = w, *St = Sl + n2, *ul = St + n2, *t = ul + n3, *p = t + n3,
                *q = p + n3, *vl = q + n3;
    for (int a = 0; a < n; ++a)
        for (int b = 0; b < n; ++b) {
            Sl[a * n + b] = S[a * n + b];
            St[a * n + b] = S[b * n + a];
        }
    for (long long e = 0; e < E; ++e) {
        for (size_t x = 0; x < n3; ++x) ul[x] = u[(size_t)e * n3 + x];
        apply_one_ld(St, St, St, ul, t, p, q, n, n, n, n, n, n);
        for (size_t x = 0; x < n3; ++x) t[x] = (long double)D[(size_t)e * n3 + x] * t[x];
        apply_one_ld(Sl, Sl, Sl, t, vl, p, q, n, n, n, n, n, n);
        for (size_t x = 0; x < n3; ++x) v[(size_t)e * n3 + x] = (double)vl[x];
    }
    free(w);
    return 0;
}

int oracle_tpo_apply_ld(const double *A, const double *B, const double *C,
                        const double *u, double *v,
                        int n0, int n1, int n2, int m0, int m1, int m2, long long E)
{
    const size_t nin = (size_t)n0 * n1 * n2, nout = (size_t)m0 * m1 * m2;
    const size_t np = (size_t)n0 * n1 * m2, nq = (size_t)n0 * m1 * m2;
    const size_t na = (size_t)m0 * n0, nb = (size_t)m1 * n1, nc = (size_t)m2 * n2;
    long double *w = (long double *)malloc((na + nb + nc + nin + nout + np + nq + 1) *
                                           sizeof(long double));
    if (!w) return -1;
    long double *Al = w, *Bl = Al + na, *Cl = Bl + nb, *ul = Cl + nc, *vl = ul + nin,
                *p = vl + nout, *q = p + np;
    for (size_t x = 0; x < na; ++x) Al[x] = A[x];
    for (size_t x = 0; x < nb; ++x) Bl[x] = B[x];
    for (size_t x = 0; x < nc; ++x) Cl[x] = C[x];
    for (long long e = 0; e < E; ++e) {
        for (size_t x = 0; x < nin; ++x) ul[x] = u[(size_t)e * nin + x];
        apply_one_ld(Al, Bl, Cl, ul, vl, p, q, n0, n1, n2, m0, m1, m2);
        for (size_t x = 0; x < nout; ++x) v[(size_t)e * nout + x] = (double)vl[x];
    }
    free(w);
    return 0;
}
