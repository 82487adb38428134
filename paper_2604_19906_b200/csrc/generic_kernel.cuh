// Run-time-sized kernels: any extents that fit in shared memory, fp64 or fp32.
//
// One CTA owns one element at a time (grid-stride loop over elements).  The element is
// staged in shared memory, the small operator matrices stay resident there for the
// life of the CTA, and the mode contractions of the lifted sums (Section 5.2) ping-pong
// between two shared buffers; only u (and D) are read from and v written to HBM.
// These kernels are the fallback for shapes that have no tuned instance.
#pragma once
#include <cuda_runtime.h>

namespace ekl {

// out[a,b,c] (extents with `axis` replaced by mo) = sum_x M(o,x) * in[...x...]
// M(o,x) = Mat[o*rs + x*cs]  (rs/cs let the same storage serve as S or S^T).
template <typename T, typename Out>
__device__ __forceinline__ void contract_axis(const T* __restrict__ in, Out* __restrict__ out,
                                              const T* __restrict__ Mat, int rs, int cs,
                                              int d0, int d1, int d2, int axis, int mo,
                                              const T* __restrict__ scale) {
    const int e0 = axis == 0 ? mo : d0, e1 = axis == 1 ? mo : d1, e2 = axis == 2 ? mo : d2;
    const int din = axis == 0 ? d0 : (axis == 1 ? d1 : d2);
    const int in_stride = axis == 0 ? d1 * d2 : (axis == 1 ? d2 : 1);
    const int total = e0 * e1 * e2;
    for (int x = threadIdx.x; x < total; x += blockDim.x) {
        const int c = x % e2, b = (x / e2) % e1, a = x / (e2 * e1);
        const int o = axis == 0 ? a : (axis == 1 ? b : c);
        const int base = axis == 0 ? b * d2 + c : (axis == 1 ? a * d1 * d2 + c : (a * d1 + b) * d2);
        T s = T(0);
        for (int y = 0; y < din; ++y) s = fma(Mat[o * rs + y * cs], in[base + y * in_stride], s);
        if (scale) s *= scale[x];
        out[x] = s;
    }
}

// v[e] = (S(x)S(x)S)(D[e] o ((S^T(x)S^T(x)S^T) u[e]))
template <typename T>
__global__ void inv_helmholtz_generic(const T* __restrict__ S, const T* __restrict__ D,
                                      const T* u, T* v, int n, long long E) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* sS = reinterpret_cast<T*>(smem_raw);
    const int n3 = n * n * n;
    T* b0 = sS + n * n;
    T* b1 = b0 + n3;
    for (int x = threadIdx.x; x < n * n; x += blockDim.x) sS[x] = S[x];
    for (long long e = blockIdx.x; e < E; e += gridDim.x) {
        const T* ue = u + e * n3;
        const T* De = D + e * n3;
        __syncthreads();  // previous element's reads of b0/b1 are done; sS is visible
        for (int x = threadIdx.x; x < n3; x += blockDim.x) b0[x] = ue[x];
        __syncthreads();
        contract_axis<T, T>(b0, b1, sS, 1, n, n, n, n, 2, n, nullptr);   // S^T on the fast axis
        __syncthreads();
        contract_axis<T, T>(b1, b0, sS, 1, n, n, n, n, 1, n, nullptr);
        __syncthreads();
        contract_axis<T, T>(b0, b1, sS, 1, n, n, n, n, 0, n, De);        // ... and times D[e]
        __syncthreads();
        contract_axis<T, T>(b1, b0, sS, n, 1, n, n, n, 2, n, nullptr);   // S on the fast axis
        __syncthreads();
        contract_axis<T, T>(b0, b1, sS, n, 1, n, n, n, 1, n, nullptr);
        __syncthreads();
        contract_axis<T, T>(b1, v + e * n3, sS, n, 1, n, n, n, 0, n, nullptr);
    }
}

// v[e] = (S0(x)S1(x)S2)(D[e] o ((S0^T(x)S1^T(x)S2^T) u[e])): one operator and one extent per
// direction, S0 on the slowest in-element axis.
template <typename T>
__global__ void inv_helmholtz3_generic(const T* __restrict__ S0, const T* __restrict__ S1,
                                       const T* __restrict__ S2, const T* __restrict__ D,
                                       const T* u, T* v, int n0, int n1, int n2, long long E) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* s0 = reinterpret_cast<T*>(smem_raw);
    T* s1 = s0 + n0 * n0;
    T* s2 = s1 + n1 * n1;
    const int n3 = n0 * n1 * n2;
    T* b0 = s2 + n2 * n2;
    T* b1 = b0 + n3;
    for (int x = threadIdx.x; x < n0 * n0; x += blockDim.x) s0[x] = S0[x];
    for (int x = threadIdx.x; x < n1 * n1; x += blockDim.x) s1[x] = S1[x];
    for (int x = threadIdx.x; x < n2 * n2; x += blockDim.x) s2[x] = S2[x];
    for (long long e = blockIdx.x; e < E; e += gridDim.x) {
        const T* ue = u + e * n3;
        const T* De = D + e * n3;
        __syncthreads();
        for (int x = threadIdx.x; x < n3; x += blockDim.x) b0[x] = ue[x];
        __syncthreads();
        contract_axis<T, T>(b0, b1, s2, 1, n2, n0, n1, n2, 2, n2, nullptr);   // S2^T, fast axis
        __syncthreads();
        contract_axis<T, T>(b1, b0, s1, 1, n1, n0, n1, n2, 1, n1, nullptr);
        __syncthreads();
        contract_axis<T, T>(b0, b1, s0, 1, n0, n0, n1, n2, 0, n0, De);        // ... and times D[e]
        __syncthreads();
        contract_axis<T, T>(b1, b0, s2, n2, 1, n0, n1, n2, 2, n2, nullptr);   // S2, fast axis
        __syncthreads();
        contract_axis<T, T>(b0, b1, s1, n1, 1, n0, n1, n2, 1, n1, nullptr);
        __syncthreads();
        contract_axis<T, T>(b1, v + e * n3, s0, n0, 1, n0, n1, n2, 0, n0, nullptr);
    }
}

// v[e] = (A(x)B(x)C) u[e], contraction order C, B, A.
template <typename T>
__global__ void apply_generic(const T* __restrict__ A, const T* __restrict__ B,
                              const T* __restrict__ C, const T* __restrict__ u,
                              T* __restrict__ v, int n0, int n1, int n2, int m0, int m1, int m2,
                              int buf_elems, long long E) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* sA = reinterpret_cast<T*>(smem_raw);
    T* sB = sA + m0 * n0;
    T* sC = sB + m1 * n1;
    T* b0 = sC + m2 * n2;
    T* b1 = b0 + buf_elems;
    for (int x = threadIdx.x; x < m0 * n0; x += blockDim.x) sA[x] = A[x];
    for (int x = threadIdx.x; x < m1 * n1; x += blockDim.x) sB[x] = B[x];
    for (int x = threadIdx.x; x < m2 * n2; x += blockDim.x) sC[x] = C[x];
    const int nin = n0 * n1 * n2;
    const long long nout = (long long)m0 * m1 * m2;
    for (long long e = blockIdx.x; e < E; e += gridDim.x) {
        const T* ue = u + e * nin;
        __syncthreads();
        for (int x = threadIdx.x; x < nin; x += blockDim.x) b0[x] = ue[x];
        __syncthreads();
        contract_axis<T, T>(b0, b1, sC, n2, 1, n0, n1, n2, 2, m2, nullptr);
        __syncthreads();
        contract_axis<T, T>(b1, b0, sB, n1, 1, n0, n1, m2, 1, m1, nullptr);
        __syncthreads();
        contract_axis<T, T>(b0, v + e * nout, sA, n0, 1, n0, m1, m2, 0, m0, nullptr);
    }
}

// F[c,e] = (I(x)I(x)D)(M[e] o P[c,0,e]) + (I(x)D(x)I)(M[e] o P[c,1,e]) + (D(x)I(x)I)(M[e] o P[c,2,e])
// for run-time extents: one CTA per (component, element) pair at a time, the three forward
// operators evaluated one after the other and summed in a shared accumulator.
template <typename T>
__global__ void convection_generic(const T* __restrict__ Dvq, const T* __restrict__ Ivq,
                                   const T* __restrict__ M, const T* __restrict__ P,
                                   T* __restrict__ F, int nq, int nv, int buf_elems, long long E) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* sD = reinterpret_cast<T*>(smem_raw);
    T* sI = sD + nv * nq;
    T* b0 = sI + nv * nq;
    T* b1 = b0 + buf_elems;
    T* acc = b1 + buf_elems;
    for (int x = threadIdx.x; x < nv * nq; x += blockDim.x) {
        sD[x] = Dvq[x];
        sI[x] = Ivq[x];
    }
    const int q3 = nq * nq * nq, v3 = nv * nv * nv;
    for (long long w = blockIdx.x; w < 3 * E; w += gridDim.x) {
        const long long c = w / E, e = w - c * E;
        const T* Me = M + e * q3;
        for (int d = 0; d < 3; ++d) {
            const T* Pd = P + ((c * 3 + d) * E + e) * q3;
            __syncthreads();  // b0, b1 and acc of the previous pass are no longer read
            for (int x = threadIdx.x; x < q3; x += blockDim.x) b0[x] = Me[x] * Pd[x];
            __syncthreads();
            // the derivative matrix sits on the fastest axis for d = 0, the slowest for d = 2
            contract_axis<T, T>(b0, b1, d == 0 ? sD : sI, nq, 1, nq, nq, nq, 2, nv, nullptr);
            __syncthreads();
            contract_axis<T, T>(b1, b0, d == 1 ? sD : sI, nq, 1, nq, nq, nv, 1, nv, nullptr);
            __syncthreads();
            contract_axis<T, T>(b0, b1, d == 2 ? sD : sI, nq, 1, nq, nv, nv, 0, nv, nullptr);
            __syncthreads();
            for (int x = threadIdx.x; x < v3; x += blockDim.x)
                acc[x] = (d == 0) ? b1[x] : acc[x] + b1[x];
        }
        __syncthreads();
        T* Fe = F + (c * E + e) * v3;
        for (int x = threadIdx.x; x < v3; x += blockDim.x) Fe[x] = acc[x];
    }
}

}  // namespace ekl
