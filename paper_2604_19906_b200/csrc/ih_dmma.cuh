// Inverse Helmholtz on the FP64 tensor path (mma.sync m8n8k4 .f64), one CTA per pair of
// elements, persistent over the element range.
//
// Every mode contraction of the lifted sums (Section 5.2) is a small GEMM
//     Out[q][o] = sum_x In[q][x] * M[x][o],   q = pencil (N*N per element), x,o in [0,N)
// computed transposed as  Out^T = M^T * In^T  so that the operator matrix is the A operand
// and lives in registers for the whole kernel, the data pencils are the B operand read
// from shared memory (8 pencils x 4 contraction indices per tile), and each lane ends up
// with one output index o and two neighbouring pencils.
//
// Shared-memory layout of a stage's input: [x][q] with the contraction axis slowest
// (stride N*N) and the pencils contiguous.  A stage whose pencils are (p1,p2) writes its
// output o to  p1*N*N + p2*N + o,  which is again of that form for the next stage: it
// contracts p1 with pencils (p2,o).  Three such stages cycle i -> j -> k and return to the
// natural [i][j][k] order, so u can be bulk-copied in untouched, D and v are addressed in
// their natural order, and for N = 2 or 6 (mod 8) every shared access is conflict-free.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace ekl {

// Set by a kernel whose bounded wait on a bulk copy gave up (never expected in practice).
__device__ int g_ih_dmma_timeout = 0;

namespace dmma {

__device__ __forceinline__ void mma_f64(double& c0, double& c1, double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(c0), "+d"(c1)
                 : "d"(a), "d"(b));
}

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)),
                 "r"(bytes)
                 : "memory");
}

// Bounded wait on a phase of the barrier; false if it gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity) {
    const uint32_t a = smem_addr(bar);
    for (unsigned it = 0; it < (1u << 24); ++it) {
        unsigned done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(a), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}

// Plain (non-multicast) bulk copy global -> this CTA's shared memory, completing on `bar`.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes,
                                          uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}

__device__ __forceinline__ void bulk_prefetch_l2(const void* src, unsigned bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

__device__ __forceinline__ void fence_async_proxy() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

template <int N>
struct Cfg {
    static constexpr int kBe = 2;                       // elements per CTA batch
    static constexpr int kN2 = N * N, kN3 = N * N * N;
    static constexpr int kTiles = kBe * kN2 / 8;        // 8-pencil tiles per stage
    static constexpr int kWarps = (N == 14) ? 7 : (N == 10 ? 5 : (N == 6 ? 3 : 4));
    static constexpr int kTilesPerWarp = (kTiles + kWarps - 1) / kWarps;
    static constexpr int kThreads = 32 * kWarps;
    static constexpr int kKSteps = (N + 3) / 4;         // last step overlaps the previous one
    static constexpr int kMTiles = (N + 7) / 8;
    static constexpr int kBufElems = kBe * kN3;
    static constexpr size_t kSmemBytes = 2 * (size_t)kBufElems * sizeof(double) + 16;
    static_assert(N % 2 == 0 && N >= 4, "even N >= 4");
    static_assert((kBe * kN2) % 8 == 0, "whole tiles");
    __host__ __device__ static constexpr int k0(int s) { return (4 * s + 4 <= N) ? 4 * s : N - 4; }
};

// One contraction stage over the CTA's batch.  MODE 0: shared -> shared.  MODE 1: shared ->
// shared with the pointwise factor (already in registers, dreg).  MODE 2: shared -> global.
template <int N, int MODE>
__device__ __forceinline__ void stage(const double* __restrict__ in, double* __restrict__ out,
                                      const double (&af)[Cfg<N>::kMTiles][Cfg<N>::kKSteps],
                                      const double* dreg, double* __restrict__ gout,
                                      int valid_pencils, int warp, int lane) {
    using C = Cfg<N>;
    const int r = lane >> 2, kk = lane & 3;
#pragma unroll
    for (int tt = 0; tt < C::kTilesPerWarp; ++tt) {
        const int t = warp * C::kTilesPerWarp + tt;
        if (t >= C::kTiles) break;
        const int q0 = 8 * t;
        // B fragments: pencil q0+r, contraction index k0(s)+kk
        const int qb = q0 + r;
        const int eb = qb / C::kN2;
        const double* src = in + eb * C::kN3 + (qb - eb * C::kN2) + kk * C::kN2;
        double b[C::kKSteps];
#pragma unroll
        for (int s = 0; s < C::kKSteps; ++s) b[s] = src[C::k0(s) * C::kN2];
        double c[C::kMTiles][2];
#pragma unroll
        for (int mt = 0; mt < C::kMTiles; ++mt) {
            c[mt][0] = 0.0;
            c[mt][1] = 0.0;
#pragma unroll
            for (int s = 0; s < C::kKSteps; ++s) mma_f64(c[mt][0], c[mt][1], af[mt][s], b[s]);
        }
        // this lane: output index o = 8*mt + r, pencils q0 + 2*kk + {0,1}
        const int qs = q0 + 2 * kk;
        const int es = qs / C::kN2;
        const int p = qs - es * C::kN2;
        if (MODE == 2) {
            if (qs < valid_pencils) {
                double* g = gout + (size_t)es * C::kN3 + p * N;
#pragma unroll
                for (int mt = 0; mt < C::kMTiles; ++mt) {
                    const int o = 8 * mt + r;
                    if (o < N) {
                        g[o] = c[mt][0];
                        g[N + o] = c[mt][1];
                    }
                }
            }
        } else {
            const int p1 = p / N, p2 = p - p1 * N;
            double* dst = out + es * C::kN3 + p1 * C::kN2 + p2 * N;
#pragma unroll
            for (int mt = 0; mt < C::kMTiles; ++mt) {
                const int o = 8 * mt + r;
                if (o < N) {
                    double v0 = c[mt][0], v1 = c[mt][1];
                    if (MODE == 1) {
                        v0 *= dreg[(tt * C::kMTiles + mt) * 2 + 0];
                        v1 *= dreg[(tt * C::kMTiles + mt) * 2 + 1];
                    }
                    dst[o] = v0;
                    dst[N + o] = v1;
                }
            }
        }
    }
}

template <int N>
__global__ void __launch_bounds__(Cfg<N>::kThreads, 2)
inv_helmholtz_dmma(const double* __restrict__ S, const double* __restrict__ D,
                   const double* u, double* v, long long E) {
    using C = Cfg<N>;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    double* bufA = reinterpret_cast<double*>(smem_raw);
    double* bufB = bufA + C::kBufElems;
    uint64_t* bar = reinterpret_cast<uint64_t*>(bufB + C::kBufElems);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = lane >> 2, kk = lane & 3;

    // Operator matrix as A fragments: forward stages apply S^T (A[o][x] = S[x][o]),
    // backward stages apply S (A[o][x] = S[o][x]).  In the overlapped last k-step only the
    // contraction indices not covered by the previous step carry values.
    double af_f[C::kMTiles][C::kKSteps], af_b[C::kMTiles][C::kKSteps];
#pragma unroll
    for (int mt = 0; mt < C::kMTiles; ++mt) {
#pragma unroll
        for (int s = 0; s < C::kKSteps; ++s) {
            const int o = 8 * mt + r, x = C::k0(s) + kk;
            const bool fresh = (s == 0) || (x >= C::k0(s - 1) + 4);
            const bool ok = (o < N) && fresh;
            af_f[mt][s] = ok ? S[x * N + o] : 0.0;
            af_b[mt][s] = ok ? S[o * N + x] : 0.0;
        }
    }

    const long long n_batches = (E + C::kBe - 1) / C::kBe;
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    long long batch = blockIdx.x;
    if (threadIdx.x == 0 && batch < n_batches) {
        const long long e0 = batch * C::kBe;
        const unsigned cnt = (unsigned)((E - e0 < C::kBe) ? (E - e0) : C::kBe);
        const unsigned bytes = cnt * C::kN3 * (unsigned)sizeof(double);
        mbar_expect_tx(bar, bytes);
        bulk_load(bufA, u + e0 * C::kN3, bytes, bar);
    }
    unsigned parity = 0;
    for (; batch < n_batches; batch += gridDim.x) {
        const long long e0 = batch * C::kBe;
        const int cnt = (int)((E - e0 < C::kBe) ? (E - e0) : C::kBe);
        const int valid = cnt * C::kN2;
        const double* Db = D + e0 * C::kN3;
        double* vb = v + e0 * C::kN3;
        const long long next = batch + gridDim.x;
        if (threadIdx.x == 0) {
            bulk_prefetch_l2(Db, (unsigned)(cnt * C::kN3 * sizeof(double)));
            if (next < n_batches) {
                const long long ne0 = next * C::kBe;
                const unsigned ncnt = (unsigned)((E - ne0 < C::kBe) ? (E - ne0) : C::kBe);
                bulk_prefetch_l2(u + ne0 * C::kN3, ncnt * C::kN3 * (unsigned)sizeof(double));
            }
        }
        // All threads take the same decision; a wait that gave up flags the error, waits
        // once more (bounded) for the copy still in flight and leaves.
        if (__syncthreads_or(mbar_wait(bar, parity) ? 0 : 1)) {
            if (threadIdx.x == 0) g_ih_dmma_timeout = 1;
            mbar_wait(bar, parity);
            break;
        }
        parity ^= 1u;
        // forward: contract i, j, k
        stage<N, 0>(bufA, bufB, af_f, nullptr, nullptr, valid, warp, lane);
        __syncthreads();
        // pointwise factor for this lane's outputs of the third stage, fetched one stage early
        double dreg[C::kTilesPerWarp * C::kMTiles * 2];
#pragma unroll
        for (int tt = 0; tt < C::kTilesPerWarp; ++tt) {
            const int t = warp * C::kTilesPerWarp + tt;
            const int qs = 8 * t + 2 * kk;
            const bool live = (t < C::kTiles) && (qs < valid);
            const int es = qs / C::kN2;
            const int p = qs - es * C::kN2;
            const double* g = Db + (size_t)es * C::kN3 + p * N;
#pragma unroll
            for (int mt = 0; mt < C::kMTiles; ++mt) {
                const int o = 8 * mt + r;
                const bool ld = live && (o < N);
                dreg[(tt * C::kMTiles + mt) * 2 + 0] = ld ? g[o] : 0.0;
                dreg[(tt * C::kMTiles + mt) * 2 + 1] = ld ? g[N + o] : 0.0;
            }
        }
        stage<N, 0>(bufB, bufA, af_f, nullptr, nullptr, valid, warp, lane);
        __syncthreads();
        stage<N, 1>(bufA, bufB, af_f, dreg, nullptr, valid, warp, lane);
        __syncthreads();
        // backward: contract i, j, k
        stage<N, 0>(bufB, bufA, af_b, nullptr, nullptr, valid, warp, lane);
        __syncthreads();
        stage<N, 0>(bufA, bufB, af_b, nullptr, nullptr, valid, warp, lane);
        __syncthreads();
        // bufA is free: bring in the next batch while the last stage streams v out
        if (threadIdx.x == 0 && next < n_batches) {
            const long long ne0 = next * C::kBe;
            const unsigned ncnt = (unsigned)((E - ne0 < C::kBe) ? (E - ne0) : C::kBe);
            const unsigned bytes = ncnt * C::kN3 * (unsigned)sizeof(double);
            fence_async_proxy();
            mbar_expect_tx(bar, bytes);
            bulk_load(bufA, u + ne0 * C::kN3, bytes, bar);
        }
        stage<N, 2>(bufB, nullptr, af_b, nullptr, vb, valid, warp, lane);
        __syncthreads();
    }
}

}  // namespace dmma
}  // namespace ekl
