// Sum-factorised tensor-product operators on the FP64 tensor path (mma.sync m8n8k4 .f64):
// persistent CTAs, each owning a small batch of elements at a time.
//
// Every mode contraction of the lifted sums (Section 5.2) is a small GEMM
//     Out[q][o] = sum_x In[q][x] * M[x][o],    q = pencil, x = contraction index, o = output index
// evaluated transposed, Out^T = M^T * In^T, so that
//   - the operator matrix is the A operand (rows o, columns x) and stays in registers,
//   - the data is the B operand, 8 pencils x 4 contraction indices per instruction, read from
//     shared memory,
//   - each lane ends up with one output index o (= 8*mt + lane/4) and two neighbouring
//     pencils (8*tile + 2*(lane%4) + {0,1}).
//
// Shared-memory layout of a stage's input, per element: [x][q], contraction axis slowest,
// pencils contiguous, q = p1*E2 + p2 over the two other axes.  The stage writes its output
// to q*O + o = p1*(E2*O) + p2*O + o, which is again of that form for the next stage: it
// contracts p1 over pencils (p2,o).  Three stages therefore cycle through the axes
// i -> j -> k and end in the natural [i][j][k] order, so the input field is bulk-copied in
// untouched and the pointwise factor and the output are addressed in their natural order.
// With N = 2 or 6 (mod 8) every shared access of the stages is bank-conflict free.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace ekl {
namespace dmma {

// Set by a kernel whose bounded wait on a bulk copy gave up (not expected in practice).
__device__ int g_bulk_wait_timeout = 0;

__device__ __forceinline__ void mma_f64(double& c0, double& c1, double a, double b) {
    asm("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
        : "+d"(c0), "+d"(c1)
        : "d"(a), "d"(b));
}

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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

// All threads of the CTA wait for the bulk copy of this phase.  Returns false, after
// flagging the error and waiting once more (bounded) for the copy still in flight, if the
// wait gave up; the decision is the same for every thread.
__device__ __forceinline__ bool wait_bulk(uint64_t* bar, unsigned parity) {
    if (__syncthreads_or(mbar_wait(bar, parity) ? 0 : 1)) {
        if (threadIdx.x == 0) g_bulk_wait_timeout = 1;
        mbar_wait(bar, parity);
        return false;
    }
    return true;
}

// One contraction stage for a batch of BE elements worked on by WARPS warps:
// input [K][E1][E2] per element, output [E1][E2][O].
template <int K_, int O_, int E1_, int E2_, int BE_, int WARPS_>
struct Stage {
    static constexpr int K = K_, O = O_, BE = BE_, WARPS = WARPS_;
    static constexpr int kP = E1_ * E2_;                  // pencils per element
    static constexpr int kIn = K * kP, kOut = O * kP;     // values per element
    static constexpr int kPencils = BE * kP;
    static constexpr int kTiles = (kPencils + 7) / 8;     // 8-pencil tiles, the last may be ragged
    static constexpr int kTilesPerWarp = (kTiles + WARPS - 1) / WARPS;
    static constexpr int kKSteps = (K + 3) / 4;
    static constexpr int kMTiles = (O + 7) / 8;
    static_assert(K >= 4, "contraction extent below one tensor step");
    static_assert(kP % 2 == 0, "pencil pairs must not straddle elements");
    // first contraction index of tensor step s; a last partial step overlaps the previous one
    __host__ __device__ static constexpr int k0(int s) { return (4 * s + 4 <= K) ? 4 * s : K - 4; }
};

// The operator matrix as this lane sees it: A[o][x], o = 8*mt + lane/4, x = k0(s) + lane%4.
template <class SS>
struct OpFrag {
    double a[SS::kMTiles][SS::kKSteps];
};

// out_major: the matrix is stored [O][K] (A[o][x] = M[o*K + x]); otherwise [K][O], i.e. the
// stage applies the transpose of the stored matrix (A[o][x] = M[x*O + o]).
template <class SS>
__device__ __forceinline__ void load_op(OpFrag<SS>& f, const double* __restrict__ M, bool out_major,
                                        int lane) {
    const int r = lane >> 2, kk = lane & 3;
#pragma unroll
    for (int mt = 0; mt < SS::kMTiles; ++mt) {
        const int o = 8 * mt + r;
#pragma unroll
        for (int s = 0; s < SS::kKSteps; ++s) {
            // an overlapping last step carries only the indices the previous one did not
            const int x = SS::k0(s) + kk;
            const bool fresh = (s == 0) || (x >= SS::k0(s - 1) + 4);
            f.a[mt][s] =
                (o < SS::O && fresh) ? __ldg(out_major ? M + o * SS::K + x : M + x * SS::O + o) : 0.0;
        }
    }
}

// Tiles are dealt to the warps round-robin; is slot `slot` of this warp a real tile?
template <class SS>
__device__ __forceinline__ bool tile_live(int warp, int slot, int& t) {
    t = warp + SS::WARPS * slot;
    return slot < SS::kTilesPerWarp && t < SS::kTiles;
}

// The pointwise factor for the outputs this lane holds of tile slot `slot`.
template <class SS>
__device__ __forceinline__ void load_factor(double (&d)[SS::kMTiles][2],
                                            const double* __restrict__ Db, int valid_pencils,
                                            int warp, int slot, int lane) {
    const int r = lane >> 2, kk = lane & 3;
    int t;
    const bool live = tile_live<SS>(warp, slot, t);
    const int qs = 8 * t + 2 * kk;
    const double* g = Db + (size_t)qs * SS::O;     // element e, pencil q: e*kOut + q*O
#pragma unroll
    for (int mt = 0; mt < SS::kMTiles; ++mt) {
        const int o = 8 * mt + r;
        const bool ld = live && (qs < valid_pencils) && (o < SS::O);
        d[mt][0] = ld ? __ldg(g + o) : 0.0;
        d[mt][1] = ld ? __ldg(g + SS::O + o) : 0.0;
    }
}

// MODE 0: shared -> shared.  MODE 1: shared -> shared, times the pointwise factor (dfac
// holds it for the warp's first tile on entry; later tiles are fetched one tile ahead from
// Db).  MODE 2: shared -> global (gout).  `valid_pencils` masks a partly filled batch.
template <class SS, int MODE>
__device__ __forceinline__ void run_stage(const double* __restrict__ in, double* __restrict__ out,
                                          const OpFrag<SS>& op, double (&dfac)[SS::kMTiles][2],
                                          const double* __restrict__ Db, double* __restrict__ gout,
                                          int valid_pencils, int warp, int lane) {
    const int r = lane >> 2, kk = lane & 3;
#pragma unroll
    for (int slot = 0; slot < SS::kTilesPerWarp; ++slot) {
        int t;
        if (!tile_live<SS>(warp, slot, t)) break;
        // B fragments: pencil 8t + r, contraction index k0(s) + kk
        int qb = 8 * t + r;
        if (qb >= SS::kPencils) qb = 0;                    // ragged last tile: any valid pencil
        const int eb = qb / SS::kP;
        const double* src = in + eb * SS::kIn + (qb - eb * SS::kP) + kk * SS::kP;
        double b[SS::kKSteps];
#pragma unroll
        for (int s = 0; s < SS::kKSteps; ++s) b[s] = src[SS::k0(s) * SS::kP];
        double dn[SS::kMTiles][2];
        if (MODE == 1 && slot + 1 < SS::kTilesPerWarp)
            load_factor<SS>(dn, Db, valid_pencils, warp, slot + 1, lane);
        double c[SS::kMTiles][2];
#pragma unroll
        for (int mt = 0; mt < SS::kMTiles; ++mt) {
            c[mt][0] = c[mt][1] = 0.0;
#pragma unroll
            for (int s = 0; s < SS::kKSteps; ++s) mma_f64(c[mt][0], c[mt][1], op.a[mt][s], b[s]);
        }
        // this lane: output index o = 8*mt + r of pencils 8t + 2*kk + {0,1}; in a batch the
        // output of element e, pencil q sits at e*kOut + q*O + o = (e*kP + q)*O + o
        const int qs = 8 * t + 2 * kk;
        const bool ok = (MODE == 2) ? (qs < valid_pencils) : (qs < SS::kPencils);
        if (ok) {
            double* dst = ((MODE == 2) ? gout : out) + (size_t)qs * SS::O;
#pragma unroll
            for (int mt = 0; mt < SS::kMTiles; ++mt) {
                const int o = 8 * mt + r;
                if (o < SS::O) {
                    dst[o] = (MODE == 1) ? c[mt][0] * dfac[mt][0] : c[mt][0];
                    dst[SS::O + o] = (MODE == 1) ? c[mt][1] * dfac[mt][1] : c[mt][1];
                }
            }
        }
        if (MODE == 1 && slot + 1 < SS::kTilesPerWarp) {
#pragma unroll
            for (int mt = 0; mt < SS::kMTiles; ++mt) {
                dfac[mt][0] = dn[mt][0];
                dfac[mt][1] = dn[mt][1];
            }
        }
    }
}

// ------------------------------------------------------------------ inverse Helmholtz

template <int N>
struct IhCfg {
    static constexpr int kBe = (N >= 16) ? 1 : ((N <= 6) ? 4 : 2);      // elements per batch
    static constexpr int kTiles = (kBe * N * N + 7) / 8;
    static constexpr int kWarps = (N == 14)           ? 8
                                  : (kTiles % 8 == 0) ? 8
                                  : (kTiles % 6 == 0) ? 6
                                  : (kTiles % 5 == 0) ? 5
                                  : (kTiles % 4 == 0) ? 4
                                                      : 8;
    using SS = Stage<N, N, N, N, kBe, kWarps>;
    static constexpr int kThreads = 32 * kWarps;
    static constexpr int kBufElems = kBe * N * N * N;
    static constexpr size_t kSmemBytes = 2 * (size_t)kBufElems * sizeof(double) + 16;
    static constexpr int kBySmem = (int)((227 * 1024) / (kSmemBytes + 1024));
    static constexpr int kByWarps = 20 / kWarps;
    static constexpr int kCtasPerSm =
        (kBySmem < kByWarps ? kBySmem : kByWarps) < 1 ? 1 : (kBySmem < kByWarps ? kBySmem : kByWarps);
    static_assert(N % 2 == 0 && N >= 4, "even N >= 4");
};

// v[e] = (S(x)S(x)S)(D[e] o ((S^T(x)S^T(x)S^T) u[e])), u's element addresses 16-byte aligned.
template <int N>
__global__ void __launch_bounds__(IhCfg<N>::kThreads, IhCfg<N>::kCtasPerSm)
inv_helmholtz_dmma(const double* __restrict__ S, const double* __restrict__ D, const double* u,
                   double* v, long long E) {
    using C = IhCfg<N>;
    using SS = typename C::SS;
    constexpr int kN3 = N * N * N;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    double* bufA = reinterpret_cast<double*>(smem_raw);
    double* bufB = bufA + C::kBufElems;
    uint64_t* bar = reinterpret_cast<uint64_t*>(bufB + C::kBufElems);

    // which warp takes the odd tile out rotates with the CTA, so that co-resident CTAs do
    // not load the same scheduler partition
    const int lane = threadIdx.x & 31;
    const int warp = ((threadIdx.x >> 5) + blockIdx.x) % C::kWarps;

    const long long n_batches = (E + C::kBe - 1) / C::kBe;
    if (threadIdx.x == 0) mbar_init(bar, 1);
    __syncthreads();

    auto batch_bytes = [&](long long b) {
        const long long e0 = b * C::kBe;
        const long long cnt = (E - e0 < C::kBe) ? (E - e0) : C::kBe;
        return (unsigned)(cnt * kN3 * sizeof(double));
    };
    long long batch = blockIdx.x;
    if (threadIdx.x == 0 && batch < n_batches) {
        mbar_expect_tx(bar, batch_bytes(batch));
        bulk_load(bufA, u + batch * C::kBe * kN3, batch_bytes(batch), bar);
    }
    unsigned parity = 0;
    for (; batch < n_batches; batch += gridDim.x) {
        const long long e0 = batch * C::kBe;
        const int cnt = (int)((E - e0 < C::kBe) ? (E - e0) : C::kBe);
        const int valid = cnt * N * N;
        const double* Db = D + e0 * kN3;
        double* vb = v + e0 * kN3;
        const long long next = batch + gridDim.x;
        if (threadIdx.x == 0 && next < n_batches) {
            bulk_prefetch_l2(u + next * C::kBe * kN3, batch_bytes(next));
            bulk_prefetch_l2(D + next * C::kBe * kN3, batch_bytes(next));
        }
        // forward stages apply S^T (t = sum_x S[x][o] in[x]); the fragments come from L1
        OpFrag<SS> op;
        load_op<SS>(op, S, false, lane);
        double dfac[SS::kMTiles][2];
        if (!wait_bulk(bar, parity)) break;
        parity ^= 1u;
        // forward: contract i, j, k
        run_stage<SS, 0>(bufA, bufB, op, dfac, nullptr, nullptr, valid, warp, lane);
        __syncthreads();
        // factor for this warp's first tile of the third stage: a whole stage hides the latency
        load_factor<SS>(dfac, Db, valid, warp, 0, lane);
        run_stage<SS, 0>(bufB, bufA, op, dfac, nullptr, nullptr, valid, warp, lane);
        __syncthreads();
        run_stage<SS, 1>(bufA, bufB, op, dfac, Db, nullptr, valid, warp, lane);
        __syncthreads();
        // backward: contract i, j, k with S itself
        load_op<SS>(op, S, true, lane);
        run_stage<SS, 0>(bufB, bufA, op, dfac, nullptr, nullptr, valid, warp, lane);
        __syncthreads();
        run_stage<SS, 0>(bufA, bufB, op, dfac, nullptr, nullptr, valid, warp, lane);
        __syncthreads();
        // bufA is free: bring in the next batch while the last stage streams v out
        if (threadIdx.x == 0 && next < n_batches) {
            fence_async_proxy();
            mbar_expect_tx(bar, batch_bytes(next));
            bulk_load(bufA, u + next * C::kBe * kN3, batch_bytes(next), bar);
        }
        run_stage<SS, 2>(bufB, nullptr, op, dfac, nullptr, vb, valid, warp, lane);
        __syncthreads();
    }
}

// ------------------------------------------------------------------ forward rectangular operator

template <int N0, int N1, int N2, int M0, int M1, int M2>
struct ApplyCfg {
    static constexpr int kBe = 2;
    static constexpr int kWarps = 4;
    using S1 = Stage<N0, M0, N1, N2, kBe, kWarps>;     // [n0][n1][n2] -> [n1][n2][m0]
    using S2 = Stage<N1, M1, N2, M0, kBe, kWarps>;     // [n1][n2][m0] -> [n2][m0][m1]
    using S3 = Stage<N2, M2, M0, M1, kBe, kWarps>;     // [n2][m0][m1] -> [m0][m1][m2]
    static constexpr int kThreads = 32 * kWarps;
    static constexpr int kU = kBe * S1::kIn;           // landing buffer of u
    static constexpr int kB = kBe * S1::kOut;          // first intermediate
    static constexpr int kA = kBe * S2::kOut;          // second intermediate
    static constexpr size_t kSmemBytes = (size_t)(kU + kB + kA) * sizeof(double) + 16;
    static constexpr int kBySmem = (int)((227 * 1024) / (kSmemBytes + 1024));
    static constexpr int kByWarps = 20 / kWarps;
    static constexpr int kCtasPerSm =
        (kBySmem < kByWarps ? kBySmem : kByWarps) < 1 ? 1 : (kBySmem < kByWarps ? kBySmem : kByWarps);
    static_assert((S1::kIn * sizeof(double)) % 16 == 0, "element size must allow bulk copies");
};

// v[e] = (A(x)B(x)C) u[e]; contraction order A, B, C (slowest axis first).
template <int N0, int N1, int N2, int M0, int M1, int M2>
__global__ void __launch_bounds__(ApplyCfg<N0, N1, N2, M0, M1, M2>::kThreads,
                                  ApplyCfg<N0, N1, N2, M0, M1, M2>::kCtasPerSm)
apply_dmma(const double* __restrict__ A, const double* __restrict__ B, const double* __restrict__ Cm,
           const double* __restrict__ u, double* __restrict__ v, long long E) {
    using C = ApplyCfg<N0, N1, N2, M0, M1, M2>;
    using S1 = typename C::S1;
    using S2 = typename C::S2;
    using S3 = typename C::S3;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    double* bufU = reinterpret_cast<double*>(smem_raw);
    double* bufB = bufU + C::kU;
    double* bufA = bufB + C::kB;
    uint64_t* bar = reinterpret_cast<uint64_t*>(bufA + C::kA);

    const int lane = threadIdx.x & 31;
    const int warp = ((threadIdx.x >> 5) + blockIdx.x) % C::kWarps;

    // all three operators stay in registers for the life of the CTA
    OpFrag<S1> opA;
    OpFrag<S2> opB;
    OpFrag<S3> opC;
    load_op<S1>(opA, A, true, lane);
    load_op<S2>(opB, B, true, lane);
    load_op<S3>(opC, Cm, true, lane);

    const long long n_batches = (E + C::kBe - 1) / C::kBe;
    if (threadIdx.x == 0) mbar_init(bar, 1);
    __syncthreads();
    auto batch_bytes = [&](long long b) {
        const long long e0 = b * C::kBe;
        const long long cnt = (E - e0 < C::kBe) ? (E - e0) : C::kBe;
        return (unsigned)(cnt * S1::kIn * sizeof(double));
    };
    long long batch = blockIdx.x;
    if (threadIdx.x == 0 && batch < n_batches) {
        mbar_expect_tx(bar, batch_bytes(batch));
        bulk_load(bufU, u + batch * C::kBe * S1::kIn, batch_bytes(batch), bar);
    }
    unsigned parity = 0;
    double none1[S1::kMTiles][2], none2[S2::kMTiles][2], none3[S3::kMTiles][2];
    for (; batch < n_batches; batch += gridDim.x) {
        const long long e0 = batch * C::kBe;
        const int cnt = (int)((E - e0 < C::kBe) ? (E - e0) : C::kBe);
        const long long next = batch + gridDim.x;
        if (!wait_bulk(bar, parity)) break;
        parity ^= 1u;
        run_stage<S1, 0>(bufU, bufB, opA, none1, nullptr, nullptr, cnt * S1::kP, warp, lane);
        __syncthreads();
        // the landing buffer is free: bring in the next batch under the remaining two stages
        if (threadIdx.x == 0 && next < n_batches) {
            fence_async_proxy();
            mbar_expect_tx(bar, batch_bytes(next));
            bulk_load(bufU, u + next * C::kBe * S1::kIn, batch_bytes(next), bar);
        }
        run_stage<S2, 0>(bufB, bufA, opB, none2, nullptr, nullptr, cnt * S2::kP, warp, lane);
        __syncthreads();
        run_stage<S3, 2>(bufA, nullptr, opC, none3, nullptr, v + e0 * S3::kOut, cnt * S3::kP, warp,
                         lane);
        // the next batch's first stage writes bufB, which this batch no longer reads
    }
}

}  // namespace dmma
}  // namespace ekl
