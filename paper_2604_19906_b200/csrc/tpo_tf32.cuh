// Single-precision inverse Helmholtz on the TF32 tensor path with split operands.
//
// The fp32 entry point has a tolerance of 1e-5, far tighter than one TF32 product (10-bit
// mantissa), so every product is taken in three tensor steps on split operands,
//     a*b ~ a_hi*b_hi + a_lo*b_hi + a_hi*b_lo,   x_hi = tf32(x), x_lo = tf32(x - x_hi),
// accumulated in fp32 by the tensor core (the dropped a_lo*b_lo term is of relative size
// 2^-22).  The fields stay fp32 in global and shared memory, which halves both kinds of traffic
// against the fp64 tensor path, and one m16n8k8 step covers all output rows (extent <= 16) and
// eight contraction indices.
//
// The stages, the cycling layouts and the tile deal are those of tpo_dmma.cuh; only the
// fragment shapes and the bank rules differ (4-byte words, 32 banks):
//   B fragment  lane (r = lane/4, kk = lane%4): contraction indices k0+kk and k0+kk+4 of pencil 8t+r,
//   A fragment  rows r, r+8 x columns k0+kk, k0+kk+4 of the operator (hi and lo parts, in registers),
//   C fragment  rows r, r+8 of pencils 8t+2kk, 8t+2kk+1.
// A warp-wide 4-byte access is conflict free when its 32 addresses fall in 32 banks: the plane
// stride (between contraction indices) is 8 or 24 (mod 32) for the loads, the row stride
// (between pencils) is 4 or 12 (mod 16) for the stores.
#pragma once
#include "tpo_dmma.cuh"

namespace ekl {
namespace tf32 {

using dmma::Stage;

__host__ __device__ constexpr int pad_row32(int o) {
    return (o % 16 == 4 || o % 16 == 12) ? o : pad_row32(o + 1);
}
__host__ __device__ constexpr int pad_plane32(int x) {
    return (x % 32 == 8 || x % 32 == 24) ? x : pad_plane32(x + 1);
}

__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], uint32_t b0,
                                         uint32_t b1) {
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// x = hi + lo with hi the nearest TF32 value; lo is exact in fp32 and is cut to TF32 by the
// tensor core when it reads the register.
__device__ __forceinline__ void split_tf32(float x, uint32_t& hi, uint32_t& lo) {
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(hi) : "f"(x));
    lo = __float_as_uint(x - __uint_as_float(hi));
}

// Eight contraction indices per tensor step; a last partial step overlaps the one before it.
template <int K>
struct Steps8 {
    static_assert(K >= 8, "contraction extent below one tensor step");
    static constexpr int kSteps = (K + 7) / 8;
    __host__ __device__ static constexpr int k0(int s) { return (8 * s + 8 <= K) ? 8 * s : K - 8; }
    // columns of step s that an earlier step already covered
    __host__ __device__ static constexpr int repeated(int s) {
        return (s > 0) ? k0(s - 1) + 8 - k0(s) : 0;
    }
};

// The operator as this lane sees it, split in hi and lo parts.
template <int KS>
struct OpFrag32 {
    uint32_t hi[KS][4];
    uint32_t lo[KS][4];
};

// out_major: A[o][x] = M[o*K + x]; otherwise the stage applies the transpose, A[o][x] = M[x*O + o].
template <class SS>
__device__ __forceinline__ void load_op32(OpFrag32<Steps8<SS::K>::kSteps>& f,
                                          const float* __restrict__ M, bool out_major, int lane) {
    using ST = Steps8<SS::K>;
    const int r = lane >> 2, kk = lane & 3;
#pragma unroll
    for (int s = 0; s < ST::kSteps; ++s) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int o = r + 8 * (j & 1);
            const int i = kk + 4 * (j >> 1);           // column within the step
            const int x = ST::k0(s) + i;
            const bool live = o < SS::O && i >= ST::repeated(s);
            const float m = live ? __ldg(out_major ? M + o * SS::K + x : M + x * SS::O + o) : 0.0f;
            split_tf32(m, f.hi[s][j], f.lo[s][j]);
        }
    }
}

// The pointwise factor for the outputs this lane holds of the warp's tile `slot`.
template <class SS>
__device__ __forceinline__ void load_factor32(float (&d)[4], const float* __restrict__ Db,
                                              int valid_pencils, int warp, int slot, int lane) {
    const int r = lane >> 2, kk = lane & 3;
    int t;
    const bool live = dmma::tile_live<SS>(warp, slot, t);
    const int qs = 8 * t + 2 * kk;
    const float* g = Db + (size_t)qs * SS::O + r;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int h = j & 1, up = j >> 1;              // c0:(r,h0) c1:(r,h1) c2:(r+8,h0) c3:(r+8,h1)
        const bool ld = live && (r + 8 * up < SS::O) && (qs + h < valid_pencils);
        d[j] = ld ? __ldg(g + h * SS::O + 8 * up) : 0.0f;
    }
}

// MODE 0: shared -> shared.  MODE 1: shared -> shared, times the pointwise factor (dfac holds it
// for the warp's first FD tiles on entry; tile i + FD is fetched into the registers tile i
// frees).  MODE 2: shared -> global (dense).
template <class SS, int MODE, int FD>
__device__ __forceinline__ void run_stage32(const float* __restrict__ in, float* __restrict__ out,
                                            float* __restrict__ gout,
                                            const OpFrag32<Steps8<SS::K>::kSteps>& op,
                                            float (&dfac)[FD][4], const float* __restrict__ Db,
                                            int valid_pencils, int warp, int lane) {
    using ST = Steps8<SS::K>;
    static_assert(SS::O <= 16 && SS::kPaired, "one row tile, even extents");
    const int r = lane >> 2, kk = lane & 3;
#pragma unroll
    for (int slot = 0; slot < SS::kTilesPerWarp; ++slot) {
        int t;
        if (!dmma::tile_live<SS>(warp, slot, t)) break;
        int qb = 8 * t + r;
        if (qb >= SS::kPencils) qb = 0;                    // ragged last tile: any valid pencil
        const int eb = qb / SS::kP;
        const int pb = qb - eb * SS::kP;
        const int pb1 = pb / SS::E2;
        const float* src =
            in + eb * SS::IN_ES + pb1 * SS::IN_RS + (pb - pb1 * SS::E2) + kk * SS::IN_PS;
        uint32_t bh[ST::kSteps][2], bl[ST::kSteps][2];
#pragma unroll
        for (int s = 0; s < ST::kSteps; ++s) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                // columns an overlapping last step repeats carry zeros in the operator: no load
                const bool fresh = kk + 4 * j >= ST::repeated(s);
                const float b = fresh ? src[(ST::k0(s) + 4 * j) * SS::IN_PS] : 0.0f;
                split_tf32(b, bh[s][j], bl[s][j]);
            }
        }
        // the two small cross terms first, then the leading one
        float c[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int s = 0; s < ST::kSteps; ++s) {
            mma_tf32(c, op.lo[s], bh[s][0], bh[s][1]);
            mma_tf32(c, op.hi[s], bl[s][0], bl[s][1]);
        }
#pragma unroll
        for (int s = 0; s < ST::kSteps; ++s) mma_tf32(c, op.hi[s], bh[s][0], bh[s][1]);
        // this lane: rows r, r+8 of pencils 8t + 2*kk + {0,1} (a pair shares row and element)
        const int qs = 8 * t + 2 * kk;
        const int limit = (MODE == 2) ? valid_pencils : SS::kPencils;
        if (qs < limit) {
            const int es = qs / SS::kP;
            const int ps = qs - es * SS::kP;
            const int ps1 = ps / SS::E2;
            const size_t off = (size_t)es * SS::OUT_ES + ps1 * SS::OUT_PS +
                               (ps - ps1 * SS::E2) * SS::OUT_RS + r;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int h = j & 1, up = j >> 1;
                if (r + 8 * up < SS::O) {
                    const size_t a = off + h * SS::OUT_RS + 8 * up;
                    if (MODE == 2)
                        gout[a] = c[j];
                    else
                        out[a] = (MODE == 1) ? c[j] * dfac[slot % FD][j] : c[j];
                }
            }
        }
        if (MODE == 1 && slot + FD < SS::kTilesPerWarp)
            load_factor32<SS>(dfac[slot % FD], Db, valid_pencils, warp, slot + FD, lane);
    }
}

// `cnt` dense elements of K planes x P floats each into the plane-padded layout, all copies
// completing on `bar`.  Called by thread 0 (LANES = 1) or by the CTA's first warp (LANES = 32,
// `lane` = threadIdx.x): lane 0 announces the bytes and the lanes issue the per-plane copies side
// by side -- one thread issuing dozens of copies in a row takes about as long as the copies
// themselves, which shows where they have little time to land (measured: 3.6 % at n = 14, 1.6 %
// at n = 16, but 6 % slower at n = 12).  A copy may complete before lane 0 has announced it: the
// phase cannot end before lane 0's arrival, and by then the byte count balances.
template <int K, int P, int PS, int ES, int LANES>
__device__ __forceinline__ void load_elements32(float* dst, const float* src, int cnt,
                                                uint64_t* bar, int lane) {
    if (lane == 0) dmma::mbar_expect_tx(bar, (unsigned)(cnt * K * P * sizeof(float)));
    if (PS == P && ES == K * P) {
        if (lane == 0) dmma::bulk_load(dst, src, (unsigned)(cnt * K * P * sizeof(float)), bar);
    } else {
        for (int i = lane; i < cnt * K; i += LANES) {
            const int e = i / K, x = i - e * K;
            dmma::bulk_load(dst + e * ES + x * PS, src + (size_t)i * P,
                            (unsigned)(P * sizeof(float)), bar);
        }
    }
}

// at most this many warps of these kernels share an SM (measured best)
constexpr int kMaxWarpsPerSm = 24;

template <int N>
struct IhCfg32 {
    static_assert(N % 2 == 0 && N >= 8 && N <= 16, "even extents from 8 to 16");
    static constexpr int kPS0 = pad_plane32(N * N), kES0 = N * kPS0;
    static constexpr int kRS = pad_row32(N), kPS = pad_plane32(N * kRS), kES = N * kPS;
    static constexpr int kElemBuf = (kES0 > kES ? kES0 : kES);
    // one element per batch in more, smaller CTAs measured 5 % (n = 8), 7 % (12), 5 % (14) and
    // 10 % (16) faster than two; n = 10 is 5 % faster with two
    static constexpr int kBe = (N == 10) ? 2 : 1;
    // threads that issue the bulk copies of u (see load_elements32)
    static constexpr int kCopyLanes = (N >= 14) ? 32 : 1;
    static constexpr int kTiles = (kBe * N * N + 7) / 8;
    // an even deal of the tiles; 4 warps (more CTAs per SM) measured 4-6 % faster for n = 8, 12,
    // and for n = 14 (25 tiles) faster than 5, 6 or 8
    static constexpr int kWarps = (N == 8 || N == 12 || N == 14) ? 4
                                  : (kTiles % 8 == 0) ? 8
                                  : (kTiles % 6 == 0) ? 6
                                  : (kTiles % 5 == 0) ? 5
                                                      : 8;
    using First = Stage<N, N, N, N, kBe, kWarps, N, kPS0, kES0, kRS, kPS, kES>;
    using Mid = Stage<N, N, N, N, kBe, kWarps, kRS, kPS, kES, kRS, kPS, kES>;
    using Last = Stage<N, N, N, N, kBe, kWarps, kRS, kPS, kES, N, N * N, N * N * N>;
    static constexpr int kThreads = 32 * kWarps;
    static constexpr int kBufElems = kBe * kElemBuf;
    static constexpr size_t kSmemBytes = 2 * (size_t)kBufElems * sizeof(float) + 16;
    static constexpr int kBySmem = (int)((227 * 1024) / (kSmemBytes + 1024));
    static constexpr int kByWarps = kMaxWarpsPerSm / kWarps;
    static constexpr int kCtasPerSm =
        (kBySmem < kByWarps ? kBySmem : kByWarps) < 1 ? 1 : (kBySmem < kByWarps ? kBySmem : kByWarps);
    // tiles of the pointwise factor held ahead in registers: deeper than this spills at the
    // 80 registers three CTAs per SM leave a thread (measured: n = 14 9 % and n = 8 12 % faster)
    // (n = 14, seven tiles per warp and stage: three ahead is another 2 % faster)
    static constexpr int kFactorDepth = (N == 8) ? 1 : (N == 14) ? 3 : 2;
};

// v[e] = (S(x)S(x)S)(D[e] o ((S^T(x)S^T(x)S^T) u[e])), fp32 fields; u must be 16-byte aligned.
template <int N>
__global__ void __launch_bounds__(IhCfg32<N>::kThreads, IhCfg32<N>::kCtasPerSm)
inv_helmholtz_tf32(const float* __restrict__ S, const float* __restrict__ D, const float* u, float* v,
                   long long E, unsigned long long* tickets) {
    using C = IhCfg32<N>;
    using First = typename C::First;
    using Mid = typename C::Mid;
    using Last = typename C::Last;
    constexpr int kN2 = N * N, kN3 = N * N * N, FD = C::kFactorDepth;
    constexpr int KS = Steps8<N>::kSteps;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float* bufA = reinterpret_cast<float*>(smem_raw);
    float* bufB = bufA + C::kBufElems;
    uint64_t* bar = reinterpret_cast<uint64_t*>(bufB + C::kBufElems);

    const int lane = threadIdx.x & 31;
    const int warp = ((threadIdx.x >> 5) + blockIdx.x) % C::kWarps;

    // forward stages apply S^T, backward stages S itself
    OpFrag32<KS> op, opb;
    load_op32<Mid>(op, S, false, lane);
    load_op32<Mid>(opb, S, true, lane);

    const long long n_batches = (E + C::kBe - 1) / C::kBe;
    __shared__ long long shared_next;
    dmma::BatchQueue q;
    q.start(tickets, &shared_next);
    if (threadIdx.x == 0) dmma::mbar_init(bar, 1);
    __syncthreads();
    auto batch_count = [&](long long b) {
        const long long e0 = b * C::kBe;
        return (int)((E - e0 < C::kBe) ? (E - e0) : C::kBe);
    };
    if (q.batch < n_batches && threadIdx.x < C::kCopyLanes)
        load_elements32<N, kN2, C::kPS0, C::kES0, C::kCopyLanes>(
            bufA, u + q.batch * C::kBe * kN3, batch_count(q.batch), bar, threadIdx.x);
    unsigned parity = 0;
    while (q.batch < n_batches) {
        q.draw();
        const long long batch = q.batch, next = q.next;
        const long long e0 = batch * C::kBe;
        const int cnt = batch_count(batch);
        const int valid = cnt * kN2;
        const float* Db = D + e0 * kN3;
        if (threadIdx.x == 0 && next < n_batches) {
            const unsigned nbytes = (unsigned)(batch_count(next) * kN3 * sizeof(float));
            dmma::bulk_prefetch_l2(u + next * C::kBe * kN3, nbytes);
            dmma::bulk_prefetch_l2(D + next * C::kBe * kN3, nbytes);
        }
        if (!dmma::wait_bulk(bar, parity)) break;
        parity ^= 1u;
        float dfac[FD][4];
        // forward: contract i, j, k
        run_stage32<First, 0, FD>(bufA, bufB, nullptr, op, dfac, Db, valid, warp, lane);
        __syncthreads();
#pragma unroll
        for (int d = 0; d < FD; ++d) load_factor32<Mid>(dfac[d], Db, valid, warp, d, lane);
        run_stage32<Mid, 0, FD>(bufB, bufA, nullptr, op, dfac, Db, valid, warp, lane);
        __syncthreads();
        run_stage32<Mid, 1, FD>(bufA, bufB, nullptr, op, dfac, Db, valid, warp, lane);
        __syncthreads();
        // backward: contract i, j, k with S itself
        run_stage32<Mid, 0, FD>(bufB, bufA, nullptr, opb, dfac, Db, valid, warp, lane);
        __syncthreads();
        run_stage32<Mid, 0, FD>(bufA, bufB, nullptr, opb, dfac, Db, valid, warp, lane);
        __syncthreads();
        // bufA is free: bring in the next batch while the last stage streams v out
        if (next < n_batches && threadIdx.x < C::kCopyLanes) {
            dmma::fence_async_proxy();
            load_elements32<N, kN2, C::kPS0, C::kES0, C::kCopyLanes>(
                bufA, u + next * C::kBe * kN3, batch_count(next), bar, threadIdx.x);
        }
        run_stage32<Last, 2, FD>(bufB, nullptr, v + e0 * kN3, opb, dfac, Db, valid, warp, lane);
        q.publish();
        __syncthreads();
        q.advance();
    }
    q.finish(n_batches);
}

// ------------------------------------------------------------------ forward rectangular operator

template <int N0, int N1, int N2, int M0, int M1, int M2>
struct ApplyCfg32 {
    static_assert(N0 >= 8 && N1 >= 8 && N2 >= 8 && M0 <= 16 && M1 <= 16 && M2 <= 16,
                  "contraction extents from 8, output extents up to 16");
    // u as it lands: [n0][n1*n2] with padded planes
    static constexpr int kPS0 = pad_plane32(N1 * N2), kES0 = N0 * kPS0;
    // after the first stage: [n1][n2][m0]
    static constexpr int kRS1 = pad_row32(M0), kPS1 = pad_plane32(N2 * kRS1), kES1 = N1 * kPS1;
    // after the second stage: [n2][m0][m1]
    static constexpr int kRS2 = pad_row32(M1), kPS2 = pad_plane32(M0 * kRS2), kES2 = N2 * kPS2;
    // one element per batch (more, smaller CTAs) from 10 points per direction on: 14 -> 14 19 %,
    // 16 -> 16 32 %, 10 -> 14 20 % faster than two; 8 -> 12 is 11 % faster with two
    static constexpr int kBe = (N0 * N1 * N2 <= 512) ? 2 : 1;
    static constexpr int kMaxTiles =
        (kBe * (N1 * N2 > N2 * M0 ? (N1 * N2 > M0 * M1 ? N1 * N2 : M0 * M1)
                                 : (N2 * M0 > M0 * M1 ? N2 * M0 : M0 * M1)) + 7) / 8;
    // 4-warp CTAs up to 48 tiles per stage (measured), 8 beyond
    static constexpr int kWarps = (kMaxTiles > 48) ? 8 : 4;
    using S1 = Stage<N0, M0, N1, N2, kBe, kWarps, N2, kPS0, kES0, kRS1, kPS1, kES1>;
    using S2 = Stage<N1, M1, N2, M0, kBe, kWarps, kRS1, kPS1, kES1, kRS2, kPS2, kES2>;
    using S3 = Stage<N2, M2, M0, M1, kBe, kWarps, kRS2, kPS2, kES2, M2, M1 * M2, M0 * M1 * M2>;
    static constexpr int kThreads = 32 * kWarps;
    static constexpr int kU = kBe * kES0, kB = kBe * kES1, kA = kBe * kES2;
    static constexpr size_t kSmemBytes = (size_t)(kU + kB + kA) * sizeof(float) + 16;
    static constexpr int kBySmem = (int)((227 * 1024) / (kSmemBytes + 1024));
    static constexpr int kByWarps = kMaxWarpsPerSm / kWarps;
    static constexpr int kCtasPerSm =
        (kBySmem < kByWarps ? kBySmem : kByWarps) < 1 ? 1 : (kBySmem < kByWarps ? kBySmem : kByWarps);
    static_assert((N1 * N2) % 4 == 0, "planes must be a whole number of 16-byte units");
};

// v[e] = (A(x)B(x)C) u[e], fp32 fields; contraction order A, B, C (slowest axis first); u must
// be 16-byte aligned.
template <int N0, int N1, int N2, int M0, int M1, int M2>
__global__ void __launch_bounds__(ApplyCfg32<N0, N1, N2, M0, M1, M2>::kThreads,
                                  ApplyCfg32<N0, N1, N2, M0, M1, M2>::kCtasPerSm)
apply_tf32(const float* __restrict__ A, const float* __restrict__ B, const float* __restrict__ Cm,
           const float* __restrict__ u, float* __restrict__ v, long long E,
           unsigned long long* tickets) {
    using C = ApplyCfg32<N0, N1, N2, M0, M1, M2>;
    using S1 = typename C::S1;
    using S2 = typename C::S2;
    using S3 = typename C::S3;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float* bufU = reinterpret_cast<float*>(smem_raw);
    float* bufB = bufU + C::kU;
    float* bufA = bufB + C::kB;
    uint64_t* bar = reinterpret_cast<uint64_t*>(bufA + C::kA);

    const int lane = threadIdx.x & 31;
    const int warp = ((threadIdx.x >> 5) + blockIdx.x) % C::kWarps;

    // all three operators, split, stay in registers for the life of the CTA
    OpFrag32<Steps8<N0>::kSteps> opA;
    OpFrag32<Steps8<N1>::kSteps> opB;
    OpFrag32<Steps8<N2>::kSteps> opC;
    load_op32<S1>(opA, A, true, lane);
    load_op32<S2>(opB, B, true, lane);
    load_op32<S3>(opC, Cm, true, lane);

    const long long n_batches = (E + C::kBe - 1) / C::kBe;
    __shared__ long long shared_next;
    dmma::BatchQueue q;
    q.start(tickets, &shared_next);
    if (threadIdx.x == 0) dmma::mbar_init(bar, 1);
    __syncthreads();
    auto batch_count = [&](long long b) {
        const long long e0 = b * C::kBe;
        return (int)((E - e0 < C::kBe) ? (E - e0) : C::kBe);
    };
    auto fetch = [&](long long b) {
        if (threadIdx.x == 0) {
            dmma::fence_async_proxy();
            load_elements32<N0, N1 * N2, C::kPS0, C::kES0, 1>(bufU, u + b * C::kBe * S1::kIn,
                                                              batch_count(b), bar, 0);
        }
    };
    if (q.batch < n_batches) fetch(q.batch);
    unsigned parity = 0;
    float none[1][4];
    while (q.batch < n_batches) {
        q.draw();
        const long long batch = q.batch;
        const long long e0 = batch * C::kBe;
        const int cnt = batch_count(batch);
        if (!dmma::wait_bulk(bar, parity)) break;
        parity ^= 1u;
        q.refresh();
        const long long next = q.next;
        run_stage32<S1, 0, 1>(bufU, bufB, nullptr, opA, none, nullptr, cnt * S1::kP, warp, lane);
        __syncthreads();
        // the landing buffer is free: bring in the next batch under the remaining two stages
        if (next < n_batches) fetch(next);
        run_stage32<S2, 0, 1>(bufB, bufA, nullptr, opB, none, nullptr, cnt * S2::kP, warp, lane);
        __syncthreads();
        run_stage32<S3, 2, 1>(bufA, nullptr, v + e0 * S3::kOut, opC, none, nullptr, cnt * S3::kP, warp,
                              lane);
        // the next batch's first stage writes bufB, which this batch no longer reads; the
        // barrier in the next iteration's wait orders the ticket handed over here
        q.publish();
        q.advance_batch();
    }
    q.finish(n_batches);
}

}  // namespace tf32
}  // namespace ekl
