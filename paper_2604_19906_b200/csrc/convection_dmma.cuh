// Volume integral of the convective flux (Eq. 1 of the paper) on the FP64 tensor path.
//
//   F[c,e] = (I(x)I(x)D)(M[e] o P[c,0,e]) + (I(x)D(x)I)(M[e] o P[c,1,e]) + (D(x)I(x)I)(M[e] o P[c,2,e])
//
// with the first Kronecker factor on the slowest in-element axis.  Sum-factorised with the
// shared contractions merged: with x_d = M o P_d,
//   stage 1 (slowest axis):  t0 = I x0,  t1 = I x1,  t2 = D x2
//   stage 2 (middle axis):   w0 = I t0,  w12 = D t1 + I t2
//   stage 3 (fastest axis):  F  = D w0 + I w12
// The two-term stages accumulate both products in the same tensor accumulators, so no
// element-wise add and no third intermediate exist.  Stages use the machinery of
// tpo_dmma.cuh (operator as register A fragments, 8-pencil B tiles from shared memory,
// cycling layouts with conflict-free padding).  M is applied while the B fragments of the
// first stage are read.  One CTA works on one element at a time: M[e] is fetched once and
// serves the three components; the P fields of the next component are bulk-copied under
// stages 2 and 3 of the current one.
#pragma once
#include "tpo_dmma.cuh"

namespace ekl {
namespace dmma {

template <int NQ, int NV>
struct ConvCfg {
    static constexpr int kWarps = 8;
    static constexpr int kThreads = 32 * kWarps;
    // fields as they land: [n][(m,l)], padded planes
    static constexpr int kPS0 = pad_plane(NQ * NQ), kES0 = NQ * kPS0;
    // after stage 1: [m][l][n']
    static constexpr int kRS1 = pad_row(NV), kPS1 = pad_plane(NQ * kRS1), kES1 = NQ * kPS1;
    // after stage 2: [l][n'][m']
    static constexpr int kRS2 = pad_row(NV), kPS2 = pad_plane(NV * kRS2), kES2 = NQ * kPS2;
    using S1 = Stage<NQ, NV, NQ, NQ, 1, kWarps, NQ, kPS0, kES0, kRS1, kPS1, kES1>;
    using S2 = Stage<NQ, NV, NQ, NV, 1, kWarps, kRS1, kPS1, kES1, kRS2, kPS2, kES2>;
    using S3 = Stage<NQ, NV, NV, NV, 1, kWarps, kRS2, kPS2, kES2, NV, NV * NV, NV * NV * NV>;
    // shared memory: M, three P fields, three stage-1 outputs, two stage-2 outputs
    static constexpr int kDoubles = 4 * kES0 + 3 * kES1 + 2 * kES2;
    static constexpr size_t kSmemBytes = (size_t)kDoubles * sizeof(double) + 16;
    static constexpr int kBySmem = (int)((227 * 1024) / (kSmemBytes + 1024));
    static constexpr int kCtasPerSm = kBySmem < 1 ? 1 : (kBySmem > 2 ? 2 : kBySmem);
    // bulk copies need planes that are whole 16-byte units; an odd nq uses 8-byte asynchronous
    // copies issued by all threads
    static constexpr bool kBulk = (NQ % 2 == 0);
    static_assert(S1::kMTiles == S2::kMTiles && S1::kKSteps == S3::kKSteps, "one fragment shape");
};

// Accumulate one (operator, input) product of tile t into c; the input may be scaled
// entry-wise by `scale` (same layout as `in`).
template <class SS, bool SCALE>
__device__ __forceinline__ void tile_accumulate(double (&c)[SS::kMTiles][2], const OpFrag<SS>& op,
                                                const double* __restrict__ in,
                                                const double* __restrict__ scale, int t, int lane) {
    const int r = lane >> 2, kk = lane & 3;
    int qb = 8 * t + r;
    if (qb >= SS::kPencils) qb = 0;
    const int pb1 = qb / SS::E2;
    const int off = pb1 * SS::IN_RS + (qb - pb1 * SS::E2) + kk * SS::IN_PS;
    double b[SS::kKSteps];
#pragma unroll
    for (int s = 0; s < SS::kKSteps; ++s) {
        b[s] = in[off + SS::k0(s) * SS::IN_PS];
        if (SCALE) b[s] *= scale[off + SS::k0(s) * SS::IN_PS];
    }
#pragma unroll
    for (int mt = 0; mt < SS::kMTiles; ++mt)
#pragma unroll
        for (int s = 0; s < SS::kKSteps; ++s) mma_f64(c[mt][0], c[mt][1], op.a[mt][s], b[s]);
}

// Write the accumulators of tile t to the stage's output layout (`out` in shared memory, or
// dense global memory when TO_GLOBAL).
template <class SS, bool TO_GLOBAL>
__device__ __forceinline__ void tile_store(const double (&c)[SS::kMTiles][2], double* out, int t,
                                           int lane) {
    const int r = lane >> 2, kk = lane & 3;
    const int qs = 8 * t + 2 * kk;
    if constexpr (SS::kPaired) {
        // even rows: the two pencils of a lane share a row, one address serves both
        if (qs >= SS::kPencils) return;
        const int ps1 = qs / SS::E2;
        double* dst = out + ps1 * SS::OUT_PS + (qs - ps1 * SS::E2) * SS::OUT_RS;
#pragma unroll
        for (int mt = 0; mt < SS::kMTiles; ++mt) {
            const int o = 8 * mt + r;
            if (o < SS::O) {
                dst[o] = c[mt][0];
                dst[SS::OUT_RS + o] = c[mt][1];
            }
        }
    } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int q = qs + h;
            if (q >= SS::kPencils) continue;
            const int ps1 = q / SS::E2;
            double* dst = out + ps1 * SS::OUT_PS + (q - ps1 * SS::E2) * SS::OUT_RS;
#pragma unroll
            for (int mt = 0; mt < SS::kMTiles; ++mt) {
                const int o = 8 * mt + r;
                if (o < SS::O) dst[o] = c[mt][h];
            }
        }
    }
}

template <int NQ, int NV>
__global__ void __launch_bounds__(ConvCfg<NQ, NV>::kThreads, ConvCfg<NQ, NV>::kCtasPerSm)
convection_dmma(const double* __restrict__ Dvq, const double* __restrict__ Ivq,
                const double* __restrict__ M, const double* __restrict__ P, double* __restrict__ F,
                long long E, unsigned long long* tickets) {
    using C = ConvCfg<NQ, NV>;
    using S1 = typename C::S1;
    using S2 = typename C::S2;
    using S3 = typename C::S3;
    constexpr int kQ3 = NQ * NQ * NQ, kV3 = NV * NV * NV;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    double* sM = reinterpret_cast<double*>(smem_raw);
    double* sX = sM + C::kES0;                  // three P fields
    double* sT = sX + 3 * C::kES0;              // t0, t1, t2
    double* sW = sT + 3 * C::kES1;              // w0, w12
    uint64_t* bar = reinterpret_cast<uint64_t*>(sW + 2 * C::kES2);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // both operators have the same shape in every stage ([nv,nq], output index major)
    OpFrag<S1> opI, opD;
    load_op<S1, double>(opI, Ivq, true, lane);
    load_op<S1, double>(opD, Dvq, true, lane);

    // elements are handed out one at a time (BatchQueue, a batch being one element)
    __shared__ long long shared_next;
    BatchQueue q;
    q.start(tickets, &shared_next);
    if (threadIdx.x == 0) mbar_init(bar, 1);
    __syncthreads();

    auto fetch = [&](int c, long long e, bool with_m) {
        const unsigned field = (unsigned)(kQ3 * sizeof(double));
        mbar_expect_tx(bar, (with_m ? 4u : 3u) * field);
        if (with_m)
            for (int x = 0; x < NQ; ++x)
                bulk_load(sM + x * C::kPS0, M + (size_t)e * kQ3 + x * NQ * NQ,
                          (unsigned)(NQ * NQ * sizeof(double)), bar);
        for (int d = 0; d < 3; ++d) {
            const double* src = P + (((size_t)c * 3 + d) * E + e) * kQ3;
            for (int x = 0; x < NQ; ++x)
                bulk_load(sX + d * C::kES0 + x * C::kPS0, src + x * NQ * NQ,
                          (unsigned)(NQ * NQ * sizeof(double)), bar);
        }
    };
    // all threads: the same transfer by 8-byte asynchronous copies, for fields whose planes are
    // not a whole number of 16-byte units (odd nq)
    auto fetch_copy = [&](int c, long long e, bool with_m) {
        if (with_m)
            copy_elements<NQ, NQ * NQ, C::kPS0, C::kES0, double>(sM, M + (size_t)e * kQ3, 1);
        for (int d = 0; d < 3; ++d)
            copy_elements<NQ, NQ * NQ, C::kPS0, C::kES0, double>(
                sX + d * C::kES0, P + (((size_t)c * 3 + d) * E + e) * kQ3, 1);
    };

    if constexpr (C::kBulk) {
        if (threadIdx.x == 0 && q.batch < E) fetch(0, q.batch, true);
    } else {
        if (q.batch < E) fetch_copy(0, q.batch, true);
    }
    unsigned parity = 0;
    bool ok = true;
    while (ok && q.batch < E) {
        q.draw();
        const long long e = q.batch;
        // ask L2 for everything this element still needs, a whole element of work ahead of
        // the bulk copies that will use it
        if (threadIdx.x == 0) {
            const unsigned field = (unsigned)(kQ3 * sizeof(double));
            for (int cd = 3; cd < 9; ++cd) bulk_prefetch_l2(P + ((size_t)cd * E + e) * kQ3, field);
        }
        // (unrolled: the compiler does not do it by itself with the early exit in the loop, and
        // the rolled loop measured 8 % slower)
#pragma unroll
        for (int c = 0; c < 3; ++c) {
            if constexpr (C::kBulk) {
                if (!wait_bulk(bar, parity)) {
                    ok = false;
                    break;
                }
                parity ^= 1u;
            } else {
                wait_copies();
            }
            if (c == 0) {
                // the barrier inside the wait orders the ticket handed over at the end of the
                // previous element; now the next element is known: ask L2 for its first fields
                q.refresh();
                const long long ne = q.next;
                if (threadIdx.x == 0 && ne < E) {
                    const unsigned field = (unsigned)(kQ3 * sizeof(double));
                    bulk_prefetch_l2(M + (size_t)ne * kQ3, field);
                    for (int d = 0; d < 3; ++d)
                        bulk_prefetch_l2(P + ((size_t)d * E + ne) * kQ3, field);
                }
            }
            // stage 1: three products, 3 * kTiles tile tasks dealt round-robin
#pragma unroll
            for (int it = 0; it < (3 * S1::kTiles + C::kWarps - 1) / C::kWarps; ++it) {
                const int task = warp + it * C::kWarps;
                if (task >= 3 * S1::kTiles) break;
                const int d = task / S1::kTiles, t = task - d * S1::kTiles;
                double acc[S1::kMTiles][2];
#pragma unroll
                for (int mt = 0; mt < S1::kMTiles; ++mt) acc[mt][0] = acc[mt][1] = 0.0;
                tile_accumulate<S1, true>(acc, d == 2 ? opD : opI, sX + d * C::kES0, sM, t, lane);
                tile_store<S1, false>(acc, sT + d * C::kES1, t, lane);
            }
            __syncthreads();
            // the P buffers (and, after the last component, M) are free: fetch what comes next
            if constexpr (C::kBulk) {
                if (threadIdx.x == 0) {
                    const bool last = (c == 2);
                    const long long ne = last ? q.next : e;
                    if (ne < E) {
                        fence_async_proxy();
                        fetch(last ? 0 : c + 1, ne, last);
                    }
                }
            } else {
                const bool last = (c == 2);
                const long long ne = last ? q.next : e;
                if (ne < E) fetch_copy(last ? 0 : c + 1, ne, last);
            }
            // stage 2: w0 = I t0 (first kTiles tasks), w12 = D t1 + I t2 (the rest)
#pragma unroll
            for (int it = 0; it < (2 * S2::kTiles + C::kWarps - 1) / C::kWarps; ++it) {
                const int task = warp + it * C::kWarps;
                if (task >= 2 * S2::kTiles) break;
                const bool dual = task >= S2::kTiles;
                const int t = dual ? task - S2::kTiles : task;
                double acc[S2::kMTiles][2];
#pragma unroll
                for (int mt = 0; mt < S2::kMTiles; ++mt) acc[mt][0] = acc[mt][1] = 0.0;
                if (dual) {
                    tile_accumulate<S2, false>(acc, opD, sT + C::kES1, nullptr, t, lane);
                    tile_accumulate<S2, false>(acc, opI, sT + 2 * C::kES1, nullptr, t, lane);
                } else {
                    tile_accumulate<S2, false>(acc, opI, sT, nullptr, t, lane);
                }
                tile_store<S2, false>(acc, sW + (dual ? C::kES2 : 0), t, lane);
            }
            __syncthreads();
            // stage 3: F = D w0 + I w12, straight to global memory in natural order
            double* Fe = F + ((size_t)c * E + e) * kV3;
#pragma unroll
            for (int it = 0; it < (S3::kTiles + C::kWarps - 1) / C::kWarps; ++it) {
                const int t = warp + it * C::kWarps;
                if (t >= S3::kTiles) break;
                double acc[S3::kMTiles][2];
#pragma unroll
                for (int mt = 0; mt < S3::kMTiles; ++mt) acc[mt][0] = acc[mt][1] = 0.0;
                tile_accumulate<S3, false>(acc, opD, sW, nullptr, t, lane);
                tile_accumulate<S3, false>(acc, opI, sW + C::kES2, nullptr, t, lane);
                tile_store<S3, true>(acc, Fe, t, lane);
            }
            // the next stage 1 writes sT, which stage 2 no longer reads; the next stage 2
            // writes sW only after the barrier that follows the next stage 1
        }
        q.publish();
        q.advance_batch();
    }
    q.finish(E);
}

}  // namespace dmma
}  // namespace ekl
