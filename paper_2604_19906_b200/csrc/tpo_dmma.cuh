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
// plane by plane and the pointwise factor and the output are addressed in their natural
// order.  Two paddings keep every shared access of the stages bank-conflict free: the row
// stride (distance between consecutive p2) is 2 or 6 (mod 8) doubles, which spreads the
// 4 pencil pairs x 4 output indices a half-warp stores, and the plane stride (distance
// between consecutive contraction indices) is 4 (mod 8), which spreads the 4 contraction
// indices x 4 pencils a half-warp loads.  For N = 14 (and 6, 10) both hold unpadded.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

namespace ekl {
namespace dmma {

// Bit 0: a kernel's bounded wait on a bulk copy gave up.  Bit 1: the ticket counter of a launch
// did not end at the value its own draws add up to, i.e. something else wrote to it while the
// kernel ran.  Neither is expected in practice.  Every translation unit that includes this
// header has its own copy and reads it with take_timeout_flag().
static __device__ int g_bulk_wait_timeout = 0;

// Host: this translation unit's flags (-1 = the query failed), cleared.
static inline int take_timeout_flag() {
    int flag = 0;
    if (cudaMemcpyFromSymbol(&flag, g_bulk_wait_timeout, sizeof(int)) != cudaSuccess) return -1;
    if (flag) {
        const int zero = 0;
        cudaMemcpyToSymbol(g_bulk_wait_timeout, &zero, sizeof(int));
    }
    return flag & 3;
}

// Hands the batches of a launch to its CTAs.  Every CTA starts on batch blockIdx.x and goes on
// to blockIdx.x + gridDim.x.  With a ticket counter (two 64-bit words in global memory that are
// zero when the kernel starts) the batches from 2 * gridDim.x on go to whichever CTA asks
// first: co-resident CTAs do not get equal shares of an SM, and a fixed round-robin share
// makes the launch wait for the slowest of them.  A CTA always knows its next batch one
// iteration ahead (it prefetches that batch), so a ticket is drawn at the top of an iteration
// and used two iterations later, and no CTA ever waits for the counter.  Without a counter
// (nullptr) the batches are dealt round-robin.
struct BatchQueue {
    unsigned long long* ticket;
    long long* shared_next;       // one value in shared memory
    long long batch, next;
    unsigned long long drawn;
    bool handed_over;             // has publish() run yet?

    __device__ __forceinline__ void start(unsigned long long* t, long long* sh) {
        ticket = t;
        shared_next = sh;
        batch = blockIdx.x;
        next = batch + gridDim.x;
        drawn = 0;
        handed_over = false;
    }
    // Top of an iteration: ask for the batch after next.
    __device__ __forceinline__ void draw() {
        if (ticket && threadIdx.x == 0) drawn = atomicAdd(ticket, 1ull);
    }
    // Before a CTA barrier at or after the end of the iteration.
    __device__ __forceinline__ void publish() {
        if (ticket && threadIdx.x == 0)
            *shared_next = 2ll * (long long)gridDim.x + (long long)drawn;
        handed_over = true;
    }
    // After that barrier.
    __device__ __forceinline__ void advance() {
        batch = next;
        next = ticket ? *shared_next : next + gridDim.x;
    }
    // For a loop whose iterations end without a barrier: advance_batch() after publish(),
    // refresh() after the first barrier of the following iteration.
    __device__ __forceinline__ void advance_batch() {
        batch = next;
        if (!ticket) next += gridDim.x;
    }
    // (the first iteration has nothing to pick up: its next batch is the fixed one)
    __device__ __forceinline__ void refresh() {
        if (ticket && handed_over) next = *shared_next;
    }
    // End of the kernel: the CTA that leaves last checks that the counter holds exactly the
    // draws of this launch (one per batch) and leaves both words
    // zero for the launch that gets this counter next.
    __device__ __forceinline__ void finish(long long n_batches) {
        if (ticket && threadIdx.x == 0) {
            __threadfence();
            const unsigned long long gone = atomicAdd(ticket + 1, 1ull);
            if (gone == gridDim.x - 1) {
                const unsigned long long draws = atomicAdd(ticket, 0ull);
                if (draws != (unsigned long long)n_batches)
                    atomicOr(&g_bulk_wait_timeout, 2);
                atomicExch(ticket, 0ull);
                atomicExch(ticket + 1, 0ull);
            }
        }
    }
};

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

// How long a wait on a bulk copy may last before it gives up (a copy takes microseconds).
constexpr unsigned long long kWaitBudgetNs = 1000ull * 1000ull * 1000ull;

__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait on a phase of the barrier; false if it gave up after about a second (the
// clock is read every 256 polls).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity) {
    const uint32_t a = smem_addr(bar);
    unsigned long long t0 = 0;
    for (unsigned it = 1;; ++it) {
        unsigned done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(a), "r"(parity)
            : "memory");
        if (done) return true;
        if ((it & 255u) == 0) {
            const unsigned long long now = global_timer_ns();
            if (t0 == 0)
                t0 = now;
            else if (now - t0 > kWaitBudgetNs)
                return false;
        }
    }
}

// Plain (non-multicast) bulk copy global -> this CTA's shared memory, completing on `bar`.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes,
                                          uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}

// L2 prefetch of a byte range; works in 16-byte granules, so a range that does not start on
// one (odd extents, odd element index) is shrunk to the granules it fully contains.
__device__ __forceinline__ void bulk_prefetch_l2(const void* src, unsigned bytes) {
    const unsigned long long a = reinterpret_cast<unsigned long long>(src);
    const unsigned lead = (unsigned)((16 - (a & 15)) & 15);
    if (bytes < lead + 16) return;
    const unsigned n = (bytes - lead) & ~15u;
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(a + lead), "r"(n) : "memory");
}

__device__ __forceinline__ void fence_async_proxy() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// All threads of the CTA wait for the bulk copy of this phase.  Returns false, after
// flagging the error and waiting once more (bounded) for the copy still in flight, if the
// wait gave up; the decision is the same for every thread.
__device__ __forceinline__ bool wait_bulk(uint64_t* bar, unsigned parity) {
    if (__syncthreads_or(mbar_wait(bar, parity) ? 0 : 1)) {
        if (threadIdx.x == 0) atomicOr(&g_bulk_wait_timeout, 1);
        mbar_wait(bar, parity);
        return false;
    }
    return true;
}

// Smallest row stride >= o whose double-word count is 2 or 6 (mod 8).
__host__ __device__ constexpr int pad_row(int o) {
    return (o % 8 == 2 || o % 8 == 6) ? o : pad_row(o + 1);
}
// Smallest plane stride >= x that is 4 (mod 8).
__host__ __device__ constexpr int pad_plane(int x) { return (x % 8 == 4) ? x : pad_plane(x + 1); }

// One contraction stage for a batch of BE elements worked on by WARPS warps: input
// [K][E1][E2] per element at  e*IN_ES + x*IN_PS + p1*IN_RS + p2,  output [E1][E2][O] at
// e*OUT_ES + p1*OUT_PS + p2*OUT_RS + o  (dense global output: OUT_RS = O, OUT_PS = E2*O).
template <int K_, int O_, int E1_, int E2_, int BE_, int WARPS_, int IN_RS_, int IN_PS_,
          int IN_ES_, int OUT_RS_, int OUT_PS_, int OUT_ES_>
struct Stage {
    static constexpr int K = K_, O = O_, E1 = E1_, E2 = E2_, BE = BE_, WARPS = WARPS_;
    static constexpr int IN_RS = IN_RS_, IN_PS = IN_PS_, IN_ES = IN_ES_;
    static constexpr int OUT_RS = OUT_RS_, OUT_PS = OUT_PS_, OUT_ES = OUT_ES_;
    static constexpr int kP = E1 * E2;                    // pencils per element
    static constexpr int kIn = K * kP, kOut = O * kP;     // values per element (dense)
    static constexpr int kPencils = BE * kP;
    static constexpr int kTiles = (kPencils + 7) / 8;     // 8-pencil tiles, the last may be ragged
    static constexpr int kTilesPerWarp = (kTiles + WARPS - 1) / WARPS;
    static constexpr int kKSteps = (K + 3) / 4;
    static constexpr int kMTiles = (O + 7) / 8;
    // do the two neighbouring pencils a lane holds always share a row (and an element)?
    static constexpr bool kPaired = (E2 % 2 == 0);
    static_assert(K >= 4, "contraction extent below one tensor step");
    // first contraction index of tensor step s; a last partial step overlaps the previous one
    __host__ __device__ static constexpr int k0(int s) { return (4 * s + 4 <= K) ? 4 * s : K - 4; }
};

// The operator matrix as this lane sees it: A[o][x], o = 8*mt + lane/4, x = k0(s) + lane%4.
template <int MT, int KS>
struct OpFragT {
    double a[MT][KS];
};
template <class SS>
using OpFrag = OpFragT<SS::kMTiles, SS::kKSteps>;

// out_major: the matrix is stored [O][K] (A[o][x] = M[o*K + x]); otherwise [K][O], i.e. the
// stage applies the transpose of the stored matrix (A[o][x] = M[x*O + o]).
template <class SS, typename T>
__device__ __forceinline__ void load_op(OpFrag<SS>& f, const T* __restrict__ M, bool out_major,
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
                (o < SS::O && fresh) ? (double)__ldg(out_major ? M + o * SS::K + x : M + x * SS::O + o)
                                     : 0.0;
        }
    }
}

// Tiles are dealt to the warps round-robin; is slot `slot` of this warp a real tile?
template <class SS>
__device__ __forceinline__ bool tile_live(int warp, int slot, int& t) {
    t = warp + SS::WARPS * slot;
    return slot < SS::kTilesPerWarp && t < SS::kTiles;
}

// The pointwise factor (dense, natural order) for the outputs this lane holds of tile `slot`.
template <class SS, typename T>
__device__ __forceinline__ void load_factor(double (&d)[SS::kMTiles][2], const T* __restrict__ Db,
                                            int valid_pencils, int warp, int slot, int lane) {
    const int r = lane >> 2, kk = lane & 3;
    int t;
    const bool live = tile_live<SS>(warp, slot, t);
    const int qs = 8 * t + 2 * kk;
    const T* g = Db + (size_t)qs * SS::O;          // element e, pencil q: e*kOut + q*O
#pragma unroll
    for (int mt = 0; mt < SS::kMTiles; ++mt) {
        const int o = 8 * mt + r;
        const bool ld = live && (o < SS::O);
        d[mt][0] = (ld && qs < valid_pencils) ? (double)__ldg(g + o) : 0.0;
        d[mt][1] = (ld && qs + 1 < valid_pencils) ? (double)__ldg(g + SS::O + o) : 0.0;
    }
}

// Where the pointwise factor of the third inverse-Helmholtz stage comes from.
struct NoFactor {
    template <class SS>
    __device__ __forceinline__ void load(double (&)[SS::kMTiles][2], int, int, int, int) const {}
};

// a stored field D[e,i,j,k] (natural order), Db pointing at the batch
template <typename T>
struct FieldFactor {
    const T* Db;
    template <class SS>
    __device__ __forceinline__ void load(double (&d)[SS::kMTiles][2], int valid_pencils, int warp,
                                         int slot, int lane) const {
        load_factor<SS, T>(d, Db, valid_pencils, warp, slot, lane);
    }
};

// formed on the fly: 1 / (((lam[i] + lam[j]) + lam[k]) + c[e]), cb pointing at the batch
struct LambdaFactor {
    const double* lam;
    const double* cb;
    template <class SS>
    __device__ __forceinline__ void load(double (&d)[SS::kMTiles][2], int valid_pencils, int warp,
                                         int slot, int lane) const {
        const int r = lane >> 2, kk = lane & 3;
        int t;
        const bool live = tile_live<SS>(warp, slot, t);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int q = 8 * t + 2 * kk + h;
            const bool ok = live && q < valid_pencils;
            const int es = ok ? q / SS::kP : 0;
            const int p = ok ? q - es * SS::kP : 0;
            const int i = p / SS::E2, j = p - i * SS::E2;
            const double base = __ldg(lam + i) + __ldg(lam + j);
            const double ce = __ldg(cb + es);
#pragma unroll
            for (int mt = 0; mt < SS::kMTiles; ++mt) {
                const int o = 8 * mt + r;
                d[mt][h] = (ok && o < SS::O) ? 1.0 / ((base + __ldg(lam + (o < SS::O ? o : 0))) + ce)
                                             : 0.0;
            }
        }
    }
};

// MODE 0: shared -> shared (out).  MODE 1: shared -> shared, times the pointwise factor (dfac
// holds it for the warp's first FD tiles on entry; the factor of tile i + FD is fetched from
// `fac` into the registers tile i frees, so a load has FD tiles to arrive: a load that misses
// L1 takes one to two thousand cycles here, several tiles' worth).  MODE 2: shared -> global
// (gout, dense, converted to the I/O type T).
// `valid_pencils` masks a partly filled batch.  All arithmetic is fp64 whatever T is.
template <class SS, int MODE, typename T, typename Factor, int FD = 1>
__device__ __forceinline__ void run_stage(const double* __restrict__ in, double* __restrict__ out,
                                          T* __restrict__ gout, const OpFrag<SS>& op,
                                          double (&dfac)[FD][SS::kMTiles][2], const Factor& fac,
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
        const int pb = qb - eb * SS::kP;
        const int pb1 = pb / SS::E2;
        const double* src =
            in + eb * SS::IN_ES + pb1 * SS::IN_RS + (pb - pb1 * SS::E2) + kk * SS::IN_PS;
        double b[SS::kKSteps];
#pragma unroll
        for (int s = 0; s < SS::kKSteps; ++s) {
            // lanes whose contraction index an overlapping last step repeats need no data:
            // their operator entries are zero
            const int repeated = (s > 0) ? SS::k0(s - 1) + 4 - SS::k0(s) : 0;
            b[s] = (kk >= repeated) ? src[SS::k0(s) * SS::IN_PS] : 0.0;
        }
        double c[SS::kMTiles][2];
#pragma unroll
        for (int mt = 0; mt < SS::kMTiles; ++mt) {
            c[mt][0] = c[mt][1] = 0.0;
#pragma unroll
            for (int s = 0; s < SS::kKSteps; ++s) mma_f64(c[mt][0], c[mt][1], op.a[mt][s], b[s]);
        }
        // this lane: output index o = 8*mt + r of pencils 8t + 2*kk + {0,1}
        const int qs = 8 * t + 2 * kk;
        const int limit = (MODE == 2) ? valid_pencils : SS::kPencils;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            // with even rows the pair shares row and element, so one address serves both
            const int q = SS::kPaired ? qs : qs + h;
            if (q >= limit) continue;
            const int es = q / SS::kP;
            const int ps = q - es * SS::kP;
            const int ps1 = ps / SS::E2;
            const size_t off = (size_t)es * SS::OUT_ES + ps1 * SS::OUT_PS +
                               (ps - ps1 * SS::E2) * SS::OUT_RS + (SS::kPaired ? h * SS::OUT_RS : 0);
#pragma unroll
            for (int mt = 0; mt < SS::kMTiles; ++mt) {
                const int o = 8 * mt + r;
                if (o < SS::O) {
                    if (MODE == 2)
                        gout[off + o] = (T)c[mt][h];
                    else
                        out[off + o] = (MODE == 1) ? c[mt][h] * dfac[slot % FD][mt][h] : c[mt][h];
                }
            }
        }
        if (MODE == 1 && slot + FD < SS::kTilesPerWarp)
            fac.template load<SS>(dfac[slot % FD], valid_pencils, warp, slot + FD, lane);
    }
}

// Thread 0: bring `cnt` dense elements of K planes x P values each from global memory into
// the (possibly plane-padded) stage-input layout, all copies completing on `bar`.
template <int K, int P, int PS, int ES>
__device__ __forceinline__ void load_elements(double* dst, const double* src, int cnt,
                                              uint64_t* bar) {
    mbar_expect_tx(bar, (unsigned)(cnt * K * P * sizeof(double)));
    if (PS == P && ES == K * P) {
        bulk_load(dst, src, (unsigned)(cnt * K * P * sizeof(double)), bar);
    } else {
        for (int e = 0; e < cnt; ++e)
            for (int x = 0; x < K; ++x)
                bulk_load(dst + e * ES + x * PS, src + (size_t)(e * K + x) * P,
                          (unsigned)(P * sizeof(double)), bar);
    }
}

// All threads: the same transfer without the bulk-copy engine, for element sizes that are not
// a multiple of 16 bytes (odd extents: 8-byte asynchronous copies) and for single-precision
// fields (plain loads, widened to fp64 on the way in).  Completed by wait_copies().
template <int K, int P, int PS, int ES, typename T>
__device__ __forceinline__ void copy_elements(double* dst, const T* __restrict__ src, int cnt) {
    const int total = cnt * K * P;
#pragma unroll 4
    for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
        const int e = idx / (K * P);
        const int rem = idx - e * (K * P);
        const int x = rem / P;
        double* d = dst + e * ES + x * PS + (rem - x * P);
        if (sizeof(T) == sizeof(double)) {
            asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_addr(d)),
                         "l"(src + idx)
                         : "memory");
        } else {
            *d = (double)__ldg(src + idx);
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

// All threads: `count` floats from global memory into a dense staging area, asynchronously.
__device__ __forceinline__ void stage_floats(float* dst, const float* __restrict__ src, int count) {
    for (int idx = threadIdx.x; idx < count; idx += blockDim.x)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_addr(dst + idx)),
                     "l"(src + idx)
                     : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
}

// All threads: widen staged fields (dense, element after element) into the stage-input layout.
template <int K, int P, int PS, int ES>
__device__ __forceinline__ void widen_elements(double* dst, const float* src, int cnt) {
    const int total = cnt * K * P;
#pragma unroll 4
    for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
        const int e = idx / (K * P);
        const int rem = idx - e * (K * P);
        const int x = rem / P;
        dst[e * ES + x * PS + (rem - x * P)] = (double)src[idx];
    }
}

__device__ __forceinline__ void wait_copies() {
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();
}

// ------------------------------------------------------------------ inverse Helmholtz

template <int N, typename T = double>
struct IhCfg {
    // natural-order input planes, padded so that the first stage loads without conflicts
    static constexpr int kPS0 = pad_plane(N * N), kES0 = N * kPS0;
    // layout between stages
    static constexpr int kRS = pad_row(N), kPS = pad_plane(N * kRS), kES = N * kPS;
    static constexpr int kElemBuf = (kES0 > kES ? kES0 : kES);
    // elements per batch: two (four for the smallest) unless that leaves room for one CTA only;
    // n = 11 and 12 measured 9 % and 2-3 % faster with one element and more, smaller CTAs
    static constexpr int kBe = (N <= 6) ? 4
                               : (N == 11 || N == 12) ? 1
                               : ((4 * kElemBuf * 8 <= 112 * 1024) ? 2 : 1);
    static constexpr int kTiles = (kBe * N * N + 7) / 8;
    // warps per CTA: an even deal of the tiles where one exists, with the measured exceptions
    // (CTAs of 5 warps load the four scheduler partitions 2,1,1,1: n = 10 and 20 run 8 % and
    // 26 % faster with 4 and 8 warps, n = 17 12 % faster with 4; n = 7 and 9 1 % and 4 % faster
    // with 4; n = 16 4 % faster with three CTAs of 8 than of 4)
    static constexpr int kWarps = (N == 14 || N == 16 || N == 20) ? 8
                                  : (N == 7 || N == 9 || N == 10 || N == 11 || N == 12 || N == 17) ? 4
                                  : (kTiles <= 36 && kTiles % 4 == 0) ? 4
                                  : (kTiles % 8 == 0) ? 8
                                  : (kTiles % 6 == 0) ? 6
                                  : (kTiles % 5 == 0) ? 5
                                  : (kTiles % 4 == 0) ? 4
                                                      : 8;
    using First = Stage<N, N, N, N, kBe, kWarps, N, kPS0, kES0, kRS, kPS, kES>;
    using Mid = Stage<N, N, N, N, kBe, kWarps, kRS, kPS, kES, kRS, kPS, kES>;
    using Last = Stage<N, N, N, N, kBe, kWarps, kRS, kPS, kES, N, N * N, N * N * N>;
    static constexpr int kThreads = 32 * kWarps;
    static constexpr int kBufElems = kBe * kElemBuf;
    // single-precision fields land asynchronously in a dense staging area of their own and are
    // widened into the stage-1 input at the start of their batch
    static constexpr size_t kStagingBytes =
        sizeof(T) == sizeof(float) ? ((size_t)kBe * N * N * N * sizeof(float) + 15) / 16 * 16 : 0;
    static constexpr size_t kSmemBytes =
        2 * (size_t)kBufElems * sizeof(double) + kStagingBytes + 16;
    static constexpr int kBySmem = (int)((227 * 1024) / (kSmemBytes + 1024));
    // at most 20 warps per SM; 24 for n = 16, where a third CTA of 8 warps fits (4 % faster)
    static constexpr int kByWarps = (N == 16 ? 24 : 20) / kWarps;
    static constexpr int kCtasPerSm =
        (kBySmem < kByWarps ? kBySmem : kByWarps) < 1 ? 1 : (kBySmem < kByWarps ? kBySmem : kByWarps);
    // bulk copies need 16-byte granules: even N; odd N uses 8-byte asynchronous copies
    static constexpr bool kBulk = (N % 2 == 0);
    // tiles of the pointwise factor held in registers ahead of their use (measured: deeper
    // than one pays only where a warp has six or seven tiles per stage)
    static constexpr int kFactorDepth = (N == 14) ? 3 : (N == 10) ? 2 : 1;
    static_assert(N >= 4, "N >= 4");
};

// v[e] = (S(x)S(x)S)(D[e] o ((S^T(x)S^T(x)S^T) u[e])).  T is the type of the fields in memory
// (double: even N needs 16-byte aligned u; float: widened on load, rounded once on store).
// LAMBDA: the factor is not read from D but formed from lam[N] and c[E] (fp64 only).
template <int N, typename T, bool LAMBDA = false>
__global__ void __launch_bounds__(IhCfg<N, T>::kThreads, IhCfg<N, T>::kCtasPerSm)
inv_helmholtz_dmma(const T* __restrict__ S, const T* __restrict__ D,
                   const double* __restrict__ lam, const double* __restrict__ cvec, const T* u,
                   T* v, long long E, unsigned long long* tickets) {
    using C = IhCfg<N, T>;
    constexpr bool kBulk = C::kBulk && sizeof(T) == sizeof(double);
    using First = typename C::First;
    using Mid = typename C::Mid;
    using Last = typename C::Last;
    constexpr int kN2 = N * N, kN3 = N * N * N;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    double* bufA = reinterpret_cast<double*>(smem_raw);
    double* bufB = bufA + C::kBufElems;
    float* staging = reinterpret_cast<float*>(bufB + C::kBufElems);
    uint64_t* bar = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(staging) +
                                                C::kStagingBytes);
    constexpr bool kStaged = sizeof(T) == sizeof(float);

    // which warp takes the odd tile out rotates with the CTA, so that co-resident CTAs do
    // not load the same scheduler partition
    const int lane = threadIdx.x & 31;
    const int warp = ((threadIdx.x >> 5) + blockIdx.x) % C::kWarps;

    // forward stages apply S^T (t = sum_x S[x][o] in[x]), backward stages S itself
    OpFrag<Mid> op, opb;
    load_op<Mid, T>(op, S, false, lane);
    load_op<Mid, T>(opb, S, true, lane);

    const long long n_batches = (E + C::kBe - 1) / C::kBe;
    __shared__ long long shared_next;
    BatchQueue q;
    q.start(tickets, &shared_next);
    if (threadIdx.x == 0) mbar_init(bar, 1);
    __syncthreads();

    auto batch_count = [&](long long b) {
        const long long e0 = b * C::kBe;
        return (int)((E - e0 < C::kBe) ? (E - e0) : C::kBe);
    };
    if (q.batch < n_batches) {
        const long long batch = q.batch;
        if (kStaged)
            stage_floats(staging, reinterpret_cast<const float*>(u) + batch * C::kBe * kN3,
                         batch_count(batch) * kN3);
        else if (!kBulk)
            copy_elements<N, kN2, C::kPS0, C::kES0, T>(bufA, u + batch * C::kBe * kN3,
                                                    batch_count(batch));
        else if (threadIdx.x == 0)
            load_elements<N, kN2, C::kPS0, C::kES0>(
                bufA, reinterpret_cast<const double*>(u) + batch * C::kBe * kN3, batch_count(batch),
                bar);
    }
    unsigned parity = 0;
    while (q.batch < n_batches) {
        q.draw();
        const long long batch = q.batch, next = q.next;
        const long long e0 = batch * C::kBe;
        const int cnt = batch_count(batch);
        const int valid = cnt * kN2;
        using Factor = typename std::conditional<LAMBDA, LambdaFactor, FieldFactor<T>>::type;
        Factor fac;
        if constexpr (LAMBDA) {
            fac.lam = lam;
            fac.cb = cvec + e0;
        } else {
            fac.Db = D + e0 * kN3;
        }
        const NoFactor none;
        if (threadIdx.x == 0 && next < n_batches) {
            const unsigned nbytes = (unsigned)(batch_count(next) * kN3 * sizeof(T));
            bulk_prefetch_l2(u + next * C::kBe * kN3, nbytes);
            if (!LAMBDA) bulk_prefetch_l2(D + next * C::kBe * kN3, nbytes);
        }
        constexpr int FD = C::kFactorDepth;
        double dfac[FD][Mid::kMTiles][2];
        if (kBulk) {
            if (!wait_bulk(bar, parity)) break;
            parity ^= 1u;
        } else {
            wait_copies();
            if (kStaged) {
                widen_elements<N, kN2, C::kPS0, C::kES0>(bufA, staging, cnt);
                __syncthreads();
            }
        }
        // forward: contract i, j, k
        run_stage<First, 0, T, NoFactor, FD>(bufA, bufB, nullptr, op, dfac, none, valid, warp, lane);
        __syncthreads();
        // factor for this warp's first tiles of the third stage: a whole stage hides the latency
#pragma unroll
        for (int d = 0; d < FD; ++d) fac.template load<Mid>(dfac[d], valid, warp, d, lane);
        run_stage<Mid, 0, T, NoFactor, FD>(bufB, bufA, nullptr, op, dfac, none, valid, warp, lane);
        __syncthreads();
        run_stage<Mid, 1, T, Factor, FD>(bufA, bufB, nullptr, op, dfac, fac, valid, warp, lane);
        __syncthreads();
        // backward: contract i, j, k with S itself
        run_stage<Mid, 0, T, NoFactor, FD>(bufB, bufA, nullptr, opb, dfac, none, valid, warp, lane);
        __syncthreads();
        run_stage<Mid, 0, T, NoFactor, FD>(bufA, bufB, nullptr, opb, dfac, none, valid, warp, lane);
        __syncthreads();
        // bufA is free: bring in the next batch while the last stage streams v out
        if (next < n_batches) {
            if (kStaged) {
                stage_floats(staging, reinterpret_cast<const float*>(u) + next * C::kBe * kN3,
                             batch_count(next) * kN3);
            } else if (!kBulk) {
                copy_elements<N, kN2, C::kPS0, C::kES0, T>(bufA, u + next * C::kBe * kN3,
                                                        batch_count(next));
            } else if (threadIdx.x == 0) {
                fence_async_proxy();
                load_elements<N, kN2, C::kPS0, C::kES0>(
                    bufA, reinterpret_cast<const double*>(u) + next * C::kBe * kN3,
                    batch_count(next), bar);
            }
        }
        run_stage<Last, 2, T, NoFactor, FD>(bufB, nullptr, v + e0 * kN3, opb, dfac, none, valid, warp, lane);
        q.publish();
        __syncthreads();
        q.advance();
    }
    q.finish(n_batches);
}

// ------------------------------------------------------------------ inverse Helmholtz, one
// operator and one extent per direction

template <int N0, int N1, int N2>
struct Ih3Cfg {
    static constexpr int cmax(int a, int b) { return a > b ? a : b; }
    // u as it lands: [n0][n1*n2] with padded planes
    static constexpr int kPS0 = pad_plane(N1 * N2), kES0 = N0 * kPS0;
    // after contracting axis 0: [n1][n2][o0]; after axis 1: [n2][o0][o1]; after axis 2 the
    // natural order [o0][o1][o2] again (kept in shared memory between the two halves)
    static constexpr int kRS1 = pad_row(N0), kPS1 = pad_plane(N2 * kRS1), kES1 = N1 * kPS1;
    static constexpr int kRS2 = pad_row(N1), kPS2 = pad_plane(N0 * kRS2), kES2 = N2 * kPS2;
    static constexpr int kRS3 = pad_row(N2), kPS3 = pad_plane(N1 * kRS3), kES3 = N0 * kPS3;
    static constexpr int kElemBuf = cmax(cmax(kES0, kES1), cmax(kES2, kES3));
    // two elements per batch unless that leaves room for one CTA per SM only, or the element is
    // large (from 14 x 12 x 8 values on one element per batch measured faster: that shape 13 %,
    // 13^3 4 %; below it two are faster by 3-20 %)
    static constexpr int kBe = (4 * kElemBuf * 8 <= 112 * 1024 && N0 * N1 * N2 < 1344) ? 2 : 1;
    static constexpr int kMaxTiles =
        (kBe * cmax(cmax(N1 * N2, N2 * N0), N0 * N1) + 7) / 8;
    static constexpr int kWarps = (kMaxTiles > 36) ? 8 : 4;
    using F1 = Stage<N0, N0, N1, N2, kBe, kWarps, N2, kPS0, kES0, kRS1, kPS1, kES1>;
    using F2 = Stage<N1, N1, N2, N0, kBe, kWarps, kRS1, kPS1, kES1, kRS2, kPS2, kES2>;
    using F3 = Stage<N2, N2, N0, N1, kBe, kWarps, kRS2, kPS2, kES2, kRS3, kPS3, kES3>;
    using B1 = Stage<N0, N0, N1, N2, kBe, kWarps, kRS3, kPS3, kES3, kRS1, kPS1, kES1>;
    using B3 = Stage<N2, N2, N0, N1, kBe, kWarps, kRS2, kPS2, kES2, N2, N1 * N2, N0 * N1 * N2>;
    static constexpr int kThreads = 32 * kWarps;
    static constexpr int kBufElems = kBe * kElemBuf;
    static constexpr size_t kSmemBytes = 2 * (size_t)kBufElems * sizeof(double) + 16;
    static constexpr int kBySmem = (int)((227 * 1024) / (kSmemBytes + 1024));
    static constexpr int kByWarps = 20 / kWarps;
    static constexpr int kCtasPerSm =
        (kBySmem < kByWarps ? kBySmem : kByWarps) < 1 ? 1 : (kBySmem < kByWarps ? kBySmem : kByWarps);
    // bulk copies need planes that are whole 16-byte units; odd planes use 8-byte asynchronous copies
    static constexpr bool kBulk = (N1 * N2) % 2 == 0;
    static_assert(N0 >= 4 && N1 >= 4 && N2 >= 4, "extents from 4 (one tensor step)");
};

// v[e] = (S0(x)S1(x)S2)(D[e] o ((S0^T(x)S1^T(x)S2^T) u[e])), fp64, u 16-byte aligned where a
// plane of u is an even number of values.  The
// operator fragments of a stage are fetched while the stage before it runs, so that two sets
// are live at a time whatever the number of distinct matrices.
template <int N0, int N1, int N2>
__global__ void __launch_bounds__(Ih3Cfg<N0, N1, N2>::kThreads, Ih3Cfg<N0, N1, N2>::kCtasPerSm)
inv_helmholtz3_dmma(const double* __restrict__ S0, const double* __restrict__ S1,
                    const double* __restrict__ S2, const double* __restrict__ D, const double* u,
                    double* v, long long E, unsigned long long* tickets) {
    using C = Ih3Cfg<N0, N1, N2>;
    using T = double;
    using F1 = typename C::F1;
    using F2 = typename C::F2;
    using F3 = typename C::F3;
    using B1 = typename C::B1;
    using B3 = typename C::B3;
    constexpr int kN3 = N0 * N1 * N2;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    double* bufA = reinterpret_cast<double*>(smem_raw);
    double* bufB = bufA + C::kBufElems;
    uint64_t* bar = reinterpret_cast<uint64_t*>(bufB + C::kBufElems);

    const int lane = threadIdx.x & 31;
    const int warp = ((threadIdx.x >> 5) + blockIdx.x) % C::kWarps;

    const long long n_batches = (E + C::kBe - 1) / C::kBe;
    __shared__ long long shared_next;
    BatchQueue q;
    q.start(tickets, &shared_next);
    if (threadIdx.x == 0) mbar_init(bar, 1);
    __syncthreads();
    auto batch_count = [&](long long b) {
        const long long e0 = b * C::kBe;
        return (int)((E - e0 < C::kBe) ? (E - e0) : C::kBe);
    };
    auto fetch = [&](long long b) {
        if constexpr (C::kBulk) {
            if (threadIdx.x == 0) {
                fence_async_proxy();
                load_elements<N0, N1 * N2, C::kPS0, C::kES0>(bufA, u + b * C::kBe * kN3,
                                                             batch_count(b), bar);
            }
        } else {
            copy_elements<N0, N1 * N2, C::kPS0, C::kES0, T>(bufA, u + b * C::kBe * kN3,
                                                            batch_count(b));
        }
    };
    if (q.batch < n_batches) fetch(q.batch);
    OpFrag<F1> f1;
    OpFrag<F2> f2;
    OpFrag<F3> f3;
    load_op<F1, T>(f1, S0, false, lane);
    unsigned parity = 0;
    double dfac[1][F3::kMTiles][2], none1[1][F1::kMTiles][2], none2[1][F2::kMTiles][2];
    const NoFactor none;
    while (q.batch < n_batches) {
        q.draw();
        const long long batch = q.batch, next = q.next;
        const long long e0 = batch * C::kBe;
        const int cnt = batch_count(batch);
        FieldFactor<T> fac;
        fac.Db = D + e0 * kN3;
        if (threadIdx.x == 0 && next < n_batches) {
            const unsigned nbytes = (unsigned)(batch_count(next) * kN3 * sizeof(T));
            bulk_prefetch_l2(u + next * C::kBe * kN3, nbytes);
            bulk_prefetch_l2(D + next * C::kBe * kN3, nbytes);
        }
        if constexpr (C::kBulk) {
            if (!wait_bulk(bar, parity)) break;
            parity ^= 1u;
        } else {
            wait_copies();
        }
        // forward: S0^T on the slowest axis, then S1^T, then S2^T
        load_op<F2, T>(f2, S1, false, lane);
        run_stage<F1, 0, T, NoFactor, 1>(bufA, bufB, nullptr, f1, none1, none, cnt * F1::kP, warp, lane);
        __syncthreads();
        load_op<F3, T>(f3, S2, false, lane);
        fac.template load<F3>(dfac[0], cnt * F3::kP, warp, 0, lane);
        run_stage<F2, 0, T, NoFactor, 1>(bufB, bufA, nullptr, f2, none2, none, cnt * F2::kP, warp, lane);
        __syncthreads();
        load_op<F1, T>(f1, S0, true, lane);
        run_stage<F3, 1, T, FieldFactor<T>, 1>(bufA, bufB, nullptr, f3, dfac, fac, cnt * F3::kP, warp, lane);
        __syncthreads();
        // backward: S0, S1, S2 themselves
        load_op<F2, T>(f2, S1, true, lane);
        run_stage<B1, 0, T, NoFactor, 1>(bufB, bufA, nullptr, f1, none1, none, cnt * B1::kP, warp, lane);
        __syncthreads();
        load_op<F3, T>(f3, S2, true, lane);
        run_stage<F2, 0, T, NoFactor, 1>(bufA, bufB, nullptr, f2, none2, none, cnt * F2::kP, warp, lane);
        __syncthreads();
        // bufA is free: bring in the next batch while the last stage streams v out
        if (next < n_batches) fetch(next);
        load_op<F1, T>(f1, S0, false, lane);
        run_stage<B3, 2, T, NoFactor, 1>(bufB, nullptr, v + e0 * kN3, f3, dfac, none, cnt * B3::kP, warp, lane);
        q.publish();
        __syncthreads();
        q.advance();
    }
    q.finish(n_batches);
}

// ------------------------------------------------------------------ forward rectangular operator

template <int N0, int N1, int N2, int M0, int M1, int M2>
struct ApplyCfg {
    // u as it lands: [n0][n1*n2] with padded planes
    static constexpr int kPS0 = pad_plane(N1 * N2), kES0 = N0 * kPS0;
    // after the first stage: [n1][n2][m0]
    static constexpr int kRS1 = pad_row(M0), kPS1 = pad_plane(N2 * kRS1), kES1 = N1 * kPS1;
    // after the second stage: [n2][m0][m1]
    static constexpr int kRS2 = pad_row(M1), kPS2 = pad_plane(M0 * kRS2), kES2 = N2 * kPS2;
    // two elements per batch for inputs of up to 8 points in the first direction, and for 10; one
    // otherwise (more, smaller CTAs).  Measured with one instead of two: 12 -> 8 15 %, 12 -> 12 7 %,
    // 9 -> 9 17 %, 11 -> 11 24 %, 13 -> 13 14 %, 7 -> 11 32 % faster; 8 -> 12 9 %, 8 -> 8 5 %,
    // 6 -> 10 19 %, 10 -> 10 7 %, 10 -> 14 7 %, 7 -> 7 13 % slower
    static constexpr bool kSmallInput = (N0 <= 8 || N0 == 10) && !(N0 == 7 && M0 > 8);
    static constexpr int kBe =
        ((kES0 + kES1 + kES2) * 2 * 8 <= 112 * 1024 && kSmallInput) ? 2 : 1;
    // the last stage has the most tiles; give every warp at most about a dozen
    static constexpr int kWarps = (kBe * M0 * M1 / 8 > 48) ? 8 : 4;
    using S1 = Stage<N0, M0, N1, N2, kBe, kWarps, N2, kPS0, kES0, kRS1, kPS1, kES1>;
    using S2 = Stage<N1, M1, N2, M0, kBe, kWarps, kRS1, kPS1, kES1, kRS2, kPS2, kES2>;
    using S3 = Stage<N2, M2, M0, M1, kBe, kWarps, kRS2, kPS2, kES2, M2, M1 * M2, M0 * M1 * M2>;
    static constexpr int kThreads = 32 * kWarps;
    static constexpr int kU = kBe * kES0;              // landing buffer of u
    static constexpr int kB = kBe * kES1;              // first intermediate
    static constexpr int kA = kBe * kES2;              // second intermediate
    static constexpr size_t kSmemBytes = (size_t)(kU + kB + kA) * sizeof(double) + 16;
    static constexpr int kBySmem = (int)((227 * 1024) / (kSmemBytes + 1024));
    static constexpr int kByWarps = 20 / kWarps;
    static constexpr int kCtasPerSm =
        (kBySmem < kByWarps ? kBySmem : kByWarps) < 1 ? 1 : (kBySmem < kByWarps ? kBySmem : kByWarps);
    // bulk copies need planes that are whole 16-byte units; odd planes use 8-byte asynchronous copies
    static constexpr bool kBulkPlanes = (N1 * N2) % 2 == 0;
};

// v[e] = (A(x)B(x)C) u[e]; contraction order A, B, C (slowest axis first).
template <int N0, int N1, int N2, int M0, int M1, int M2, typename T>
__global__ void __launch_bounds__(ApplyCfg<N0, N1, N2, M0, M1, M2>::kThreads,
                                  ApplyCfg<N0, N1, N2, M0, M1, M2>::kCtasPerSm)
apply_dmma(const T* __restrict__ A, const T* __restrict__ B, const T* __restrict__ Cm,
           const T* __restrict__ u, T* __restrict__ v, long long E, unsigned long long* tickets) {
    using C = ApplyCfg<N0, N1, N2, M0, M1, M2>;
    constexpr bool kBulk = sizeof(T) == sizeof(double) && C::kBulkPlanes;
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
    load_op<S1, T>(opA, A, true, lane);
    load_op<S2, T>(opB, B, true, lane);
    load_op<S3, T>(opC, Cm, true, lane);

    const long long n_batches = (E + C::kBe - 1) / C::kBe;
    __shared__ long long shared_next;
    BatchQueue q;
    q.start(tickets, &shared_next);
    if (threadIdx.x == 0) mbar_init(bar, 1);
    __syncthreads();
    auto batch_count = [&](long long b) {
        const long long e0 = b * C::kBe;
        return (int)((E - e0 < C::kBe) ? (E - e0) : C::kBe);
    };
    auto fetch = [&](long long b) {
        if (!kBulk) {
            copy_elements<N0, N1 * N2, C::kPS0, C::kES0, T>(bufU, u + b * C::kBe * S1::kIn,
                                                            batch_count(b));
        } else if (threadIdx.x == 0) {
            fence_async_proxy();
            load_elements<N0, N1 * N2, C::kPS0, C::kES0>(
                bufU, reinterpret_cast<const double*>(u) + b * C::kBe * S1::kIn, batch_count(b), bar);
        }
    };
    if (q.batch < n_batches) fetch(q.batch);
    unsigned parity = 0;
    double none1[1][S1::kMTiles][2], none2[1][S2::kMTiles][2], none3[1][S3::kMTiles][2];
    while (q.batch < n_batches) {
        q.draw();
        const long long batch = q.batch;
        const long long e0 = batch * C::kBe;
        const int cnt = batch_count(batch);
        if (kBulk) {
            if (!wait_bulk(bar, parity)) break;
            parity ^= 1u;
        } else {
            wait_copies();
        }
        q.refresh();
        const long long next = q.next;
        run_stage<S1, 0, T>(bufU, bufB, nullptr, opA, none1, NoFactor(), cnt * S1::kP, warp, lane);
        __syncthreads();
        // the landing buffer is free: bring in the next batch under the remaining two stages
        if (next < n_batches) fetch(next);
        run_stage<S2, 0, T>(bufB, bufA, nullptr, opB, none2, NoFactor(), cnt * S2::kP, warp, lane);
        __syncthreads();
        run_stage<S3, 2, T>(bufA, nullptr, v + e0 * S3::kOut, opC, none3, NoFactor(), cnt * S3::kP,
                            warp, lane);
        // the next batch's first stage writes bufB, which this batch no longer reads; the
        // barrier in the next iteration's wait orders the ticket handed over here
        q.publish();
        q.advance_batch();
    }
    q.finish(n_batches);
}

}  // namespace dmma
}  // namespace ekl
