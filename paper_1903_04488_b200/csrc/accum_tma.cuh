// accum_tma.cuh -- the streaming form of Algorithm 3 lines 5-7 used by ssgd_step on sm_100a.
//
// Persistent CTAs (one per SM) own tiles of KT_TC consecutive coordinates.  For a tile it walks the W workers;
// each (tile, worker) is one pipeline stage: three bulk asynchronous copies (cp.async.bulk, the TMA
// engine) bring that worker's g, u and v slices into a ring of shared-memory slots, completion is
// signalled on an mbarrier.  A dedicated producer warp keeps the ring full, so the bytes in flight do
// not depend on what the consumer warps are doing; eight consumer warps take a slot, compute
//     u' = fma(rho, u, g),  v' = v + u',  x += v'        (x: sum over workers, in worker order)
// write u', v' straight back to global memory (coalesced 128-bit stores) and release the slot.
// After the last worker each consumer thread hashes its four coordinates and issues the r reductions
// per coordinate into the L2-resident merged table (sum_w S(v_w) = S(sum_w v_w), Section 3).
// The producer runs ahead into the next tile while the consumers issue a tile's reductions.
// Tiles are dealt out round robin, so that at any moment the CTAs read neighbouring tiles: one contiguous range
// per CTA (no partial last round) measured slower, 9.45 against 9.38 ms at W = 256 and 4.81 against 4.71 at W = 128.
// Cache hints, measured at W = 256 / 128 (ms per step): bulk loads with an L2 evict-first policy and streaming
// (.cs) stores 9.53 / 4.86; loads without a hint 9.47 / 4.81; loads without a hint and plain stores 9.43 / 4.80 (kept).
// The results leave through 128-bit stores of the consumer threads: written into the slot in place and
// sent by bulk stores (16 KB pieces, issued by the producer before it refills the slot) measured 9.40 ms with 3
// slots and 9.46 ms with 4 against 9.37 ms at W = 256.
//
// Every mbarrier wait is bounded: after `wait_ns` nanoseconds (an argument; ssgd_set_wait_limit_ns) the waiter
// records ERR_TIMEOUT in the error word, raises the CTA's abort flag and leaves; whatever happened, the producer
// waits (bounded again) for the copies it still has in flight before it leaves, so that none lands in a CTA
// that is gone.
#pragma once
#include <stdint.h>

#include "hash.cuh"

namespace ssgd {

constexpr int ERR_BAD_INDEX = 1;
constexpr int ERR_TIMEOUT = 2;

struct AccumArgs {
    const float* g; int64_t ld_g;
    float* u; float* v; int64_t ld;
    int32_t W; int64_t d; float rho;
    float* table;        // merged [r][c], or per-worker [W][r][c]
    int64_t c;
    HashParams hp; Bucketizer bk;
    // plain-load merged mode only: insert rows [0, rows_here) in this kernel (k_insert_rows does the others)
    int32_t rows_here;
    // plain-load kernel: 1 = read g, u, v with the evict-first operator (.cs), 0 = cached in L2 only (.cg)
    int32_t loads_evict_first;
    // merged modes: if not NULL, the per-coordinate sum over workers of the new v (fp64 accumulation in worker
    // order, rounded once) is also written to xsum[d]: the second round's exact sums, and k_insert_rows' input
    float* xsum;
    // d-bit map of coordinates whose zero-out (Algorithm 3 line 13) is still pending from the previous step: their
    // u and v are read as +0.  NULL: nothing is pending.
    const uint32_t* pending;
    uint64_t wait_ns;    // limit of every wait inside the kernel (bulk-copy pipeline only)
    int32_t withhold;    // test hook (bulk-copy pipeline only): the producer of CTA (withhold - 1) issues nothing
};

constexpr int KT_CONSUMER_WARPS = 8;
constexpr int KT_CONSUMERS = KT_CONSUMER_WARPS * 32;
constexpr int KT_THREADS = KT_CONSUMERS + 32;       // + one producer warp
// Tile shape.  What matters is the length of the contiguous piece each bulk copy takes from one worker's row: with
// W workers the kernel reads 3 W interleaved streams, and DRAM serves long pieces better than short ones.  Measured
// on B200 at d = 11,173,962 (TB/s of 20 W d bytes; groups per thread x ring slots; piece = 4 KB x groups):
//   W = 256:  1 x 6  5.72    2 x 4  5.93    4 x 4  6.09    4 x 3  6.13    6 x 2  6.14    8 x 2  6.11
//   W = 128:  1 x 6  5.70    2 x 4  5.90    4 x 3  6.06        W = 64:  4 x 3  5.91  (plain-load kernel 5.88)
//   16 consumer warps x 2 groups x 3 slots: 6.12; 4 warps x 8 x 3: 6.01.
constexpr int KT_VEC = 4;                           // float4 groups per consumer thread and stage
constexpr int KT_TC = KT_CONSUMERS * 4 * KT_VEC;    // 4096 coordinates per tile: 16 KB pieces
constexpr int KT_STAGES = 3;                        // ring slots of 3 * 4 * KT_TC = 48 KB each (one CTA per SM)

struct alignas(128) KtSlot { float g[KT_TC]; float u[KT_TC]; float v[KT_TC]; };
struct KtShared {
    KtSlot slot[KT_STAGES];
    uint64_t full[KT_STAGES];
    uint64_t empty[KT_STAGES];
    volatile int abort;
};

#ifdef __CUDACC__
// The four pending bits of the float4 group that starts at coordinate i0 (a multiple of 4).
__device__ __forceinline__ uint32_t pending_bits4(const uint32_t* __restrict__ pending, int64_t i0) {
    return pending ? (__ldg(pending + (i0 >> 5)) >> (i0 & 31)) & 0xFu : 0u;
}
__device__ __forceinline__ bool pending_bit(const uint32_t* __restrict__ pending, int64_t i) {
    return pending && ((__ldg(pending + (i >> 5)) >> (i & 31)) & 1u);
}
// Applies the pending zero-out to one worker's u, v of that group before they are used.
__device__ __forceinline__ void drop_pending(uint32_t bits, float4& u4, float4& v4) {
    if (bits & 1u) { u4.x = 0.f; v4.x = 0.f; }
    if (bits & 2u) { u4.y = 0.f; v4.y = 0.f; }
    if (bits & 4u) { u4.z = 0.f; v4.z = 0.f; }
    if (bits & 8u) { u4.w = 0.f; v4.w = 0.f; }
}

__device__ __forceinline__ void red_add(float* addr, float x) {
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(addr), "f"(x) : "memory");
}
// The same with an L2 eviction policy for the line it touches (table_policy: the table's lines are the last to go)
__device__ __forceinline__ void red_add_hint(float* addr, float x, uint64_t policy) {
    asm volatile("red.global.add.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(addr), "f"(x), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t table_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait; false if it gave up (wait_ns elapsed) or the CTA is aborting.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort, uint64_t wait_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0) {
            if (*abort || global_ns() - t0 > wait_ns) return false;
            __nanosleep(64);
        }
    }
}
// global -> shared bulk copy; src, dst 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

template <int R, bool POW2>
__global__ void __launch_bounds__(KT_THREADS)
k_accum_insert_tma(const AccumArgs A, int32_t* __restrict__ errflag) {
    extern __shared__ __align__(128) unsigned char kt_raw[];
    KtShared& S = *reinterpret_cast<KtShared*>(kt_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t d_main = A.d & ~(int64_t)3;                      // bulk copies cover whole float4 groups
    const int64_t ntiles = (d_main + KT_TC - 1) / KT_TC;

    pdl_trigger();
    if (tid == 0) {
        for (int s = 0; s < KT_STAGES; ++s) { mbar_init(&S.full[s], 1); mbar_init(&S.empty[s], KT_CONSUMER_WARPS); }
        S.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_wait();
    __syncthreads();

    if (warp == KT_CONSUMER_WARPS) {
        // ---------------- producer warp: one thread feeds the ring ----------------
        if (lane == 0) {
            uint32_t n = 0;
            bool ok = true;
            const bool withheld = A.withhold && (int)blockIdx.x == A.withhold - 1;
            for (int64_t tile = blockIdx.x; tile < ntiles && ok && !withheld; tile += gridDim.x) {
                const int64_t i0 = tile * KT_TC;
                const uint32_t bytes = (uint32_t)((d_main - i0 < KT_TC ? d_main - i0 : KT_TC) * 4);
                for (int w = 0; w < A.W; ++w, ++n) {
                    const int s = n % KT_STAGES;
                    if (n >= KT_STAGES && !mbar_wait(&S.empty[s], ((n / KT_STAGES) - 1) & 1, &S.abort, A.wait_ns)) { ok = false; break; }
                    mbar_expect_tx(&S.full[s], 3 * bytes);
                    bulk_load(S.slot[s].g, A.g + (int64_t)w * A.ld_g + i0, bytes, &S.full[s]);
                    bulk_load(S.slot[s].u, A.u + (int64_t)w * A.ld + i0, bytes, &S.full[s]);
                    bulk_load(S.slot[s].v, A.v + (int64_t)w * A.ld + i0, bytes, &S.full[s]);
                }
            }
            if (!ok) {                                     // give up: report and tell the consumers
                atomicExch(errflag, ERR_TIMEOUT);
                S.abort = 1;
            }
            // the copies of the last stages issued must have landed before this CTA may go away, whether the
            // consumers took them or gave up (returns at once for stages that completed long ago)
            const uint32_t first = n > KT_STAGES ? n - KT_STAGES : 0;
            for (uint32_t m = first; m < n; ++m) {
                uint64_t* bar = &S.full[m % KT_STAGES];
                const uint64_t t0 = global_ns();
                while (!mbar_try_wait(bar, (m / KT_STAGES) & 1) && global_ns() - t0 < A.wait_ns) __nanosleep(64);
            }
        }
    } else {
        // ---------------- consumer warps ----------------
        const uint64_t tpol = table_policy();
        uint32_t n = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
            // this thread's float4 groups of the tile: group v starts at coordinate tile * KT_TC + 4 * (tid + v * KT_CONSUMERS)
            const int64_t t0 = tile * KT_TC;
            double xs[KT_VEC][4];                           // sum over workers of the new v: fp64, worker order
            uint32_t pend[KT_VEC];
            bool active[KT_VEC];
#pragma unroll
            for (int v = 0; v < KT_VEC; ++v) {
                const int64_t i0 = t0 + 4 * (tid + v * KT_CONSUMERS);
                active[v] = i0 < d_main;
                pend[v] = active[v] ? pending_bits4(A.pending, i0) : 0u;
                xs[v][0] = xs[v][1] = xs[v][2] = xs[v][3] = 0.;
            }
            for (int w = 0; w < A.W; ++w, ++n) {
                const int s = n % KT_STAGES;
                if (!mbar_wait(&S.full[s], (n / KT_STAGES) & 1, &S.abort, A.wait_ns)) { ok = false; break; }
#pragma unroll
                for (int v = 0; v < KT_VEC; ++v) {
                    if (!active[v]) continue;
                    const int at = 4 * (tid + v * KT_CONSUMERS);
                    const int64_t i0 = t0 + at;
                    const float4 g4 = *reinterpret_cast<const float4*>(&S.slot[s].g[at]);
                    float4 u4 = *reinterpret_cast<const float4*>(&S.slot[s].u[at]);
                    float4 v4 = *reinterpret_cast<const float4*>(&S.slot[s].v[at]);
                    if (pend[v]) drop_pending(pend[v], u4, v4);
                    float4 un, vn;
                    un.x = __fmaf_rn(A.rho, u4.x, g4.x); vn.x = __fadd_rn(v4.x, un.x);
                    un.y = __fmaf_rn(A.rho, u4.y, g4.y); vn.y = __fadd_rn(v4.y, un.y);
                    un.z = __fmaf_rn(A.rho, u4.z, g4.z); vn.z = __fadd_rn(v4.z, un.z);
                    un.w = __fmaf_rn(A.rho, u4.w, g4.w); vn.w = __fadd_rn(v4.w, un.w);
                    *reinterpret_cast<float4*>(A.u + (int64_t)w * A.ld + i0) = un;
                    *reinterpret_cast<float4*>(A.v + (int64_t)w * A.ld + i0) = vn;
                    xs[v][0] = __dadd_rn(xs[v][0], (double)vn.x); xs[v][1] = __dadd_rn(xs[v][1], (double)vn.y);
                    xs[v][2] = __dadd_rn(xs[v][2], (double)vn.z); xs[v][3] = __dadd_rn(xs[v][3], (double)vn.w);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&S.empty[s]);
            }
            if (!ok) break;
#pragma unroll
            for (int v = 0; v < KT_VEC; ++v) {
                if (!active[v]) continue;
                const int64_t i0 = t0 + 4 * (tid + v * KT_CONSUMERS);
                const float x[4] = {(float)xs[v][0], (float)xs[v][1], (float)xs[v][2], (float)xs[v][3]};
                if (A.xsum) __stcs(reinterpret_cast<float4*>(A.xsum + i0), make_float4(x[0], x[1], x[2], x[3]));
#pragma unroll
                for (int j = 0; j < R; ++j) {
                    uint32_t hb[4];
                    row_hashes<POW2, 4>(A.hp.row[j], A.bk, (uint32_t)i0, hb);
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (x[e] != 0.0f) red_add_hint(A.table + (int64_t)j * A.c + (hb[e] & P31), apply_sign(x[e], hb[e]), tpol);
                }
            }
        }
        if (!ok && lane == 0) { atomicExch(errflag, ERR_TIMEOUT); S.abort = 1; }
        // ragged tail (d not a multiple of 4): at most three coordinates, plain loads, one thread
        if (ok && blockIdx.x == 0 && tid == 0) {
            for (int64_t i = d_main; i < A.d; ++i) {
                double xd = 0.;
                const bool pend = pending_bit(A.pending, i);
                for (int64_t w = 0; w < A.W; ++w) {
                    const float un = __fmaf_rn(A.rho, pend ? 0.f : A.u[w * A.ld + i], A.g[w * A.ld_g + i]);
                    const float vn = __fadd_rn(pend ? 0.f : A.v[w * A.ld + i], un);
                    A.u[w * A.ld + i] = un;
                    A.v[w * A.ld + i] = vn;
                    xd = __dadd_rn(xd, (double)vn);
                }
                const float x = (float)xd;
                if (A.xsum) A.xsum[i] = x;
                for (int j = 0; j < R; ++j) {
                    uint32_t hb[1];
                    row_hashes<POW2, 1>(A.hp.row[j], A.bk, (uint32_t)i, hb);
                    if (x != 0.0f) red_add(A.table + (int64_t)j * A.c + (hb[0] & P31), apply_sign(x, hb[0]));
                }
            }
        }
    }
}

#endif  // __CUDACC__
}  // namespace ssgd
