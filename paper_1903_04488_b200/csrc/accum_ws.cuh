// accum_ws.cuh -- warp-specialised form of Algorithm 3 lines 5-7: stream and sketch run on different warps.
//
// The accumulate+insert work has two halves that want different things from an SM: streaming g, u, v
// (HBM-bound, wants bytes in flight) and r scattered reductions per coordinate (bound by the load/store
// unit's rate for scattered sectors).  When the same warps do both, one half waits for the other; with few
// workers per coordinate (W <= 16) the reductions are a large part of the total.  Here a CTA has
//   warp 0        producer: bulk asynchronous copies (cp.async.bulk) of one worker's g/u/v tile slices into
//                 a ring of shared-memory slots, full/empty mbarriers (as in accum_tma.cuh)
//   warps 1-8     stream: take a slot, compute u' = fma(rho,u,g), v' = v+u', store them (128-bit, streaming),
//                 keep x = sum_w v' in registers; after the last worker of a tile hand x over through a
//                 double-buffered shared-memory vector and go straight on to the next tile
//   warps 9-12    sketch: take a finished x vector, hash its coordinates (h_j, s_j for the r rows) and issue
//                 the reductions into the L2-resident merged table
// so that loads (TMA), stores and reductions (load/store unit) and the hash arithmetic overlap inside one CTA.
// All waits are bounded (two seconds), as in accum_tma.cuh: error word, abort flag, drain of copies in flight.
#pragma once
#include <stdint.h>

#include "accum_tma.cuh"

namespace ssgd {

#ifndef SSGD_WS_STAGES
#define SSGD_WS_STAGES 5
#endif
#ifndef SSGD_WS_STREAM_WARPS
#define SSGD_WS_STREAM_WARPS 8
#endif
#ifndef SSGD_WS_SKETCH_WARPS
#define SSGD_WS_SKETCH_WARPS 4
#endif
constexpr int WS_STREAM_WARPS = SSGD_WS_STREAM_WARPS;
constexpr int WS_SKETCH_WARPS = SSGD_WS_SKETCH_WARPS;
constexpr int WS_STREAM_THREADS = WS_STREAM_WARPS * 32;
constexpr int WS_SKETCH_THREADS = WS_SKETCH_WARPS * 32;
constexpr int WS_THREADS = 32 + WS_STREAM_THREADS + WS_SKETCH_THREADS;
constexpr int WS_TC = WS_STREAM_THREADS * 4;          // coordinates per tile
constexpr int WS_STAGES = SSGD_WS_STAGES;
constexpr int WS_GROUPS_PER_SKETCH_THREAD = WS_TC / 4 / WS_SKETCH_THREADS;   // float4 groups of x per sketch thread

struct alignas(128) WsSlot { float g[WS_TC]; float u[WS_TC]; float v[WS_TC]; };
struct WsShared {
    WsSlot slot[WS_STAGES];
    alignas(16) float x[2][WS_TC];      // finished tile sums, double-buffered
    uint64_t full[WS_STAGES];
    uint64_t empty[WS_STAGES];
    uint64_t x_full[2];
    uint64_t x_empty[2];
    volatile int abort;
};

#ifdef __CUDACC__

template <int R, bool POW2>
__global__ void __launch_bounds__(WS_THREADS)
k_accum_insert_ws(const AccumArgs A, int32_t* __restrict__ errflag) {
    extern __shared__ __align__(128) unsigned char ws_raw[];
    WsShared& S = *reinterpret_cast<WsShared*>(ws_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t d_main = A.d & ~(int64_t)3;
    const int64_t ntiles = (d_main + WS_TC - 1) / WS_TC;

    pdl_trigger();
    if (tid == 0) {
        for (int s = 0; s < WS_STAGES; ++s) { mbar_init(&S.full[s], 1); mbar_init(&S.empty[s], WS_STREAM_WARPS); }
        for (int b = 0; b < 2; ++b) { mbar_init(&S.x_full[b], WS_STREAM_WARPS); mbar_init(&S.x_empty[b], WS_SKETCH_WARPS); }
        S.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_wait();
    __syncthreads();

    if (warp == 0) {
        // ---------------- producer ----------------
        if (lane == 0) {
            const uint64_t pol = policy_evict_first();
            uint32_t n = 0;
            bool ok = true;
            for (int64_t tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                const int64_t i0 = tile * WS_TC;
                const uint32_t bytes = (uint32_t)((d_main - i0 < WS_TC ? d_main - i0 : WS_TC) * 4);
                for (int w = 0; w < A.W; ++w, ++n) {
                    const int s = n % WS_STAGES;
                    if (n >= WS_STAGES && !mbar_wait(&S.empty[s], ((n / WS_STAGES) - 1) & 1, &S.abort)) { ok = false; break; }
                    mbar_expect_tx(&S.full[s], 3 * bytes);
                    bulk_load(S.slot[s].g, A.g + (int64_t)w * A.ld_g + i0, bytes, &S.full[s], pol);
                    bulk_load(S.slot[s].u, A.u + (int64_t)w * A.ld + i0, bytes, &S.full[s], pol);
                    bulk_load(S.slot[s].v, A.v + (int64_t)w * A.ld + i0, bytes, &S.full[s], pol);
                }
            }
            if (!ok) {
                atomicExch(errflag, ERR_TIMEOUT);
                S.abort = 1;
                const uint32_t first = n > WS_STAGES ? n - WS_STAGES : 0;
                for (uint32_t m = first; m < n; ++m) {
                    uint64_t* bar = &S.full[m % WS_STAGES];
                    const uint64_t t0 = global_ns();
                    while (!mbar_try_wait(bar, (m / WS_STAGES) & 1) && global_ns() - t0 < KT_WAIT_NS) __nanosleep(64);
                }
            }
        }
    } else if (warp <= WS_STREAM_WARPS) {
        // ---------------- stream warps ----------------
        const int st = tid - 32;                              // 0 .. WS_STREAM_THREADS-1
        uint32_t n = 0, nt = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++nt) {
            const int64_t i0 = tile * WS_TC + 4 * st;
            const bool active = i0 < d_main;
            double x0 = 0., x1 = 0., x2 = 0., x3 = 0.;
            const uint32_t pend = active ? pending_bits4(A.pending, i0) : 0u;
            for (int w = 0; w < A.W; ++w, ++n) {
                const int s = n % WS_STAGES;
                if (!mbar_wait(&S.full[s], (n / WS_STAGES) & 1, &S.abort)) { ok = false; break; }
                if (active) {
                    const float4 g4 = *reinterpret_cast<const float4*>(&S.slot[s].g[4 * st]);
                    float4 u4 = *reinterpret_cast<const float4*>(&S.slot[s].u[4 * st]);
                    float4 v4 = *reinterpret_cast<const float4*>(&S.slot[s].v[4 * st]);
                    if (pend) drop_pending(pend, u4, v4);
                    float4 un, vn;
                    un.x = __fmaf_rn(A.rho, u4.x, g4.x); vn.x = __fadd_rn(v4.x, un.x);
                    un.y = __fmaf_rn(A.rho, u4.y, g4.y); vn.y = __fadd_rn(v4.y, un.y);
                    un.z = __fmaf_rn(A.rho, u4.z, g4.z); vn.z = __fadd_rn(v4.z, un.z);
                    un.w = __fmaf_rn(A.rho, u4.w, g4.w); vn.w = __fadd_rn(v4.w, un.w);
                    __stcs(reinterpret_cast<float4*>(A.u + (int64_t)w * A.ld + i0), un);
                    __stcs(reinterpret_cast<float4*>(A.v + (int64_t)w * A.ld + i0), vn);
                    x0 = __dadd_rn(x0, (double)vn.x); x1 = __dadd_rn(x1, (double)vn.y);
                    x2 = __dadd_rn(x2, (double)vn.z); x3 = __dadd_rn(x3, (double)vn.w);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&S.empty[s]);
            }
            if (!ok) break;
            // hand the tile's sums to the sketch warps
            const int b = nt & 1;
            if (nt >= 2 && !mbar_wait(&S.x_empty[b], ((nt >> 1) - 1) & 1, &S.abort)) { ok = false; break; }
            const float4 xf = make_float4((float)x0, (float)x1, (float)x2, (float)x3);
            *reinterpret_cast<float4*>(&S.x[b][4 * st]) = xf;
            if (active && A.xsum) __stcs(reinterpret_cast<float4*>(A.xsum + i0), xf);
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.x_full[b]);
        }
        if (!ok && lane == 0) { atomicExch(errflag, ERR_TIMEOUT); S.abort = 1; }
        // ragged tail (d not a multiple of 4): at most three coordinates, plain loads, one thread
        if (ok && blockIdx.x == 0 && st == 0) {
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
    } else {
        // ---------------- sketch warps ----------------
        const int sk = tid - 32 - WS_STREAM_THREADS;          // 0 .. WS_SKETCH_THREADS-1
        uint32_t nt = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++nt) {
            const int b = nt & 1;
            if (!mbar_wait(&S.x_full[b], (nt >> 1) & 1, &S.abort)) { ok = false; break; }
#pragma unroll
            for (int q = 0; q < WS_GROUPS_PER_SKETCH_THREAD; ++q) {
                const int grp = sk + q * WS_SKETCH_THREADS;   // float4 group inside the tile
                const int64_t i0 = tile * WS_TC + 4 * grp;
                if (i0 < d_main) {
                    const float4 xv = *reinterpret_cast<const float4*>(&S.x[b][4 * grp]);
                    const float x[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                    for (int j = 0; j < R; ++j) {
                        uint32_t hb[4];
                        row_hashes<POW2, 4>(A.hp.row[j], A.bk, (uint32_t)i0, hb);
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (x[e] != 0.0f) red_add(A.table + (int64_t)j * A.c + (hb[e] & P31), apply_sign(x[e], hb[e]));
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.x_empty[b]);
        }
        if (!ok && lane == 0) { atomicExch(errflag, ERR_TIMEOUT); S.abort = 1; }
    }
}

#endif  // __CUDACC__
}  // namespace ssgd
