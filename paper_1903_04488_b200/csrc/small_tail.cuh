// small_tail.cuh -- Algorithm 3 lines 9-13 in ONE kernel, for problems so small that a chain of short launches
// costs more than the work itself (d up to a few million coordinates, at most SMALL_MAX_NCAND candidates).
//
// The grid is co-resident (one CTA per SM, launched cooperatively) and its CTAs meet at four grid-wide barriers:
//
//   phase 1   every CTA estimates its share of the coordinates (Algorithm 4 estimate: median of the r signed
//             buckets), stores est[i] and counts the top 12 bits of |est| in a shared-memory histogram -> H1.
//             As many rows of the table as fit one CTA's shared memory are copied there first and looked up there
//             (3.5 random 4-byte reads per clock per SM against 1.1 from L2, measured), provided the CTA has
//             enough lookups to do for the copy to pay; the other rows are read from L2.  A table split over the shared memory of a
//             thread-block cluster was measured and dropped: random reads of another CTA's shared memory run at
//             0.7 per clock per SM in a cluster of 2 and 0.4 in clusters of 4 to 16 -- slower than L2.
//   barrier   H1 complete: every CTA finds the first threshold digit d1 for itself
//   phase 2   histogram H2 of the next 11 key bits among the items inside d1
//   barrier   -> second digit d2
//   phase 3   histogram H3 of the last 8 key bits among the items matching the 23-bit prefix
//   barrier   -> threshold key T and tie quota Q
//   phase 4   every warp counts, per segment of 128 consecutive coordinates, those above T and those equal to T
//   barrier   -> with the counts of everything before it, every warp emits its candidates to their final slots:
//             cand_idx ascending, ties at T to the smallest coordinates (line 9), and reads each candidate's exact
//             sum over the workers right there (line 10).  The CTA that draws the last ticket goes on alone
//             (nobody waits for it):
//   phase 5   exact top-k of |xs| in shared memory, 12 + 11 + 8 bits, ordered emit of out_idx / out_val (line 11);
//             line 13 as marks in the pending map (deferred) or as zeros written to u and v (eager, small k*W).
// (An earlier form marked the candidates in two d-bit maps and let the last CTA walk them in order: 13 us of
// instruction issue on one SM at d = 2^20, growing with d; the distributed form costs one more barrier.)
//
// Every wait at a barrier is bounded: after `wait_ns` the waiting CTA records ERR_TIMEOUT in the error word,
// raises the abort flag so that the others stop waiting too, and returns.
#pragma once
#include <stdint.h>

#include "accum_tma.cuh"
#include "estimate.cuh"
#include "hash.cuh"
#include "select.cuh"

namespace ssgd {

constexpr int ST_THREADS = 512;
constexpr int ST_WARPS = ST_THREADS / 32;
constexpr int64_t SMALL_MAX_NCAND = 16384;               // candidates the last CTA holds in shared memory
constexpr int64_t SMALL_MAX_D = (int64_t)1 << 22;        // coordinates (the last CTA walks two d-bit maps)
constexpr size_t SMALL_TABLE_SMEM_MAX = 200 * 1024;      // table slice per CTA (next to a 16 KiB histogram)

struct SmallState {          // zeroed before the step
    uint32_t bar;            // arrivals at the grid barriers (monotonic: barrier n completes at n * gridDim.x)
    uint32_t abort;          // a wait gave up
    uint32_t ticket;         // CTAs that finished phase 4
    uint32_t pad;
    uint64_t trace[12];      // globaltimer stamps of CTA 0 (slots 0-5) and of the last CTA (6-10), for diagnostics
    // coordinates above / at the threshold per super-segment (64 segments of 128 coordinates), counted in phase 4
    uint32_t sup_a[ST_THREADS], sup_b[ST_THREADS];
};

struct SmallArgs {
    const float* table; int64_t c; int64_t d;
    HashParams hp; Bucketizer bk;
    float* est;              // [d], 16-byte aligned
    uint32_t* h1; uint32_t* h2; uint32_t* h3;   // global histograms of the candidate selection, zeroed
    SmallState* st;
    uint32_t* map_a; uint32_t* map_b;           // [>= ceil(d/128)] words each: per-segment counts, written before they are read
    const float* xsum;       // [d] per-coordinate sums over the workers of the new v
    int32_t* cand_idx; float* xs;               // [ncand] (kept for inspection)
    uint32_t ncand, k;
    int32_t* out_idx; float* out_val;           // [k]
    uint32_t* pending;       // the pending map of a deferred line 13: emptied in phase 1 (the accumulate kernel has
    int64_t pending_words;   // consumed it), marked again in phase 5 if mark_pending != 0
    int32_t mark_pending;
    float* u; float* v; int64_t ld; int32_t W;  // eager line 13 written here when zero_inline != 0
    int32_t zero_inline;
    int32_t rows_smem;       // every CTA copies rows [0, rows_smem) of the table into its shared memory and looks up there
    uint64_t wait_ns;        // limit of a barrier wait
    int32_t withhold;        // test hook: CTA (withhold - 1) leaves before the first barrier, so the others' wait runs out
    int32_t* errflag;
};

#ifdef __CUDACC__

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// n-th (1-based) grid barrier.  False, in every thread of the CTA, if the wait ran out or another CTA gave up.
__device__ __forceinline__ bool small_grid_barrier(const SmallArgs& A, uint32_t nth, uint32_t* s_flag) {
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t ok = 1;
        __threadfence();
        atomicAdd(&A.st->bar, 1u);
        const uint32_t target = nth * gridDim.x;
        const uint64_t t0 = global_ns();
        for (uint32_t it = 1; ld_acquire_u32(&A.st->bar) < target; ++it) {
            if ((it & 15u) == 0 && (ld_acquire_u32(&A.st->abort) != 0u || global_ns() - t0 > A.wait_ns)) { ok = 0; break; }
        }
        if (!ok) { atomicExch(&A.st->abort, 1u); atomicExch(A.errflag, ERR_TIMEOUT); }
        __threadfence();
        *s_flag = ok;
    }
    __syncthreads();
    return *s_flag != 0;
}

// Largest bin D of a shared-memory histogram with count(bins > D) < want <= count(bins >= D); rem = want - count(bins > D).
// All ST_THREADS threads call.  1 <= want <= total count.
template <int NBINS>
__device__ __forceinline__ void smem_find_from_top(const uint32_t* hist, uint32_t want, uint32_t* s_warp, uint32_t* s_found,
                                                   uint32_t& digit, uint32_t& rem) {
    constexpr int NT = NBINS < ST_THREADS ? NBINS : ST_THREADS;   // searching threads
    constexpr int PER = NBINS / NT;
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    if (t == 0) { s_found[0] = 0; s_found[1] = 1; }
    uint32_t sum = 0, incl = 0;
    if (t < NT) {
#pragma unroll
        for (int s = 0; s < PER; ++s) sum += hist[t * PER + s];
    }
    incl = sum;                                            // sum over the lanes >= lane of this warp
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t o = __shfl_down_sync(0xFFFFFFFFu, incl, off);
        if (lane + off < 32) incl += o;
    }
    if (lane == 0) s_warp[warp] = incl;
    __syncthreads();
    if (t < NT) {
        uint32_t above = incl - sum;
        for (int w2 = warp + 1; w2 < ST_WARPS; ++w2) above += s_warp[w2];
        if (above < want && want <= above + sum) {
            uint32_t acc = above;
            for (int b = t * PER + PER - 1; b >= t * PER; --b) {
                const uint32_t h = hist[b];
                if (acc + h >= want) { s_found[0] = (uint32_t)b; s_found[1] = want - acc; break; }
                acc += h;
            }
        }
    }
    __syncthreads();
    digit = s_found[0];
    rem = s_found[1];
    __syncthreads();
}

// Exclusive block-wide scan of two counters per thread (ST_THREADS threads).
__device__ __forceinline__ void block_excl_scan2(uint32_t a, uint32_t b, uint32_t* s_a, uint32_t* s_b, uint32_t& ea, uint32_t& eb) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t ia = a, ib = b;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t oa = __shfl_up_sync(0xFFFFFFFFu, ia, off), ob = __shfl_up_sync(0xFFFFFFFFu, ib, off);
        if (lane >= off) { ia += oa; ib += ob; }
    }
    __syncthreads();
    if (lane == 31) { s_a[warp] = ia; s_b[warp] = ib; }
    __syncthreads();
    ea = ia - a; eb = ib - b;
    for (int w = 0; w < warp; ++w) { ea += s_a[w]; eb += s_b[w]; }
    __syncthreads();
}

template <int R, bool POW2>
__global__ void __launch_bounds__(ST_THREADS, 1)
k_small_tail(const SmallArgs A) {
    extern __shared__ __align__(16) unsigned char st_dyn[];   // table slice, later the candidates and their sums
    __shared__ SelShared sh;
    __shared__ uint32_t s_flag, s_warp_a[ST_WARPS], s_warp_b[ST_WARPS], s_found[2];
    const int tid = threadIdx.x;
    const int64_t groups = (A.d + 3) >> 2;
    const int64_t gstride = (int64_t)gridDim.x * ST_THREADS;
    const int64_t gtid = (int64_t)blockIdx.x * ST_THREADS + tid;
    auto stamp = [&](int slot, bool mine) { if (mine && tid == 0) A.st->trace[slot] = global_ns(); };
    const bool first_cta = blockIdx.x == 0;
    stamp(0, first_cta);

    // ---------------- phase 1: table slice -> shared memory; estimates, H1 ----------------
    for (int b = tid; b < H1_BINS; b += ST_THREADS) sh.hist[b] = 0;
    if (A.pending)
        for (int64_t t = gtid; t < A.pending_words; t += gstride) A.pending[t] = 0u;   // consumed by the accumulate kernel
    const float* slice = reinterpret_cast<const float*>(st_dyn);
    if (A.rows_smem > 0) {
        const int64_t n = (int64_t)A.rows_smem * A.c;      // the first rows are one contiguous piece of the table
        if ((A.c & 3) == 0) {
            float4* dst = reinterpret_cast<float4*>(st_dyn);
            const float4* src = reinterpret_cast<const float4*>(A.table);
            for (int64_t b0 = tid; b0 < (n >> 2); b0 += ST_THREADS * 8) {
                float4 t[8];
#pragma unroll
                for (int s8 = 0; s8 < 8; ++s8) {
                    const int64_t at = b0 + s8 * ST_THREADS;
                    t[s8] = __ldcg(src + (at < (n >> 2) ? at : 0));
                }
#pragma unroll
                for (int s8 = 0; s8 < 8; ++s8) if (b0 + s8 * ST_THREADS < (n >> 2)) dst[b0 + s8 * ST_THREADS] = t[s8];
            }
        } else {
            float* dst = reinterpret_cast<float*>(st_dyn);
            for (int64_t b0 = tid; b0 < n; b0 += ST_THREADS * 8) {
                float t[8];
#pragma unroll
                for (int s8 = 0; s8 < 8; ++s8) {
                    const int64_t at = b0 + s8 * ST_THREADS;
                    t[s8] = __ldcg(A.table + (at < n ? at : 0));
                }
#pragma unroll
                for (int s8 = 0; s8 < 8; ++s8) if (b0 + s8 * ST_THREADS < n) dst[b0 + s8 * ST_THREADS] = t[s8];
            }
        }
    }
    __syncthreads();
    stamp(1, first_cta);
    for (int64_t q = gtid; q < groups; q += gstride) {
        const int64_t i0 = q << 2;
        float rowv[4][R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            uint32_t hb[4];
            row_hashes<POW2, 4>(A.hp.row[j], A.bk, (uint32_t)i0, hb);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int64_t at = (int64_t)j * A.c + (hb[e] & P31);
                rowv[e][j] = apply_sign(j < A.rows_smem ? slice[at] : table_load(A.table + at), hb[e]);
            }
        }
        float m[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) m[e] = median_of<R>(rowv[e]);
        if (i0 + 3 < A.d) {
            *reinterpret_cast<float4*>(A.est + i0) = make_float4(m[0], m[1], m[2], m[3]);
#pragma unroll
            for (int e = 0; e < 4; ++e) atomicAdd(&sh.hist[key_of(m[e]) >> H1_SHIFT], 1u);
        } else {
            for (int e = 0; e < 4 && i0 + e < A.d; ++e) {
                A.est[i0 + e] = m[e];
                atomicAdd(&sh.hist[key_of(m[e]) >> H1_SHIFT], 1u);
            }
        }
    }
    __syncthreads();
    flush_hist<H1_BINS>(sh.hist, A.h1);
    if (A.withhold && (int)blockIdx.x == A.withhold - 1) return;
    stamp(2, first_cta);
    if (!small_grid_barrier(A, 1, &s_flag)) return;
    stamp(3, first_cta);

    // keys of this thread's coordinates, re-read from est (L2) in each of the later phases, four groups per round
    // trip (the loads are unconditional so that they are all in flight before the first is used)
    auto for_my_keys = [&](auto&& f) {
        for (int64_t q0 = gtid; q0 < groups; q0 += 4 * gstride) {
            float4 t[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int64_t i0 = (q0 + b * gstride) << 2;
                t[b] = __ldcg(reinterpret_cast<const float4*>(A.est + (i0 + 3 < A.d ? i0 : 0)));
            }
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int64_t i0 = (q0 + b * gstride) << 2;
                if (i0 >= A.d) continue;
                uint32_t key[4];
                if (i0 + 3 < A.d) {
                    key[0] = key_of(t[b].x); key[1] = key_of(t[b].y); key[2] = key_of(t[b].z); key[3] = key_of(t[b].w);
                } else {                                   // the ragged last group
#pragma unroll
                    for (int e = 0; e < 4; ++e) key[e] = i0 + e < A.d ? key_of(__ldcg(A.est + i0 + e)) : NO_ITEM;
                }
                f(i0, key);
            }
        }
    };

    // ---------------- phase 2: second digit ----------------
    uint32_t d1, rem1, d2, rem2, d3, rem3;
    block_find_from_top<H1_BINS>(A.h1, A.ncand, sh, d1, rem1);
    for (int b = tid; b < H2_BINS; b += ST_THREADS) sh.hist[b] = 0;
    __syncthreads();
    for_my_keys([&](int64_t, const uint32_t (&key)[4]) {
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (key[e] != NO_ITEM && (key[e] >> H1_SHIFT) == d1) atomicAdd(&sh.hist[(key[e] >> H2_SHIFT) & (H2_BINS - 1)], 1u);
    });
    __syncthreads();
    flush_hist<H2_BINS>(sh.hist, A.h2);
    if (!small_grid_barrier(A, 2, &s_flag)) return;
    stamp(4, first_cta);

    // ---------------- phase 3: third digit ----------------
    block_find_from_top<H2_BINS>(A.h2, rem1, sh, d2, rem2);
    const uint32_t prefix = (d1 << H2_BITS) | d2;
    for (int b = tid; b < H3_BINS; b += ST_THREADS) sh.hist[b] = 0;
    __syncthreads();
    for_my_keys([&](int64_t, const uint32_t (&key)[4]) {
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (key[e] != NO_ITEM && (key[e] >> H2_SHIFT) == prefix) atomicAdd(&sh.hist[key[e] & (H3_BINS - 1)], 1u);
    });
    __syncthreads();
    flush_hist<H3_BINS>(sh.hist, A.h3);
    if (!small_grid_barrier(A, 3, &s_flag)) return;
    stamp(5, first_cta);

    // ---------------- phase 4: ordered candidates (line 9) and the second round (line 10), by every CTA ----------------
    // A warp owns, in each of its iterations, one SEGMENT of 128 consecutive coordinates (its 32 lanes hold 32
    // consecutive groups of four).  4a: count the segment's coordinates above T (a) and equal to T (b); the counts go
    // to seg_a / seg_b and are added to the counters of the segment's SUPER-segment (64 segments).  Grid barrier.
    // 4b: a candidate's slot is the number of a's before it plus min(number of b's before it, Q) -- ties at T go to the
    // smallest coordinates -- and "before it" = whole super-segments (block-wide scan of at most 512 counters) +
    // earlier segments of its super-segment (64 counts, two loads per lane) + earlier lanes of its segment (warp
    // scan).  The candidate list comes out ascending, each candidate's exact sum is read right where it is emitted.
    block_find_from_top<H3_BINS>(A.h3, rem2, sh, d3, rem3);
    const uint32_t T = (d1 << H1_SHIFT) | (d2 << H2_SHIFT) | d3, Q = rem3;
    const int lane = tid & 31;
    uint32_t* seg_a = A.map_a;                             // [ceil(d / 128)] of each, written by the owning warps
    uint32_t* seg_b = A.map_b;
    // keys of one segment's share of this lane: gt / eq masks over its four coordinates
    auto lane_masks = [&](int64_t q, uint32_t& gt, uint32_t& eq) {
        const int64_t i0 = q << 2;
        uint32_t key[4];
        if (i0 + 3 < A.d) {
            const float4 t = __ldcg(reinterpret_cast<const float4*>(A.est + i0));
            key[0] = key_of(t.x); key[1] = key_of(t.y); key[2] = key_of(t.z); key[3] = key_of(t.w);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) key[e] = i0 + e < A.d ? key_of(__ldcg(A.est + i0 + e)) : NO_ITEM;
        }
        gt = 0; eq = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (key[e] == NO_ITEM) continue;
            gt |= (key[e] > T ? 1u : 0u) << e;
            eq |= (key[e] == T ? 1u : 0u) << e;
        }
    };
    for (int64_t q = gtid; q - lane < groups; q += gstride) {          // warp-uniform trip count
        uint32_t gt, eq;
        lane_masks(q, gt, eq);
        const uint32_t ta = __reduce_add_sync(0xFFFFFFFFu, (uint32_t)__popc(gt));
        const uint32_t tb = __reduce_add_sync(0xFFFFFFFFu, (uint32_t)__popc(eq));
        if (lane == 0) {
            const int64_t seg = q >> 5;
            seg_a[seg] = ta; seg_b[seg] = tb;
            if (ta) atomicAdd(&A.st->sup_a[seg >> 6], ta);
            if (tb) atomicAdd(&A.st->sup_b[seg >> 6], tb);
        }
    }
    if (!small_grid_barrier(A, 4, &s_flag)) return;
    stamp(11, first_cta);
    {
        uint32_t* s_sup_a = sh.hist;                       // exclusive prefixes over the super-segments
        uint32_t* s_sup_b = sh.hist + ST_THREADS;
        const int64_t nsuper = (((A.d + 127) >> 7) + 63) >> 6;         // <= ST_THREADS since d <= SMALL_MAX_D
        const uint32_t ca = tid < nsuper ? __ldcg(&A.st->sup_a[tid]) : 0u, cb = tid < nsuper ? __ldcg(&A.st->sup_b[tid]) : 0u;
        uint32_t ea, eb;
        block_excl_scan2(ca, cb, s_warp_a, s_warp_b, ea, eb);
        s_sup_a[tid] = ea; s_sup_b[tid] = eb;
        __syncthreads();
        for (int64_t q = gtid; q - lane < groups; q += gstride) {
            uint32_t gt, eq;
            lane_masks(q, gt, eq);
            const int64_t seg = (q - lane) >> 5, sup = seg >> 6;
            const int within = (int)(seg & 63);
            // a's and b's in the earlier segments of this super-segment
            uint32_t pa = (lane < within ? __ldcg(seg_a + (sup << 6) + lane) : 0u) + (lane + 32 < within ? __ldcg(seg_a + (sup << 6) + 32 + lane) : 0u);
            uint32_t pb = (lane < within ? __ldcg(seg_b + (sup << 6) + lane) : 0u) + (lane + 32 < within ? __ldcg(seg_b + (sup << 6) + 32 + lane) : 0u);
            pa = __reduce_add_sync(0xFFFFFFFFu, pa);
            pb = __reduce_add_sync(0xFFFFFFFFu, pb);
            if (__ballot_sync(0xFFFFFFFFu, (gt | eq) != 0u) == 0u) continue;      // nothing to emit in this segment
            const uint32_t packed = (uint32_t)__popc(gt) | ((uint32_t)__popc(eq) << 16);   // at most 4 each
            uint32_t incl = packed;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += o;
            }
            uint32_t a = s_sup_a[sup] + pa + ((incl - packed) & 0xFFFFu), b = s_sup_b[sup] + pb + ((incl - packed) >> 16);
            uint32_t bits = gt | eq;
            while (bits) {
                const int e = __ffs(bits) - 1;
                bits &= bits - 1;
                uint32_t slot = 0xFFFFFFFFu;
                if ((gt >> e) & 1u) { slot = a + (b < Q ? b : Q); ++a; }
                else { if (b < Q) slot = a + b; ++b; }
                if (slot < A.ncand) {
                    const int64_t coord = (q << 2) + e;
                    A.cand_idx[slot] = (int32_t)coord;
                    A.xs[slot] = __ldcg(A.xsum + coord);   // line 10: the accumulate kernel's sum over the workers
                }
            }
        }
    }
    if (!block_is_last(&A.st->ticket, sh)) return;

    // ---------------- phase 5 (one CTA): final top-k (line 11) and line 13 ----------------
    stamp(6, true);
    int32_t* cand_s = reinterpret_cast<int32_t*>(st_dyn);
    float* xs_s = reinterpret_cast<float*>(st_dyn) + A.ncand;
    for (int b = tid; b < H1_BINS; b += ST_THREADS) sh.hist[b] = 0;
    __syncthreads();
    stamp(7, true);
    for (uint32_t m = tid; m < A.ncand; m += ST_THREADS) {
        const uint32_t i = (uint32_t)__ldcg(A.cand_idx + m);
        const bool ok = (int64_t)i < A.d;                  // consistent histograms fill every slot with a coordinate
        const float x = ok ? __ldcg(A.xs + m) : 0.0f;
        cand_s[m] = ok ? (int32_t)i : 0;
        xs_s[m] = x;
        atomicAdd(&sh.hist[key_of(x) >> H1_SHIFT], 1u);
    }
    __syncthreads();
    stamp(8, true);
    // line 11: exact top-k of |xs| among the candidates, all in shared memory
    uint32_t e1, r1, e2, r2, e3, r3;
    smem_find_from_top<H1_BINS>(sh.hist, A.k, s_warp_a, s_found, e1, r1);
    for (int b = tid; b < H2_BINS; b += ST_THREADS) sh.hist[b] = 0;
    __syncthreads();
    for (uint32_t m = tid; m < A.ncand; m += ST_THREADS) {
        const uint32_t key = key_of(xs_s[m]);
        if ((key >> H1_SHIFT) == e1) atomicAdd(&sh.hist[(key >> H2_SHIFT) & (H2_BINS - 1)], 1u);
    }
    __syncthreads();
    smem_find_from_top<H2_BINS>(sh.hist, r1, s_warp_a, s_found, e2, r2);
    const uint32_t prefix2 = (e1 << H2_BITS) | e2;
    for (int b = tid; b < H3_BINS; b += ST_THREADS) sh.hist[b] = 0;
    __syncthreads();
    for (uint32_t m = tid; m < A.ncand; m += ST_THREADS) {
        const uint32_t key = key_of(xs_s[m]);
        if ((key >> H2_SHIFT) == prefix2) atomicAdd(&sh.hist[key & (H3_BINS - 1)], 1u);
    }
    __syncthreads();
    smem_find_from_top<H3_BINS>(sh.hist, r2, s_warp_a, s_found, e3, r3);
    const uint32_t T2 = (e1 << H1_SHIFT) | (e2 << H2_SHIFT) | e3, Q2 = r3;
    stamp(9, true);
    // ordered emit: thread t owns the candidates [t * per2, (t + 1) * per2)
    const uint32_t per2 = (A.ncand + ST_THREADS - 1) / ST_THREADS;
    const uint32_t m_lo = tid * per2 < A.ncand ? tid * per2 : A.ncand;
    const uint32_t m_hi = m_lo + per2 < A.ncand ? m_lo + per2 : A.ncand;
    uint32_t cg = 0, ce = 0;
    for (uint32_t m = m_lo; m < m_hi; ++m) {
        const uint32_t key = key_of(xs_s[m]);
        cg += key > T2 ? 1u : 0u;
        ce += key == T2 ? 1u : 0u;
    }
    uint32_t g_before, e_before;
    block_excl_scan2(cg, ce, s_warp_a, s_warp_b, g_before, e_before);
    for (uint32_t m = m_lo; m < m_hi; ++m) {
        const float x = xs_s[m];
        const uint32_t key = key_of(x);
        uint32_t slot = 0xFFFFFFFFu;
        if (key > T2) { slot = g_before + (e_before < Q2 ? e_before : Q2); ++g_before; }
        else if (key == T2) { if (e_before < Q2) slot = g_before + e_before; ++e_before; }
        if (slot < A.k) {
            const int32_t i = cand_s[m];
            A.out_idx[slot] = i;
            A.out_val[slot] = x;
            if (A.mark_pending) atomicOr(A.pending + (i >> 5), 1u << (i & 31));  // deferred line 13
            if (A.zero_inline)
                for (int64_t w = 0; w < A.W; ++w) { A.u[w * A.ld + i] = 0.0f; A.v[w * A.ld + i] = 0.0f; }
        }
    }
    __syncthreads();
    stamp(10, true);
}

#endif  // __CUDACC__
}  // namespace ssgd
