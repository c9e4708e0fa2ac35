// sparse_select.cuh -- Algorithm 3 line 9 with early termination: "query every coordinate, keep the
// ncand largest |estimate|" without paying r table reads for coordinates that provably cannot make it.
//
// The unsketch kernel is bound by scattered 4-byte reads of the L2-resident table (one sector per read,
// about one sector per clock per SM), so the way to make it faster is to read less:
//
//   * |median of r values| >= t  implies  at least (r+1)/2 of the r values have magnitude >= t.
//     So once a coordinate cannot reach (r+1)/2 "big" row estimates any more, its remaining rows need
//     not be read: it is certainly below t.
//   * A safe t comes from a sample: k_unsketch_sample computes exact estimates for 1/64 of the
//     float4 groups (pseudo-randomly placed), histograms them, and takes the histogram-bin edge `bin_lo`
//     below which fewer than  ncand/64 + 6*sqrt(ncand/64) + 16  sampled estimates remain ... i.e. a
//     threshold the full vector exceeds at least ncand times except with negligible probability.
//   * k_unsketch_pruned evaluates every coordinate with that early exit and appends the survivors
//     (exact estimate in a bin >= bin_lo) to a compact list.  The survivor set does not depend on how the
//     pruning went: it is exactly { i : bin(|est_i|) >= bin_lo }.
//   * If the list holds at least ncand entries (and fits), the top-ncand of all d coordinates is the
//     top-ncand of the list: k_select_sparse, one 8-CTA cluster, runs the radix select on the list
//     (histograms reduced through distributed shared memory), breaks ties at the threshold by coordinate
//     index, marks the selected coordinates in a d-bit map and compacts the map in order, so cand_idx
//     comes out ascending exactly as the dense path produces it.
//   * Otherwise a flag opens the gate of the dense path (k_unsketch + select.cuh), whose kernels are
//     always enqueued behind and return at once when the gate is closed.
#pragma once
#include <cooperative_groups.h>
#include <stdint.h>

#include "estimate.cuh"
#include "hash.cuh"
#include "select.cuh"

namespace ssgd {

// measured at C2/C3/C4: 1/32 0.210/0.345/1.524 ms (sample + early-exit kernel), 1/64 0.207, 1/128 0.205, 1/256 0.208/0.338/1.467
#ifndef SSGD_SAMPLE_SHIFT
#define SSGD_SAMPLE_SHIFT 6
#endif
constexpr int SPARSE_SAMPLE_SHIFT = SSGD_SAMPLE_SHIFT;   // one float4 group in 2^shift is sampled
constexpr int SPARSE_CLUSTER = 8;                 // CTAs in the selection cluster (portable maximum)
constexpr int SPARSE_THREADS = 1024;
constexpr int SPARSE_MAX_TIES = 2048;             // ties at the threshold handled in shared memory

struct SparseState {                              // zeroed before the step
    uint32_t bin_lo;       // prune threshold: H1 bin index; 0 = nothing can be pruned
    uint32_t n_surv;       // survivors appended (may exceed the capacity; entries beyond it are dropped)
    uint32_t fallback;     // != 0: the dense path must run (this word is the dense kernels' gate)
    uint32_t d1, rem1;     // first threshold digit of the survivors' histogram
    uint32_t ticket[2];
    uint32_t pad[9];
};

struct SparseBuffers {
    uint32_t* h1_sample;   // [H1_BINS] zeroed
    uint32_t* h1;          // [H1_BINS] zeroed: histogram of the survivors' estimates
    SparseState* state;
    int32_t* list_idx;     // [cap]
    float* list_est;       // [cap]
    uint32_t cap;
    uint32_t* bitmap;      // [ceil(d/32)] zeroed
};

struct SparseArgs {
    const float* table; int64_t c; int64_t d;
    HashParams hp; Bucketizer bk;
    SparseBuffers sp;
    uint32_t ncand;
    uint32_t want_sample;  // rank (from the top) in the sample's histogram that defines bin_lo
};

#ifdef __CUDACC__
namespace cg = cooperative_groups;

__device__ __forceinline__ uint32_t mix32(uint32_t x) {
    x ^= x >> 16; x *= 0x7FEB352Du; x ^= x >> 15; x *= 0x846CA68Bu; x ^= x >> 16;
    return x;
}

// ---- sample: exact estimates of one group in 32, histogram, prune threshold ------------------------
template <int R, bool POW2>
__global__ void __launch_bounds__(SEL_THREADS)
k_unsketch_sample(const SparseArgs A) {
    __shared__ SelShared sh;
    pdl_trigger();
    for (int b = threadIdx.x; b < H1_BINS; b += SEL_THREADS) sh.hist[b] = 0;
    pdl_wait();
    __syncthreads();
    const int64_t groups = (A.d + 3) >> 2;
    const int64_t windows = (groups + (1 << SPARSE_SAMPLE_SHIFT) - 1) >> SPARSE_SAMPLE_SHIFT;
    const int64_t stride = (int64_t)gridDim.x * SEL_THREADS;
    for (int64_t s = (int64_t)blockIdx.x * SEL_THREADS + threadIdx.x; s < windows; s += stride) {
        const int64_t q = (s << SPARSE_SAMPLE_SHIFT) + (mix32((uint32_t)s) & ((1u << SPARSE_SAMPLE_SHIFT) - 1));
        const int64_t i0 = q << 2;
        if (i0 >= A.d) continue;
        float rowv[4][R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            uint32_t hb[4];
            row_hashes<POW2, 4>(A.hp.row[j], A.bk, (uint32_t)i0, hb);
#pragma unroll
            for (int e = 0; e < 4; ++e)
                rowv[e][j] = apply_sign(table_load(A.table + (int64_t)j * A.c + (hb[e] & P31)), hb[e]);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (i0 + e < A.d) atomicAdd(&sh.hist[key_of(median_of<R>(rowv[e])) >> H1_SHIFT], 1u);
    }
    __syncthreads();
    flush_hist<H1_BINS>(sh.hist, A.sp.h1_sample);
    if (block_is_last(&A.sp.state->ticket[0], sh)) {
        // total sampled; if the sample is too small to place the rank, prune nothing (bin_lo stays 0)
        uint32_t digit = 0, rem = 0;
        block_find_from_top<H1_BINS>(A.sp.h1_sample, A.want_sample, sh, digit, rem);
        uint32_t part = 0;
        for (int b = threadIdx.x; b < H1_BINS; b += SEL_THREADS) part += __ldcg(A.sp.h1_sample + b);
        for (int off = 16; off; off >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, off);
        if ((threadIdx.x & 31) == 0) sh.warp_sum[threadIdx.x >> 5] = part;
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t total = 0;
            for (int w = 0; w < SEL_WARPS; ++w) total += sh.warp_sum[w];
            A.sp.state->bin_lo = (A.want_sample >= 1 && A.want_sample <= total) ? digit : 0u;
        }
    }
}

// ---- every coordinate, with early exit; survivors appended to the list -----------------------------
#ifndef SSGD_PRUNED_MINBLOCKS
#define SSGD_PRUNED_MINBLOCKS 1
#endif
#ifndef SSGD_PRUNED_NC
#define SSGD_PRUNED_NC 4
#endif
template <int R, bool POW2>
__global__ void __launch_bounds__(SEL_THREADS, SSGD_PRUNED_MINBLOCKS)
k_unsketch_pruned(const SparseArgs A) {
    __shared__ SelShared sh;
    constexpr int NEED = (R + 1) / 2;      // big row estimates a survivor must have
    pdl_trigger();
    for (int b = threadIdx.x; b < H1_BINS; b += SEL_THREADS) sh.hist[b] = 0;
    pdl_wait();
    const uint32_t bin_lo = A.sp.state->bin_lo;
    __syncthreads();
    const int lane = threadIdx.x & 31;
    constexpr int NC = SSGD_PRUNED_NC;                     // consecutive coordinates per thread
    const int64_t groups = (A.d + NC - 1) / NC;
    const int64_t stride = (int64_t)gridDim.x * SEL_THREADS;
    // warp-uniform trip count: the append below uses warp-wide shuffles
    for (int64_t base = (int64_t)blockIdx.x * SEL_THREADS + (threadIdx.x & ~31); base < groups; base += stride) {
        const int64_t q = base + lane;
        const int64_t i0 = q * NC;
        float rowv[NC][R];
        int cnt[NC];
        bool alive[NC];
        bool any = false;
#pragma unroll
        for (int e = 0; e < NC; ++e) { cnt[e] = 0; alive[e] = q < groups && i0 + e < A.d; any = any || alive[e]; }
        if (any) {
#pragma unroll
            for (int j = 0; j < NEED; ++j) {
                uint32_t hb[NC];
                row_hashes<POW2, NC>(A.hp.row[j], A.bk, (uint32_t)i0, hb);
#pragma unroll
                for (int e = 0; e < NC; ++e) {
                    const float val = apply_sign(table_load(A.table + (int64_t)j * A.c + (hb[e] & P31)), hb[e]);
                    rowv[e][j] = val;
                    cnt[e] += (key_of(val) >> H1_SHIFT) >= bin_lo ? 1 : 0;
                }
            }
#pragma unroll
            for (int e = 0; e < NC; ++e) alive[e] = alive[e] && cnt[e] + (R - NEED) >= NEED;
#pragma unroll
            for (int j = NEED; j < R; ++j) {
                any = false;
#pragma unroll
                for (int e = 0; e < NC; ++e) any = any || alive[e];
                if (any) {
                    uint32_t hb[NC];
                    row_hashes<POW2, NC>(A.hp.row[j], A.bk, (uint32_t)i0, hb);
#pragma unroll
                    for (int e = 0; e < NC; ++e) {
                        if (alive[e]) {
                            const float val = apply_sign(table_load(A.table + (int64_t)j * A.c + (hb[e] & P31)), hb[e]);
                            rowv[e][j] = val;
                            cnt[e] += (key_of(val) >> H1_SHIFT) >= bin_lo ? 1 : 0;
                            alive[e] = cnt[e] + (R - 1 - j) >= NEED;
                        }
                    }
                }
            }
        }
        float m[NC];
        int ns = 0;
#pragma unroll
        for (int e = 0; e < NC; ++e) {
            m[e] = 0.f;
            if (alive[e]) {
                m[e] = median_of<R>(rowv[e]);
                alive[e] = (key_of(m[e]) >> H1_SHIFT) >= bin_lo;
                ns += alive[e] ? 1 : 0;
            }
        }
        if (__ballot_sync(0xFFFFFFFFu, ns > 0)) {
            int incl = ns;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += o;
            }
            const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
            uint32_t wbase = 0;
            if (lane == 0) wbase = atomicAdd(&A.sp.state->n_surv, (uint32_t)total);
            wbase = __shfl_sync(0xFFFFFFFFu, wbase, 0);
            uint32_t pos = wbase + (uint32_t)(incl - ns);
#pragma unroll
            for (int e = 0; e < NC; ++e) {
                if (alive[e]) {
                    if (pos < A.sp.cap) { A.sp.list_idx[pos] = (int32_t)(i0 + e); A.sp.list_est[pos] = m[e]; }
                    ++pos;
                    atomicAdd(&sh.hist[key_of(m[e]) >> H1_SHIFT], 1u);
                }
            }
        }
    }
    __syncthreads();
    flush_hist<H1_BINS>(sh.hist, A.sp.h1);
    if (block_is_last(&A.sp.state->ticket[1], sh)) {
        const uint32_t n = __ldcg(&A.sp.state->n_surv);
        const bool fb = n < A.ncand || n > A.sp.cap;
        uint32_t d1 = 0, rem1 = 1;
        if (!fb) block_find_from_top<H1_BINS>(A.sp.h1, A.ncand, sh, d1, rem1);
        if (threadIdx.x == 0) { A.sp.state->fallback = fb ? 1u : 0u; A.sp.state->d1 = d1; A.sp.state->rem1 = rem1; }
    }
}

// ---- one cluster: radix select on the survivor list, ties by index, bitmap, ordered emit -----------
struct SparseShared {
    uint32_t hist[H2_BINS];              // H2, then H3 (in CTA 0: the cluster-wide sums)
    uint32_t wsum[32];
    uint32_t found[2];
    uint32_t thr[2][2];                  // per pass: prefix/threshold and remaining count (valid in CTA 0)
    uint32_t n_ties;                     // CTA 0
    int32_t ties[SPARSE_MAX_TIES];       // CTA 0: coordinates with key == T
    uint32_t cta_total[SPARSE_CLUSTER];  // CTA 0: selected bits per CTA range
    uint32_t bail;                       // CTA 0
};

// Largest digit D with count(bins > D) < want <= count(bins >= D) over a shared-memory histogram;
// all SPARSE_THREADS threads call.  nbins is a multiple of 32 and at most H2_BINS.
__device__ __forceinline__ void cta_find_from_top(SparseShared& sh, int nbins, uint32_t want, uint32_t& digit, uint32_t& rem) {
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int per_warp = nbins / 32;                   // 64 or 8 bins per warp
    uint32_t part = 0;
    for (int b = lane; b < per_warp; b += 32) part += sh.hist[warp * per_warp + b];
    for (int off = 16; off; off >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, off);
    if (lane == 0) sh.wsum[warp] = part;
    if (t == 0) { sh.found[0] = 0; sh.found[1] = 1; }
    __syncthreads();
    if (warp == 0) {
        // lane = index of a warp-sized chunk; suffix sums over chunks above this one
        const uint32_t mine = sh.wsum[lane];
        uint32_t incl = mine;
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t o = __shfl_down_sync(0xFFFFFFFFu, incl, off);
            if (lane + off < 32) incl += o;
        }
        const uint32_t above = incl - mine;
        if (above < want && want <= above + mine) {
            uint32_t acc = above;
            for (int b = lane * per_warp + per_warp - 1; b >= lane * per_warp; --b) {
                const uint32_t h = sh.hist[b];
                if (acc + h >= want) { sh.found[0] = (uint32_t)b; sh.found[1] = want - acc; break; }
                acc += h;
            }
        }
    }
    __syncthreads();
    digit = sh.found[0];
    rem = sh.found[1];
    __syncthreads();
}

// LB list entries per thread are loaded together (independent loads in flight), then processed.
constexpr int LB = 8;
constexpr uint32_t NO_KEY = 0xFFFFFFFFu;                    // marks "past the end of the list"
__device__ __forceinline__ void list_keys(const float* __restrict__ est, uint32_t n, uint32_t i0, uint32_t step,
                                          uint32_t (&keys)[LB]) {
#pragma unroll
    for (int u = 0; u < LB; ++u) {
        const uint32_t i = i0 + (uint32_t)u * step;
        keys[u] = i < n ? key_of(__ldcg(est + i)) : NO_KEY;
    }
}

__global__ void __launch_bounds__(SPARSE_THREADS)
k_select_sparse(SparseBuffers sp, int64_t d, uint32_t ncand, int32_t* __restrict__ cand_idx) {
    __shared__ SparseShared sh;
    cg::cluster_group cluster = cg::this_cluster();
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const unsigned rank = cluster.block_rank();
    const int gthreads = SPARSE_CLUSTER * SPARSE_THREADS;
    const int gt = rank * SPARSE_THREADS + t;
    SparseShared* sh0 = cluster.map_shared_rank(&sh, 0);
    pdl_trigger();
    pdl_wait();
    if (__ldcg(&sp.state->fallback) != 0) return;          // uniform over the cluster: the dense path runs instead
    const uint32_t n = __ldcg(&sp.state->n_surv);
    const uint32_t d1 = sp.state->d1, rem1 = sp.state->rem1;

    // ---- H2 and H3 over the list: per-CTA histogram, summed into CTA 0 through distributed shared memory
    uint32_t prefix = d1, want = rem1;
    uint32_t T = 0, Q = 0;
    for (int pass = 0; pass < 2; ++pass) {
        const int nbins = pass == 0 ? H2_BINS : H3_BINS;
        for (int b = t; b < H2_BINS; b += SPARSE_THREADS) sh.hist[b] = 0;
        if (pass == 0 && rank == 0 && t == 0) { sh.n_ties = 0; sh.bail = 0; }
        __syncthreads();
        for (uint32_t i0 = gt; i0 < n; i0 += gthreads * LB) {
            uint32_t keys[LB];
            list_keys(sp.list_est, n, i0, gthreads, keys);
#pragma unroll
            for (int u = 0; u < LB; ++u) {
                const uint32_t key = keys[u];
                if (key == NO_KEY) continue;
                if (pass == 0) { if ((key >> H1_SHIFT) == prefix) atomicAdd(&sh.hist[(key >> H2_SHIFT) & (H2_BINS - 1)], 1u); }
                else           { if ((key >> H2_SHIFT) == prefix) atomicAdd(&sh.hist[key & (H3_BINS - 1)], 1u); }
            }
        }
        cluster.sync();                                     // every CTA's private histogram is complete
        if (rank == 0) {
            // CTA 0 sums the eight histograms through distributed shared memory, then finds the digit
            uint32_t acc[H2_BINS / SPARSE_THREADS];
#pragma unroll
            for (int q = 0; q < H2_BINS / SPARSE_THREADS; ++q) {
                const int b = t + q * SPARSE_THREADS;
                acc[q] = 0;
                if (b < nbins)
                    for (unsigned r2 = 0; r2 < SPARSE_CLUSTER; ++r2) acc[q] += cluster.map_shared_rank(&sh, r2)->hist[b];
            }
            __syncthreads();
#pragma unroll
            for (int q = 0; q < H2_BINS / SPARSE_THREADS; ++q) {
                const int b = t + q * SPARSE_THREADS;
                if (b < nbins) sh.hist[b] = acc[q];
            }
            __syncthreads();
            uint32_t digit, rem;
            cta_find_from_top(sh, nbins, want, digit, rem);
            if (t == 0) {
                sh.thr[pass][0] = (prefix << (pass == 0 ? H2_BITS : H3_BITS)) | digit;
                sh.thr[pass][1] = rem;
            }
        }
        cluster.sync();                                     // thr[pass] is published; the histograms may be reused
        prefix = sh0->thr[pass][0];
        want = sh0->thr[pass][1];
    }
    T = prefix;
    Q = want;

    // ---- ties at the threshold: the Q smallest coordinates win ---------------------------------------
    for (uint32_t i0 = gt; i0 < n; i0 += gthreads * LB) {
        uint32_t keys[LB];
        list_keys(sp.list_est, n, i0, gthreads, keys);
#pragma unroll
        for (int u = 0; u < LB; ++u) {
            if (keys[u] == T) {                                 // NO_KEY is never a threshold (bit 31 set)
                const uint32_t slot = atomicAdd(&sh0->n_ties, 1u);
                if (slot < SPARSE_MAX_TIES) sh0->ties[slot] = sp.list_idx[i0 + (uint32_t)u * gthreads];
            }
        }
    }
    cluster.sync();
    const uint32_t n_ties = sh0->n_ties;
    if (n_ties > SPARSE_MAX_TIES) {
        // too many equal magnitudes to rank here: hand over to the dense path (nothing written yet)
        if (rank == 0 && t == 0) sp.state->fallback = 1u;
        cluster.sync();
        return;
    }
    // every CTA takes its own copy of the tied coordinates (remote shared memory is slow to scan)
    if (rank != 0)
        for (uint32_t s = t; s < n_ties; s += SPARSE_THREADS) sh.ties[s] = sh0->ties[s];
    __syncthreads();
    // selected: key > T, or key == T and fewer than Q tied coordinates are smaller
    for (uint32_t i0 = gt; i0 < n; i0 += gthreads * LB) {
        uint32_t keys[LB];
        int32_t idxs[LB];
        list_keys(sp.list_est, n, i0, gthreads, keys);
#pragma unroll
        for (int u = 0; u < LB; ++u) {
            const uint32_t i = i0 + (uint32_t)u * gthreads;
            idxs[u] = i < n ? sp.list_idx[i] : 0;
        }
#pragma unroll
        for (int u = 0; u < LB; ++u) {
            const uint32_t key = keys[u];
            if (key == NO_KEY) continue;
            const int32_t idx = idxs[u];
            bool sel = key > T;
            if (key == T) {
                uint32_t smaller = 0;
                for (uint32_t s = 0; s < n_ties; ++s) smaller += sh.ties[s] < idx ? 1u : 0u;
                sel = smaller < Q;
            }
            if (sel) atomicOr(&sp.bitmap[(uint32_t)idx >> 5], 1u << ((uint32_t)idx & 31));
        }
    }
    __threadfence();
    cluster.sync();

    // ---- ordered compaction of the bitmap: each warp owns a contiguous run of words, read 32 at a time
    const int64_t nwords = (d + 31) >> 5;
    const int nwarps = gthreads / 32;
    const int64_t per_warp = ((nwords + nwarps - 1) / nwarps + 31) / 32 * 32;
    const int64_t w_lo = (int64_t)(gt >> 5) * per_warp;
    const int64_t w_hi = w_lo + per_warp < nwords ? w_lo + per_warp : nwords;
    constexpr int BATCH = 8;                                // bitmap words in flight per lane
    uint32_t mine = 0;
    for (int64_t wb = w_lo; wb < w_hi; wb += 32 * BATCH) {
        uint32_t bits[BATCH];
#pragma unroll
        for (int u = 0; u < BATCH; ++u) {
            const int64_t w = wb + u * 32 + lane;
            bits[u] = w < w_hi ? __ldcg(sp.bitmap + w) : 0u;
        }
#pragma unroll
        for (int u = 0; u < BATCH; ++u) mine += __popc(bits[u]);
    }
    for (int off = 16; off; off >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, off);   // warp total
    if (lane == 0) sh.wsum[warp] = mine;
    __syncthreads();
    uint32_t before = 0, cta_sum = 0;
    for (int w2 = 0; w2 < SPARSE_THREADS / 32; ++w2) { const uint32_t s2 = sh.wsum[w2]; if (w2 < warp) before += s2; cta_sum += s2; }
    if (t == 0) sh0->cta_total[rank] = cta_sum;
    cluster.sync();
    for (unsigned r2 = 0; r2 < rank; ++r2) before += sh0->cta_total[r2];
    uint32_t run = before;                                  // selected coordinates before this warp's next word group
    for (int64_t wb = w_lo; wb < w_hi; wb += 32 * BATCH) {
        uint32_t bits[BATCH];
#pragma unroll
        for (int u = 0; u < BATCH; ++u) {
            const int64_t w = wb + u * 32 + lane;
            bits[u] = w < w_hi ? __ldcg(sp.bitmap + w) : 0u;
        }
#pragma unroll
        for (int u = 0; u < BATCH; ++u) {
            const int64_t w = wb + u * 32 + lane;
            uint32_t b32 = bits[u];
            const uint32_t c = __popc(b32);
            uint32_t incl = c;
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += o;
            }
            uint32_t slot = run + incl - c;
            while (b32) {
                const int b = __ffs(b32) - 1;
                b32 &= b32 - 1;
                if (slot < ncand) cand_idx[slot] = (int32_t)((w << 5) + b);
                ++slot;
            }
            run += __shfl_sync(0xFFFFFFFFu, incl, 31);
        }
    }
    cluster.sync();                                         // CTA 0's shared memory stays alive until all are done
}

#endif  // __CUDACC__
}  // namespace ssgd
