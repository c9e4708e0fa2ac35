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
//   * If the list holds at least ncand entries, the top-ncand of all d coordinates is the top-ncand of the
//     list, which the kernels of list_select.cuh extract (cand_idx comes out ascending, exactly as the dense
//     path produces it).
//   * Otherwise (the sample misjudged the threshold) the last block of k_unsketch_pruned resets the list
//     and raises a flag; a second launch of the same kernel, always enqueued behind and returning at once
//     unless the flag is up, redoes the pass without pruning.  The list has room for all d coordinates.
#pragma once
#include <stdint.h>

#include "estimate.cuh"
#include "hash.cuh"
#include "select.cuh"

namespace ssgd {

// measured at C2/C3/C4: 1/32 0.210/0.345/1.524 ms (sample + early-exit kernel), 1/64 0.207, 1/128 0.205, 1/256 0.208/0.338/1.467
constexpr int SPARSE_SAMPLE_SHIFT = 6;   // one float4 group in 2^shift is sampled

struct SparseState {                              // zeroed before the step
    uint32_t bin_lo;       // prune threshold: H1 bin index; 0 = nothing can be pruned
    uint32_t n_surv;       // survivors appended to the list
    uint32_t fallback;     // 1: too few survivors, the unpruned pass must run; 2: it has run
    uint32_t d1, rem1;     // first threshold digit of the survivors' histogram H1 and the count wanted inside it
    uint32_t thr_key;      // T: the exact 31-bit threshold key
    uint32_t quota_eq;     // Q: how many items with key == T are selected (smallest coordinates first)
    uint32_t ticket[6];    // finished-block counters: sample, first pass, unpruned rerun, list histogram, map count, fold
    uint32_t fold_ones;    // set bits of the bucket bitmap whose density is measured: the folded one, or the unfolded one
                           // when it is used row by row (filter_unsketch.cuh, rowbits_unsketch.cuh)
    uint32_t use_table;    // 1: that bitmap is too dense to prune; the first pass reads the table instead
    uint32_t pad[1];
};

struct SparseBuffers {
    uint32_t* h1_sample;   // [H1_BINS] zeroed
    uint32_t* h1;          // [H1_BINS] zeroed: histogram of the survivors' estimates
    SparseState* state;
    uint32_t* h2;          // [H2_BINS] zeroed: next 11 key bits of the list items inside the first digit
    uint32_t* h19;         // [2^19] zeroed: the low 19 key bits of the same items
    int32_t* list_idx;     // [cap], cap >= d
    float* list_est;       // [cap]
    uint32_t cap;
    uint32_t* map_a;       // [ceil(d/32)] zeroed: coordinates above the threshold
    uint32_t* map_b;       // [ceil(d/32)] zeroed: coordinates at the threshold (ties)
    uint32_t* chunk_a;     // [map chunks] marks per chunk of map words, then exclusive offsets
    uint32_t* chunk_b;
};

struct SparseArgs {
    const float* table; int64_t c; int64_t d;
    HashParams hp; Bucketizer bk;
    SparseBuffers sp;
    uint32_t ncand;
    uint32_t want_sample;  // rank (from the top) in the sample's histogram that defines bin_lo
    uint32_t n_sampled_min; // a lower bound of the number of sampled coordinates: 4 * (windows - 2)
    int32_t rerun;         // 0: the pruned pass; 1: the unpruned pass behind it (runs only if fallback == 1)
    int32_t gated;         // 1: the pruned pass runs only if use_table is set (it follows a bitmap filter that declined)
};

#ifdef __CUDACC__
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
        // if the sample is too small to place the rank, prune nothing (bin_lo stays 0); the number of sampled
        // coordinates is a function of d alone: every window holds one group of 4, the last group may be short
        uint32_t digit = 0, rem = 0;
        block_find_from_top<H1_BINS>(A.sp.h1_sample, A.want_sample, sh, digit, rem);
        if (threadIdx.x == 0)
            A.sp.state->bin_lo = (A.want_sample >= 1 && A.want_sample <= A.n_sampled_min) ? digit : 0u;
    }
}

// ---- every coordinate, with early exit; survivors appended to the list -----------------------------
constexpr int PRUNED_NC = 4;                             // consecutive coordinates per thread
template <int R, bool POW2>
__global__ void __launch_bounds__(SEL_THREADS)
k_unsketch_pruned(const SparseArgs A) {
    __shared__ SelShared sh;
    constexpr int NEED = (R + 1) / 2;      // big row estimates a survivor must have
    pdl_trigger();
    for (int b = threadIdx.x; b < H1_BINS; b += SEL_THREADS) sh.hist[b] = 0;
    pdl_wait();
    if (A.rerun && __ldcg(&A.sp.state->fallback) != 1u) return;
    if (A.gated && __ldcg(&A.sp.state->use_table) == 0u) return;
    const uint32_t bin_lo = A.rerun ? 0u : A.sp.state->bin_lo;
    __syncthreads();
    const int lane = threadIdx.x & 31;
    constexpr int NC = PRUNED_NC;
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
    if (block_is_last(&A.sp.state->ticket[A.rerun ? 2 : 1], sh)) {
        const uint32_t n = __ldcg(&A.sp.state->n_surv);
        if (!A.rerun && n < A.ncand) {
            // the sampled threshold was too high: empty the list and its histogram for the unpruned pass
            for (int b = threadIdx.x; b < H1_BINS; b += SEL_THREADS) A.sp.h1[b] = 0;
            if (threadIdx.x == 0) { A.sp.state->n_surv = 0; A.sp.state->fallback = 1u; }
        } else {
            uint32_t d1 = 0, rem1 = 1;
            block_find_from_top<H1_BINS>(A.sp.h1, A.ncand, sh, d1, rem1);
            if (threadIdx.x == 0) {
                A.sp.state->d1 = d1; A.sp.state->rem1 = rem1;
                if (A.rerun) A.sp.state->fallback = 2u;
            }
        }
    }
}

#endif  // __CUDACC__
}  // namespace ssgd
