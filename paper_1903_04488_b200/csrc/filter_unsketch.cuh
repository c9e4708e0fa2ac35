// filter_unsketch.cuh -- Algorithm 3 line 9, first pass over all d coordinates, with the sketch table replaced
// by one bit per bucket held in shared memory.
//
// The early-exit unsketch of sparse_select.cuh still pays three or more scattered reads of the L2-resident table
// per coordinate, and the load/store unit's rate for such reads (about one 32-byte sector per clock per SM) is
// what bounds it.  The test it applies to each value read, "is |table[j][h_j(i)]| in a histogram bin >= bin_lo",
// depends on the bucket alone, so it can be evaluated once per bucket instead of once per (coordinate, row):
//
//   k_bitmap_build     bit (j, b) = 1 iff the magnitude of table[j][b] lies in a bin >= bin_lo   (r*c bits)
//   k_bitmap_fold      if r*c bits exceed the shared memory of an SM: OR 2^s neighbouring buckets into one bit,
//                      s <= 5 (a coarser, still necessary, condition; the full bitmap stays in global memory)
//   k_unsketch_filter  one block per SM copies the (folded) bitmap into shared memory; every thread walks a run of
//                      consecutive coordinates (one add + conditional subtract per row hash) and counts, per
//                      coordinate, the rows whose bit is set.  |median of r| >= t needs (r+1)/2 rows of magnitude
//                      >= t, so a coordinate with fewer set bits is certainly below the threshold and is dropped
//                      without a single read of global memory.  The few that pass (2 % at C2's shape) are queued
//                      per warp in shared memory and processed 32 at a time: folded bitmaps are re-checked against
//                      the full bitmap first (second queue), then the exact estimate is computed from the table
//                      and the coordinate is appended to the survivor list iff its own bin is >= bin_lo.
//
// The survivor set is therefore exactly { i : bin(|est_i|) >= bin_lo }, as with the early-exit kernel, and the rest
// of the stage (too-few-survivors rerun, selection on the list) is unchanged.
#pragma once
#include <stdint.h>

#include "estimate.cuh"
#include "hash.cuh"
#include "select.cuh"
#include "sparse_select.cuh"

namespace ssgd {

// Measured on B200 (C2; sample + bitmap + filter + the skipped rerun launch): 256 threads x 4 coordinates per
// iteration 0.092 ms; 512 x 1, 2, 4: 0.073, 0.071, 0.073; 1024 x 1, 2: 0.070, 0.067.  With a folded bitmap the
// kernel needs more than the 64 registers that 1024 threads leave it (d = 2e7, c = 2^20: 0.41 ms against 0.26 ms).
constexpr int FILTER_THREADS = 512;
constexpr int FILTER_NC = 2;                             // coordinates per loop iteration (independent lookups)
constexpr int FILTER_WARPS = FILTER_THREADS / 32;
constexpr int FILTER_QUEUE = 64;                         // entries per warp queue (at most 31 + 32 are ever held)
constexpr int FILTER_MAX_WORDS = 49152;                  // 192 KiB of bitmap per SM (+ 16 KiB of queues + 16 KiB histogram)
constexpr int FILTER_MAX_FOLD = 5;                       // a folded bit covers at most one word of the full bitmap
// Shared memory of the filter kernel besides its static SelShared: the bitmap, then two queues per warp.
constexpr size_t FILTER_QUEUE_BYTES = (size_t)FILTER_WARPS * 2 * (2 * FILTER_QUEUE) * 4;   // (value, tag) entries

struct FilterArgs {
    SparseArgs A;
    uint32_t* bm_full;        // [r][stride_full] words: bit b of row j at word b >> 5, bit b & 31
    uint32_t* bm_fold;        // [r][stride_fold] words (unused when fold == 0)
    int32_t stride_full;      // words per row, a multiple of 4
    int32_t stride_fold;      // words per row of the folded bitmap, a multiple of 4
    int32_t fold;             // s: a folded bit covers buckets [q << s, (q + 1) << s)
    int32_t r;
    // 1: the bitmap is used unfolded, row by row (rowbits_unsketch.cuh); k_bitmap_build then counts the set bits and
    // its last block decides between that filter and the table kernel (k_bitmap_fold does it for folded bitmaps)
    int32_t decide_in_build;
    float max_pass;           // decide_in_build: largest expected share of passing coordinates the filter is used for
};

#ifdef __CUDACC__

// Probability that at least `need` of r independent bits of density p are set.
__device__ __forceinline__ float binomial_tail(int r, int need, float p) {
    float tail = 0.f;
    for (int k = need; k <= r; ++k) {
        float term = 1.f;                                  // C(r, k) p^k (1-p)^(r-k)
        for (int t = 0; t < k; ++t) term *= p * (float)(r - t) / (float)(k - t);
        for (int t = 0; t < r - k; ++t) term *= 1.f - p;
        tail += term;
    }
    return tail;
}

// ---- bit per bucket ------------------------------------------------------------------------------------------
// One warp per 32 words (1024 buckets) of one row: 32 coalesced loads, a ballot each; lane k keeps ballot k.
static __global__ void __launch_bounds__(SEL_THREADS)
k_bitmap_build(const FilterArgs F) {
    __shared__ uint32_t s_last;
    pdl_trigger();
    pdl_wait();
    uint32_t ones = 0;
    const uint32_t bin_lo = __ldcg(&F.A.sp.state->bin_lo);
    const int lane = threadIdx.x & 31;
    const int64_t tasks_per_row = (F.stride_full + 31) / 32;
    const int64_t tasks = tasks_per_row * F.r;
    const int64_t nwarps = (int64_t)gridDim.x * SEL_WARPS;
    for (int64_t task = (int64_t)blockIdx.x * SEL_WARPS + (threadIdx.x >> 5); task < tasks; task += nwarps) {
        const int64_t j = task / tasks_per_row;
        const int64_t w0 = (task - j * tasks_per_row) * 32;          // first word of this task in row j
        const float* row = F.A.table + j * F.A.c;
        uint32_t mine = 0;
        uint32_t key[32];                                    // all 32 loads in flight: one L2 round trip per task
#pragma unroll
        for (int k = 0; k < 32; ++k) {
            const int64_t b = (w0 + k) * 32 + lane;
            key[k] = b < F.A.c ? key_of(__ldcg(row + b)) : 0xFFFFFFFFu;
        }
#pragma unroll
        for (int k = 0; k < 32; ++k) {
            const bool big = key[k] != 0xFFFFFFFFu && (key[k] >> H1_SHIFT) >= bin_lo;
            const uint32_t bal = __ballot_sync(0xFFFFFFFFu, big);
            if (lane == k) mine = bal;
        }
        if (w0 + lane < F.stride_full) F.bm_full[j * F.stride_full + w0 + lane] = mine;
        ones += __popc(mine);
    }
    if (F.decide_in_build) {                               // density of the unfolded bitmap -> filter or table kernel
        for (int off = 16; off; off >>= 1) ones += __shfl_xor_sync(0xFFFFFFFFu, ones, off);
        if (lane == 0 && ones) atomicAdd(&F.A.sp.state->fold_ones, ones);
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) s_last = atomicAdd(&F.A.sp.state->ticket[5], 1u) == gridDim.x - 1 ? 1u : 0u;
        __syncthreads();
        if (s_last && threadIdx.x == 0) {
            const float p = fminf(1.f, (float)__ldcg(&F.A.sp.state->fold_ones) / ((float)F.r * (float)F.A.c));
            F.A.sp.state->use_table = binomial_tail(F.r, (F.r + 1) / 2, p) > F.max_pass ? 1u : 0u;
        }
    }
}

// A folded bitmap is used only if it passes at most this share of the coordinates (estimated from its density as
// a binomial tail); otherwise the first pass reads the table.  Measured on B200, r = 5, whole step in ms with the
// filter / with the table kernel, by estimated share: 0.63 (d = 2e7, c = 2^20, 4 buckets per bit) 2.70 / 2.84;
// 0.77 (same, ncand doubled) 2.79 / 2.89; 0.88 (d = 9e7, c = 1e6, 4 per bit) 4.82 / 4.91; 0.90 (d = 9e7, c = 2^22,
// 16 per bit, ncand = 5e4) 7.49 / 7.85; 0.96 (d = 2e7, c = 2^20, ncand = 1.6e6) 2.65 / 2.60; 0.99 (d = 9e7, c = 2^22,
// ncand = 2e5) 7.97 / 7.99; r = 15, 0.95 (d = 9e7, c = 180,000, 2 per bit) 16.7 / 12.5.
constexpr float FILTER_MAX_PASS = 0.93f;

// One thread per folded word: 32 folded bits, each the OR of 2^s consecutive bits of the full bitmap.  The last
// block to finish turns the density of the folded bitmap into the decision between the two first-pass kernels.
static __global__ void __launch_bounds__(SEL_THREADS)
k_bitmap_fold(const FilterArgs F) {
    __shared__ uint32_t s_last;
    pdl_trigger();
    pdl_wait();
    const int s = F.fold;
    const int64_t total = (int64_t)F.r * F.stride_fold;
    const uint32_t group = s >= 5 ? 0xFFFFFFFFu : ((1u << (1 << s)) - 1u);
    uint32_t ones = 0;
    for (int64_t t = (int64_t)blockIdx.x * SEL_THREADS + threadIdx.x; t < total; t += (int64_t)gridDim.x * SEL_THREADS) {
        const int64_t j = t / F.stride_fold;
        const int64_t fw = t - j * F.stride_fold;
        const uint32_t* src = F.bm_full + j * F.stride_full;
        uint32_t out = 0;
        for (int q = 0; q < 32; ++q) {
            const int64_t w = (fw << s) + (q >> (5 - s));            // word of the full row holding this group
            const int off = (q << s) & 31;
            const uint32_t word = w < F.stride_full ? __ldcg(src + w) : 0u;
            out |= (((word >> off) & group) != 0u ? 1u : 0u) << q;
        }
        F.bm_fold[t] = out;
        ones += __popc(out);
    }
    for (int off = 16; off; off >>= 1) ones += __shfl_xor_sync(0xFFFFFFFFu, ones, off);
    if ((threadIdx.x & 31) == 0 && ones) atomicAdd(&F.A.sp.state->fold_ones, ones);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(&F.A.sp.state->ticket[5], 1u) == gridDim.x - 1 ? 1u : 0u;
    __syncthreads();
    if (s_last && threadIdx.x == 0) {
        const float bits = (float)F.r * (float)((F.A.c + (1 << s) - 1) >> s);
        const float p = fminf(1.f, (float)__ldcg(&F.A.sp.state->fold_ones) / bits);
        F.A.sp.state->use_table = binomial_tail(F.r, (F.r + 1) / 2, p) > FILTER_MAX_PASS ? 1u : 0u;
    }
}

// ---- the filter pass ---------------------------------------------------------------------------------------------
struct WarpQueue {
    uint32_t* buf;     // FILTER_QUEUE entries of this warp in shared memory, then FILTER_QUEUE tags
    int count;         // warp-uniform
    // every lane calls; lanes with `take` append (value, tag)
    __device__ __forceinline__ void push(bool take, uint32_t value, uint32_t tag, int lane) {
        const uint32_t bal = __ballot_sync(0xFFFFFFFFu, take);
        if (bal == 0u) return;
        if (take) {
            const int pos = count + __popc(bal & ((1u << lane) - 1u));
            buf[pos] = value;
            buf[FILTER_QUEUE + pos] = tag;
        }
        count += __popc(bal);
        __syncwarp();
    }
    // every lane calls; removes up to 32 entries from the top; returns whether this lane got one
    __device__ __forceinline__ bool pop(uint32_t& value, uint32_t& tag, int lane) {
        const int n = count < 32 ? count : 32;
        const bool got = lane < n;
        if (got) { value = buf[count - n + lane]; tag = buf[FILTER_QUEUE + count - n + lane]; }
        count -= n;
        __syncwarp();
        return got;
    }
};

template <int R, bool POW2, bool FOLD>
__global__ void __launch_bounds__(FILTER_THREADS, 1)
k_unsketch_filter(const FilterArgs F) {
    __shared__ SelShared sh;
    extern __shared__ __align__(16) uint32_t dyn[];
    constexpr int NEED = (R + 1) / 2;
    const SparseArgs& A = F.A;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int fold = FOLD ? F.fold : 0;                  // FOLD == (F.fold != 0)
    const int stride_s = fold ? F.stride_fold : F.stride_full;
    const int nw = R * stride_s;
    uint32_t* bm = dyn;
    WarpQueue q2{dyn + nw + (warp * 2 + 0) * (2 * FILTER_QUEUE), 0};
    WarpQueue q3{dyn + nw + (warp * 2 + 1) * (2 * FILTER_QUEUE), 0};
    pdl_trigger();
    for (int b = threadIdx.x; b < H1_BINS; b += FILTER_THREADS) sh.hist[b] = 0;
    pdl_wait();
    if (FOLD && __ldcg(&A.sp.state->use_table) != 0u) return;   // too dense to prune: the table kernel behind runs
    const uint32_t bin_lo = __ldcg(&A.sp.state->bin_lo);
    {
        // asynchronous 16-byte copies, all in flight at once: the fill costs one L2 round trip, not one per piece
        // (measured at C2: five 32 KiB bulk copies issued by one thread and awaited on an mbarrier take 2.5 us longer)
        const uint4* src = reinterpret_cast<const uint4*>(fold ? F.bm_fold : F.bm_full);
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(bm);
        for (int w = threadIdx.x; w < nw / 4; w += FILTER_THREADS)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (uint32_t)w * 16u), "l"(src + w) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();

    // unfolded bitmaps (q3 is free): kept coordinates wait in q3 and go to the list 32 at a time, one reservation
    // and two coalesced stores each -- reservations all hit one counter, and one per batch with a kept coordinate
    // in it is what bounds the kernel when many pass (measured at 5 x 180,000, d = 7.3e7)
    auto flush_kept = [&](int at_least) {
        while (q3.count >= at_least) {
            const int n = q3.count < 32 ? q3.count : 32;
            uint32_t c = 0, mbits = 0;
            const bool got = q3.pop(c, mbits, lane);
            uint32_t base = 0;
            if (lane == 0) base = atomicAdd(&A.sp.state->n_surv, (uint32_t)n);
            base = __shfl_sync(0xFFFFFFFFu, base, 0);
            const uint32_t pos = base + (uint32_t)lane;
            if (got && pos < A.sp.cap) { A.sp.list_idx[pos] = (int32_t)c; A.sp.list_est[pos] = __uint_as_float(mbits); }
        }
    };
    // exact estimate of one queued coordinate; append to the list iff its bin is >= bin_lo
    auto exact = [&](uint32_t i, bool have) {
        float m = 0.f;
        bool keep = false;
        if (have) {
            float rowv[R];
#pragma unroll
            for (int j = 0; j < R; ++j) {
                uint32_t hb[1];
                row_hashes<POW2, 1>(A.hp.row[j], A.bk, i, hb);
                rowv[j] = apply_sign(table_load(A.table + (int64_t)j * A.c + (hb[0] & P31)), hb[0]);
            }
            m = median_of<R>(rowv);
            keep = (key_of(m) >> H1_SHIFT) >= bin_lo;
        }
        if (keep) atomicAdd(&sh.hist[key_of(m) >> H1_SHIFT], 1u);
        if (!FOLD) {
            q3.push(keep, i, __float_as_uint(m), lane);
            flush_kept(32);
            return;
        }
        const uint32_t bal = __ballot_sync(0xFFFFFFFFu, keep);
        if (bal == 0u) return;
        uint32_t base = 0;
        if (lane == 0) base = atomicAdd(&A.sp.state->n_surv, (uint32_t)__popc(bal));
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        if (keep) {
            const uint32_t pos = base + __popc(bal & ((1u << lane) - 1u));
            if (pos < A.sp.cap) { A.sp.list_idx[pos] = (int32_t)i; A.sp.list_est[pos] = m; }
        }
    };
    // folded bitmaps only: the rows whose folded bit was set (`rows`) are looked up in the full bitmap (global
    // memory, L2-resident); the other rows are known to be below the threshold
    auto recheck = [&](uint32_t i, uint32_t rows, bool have) {
        bool pass = false;
        if (have) {
            uint32_t word[R], b[R];
#pragma unroll
            for (int j = 0; j < R; ++j) {                // all loads issued before any is used
                b[j] = bucket_of<POW2>(lin_hash(A.hp.row[j].a, A.hp.row[j].b, i), A.bk);
                word[j] = 0u;
                if ((rows >> j) & 1u) word[j] = __ldg(F.bm_full + (int64_t)j * F.stride_full + (b[j] >> 5));
            }
            int cnt = 0;
#pragma unroll
            for (int j = 0; j < R; ++j) cnt += (int)(__funnelshift_r(word[j], 0u, b[j]) & 1u);
            pass = cnt >= NEED;
        }
        q3.push(pass, i, 0u, lane);
        if (q3.count >= 32) { uint32_t c = 0, tag = 0; const bool got = q3.pop(c, tag, lane); exact(c, got); }
    };
    auto drain2 = [&]() {
        uint32_t c = 0, rows = 0;
        const bool got = q2.pop(c, rows, lane);
        if (FOLD) recheck(c, rows, got); else exact(c, got);
    };

    // this thread's run of consecutive coordinates, 32 at a time: row j's bits of the 32 are shifted into one word
    // (two funnel shifts per lookup), the rows are counted with a bit-sliced adder, and only the coordinates with
    // at least NEED set bits are looked at one by one
    const uint32_t total_threads = gridDim.x * FILTER_THREADS;
    constexpr uint32_t NC = FILTER_NC;
    const uint32_t per = (uint32_t)((A.d + total_threads - 1) / total_threads + NC - 1) / NC * NC;
    const uint32_t gtid = blockIdx.x * FILTER_THREADS + threadIdx.x;
    const uint64_t begin64 = (uint64_t)gtid * per;
    const uint32_t i_begin = begin64 < (uint64_t)A.d ? (uint32_t)begin64 : (uint32_t)A.d;
    const uint32_t i_end = begin64 + per < (uint64_t)A.d ? (uint32_t)(begin64 + per) : (uint32_t)A.d;
    uint32_t y[R];
    const uint32_t* row_base[R];
#pragma unroll
    for (int j = 0; j < R; ++j) { y[j] = lin_hash(A.hp.row[j].a, A.hp.row[j].b, i_begin); row_base[j] = bm + j * stride_s; }
    for (uint32_t t0 = 0; t0 < per; t0 += 32u) {         // warp-uniform trip counts, here and below
        const uint32_t n_this = per - t0 < 32u ? per - t0 : 32u;     // a multiple of NC
        uint32_t w[R];                                   // bit e of w[j]: row j's bit of coordinate i_begin + t0 + e
#pragma unroll
        for (int j = 0; j < R; ++j) w[j] = 0u;
        for (uint32_t t = 0; t < n_this; t += NC) {
#pragma unroll
            for (uint32_t e = 0; e < NC; ++e) {
#pragma unroll
                for (int j = 0; j < R; ++j) {
                    const uint32_t b = bucket_of<POW2>(y[j], A.bk) >> fold;
                    const uint32_t bits = __funnelshift_r(row_base[j][b >> 5], 0u, b);   // shift amount taken mod 32
                    w[j] = __funnelshift_r(w[j], bits, 1);                               // lowest bit of `bits` enters at the top
                    y[j] = next_hash(y[j], A.hp.row[j].a);
                }
            }
        }
        if (n_this < 32u) {
#pragma unroll
            for (int j = 0; j < R; ++j) w[j] >>= 32u - n_this;
        }
        // bit-sliced count (4 planes: r <= 15) of the rows whose bit is set; pass = count >= NEED
        uint32_t c0 = 0, c1 = 0, c2 = 0, c3 = 0;
#pragma unroll
        for (int j = 0; j < R; ++j) {
            uint32_t carry = w[j], x;
            x = c0 & carry; c0 ^= carry; carry = x;
            x = c1 & carry; c1 ^= carry; carry = x;
            x = c2 & carry; c2 ^= carry; carry = x;
            c3 ^= carry;
        }
        const uint32_t plane[4] = {c0, c1, c2, c3};
        uint32_t gt = 0u, eq = 0xFFFFFFFFu;
#pragma unroll
        for (int p = 3; p >= 0; --p) {
            if ((NEED >> p) & 1) { eq &= plane[p]; }
            else { gt |= eq & plane[p]; eq &= ~plane[p]; }
        }
        const uint32_t first = i_begin + t0;
        const uint32_t nvalid = i_end > first ? (i_end - first < 32u ? i_end - first : 32u) : 0u;
        uint32_t pass = (gt | eq) & (nvalid >= 32u ? 0xFFFFFFFFu : (1u << nvalid) - 1u);
        while (__any_sync(0xFFFFFFFFu, pass != 0u)) {
            const bool have = pass != 0u;
            const int bit = have ? __ffs(pass) - 1 : 0;
            pass &= pass - 1u;                           // (0 stays 0)
            uint32_t rows = 0u;                          // folded bitmaps: which rows had their folded bit set
            if (FOLD) {
#pragma unroll
                for (int j = 0; j < R; ++j) rows |= ((w[j] >> bit) & 1u) << j;
            }
            q2.push(have, first + (uint32_t)bit, rows, lane);
            if (q2.count >= 32) drain2();
        }
    }
    if (q2.count > 0) drain2();
    if (FOLD && q3.count > 0) { uint32_t c = 0, tag = 0; const bool got = q3.pop(c, tag, lane); exact(c, got); }
    if (!FOLD) flush_kept(1);

    __syncthreads();
    flush_hist<H1_BINS>(sh.hist, A.sp.h1);
    if (block_is_last(&A.sp.state->ticket[1], sh)) {
        const uint32_t n = __ldcg(&A.sp.state->n_surv);
        if (n < A.ncand) {
            // the sampled threshold was too high: empty the list and its histogram for the unpruned pass
            for (int b = threadIdx.x; b < H1_BINS; b += FILTER_THREADS) A.sp.h1[b] = 0;
            if (threadIdx.x == 0) { A.sp.state->n_surv = 0; A.sp.state->fallback = 1u; }
        } else {
            uint32_t d1 = 0, rem1 = 1;
            block_find_from_top<H1_BINS>(A.sp.h1, A.ncand, sh, d1, rem1);
            if (threadIdx.x == 0) { A.sp.state->d1 = d1; A.sp.state->rem1 = rem1; }
        }
    }
}

#endif  // __CUDACC__
}  // namespace ssgd
