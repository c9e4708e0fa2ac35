// rowbits_unsketch.cuh -- Algorithm 3 line 9, first pass over all d coordinates, for sketches whose one-bit-per-
// bucket filter (filter_unsketch.cuh) does not fit one SM's shared memory as a whole but does fit ROW BY ROW, or a row
// in up to RB_MAX_SLICES slices.
//
// The folded filter of filter_unsketch.cuh ORs neighbouring buckets into one bit until all r rows fit; what passes
// the coarser test has to be re-checked on the full bitmap in global memory, r scattered L2 reads each, and with 4 or
// more buckets per bit most coordinates pass.  Here nothing is folded:
//
//   k_row_bits          a thread block holds ONE row of the full bitmap (c bits <= 192 KiB) in shared memory and
//                       evaluates that row's bit for every coordinate of its range: of each 1024 coordinates a
//                       warp takes, lane l walks the 32 consecutive ones of result word l (one add + conditional
//                       subtract per hash, one shared-memory load, two funnel shifts to append the bit), then
//                       the warp stores its 32 words with one coalesced 128-byte store.  A row longer than shared
//                       memory is cut into slices, one block each: a block sets the bits of the coordinates whose
//                       bucket lies in its slice, into a result row of its own.
//   k_rowbits_combine   reads the r result words of 32 coordinates (coalesced; ORs a row's slices), counts per coordinate how many rows
//                       have their bit set with a bit-sliced adder, and for the few coordinates with at least (r+1)/2
//                       set bits computes the exact estimate from the table (the warp's passing coordinates are
//                       compacted in shared memory first, so that every lane has one) and appends it to the
//                       survivor list iff its own bin is >= bin_lo: one reservation per warp and 1024 coordinates.
//
// The survivor set is exactly { i : bin(|est_i|) >= bin_lo }, as with the other first-pass kernels, and the rest of
// the stage (too-few-survivors rerun, selection on the list) is unchanged.  k_bitmap_build's last block measures the
// bitmap's density; if so many buckets are above the threshold that most coordinates would pass, both kernels return
// at once and the table-reading kernel enqueued behind them does the first pass.
#pragma once
#include <stdint.h>

#include "estimate.cuh"
#include "filter_unsketch.cuh"
#include "hash.cuh"
#include "select.cuh"
#include "sparse_select.cuh"

namespace ssgd {

constexpr int RB_MAX_THREADS = 1024;
constexpr int RB_MAX_SLICES = 4;       // a row in more slices costs more hash evaluations than the folded filter saves
// The row-by-row filter is used if at most this share of the coordinates is expected to pass it (binomial tail of
// the bitmap's density): beyond, exact estimates for nearly everyone cost more than the early-exit table kernel.
// Measured on B200, whole step in ms with this filter / with the table kernel, by density of the bitmap (share
// expected to pass): 5 x 1,000,000 at d = 9e7: 0.28 (0.14) 3.43 / 4.47, 0.35 (0.24) 3.68 / 4.58, 0.46 (0.42)
// 4.14 / 4.70, 0.60 (0.68) 4.98 / 5.38; 5 x 2^20 at d = 2e7: 0.15 2.21 / 2.37, 0.44 2.48 / 2.59; 5 x 2^22 in
// three slices at d = 9e7: 0.08 7.18 / 7.42, 0.25 7.61 / 8.25.
constexpr float ROWBITS_MAX_PASS = 0.7f;

struct RowBitsArgs {
    FilterArgs F;
    uint32_t* rowbits;        // [slices][r][words_per_row]: bit i of row j = "row j's bucket of coordinate i lies in
                              // this slice and is above the threshold"
    int64_t words_per_row;    // ceil(d / 32)
    int32_t ranges;           // blocks per row and slice: block b works on row b % r, slice (b / r) % slices,
                              // coordinate range b / (r * slices)
    int32_t slices;           // pieces a bitmap row is cut into (1: the row fits shared memory)
    int32_t slice_words;      // words per slice (a multiple of 4; the last slice may be shorter)
};

#ifdef __CUDACC__

template <bool POW2, bool SLICED>
__global__ void __launch_bounds__(RB_MAX_THREADS)
k_row_bits(const RowBitsArgs B) {
    extern __shared__ __align__(16) uint32_t rb_bm[];      // row j of the full bitmap (SLICED: words [lo, lo + nw) of it)
    const SparseArgs& A = B.F.A;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthreads = blockDim.x, nwarps = nthreads >> 5;
    pdl_trigger();
    pdl_wait();
    if (__ldcg(&A.sp.state->use_table) != 0u) return;      // too dense to prune: the table kernel behind runs
    const int j = (int)(blockIdx.x % (unsigned)B.F.r);
    const int sl = SLICED ? (int)((blockIdx.x / (unsigned)B.F.r) % (unsigned)B.slices) : 0;
    const int64_t rho = blockIdx.x / ((unsigned)B.F.r * (unsigned)(SLICED ? B.slices : 1));
    const uint32_t lo = (uint32_t)sl * (uint32_t)B.slice_words;
    const uint32_t nw = SLICED ? ((uint32_t)B.F.stride_full - lo < (uint32_t)B.slice_words ? (uint32_t)B.F.stride_full - lo
                                                                                          : (uint32_t)B.slice_words)
                               : (uint32_t)B.F.stride_full;
    {
        const uint4* src = reinterpret_cast<const uint4*>(B.F.bm_full + (int64_t)j * B.F.stride_full + lo);
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(rb_bm);
        for (int w = tid; w < (int)(nw / 4); w += nthreads)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (uint32_t)w * 16u), "l"(src + w) : "memory");
        if (SLICED && tid == 0) rb_bm[nw] = 0u;            // what buckets outside the slice read
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    // chunks of 1024 coordinates; this block's chunks, then this warp's share of them (contiguous: the hash runs on)
    const int64_t nchunks = (A.d + 1023) >> 10;
    const int64_t per_cta = (nchunks + B.ranges - 1) / B.ranges;
    const int64_t c_lo = rho * per_cta, c_hi = c_lo + per_cta < nchunks ? c_lo + per_cta : nchunks;
    if (c_lo >= c_hi) return;
    const int64_t per_warp = (c_hi - c_lo + nwarps - 1) / nwarps;
    const int64_t w_lo = c_lo + warp * per_warp, w_hi = w_lo + per_warp < c_hi ? w_lo + per_warp : c_hi;
    if (w_lo >= w_hi) return;
    // lane l owns the 32 consecutive coordinates s .. s + 31 of each chunk, i.e. one result word: the hash advances
    // by one add and a conditional subtract per coordinate, the bit is shifted into the word from the top
    const HashRow hr = A.hp.row[j];
    uint32_t s = (uint32_t)(w_lo << 10) + (uint32_t)lane * 32u;
    uint32_t y = lin_hash(hr.a, hr.b, s);
    const uint32_t skip = mod_p31((uint64_t)hr.a * 992ull);   // from s + 32 to the lane's word of the next chunk
    const uint32_t d32 = (uint32_t)A.d;
    uint32_t* out = B.rowbits + ((int64_t)sl * B.F.r + j) * B.words_per_row;
    for (int64_t chunk = w_lo; chunk < w_hi; ++chunk) {
        uint32_t word = 0;
#pragma unroll
        for (int t = 0; t < 32; ++t) {
            const uint32_t b = bucket_of<POW2>(y, A.bk);
            uint32_t bits;                                                   // bucket b's bit lowest (shift taken mod 32)
            if (SLICED) {
                const uint32_t wi = (b >> 5) - lo;                           // wraps to a large value below the slice
                bits = __funnelshift_r(rb_bm[wi < nw ? wi : nw], 0u, b);     // word nw is zero: no branch, a broadcast read
            } else {
                bits = __funnelshift_r(rb_bm[b >> 5], 0u, b);
            }
            word = __funnelshift_r(word, bits, 1);                           // word >> 1 | lowest bit of `bits` << 31
            y = next_hash(y, hr.a);
        }
        y = next_hash(y, skip);
        const uint32_t valid = d32 > s ? d32 - s : 0u;       // coordinates of this word below d
        if (valid < 32u) word &= (1u << valid) - 1u;
        const int64_t widx = (chunk << 5) + lane;
        if (widx < B.words_per_row) out[widx] = word;
        s += 1024u;
    }
}

// Per warp: the passing coordinates of 1024 (at most all of them) and the estimates of those that are kept.
constexpr int RBC_QUEUE = 1024;
constexpr size_t RBC_SMEM = (size_t)SEL_WARPS * RBC_QUEUE * 2 * 4;

template <int R, bool POW2>
__global__ void __launch_bounds__(SEL_THREADS)
k_rowbits_combine(const RowBitsArgs B) {
    extern __shared__ __align__(16) uint32_t rbc_smem[];
    __shared__ SelShared sh;
    constexpr int NEED = (R + 1) / 2;
    const SparseArgs& A = B.F.A;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* q = rbc_smem + (size_t)warp * (RBC_QUEUE * 2);          // coordinates: passing ones, then (in place) kept ones
    float* e = reinterpret_cast<float*>(q + RBC_QUEUE);                 // estimates of the kept ones
    pdl_trigger();
    for (int b = threadIdx.x; b < H1_BINS; b += SEL_THREADS) sh.hist[b] = 0;
    pdl_wait();
    if (__ldcg(&A.sp.state->use_table) != 0u) return;
    const uint32_t bin_lo = __ldcg(&A.sp.state->bin_lo);
    __syncthreads();
    const int64_t stride = (int64_t)gridDim.x * SEL_THREADS;
    // warp-uniform trip count: the queue is the warp's
    for (int64_t w0 = (int64_t)blockIdx.x * SEL_THREADS + (threadIdx.x & ~31); w0 < B.words_per_row; w0 += stride) {
        const int64_t w = w0 + lane;
        // bit-sliced count (4 planes: r <= 15) of the rows whose bit is set, for 32 coordinates at once
        uint32_t c0 = 0, c1 = 0, c2 = 0, c3 = 0;
        uint32_t rows[R];
#pragma unroll
        for (int j = 0; j < R; ++j) rows[j] = 0u;
        if (w < B.words_per_row) {
            for (int sl = 0; sl < B.slices; ++sl) {
#pragma unroll
                for (int j = 0; j < R; ++j) rows[j] |= __ldcs(B.rowbits + ((int64_t)sl * R + j) * B.words_per_row + w);
            }
        }
#pragma unroll
        for (int j = 0; j < R; ++j) {
            uint32_t carry = rows[j], t;
            t = c0 & carry; c0 ^= carry; carry = t;
            t = c1 & carry; c1 ^= carry; carry = t;
            t = c2 & carry; c2 ^= carry; carry = t;
            c3 ^= carry;
        }
        // pass = (count >= NEED), compared plane by plane from the top
        const uint32_t plane[4] = {c0, c1, c2, c3};
        uint32_t gt = 0u, eq = 0xFFFFFFFFu;
#pragma unroll
        for (int p = 3; p >= 0; --p) {
            if ((NEED >> p) & 1) { eq &= plane[p]; }
            else { gt |= eq & plane[p]; eq &= ~plane[p]; }
        }
        uint32_t pass = gt | eq;
        // the warp's passing coordinates, compacted: every lane then computes one exact estimate per round
        const uint32_t mine = (uint32_t)__popc(pass);
        uint32_t incl = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += up;
        }
        const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 31);
        if (total == 0u) continue;
        uint32_t at = incl - mine;
        while (pass) {
            const int bit = __ffs(pass) - 1;
            pass &= pass - 1u;
            q[at++] = (uint32_t)(w << 5) + (uint32_t)bit;
        }
        __syncwarp();
        uint32_t nk = 0;                                     // kept so far (<= coordinates read so far: in place)
        for (uint32_t t0 = 0; t0 < total; t0 += 32u) {
            const bool have = t0 + (uint32_t)lane < total;
            const uint32_t i = have ? q[t0 + lane] : 0u;
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
            const uint32_t bal = __ballot_sync(0xFFFFFFFFu, keep);
            __syncwarp();
            if (keep) {
                const uint32_t pos = nk + (uint32_t)__popc(bal & ((1u << lane) - 1u));
                q[pos] = i;
                e[pos] = m;
                atomicAdd(&sh.hist[key_of(m) >> H1_SHIFT], 1u);
            }
            nk += (uint32_t)__popc(bal);
        }
        __syncwarp();
        if (nk) {                                            // one reservation and coalesced stores per 1024 coordinates
            uint32_t base = 0;
            if (lane == 0) base = atomicAdd(&A.sp.state->n_surv, nk);
            base = __shfl_sync(0xFFFFFFFFu, base, 0);
            for (uint32_t t = (uint32_t)lane; t < nk; t += 32u) {
                const uint32_t pos = base + t;
                if (pos < A.sp.cap) { A.sp.list_idx[pos] = (int32_t)q[t]; A.sp.list_est[pos] = e[t]; }
            }
        }
        __syncwarp();
    }
    __syncthreads();
    flush_hist<H1_BINS>(sh.hist, A.sp.h1);
    if (block_is_last(&A.sp.state->ticket[1], sh)) {
        const uint32_t n = __ldcg(&A.sp.state->n_surv);
        if (n < A.ncand) {
            // the sampled threshold was too high: empty the list and its histogram for the unpruned pass
            for (int b = threadIdx.x; b < H1_BINS; b += SEL_THREADS) A.sp.h1[b] = 0;
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
