// select.cuh -- exact top-m selection by magnitude (Algorithm 3 lines 9 and 11).
//
// Items are positions 0..n-1 of an fp32 array; the key of an item is the bit pattern of |value|
// (31 bits, monotone in the magnitude, -0 == +0).  The m selected items are the first m under the
// total order "larger key first, then smaller position first".  The method is a most-significant-
// digit radix select on 12 + 11 + 8 key bits:
//
//   producer kernel   histogram H1 of key bits 30..19          (fused into the kernel that makes the values)
//   k_sel_pass2       histogram H2 of bits 18..8 among items whose top digit is the threshold digit
//   k_sel_pass3       histogram H3 of bits 7..0 among items matching the 23-bit threshold prefix
//   k_sel_count       threshold key T and tie quota Q are now known: per-chunk counts of key > T, key == T;
//                     its last block turns the counts into exclusive offsets
//   emit kernel       item i is selected iff key > T or (key == T and #equal before i < Q); its output
//                     slot is #greater before i + min(#equal before i, Q): outputs come out in position
//                     order, with no atomics and no dependence on scheduling.
//
// Each histogram is turned into its threshold digit by the LAST block of the kernel that filled it
// (a fence + ticket counter tells a block that it is the last one to finish; nobody waits), so no
// single-block "find threshold" launch sits between the passes.
#pragma once
#include <stdint.h>

namespace ssgd {

constexpr int SEL_THREADS = 256;
constexpr int SEL_WARPS = SEL_THREADS / 32;
constexpr int SEL_ITEMS = 16;                          // items per thread in count/emit
constexpr int SEL_CHUNK = SEL_THREADS * SEL_ITEMS;     // 4096 items per chunk (one block)
constexpr int H1_BITS = 12, H2_BITS = 11, H3_BITS = 8;
constexpr int H1_BINS = 1 << H1_BITS, H2_BINS = 1 << H2_BITS, H3_BINS = 1 << H3_BITS;
constexpr int H1_SHIFT = 31 - H1_BITS;                 // 19
constexpr int H2_SHIFT = H1_SHIFT - H2_BITS;           // 8
constexpr int SEL_HIST_WORDS = H1_BINS + H2_BINS + H3_BINS;
constexpr int H19_BITS = H2_BITS + H3_BITS;            // 19: the key bits below the first digit
constexpr int H19_BINS = 1 << H19_BITS;
constexpr int SEL_ITEMS_SMALL = 4;                     // items per thread in count/emit of short inputs (more blocks)
constexpr int SEL_CHUNK_SMALL = SEL_THREADS * SEL_ITEMS_SMALL;

// Per-selection state, zeroed before the producer runs.
struct SelState {
    uint32_t d1, rem1;   // threshold digit of H1 and how many items are still wanted inside it
    uint32_t d2, rem2;   // same for H2
    uint32_t thr_key;    // T: the full 31-bit threshold key
    uint32_t quota_eq;   // Q >= 1: how many items with key == T are selected
    uint32_t ticket[4];  // finished-block counters of the three histogram kernels and of the count kernel
    uint32_t pad[6];
};

struct SelBuffers {
    uint32_t* h1;        // [H1_BINS]   zeroed before the producer runs
    uint32_t* h2;        // [H2_BINS]   zeroed
    uint32_t* h3;        // [H3_BINS]   zeroed
    SelState* state;
    uint32_t* chunk_gt;  // [nchunks] counts, then exclusive offsets
    uint32_t* chunk_eq;  // [nchunks]
    uint32_t* h19;       // [H19_BINS] zeroed, or NULL: with it, k_sel_pass23 replaces k_sel_pass2 + k_sel_pass3
    // optional gate: if not NULL, the selection's kernels do nothing unless *gate > gate_above (a selection that is
    // enqueued unconditionally but needed only in a case the device decides)
    const uint32_t* gate;
    uint32_t gate_above;
};

#ifdef __CUDACC__

__device__ __forceinline__ uint32_t key_of(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }
__device__ __forceinline__ bool sel_gated_off(const SelBuffers& sb) { return sb.gate && __ldcg(sb.gate) <= sb.gate_above; }

// Histogram passes load SEL_BATCH items per thread before touching shared memory, so that a pass costs a few
// L2 round trips instead of one per item (the shared-memory atomics keep the compiler from hoisting loads).
constexpr int SEL_BATCH = 8;
constexpr uint32_t NO_ITEM = 0xFFFFFFFFu;                  // keys have bit 31 clear
__device__ __forceinline__ void load_keys(const float* __restrict__ val, int64_t n, int64_t i0, int64_t step,
                                          uint32_t (&keys)[SEL_BATCH]) {
#pragma unroll
    for (int u = 0; u < SEL_BATCH; ++u) {
        const int64_t i = i0 + u * step;
        keys[u] = i < n ? key_of(val[i]) : NO_ITEM;
    }
}


struct SelShared {
    uint32_t hist[H1_BINS];
    uint32_t warp_sum[SEL_WARPS];
    uint32_t found[2];
    uint32_t last;
};

// True, in every thread of the block, iff this block is the last of the grid to get here.  Everything
// the other blocks wrote to global memory before their own call is then visible to this block.
__device__ __forceinline__ bool block_is_last(uint32_t* ticket, SelShared& sh) {
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) sh.last = (atomicAdd(ticket, 1u) == gridDim.x - 1) ? 1u : 0u;
    __syncthreads();
    return sh.last != 0;
}

// Largest digit D with count(bins > D) < want <= count(bins >= D); rem = want - count(bins > D).
// The whole block must call (SEL_THREADS threads or more; the first SEL_THREADS do the search).
// Requires 1 <= want <= total count.
template <int NBINS>
__device__ __forceinline__ void block_find_from_top(const uint32_t* __restrict__ gh, uint32_t want,
                                                    SelShared& sh, uint32_t& digit, uint32_t& rem) {
    constexpr int PER = NBINS / SEL_THREADS;  // 16, 8, 1
    static_assert(PER >= 1 && PER * SEL_THREADS == NBINS, "bins must be a multiple of the block");
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const bool searcher = t < SEL_THREADS;    // warp-uniform
    for (int b = t; b < NBINS; b += blockDim.x) sh.hist[b] = __ldcg(gh + b);  // L2: other blocks' atomics
    if (t == 0) { sh.found[0] = 0; sh.found[1] = 1; }
    __syncthreads();
    uint32_t sum = 0, incl = 0;
    if (searcher) {
#pragma unroll
        for (int s = 0; s < PER; ++s) sum += sh.hist[t * PER + ((s + t) % PER)];  // rotated: no bank conflicts
        incl = sum;  // sum over lanes >= lane of this warp
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t o = __shfl_down_sync(0xFFFFFFFFu, incl, off);
            if (lane + off < 32) incl += o;
        }
        if (lane == 0) sh.warp_sum[warp] = incl;
    }
    __syncthreads();
    if (searcher) {
        uint32_t above = incl - sum;
        for (int w2 = warp + 1; w2 < SEL_WARPS; ++w2) above += sh.warp_sum[w2];
        if (above < want && want <= above + sum) {
            uint32_t acc = above;
            for (int b = t * PER + PER - 1; b >= t * PER; --b) {
                const uint32_t h = sh.hist[b];
                if (acc + h >= want) { sh.found[0] = (uint32_t)b; sh.found[1] = want - acc; break; }
                acc += h;
            }
        }
    }
    __syncthreads();
    digit = sh.found[0];
    rem = sh.found[1];
    __syncthreads();  // sh.hist may be reused by the caller
}

// Adds a block-private histogram (shared memory) into the global one, skipping empty bins.
template <int NBINS>
__device__ __forceinline__ void flush_hist(const uint32_t* s_hist, uint32_t* __restrict__ gh) {
    for (int b = threadIdx.x; b < NBINS; b += blockDim.x) {
        const uint32_t h = s_hist[b];
        if (h) atomicAdd(&gh[b], h);
    }
}

// ---- pass 2: H2 over items whose top digit equals the threshold digit -----------------------------
static __global__ void __launch_bounds__(SEL_THREADS)
k_sel_pass2(const float* __restrict__ val, int64_t n, SelBuffers sb) {
    __shared__ SelShared sh;
    pdl_trigger();
    for (int b = threadIdx.x; b < H2_BINS; b += SEL_THREADS) sh.hist[b] = 0;
    pdl_wait();
    const uint32_t d1 = sb.state->d1;
    __syncthreads();
    const int64_t stride = (int64_t)gridDim.x * SEL_THREADS;
    for (int64_t i0 = (int64_t)blockIdx.x * SEL_THREADS + threadIdx.x; i0 < n; i0 += stride * SEL_BATCH) {
        uint32_t keys[SEL_BATCH];
        load_keys(val, n, i0, stride, keys);
#pragma unroll
        for (int u = 0; u < SEL_BATCH; ++u)
            if (keys[u] != NO_ITEM && (keys[u] >> H1_SHIFT) == d1) atomicAdd(&sh.hist[(keys[u] >> H2_SHIFT) & (H2_BINS - 1)], 1u);
    }
    __syncthreads();
    flush_hist<H2_BINS>(sh.hist, sb.h2);
    if (block_is_last(&sb.state->ticket[1], sh)) {
        uint32_t d2, rem2;
        block_find_from_top<H2_BINS>(sb.h2, sb.state->rem1, sh, d2, rem2);
        if (threadIdx.x == 0) { sb.state->d2 = d2; sb.state->rem2 = rem2; }
    }
}

// ---- pass 3: H3 over items matching the 23-bit prefix; its last block publishes T and Q -----------
static __global__ void __launch_bounds__(SEL_THREADS)
k_sel_pass3(const float* __restrict__ val, int64_t n, SelBuffers sb) {
    __shared__ SelShared sh;
    pdl_trigger();
    for (int b = threadIdx.x; b < H3_BINS; b += SEL_THREADS) sh.hist[b] = 0;
    pdl_wait();
    const uint32_t d1 = sb.state->d1, d2 = sb.state->d2;
    const uint32_t prefix = (d1 << H2_BITS) | d2;
    __syncthreads();
    const int64_t stride = (int64_t)gridDim.x * SEL_THREADS;
    for (int64_t i0 = (int64_t)blockIdx.x * SEL_THREADS + threadIdx.x; i0 < n; i0 += stride * SEL_BATCH) {
        uint32_t keys[SEL_BATCH];
        load_keys(val, n, i0, stride, keys);
#pragma unroll
        for (int u = 0; u < SEL_BATCH; ++u)
            if (keys[u] != NO_ITEM && (keys[u] >> H2_SHIFT) == prefix) atomicAdd(&sh.hist[keys[u] & (H3_BINS - 1)], 1u);
    }
    __syncthreads();
    flush_hist<H3_BINS>(sh.hist, sb.h3);
    if (block_is_last(&sb.state->ticket[2], sh)) {
        uint32_t d3, rem3;
        block_find_from_top<H3_BINS>(sb.h3, sb.state->rem2, sh, d3, rem3);
        if (threadIdx.x == 0) {
            sb.state->thr_key = (d1 << H1_SHIFT) | (d2 << H2_SHIFT) | d3;
            sb.state->quota_eq = rem3;
        }
    }
}

// ---- passes 2 and 3 in one: H2 in shared memory and, in the same pass, the low 19 key bits of the items inside
// the first digit in a 2^19-bin table in global memory (few items: the first digit has already cut the input
// down to one bin in 4096).  The last block finds the second digit in H2 and the third among the 256 bins of the
// big table under it: the exact threshold key T and the tie quota Q.
static __global__ void __launch_bounds__(SEL_THREADS)
k_sel_pass23(const float* __restrict__ val, int64_t n, SelBuffers sb) {
    __shared__ SelShared sh;
    pdl_trigger();
    for (int b = threadIdx.x; b < H2_BINS; b += SEL_THREADS) sh.hist[b] = 0;
    pdl_wait();
    if (sel_gated_off(sb)) return;
    const uint32_t d1 = sb.state->d1;
    __syncthreads();
    const int64_t stride = (int64_t)gridDim.x * SEL_THREADS;
    for (int64_t i0 = (int64_t)blockIdx.x * SEL_THREADS + threadIdx.x; i0 < n; i0 += stride * SEL_BATCH) {
        uint32_t keys[SEL_BATCH];
        load_keys(val, n, i0, stride, keys);
#pragma unroll
        for (int u = 0; u < SEL_BATCH; ++u) {
            if (keys[u] != NO_ITEM && (keys[u] >> H1_SHIFT) == d1) {
                atomicAdd(&sh.hist[(keys[u] >> H2_SHIFT) & (H2_BINS - 1)], 1u);
                atomicAdd(&sb.h19[keys[u] & (H19_BINS - 1)], 1u);
            }
        }
    }
    __syncthreads();
    flush_hist<H2_BINS>(sh.hist, sb.h2);
    if (block_is_last(&sb.state->ticket[1], sh)) {
        uint32_t d2, rem2, d3, rem3;
        block_find_from_top<H2_BINS>(sb.h2, sb.state->rem1, sh, d2, rem2);
        block_find_from_top<H3_BINS>(sb.h19 + ((size_t)d2 << H3_BITS), rem2, sh, d3, rem3);
        if (threadIdx.x == 0) {
            sb.state->d2 = d2; sb.state->rem2 = rem2;
            sb.state->thr_key = (d1 << H1_SHIFT) | (d2 << H2_SHIFT) | d3;
            sb.state->quota_eq = rem3;
        }
    }
}

// For producer kernels (SEL_THREADS threads, histogram H1 already flushed): the last block turns H1
// into the first threshold digit.  `want` = how many items the selection keeps.
__device__ __forceinline__ void producer_epilogue(const SelBuffers& sb, uint32_t want, SelShared& sh) {
    if (block_is_last(&sb.state->ticket[0], sh)) {
        uint32_t d1, rem1;
        block_find_from_top<H1_BINS>(sb.h1, want, sh, d1, rem1);
        if (threadIdx.x == 0) { sb.state->d1 = d1; sb.state->rem1 = rem1; }
    }
}

// A chunk is SEL_THREADS * ITEMS items (one block's share); warp w of the block owns items
// [chunk_base + w*32*ITEMS, +32*ITEMS), read 32 at a time (coalesced).
// Returns, as ballots per iteration, which lanes hold key > T (bg) and key == T (be).
template <int ITEMS>
__device__ __forceinline__ void chunk_ballots(const float* __restrict__ val, int64_t n, int64_t warp_base,
                                              uint32_t T, uint32_t (&bg)[ITEMS], uint32_t (&be)[ITEMS],
                                              uint32_t& ngt, uint32_t& neq) {
    const int lane = threadIdx.x & 31;
    ngt = 0; neq = 0;
    uint32_t keys[ITEMS];                                   // all of the lane's items are loaded before any is used
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
        const int64_t i = warp_base + it * 32 + lane;
        keys[it] = i < n ? key_of(val[i]) : NO_ITEM;
    }
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
        const bool ok = keys[it] != NO_ITEM;
        bg[it] = __ballot_sync(0xFFFFFFFFu, ok && keys[it] > T);
        be[it] = __ballot_sync(0xFFFFFFFFu, ok && keys[it] == T);
        ngt += __popc(bg[it]);
        neq += __popc(be[it]);
    }
}

// ---- count: per-chunk numbers of key > T and key == T; the last block turns them into offsets ------
// Exclusive scan of the chunk counts in place, by one block of SEL_THREADS threads.
__device__ __forceinline__ void block_scan_chunks(const SelBuffers& sb, int64_t nchunks, SelShared& sh) {
    uint32_t* s_g = sh.hist;                 // [SEL_WARPS + 1] warp totals, then exclusive + tile total
    uint32_t* s_e = sh.hist + 32;
    uint32_t* carry = sh.hist + 64;          // [2]
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    if (t == 0) { carry[0] = 0; carry[1] = 0; }
    __syncthreads();
    for (int64_t base = 0; base < nchunks; base += SEL_THREADS) {
        const int64_t i = base + t;
        const uint32_t g = i < nchunks ? __ldcg(sb.chunk_gt + i) : 0, e = i < nchunks ? __ldcg(sb.chunk_eq + i) : 0;
        uint32_t ig = g, ie = e;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t og = __shfl_up_sync(0xFFFFFFFFu, ig, off), oe = __shfl_up_sync(0xFFFFFFFFu, ie, off);
            if (lane >= off) { ig += og; ie += oe; }
        }
        if (lane == 31) { s_g[warp] = ig; s_e[warp] = ie; }
        __syncthreads();
        if (t == 0) {
            uint32_t ag = 0, ae = 0;
            for (int w = 0; w < SEL_WARPS; ++w) {
                const uint32_t tg = s_g[w], te = s_e[w];
                s_g[w] = ag; s_e[w] = ae;
                ag += tg; ae += te;
            }
            s_g[SEL_WARPS] = ag; s_e[SEL_WARPS] = ae;   // tile totals
        }
        __syncthreads();
        if (i < nchunks) {
            sb.chunk_gt[i] = carry[0] + s_g[warp] + ig - g;
            sb.chunk_eq[i] = carry[1] + s_e[warp] + ie - e;
        }
        __syncthreads();
        if (t == 0) { carry[0] += s_g[SEL_WARPS]; carry[1] += s_e[SEL_WARPS]; }
        __syncthreads();
    }
}

template <int ITEMS>
__global__ void __launch_bounds__(SEL_THREADS)
k_sel_count(const float* __restrict__ val, int64_t n, SelBuffers sb, int64_t nchunks) {
    __shared__ SelShared sh;
    pdl_trigger();
    pdl_wait();
    if (sel_gated_off(sb)) return;
    const uint32_t T = sb.state->thr_key;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
        uint32_t bg[ITEMS], be[ITEMS], ngt, neq;
        chunk_ballots<ITEMS>(val, n, (chunk * SEL_THREADS + warp * 32) * ITEMS, T, bg, be, ngt, neq);
        if (lane == 0) { sh.hist[warp] = ngt; sh.hist[SEL_WARPS + warp] = neq; }
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t a = 0, b = 0;
            for (int w = 0; w < SEL_WARPS; ++w) { a += sh.hist[w]; b += sh.hist[SEL_WARPS + w]; }
            sb.chunk_gt[chunk] = a;
            sb.chunk_eq[chunk] = b;
        }
        __syncthreads();
    }
    if (block_is_last(&sb.state->ticket[3], sh)) block_scan_chunks(sb, nchunks, sh);
}

// ---- emit: ordered compaction of the selected items -----------------------------------------------
// `sink(slot, i)` is called once for every selected item i with its output slot (0 .. m-1).
template <int ITEMS, typename Sink>
__device__ __forceinline__ void sel_emit_chunks(const float* __restrict__ val, int64_t n, const SelBuffers& sb,
                                                int64_t nchunks, Sink sink) {
    __shared__ uint32_t s_wg[SEL_WARPS], s_we[SEL_WARPS];
    pdl_trigger();
    pdl_wait();
    if (sel_gated_off(sb)) return;
    const uint32_t T = sb.state->thr_key, Q = sb.state->quota_eq;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
    const int64_t warp_base = (chunk * SEL_THREADS + warp * 32) * ITEMS;
    uint32_t bg[ITEMS], be[ITEMS], ngt, neq;
    chunk_ballots<ITEMS>(val, n, warp_base, T, bg, be, ngt, neq);
    __syncthreads();                       // the previous chunk's readers are done with s_wg, s_we
    if (lane == 0) { s_wg[warp] = ngt; s_we[warp] = neq; }
    __syncthreads();
    uint32_t gt_before = sb.chunk_gt[chunk], eq_before = sb.chunk_eq[chunk];
    for (int w = 0; w < warp; ++w) { gt_before += s_wg[w]; eq_before += s_we[w]; }
    const uint32_t lt_mask = (1u << lane) - 1u;
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
        const uint32_t g = gt_before + __popc(bg[it] & lt_mask);
        const uint32_t e = eq_before + __popc(be[it] & lt_mask);
        const bool is_gt = (bg[it] >> lane) & 1u, is_eq = (be[it] >> lane) & 1u;
        if (is_gt || (is_eq && e < Q)) sink(g + (e < Q ? e : Q), warp_base + it * 32 + lane);
        gt_before += __popc(bg[it]);
        eq_before += __popc(be[it]);
    }
  }
}

#endif  // __CUDACC__
}  // namespace ssgd
