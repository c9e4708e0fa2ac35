// list_select.cuh -- exact top-ncand of the survivor list written by k_unsketch_pruned (Algorithm 3 line 9),
// emitted in ascending coordinate order.
//
// The list is short (1-2 x ncand entries out of d coordinates) and unordered.  Three grid-wide launches:
//
//   k_list_hist     one pass over the list: for the items inside the first threshold digit (12 bits, found by
//                   the producer's last block) count the next 11 key bits in H2 and the low 19 key bits in a
//                   2^19-bin table; the last block finds the second digit in H2 and the third among the 256
//                   bins of the big table under it: the exact threshold key T and the tie quota Q.
//   k_list_mark     items above T set their coordinate's bit in map A, items equal to T in map B, and count
//                   themselves on their chunk of map words; the last block turns the counts into exclusive offsets.
//   k_map_emit      walks the maps in coordinate order: an A bit with a A-bits and b B-bits before it goes to
//                   slot a + min(b, Q); a B bit with b < Q to slot a + b.  Ties at the threshold therefore go
//                   to the smallest coordinates, without a sort and without a limit on their number.  In ssgd_step
//                   the second round's read of each candidate's exact sum rides on this kernel.
//
// Nothing here waits on another block: "last block" means the block that draws the last ticket after a fence.
#pragma once
#include <stdint.h>

#include "select.cuh"
#include "sparse_select.cuh"

namespace ssgd {

constexpr int MAP_CHUNK_WORDS = SEL_THREADS * 8;       // map words per block in count/emit (8 per thread)

#ifdef __CUDACC__

// ---- histogram pass over the list; its last block publishes T and Q --------------------------------------
static __global__ void __launch_bounds__(SEL_THREADS)
k_list_hist(SparseBuffers sp) {
    __shared__ SelShared sh;
    pdl_trigger();
    for (int b = threadIdx.x; b < H2_BINS; b += SEL_THREADS) sh.hist[b] = 0;
    pdl_wait();
    const uint32_t n = __ldcg(&sp.state->n_surv);
    const uint32_t d1 = __ldcg(&sp.state->d1);
    __syncthreads();
    const int64_t stride = (int64_t)gridDim.x * SEL_THREADS;
    for (int64_t i0 = (int64_t)blockIdx.x * SEL_THREADS + threadIdx.x; i0 < n; i0 += stride * SEL_BATCH) {
        uint32_t keys[SEL_BATCH];
        load_keys(sp.list_est, n, i0, stride, keys);
#pragma unroll
        for (int u = 0; u < SEL_BATCH; ++u) {
            if (keys[u] != NO_ITEM && (keys[u] >> H1_SHIFT) == d1) {
                atomicAdd(&sh.hist[(keys[u] >> H2_SHIFT) & (H2_BINS - 1)], 1u);
                atomicAdd(&sp.h19[keys[u] & (H19_BINS - 1)], 1u);
            }
        }
    }
    __syncthreads();
    flush_hist<H2_BINS>(sh.hist, sp.h2);
    if (block_is_last(&sp.state->ticket[3], sh)) {
        uint32_t d2, rem2, d3, rem3;
        block_find_from_top<H2_BINS>(sp.h2, __ldcg(&sp.state->rem1), sh, d2, rem2);
        block_find_from_top<H3_BINS>(sp.h19 + ((size_t)d2 << H3_BITS), rem2, sh, d3, rem3);
        if (threadIdx.x == 0) {
            sp.state->thr_key = (d1 << H1_SHIFT) | (d2 << H2_SHIFT) | d3;
            sp.state->quota_eq = rem3;
        }
    }
}

// ---- mark: coordinates above the threshold in map A, at the threshold in map B; marks per chunk of map words ---
// Every list item is a distinct coordinate, so the marks a chunk of the maps receives can be counted here, one
// atomic per marked item on the chunk's counter (zeroed with the maps); the last block turns the counts into
// exclusive offsets for k_map_emit.
static __global__ void __launch_bounds__(SEL_THREADS)
k_list_mark(SparseBuffers sp, int64_t nchunks) {
    __shared__ SelShared sh;
    // chunk counters are hot addresses (a few hundred of them for 1e5 marks): count in shared memory first
    const bool local = 2 * nchunks <= H1_BINS;
    pdl_trigger();
    if (local) for (int b = threadIdx.x; b < 2 * nchunks; b += SEL_THREADS) sh.hist[b] = 0;
    pdl_wait();
    const uint32_t n = __ldcg(&sp.state->n_surv);
    const uint32_t T = __ldcg(&sp.state->thr_key);
    __syncthreads();
    const int64_t stride = (int64_t)gridDim.x * SEL_THREADS;
    for (int64_t i0 = (int64_t)blockIdx.x * SEL_THREADS + threadIdx.x; i0 < n; i0 += stride * SEL_BATCH) {
        uint32_t keys[SEL_BATCH];
        load_keys(sp.list_est, n, i0, stride, keys);
#pragma unroll
        for (int u = 0; u < SEL_BATCH; ++u) {
            if (keys[u] == NO_ITEM || keys[u] < T) continue;
            const uint32_t c = (uint32_t)sp.list_idx[i0 + u * stride];
            const bool above = keys[u] > T;
            atomicOr((above ? sp.map_a : sp.map_b) + (c >> 5), 1u << (c & 31));
            const uint32_t chunk = (c >> 5) / MAP_CHUNK_WORDS;
            if (local) atomicAdd(&sh.hist[(above ? 0 : nchunks) + chunk], 1u);
            else atomicAdd((above ? sp.chunk_a : sp.chunk_b) + chunk, 1u);
        }
    }
    if (local) {
        __syncthreads();
        for (int b = threadIdx.x; b < 2 * nchunks; b += SEL_THREADS) {
            const uint32_t h = sh.hist[b];
            if (h) atomicAdd(b < nchunks ? sp.chunk_a + b : sp.chunk_b + (b - nchunks), h);
        }
    }
    if (block_is_last(&sp.state->ticket[4], sh)) {
        SelBuffers sb{};
        sb.chunk_gt = sp.chunk_a;
        sb.chunk_eq = sp.chunk_b;
        block_scan_chunks(sb, nchunks, sh);
    }
}

// A block's 8 words per thread of both maps, word = chunk_base + it*SEL_THREADS + tid (coalesced)
__device__ __forceinline__ void load_map_words(const SparseBuffers& sp, int64_t nwords, int64_t chunk_base,
                                               uint32_t (&wa)[8], uint32_t (&wb)[8]) {
#pragma unroll
    for (int it = 0; it < 8; ++it) {
        const int64_t w = chunk_base + it * SEL_THREADS + threadIdx.x;
        wa[it] = w < nwords ? __ldcg(sp.map_a + w) : 0u;
        wb[it] = w < nwords ? __ldcg(sp.map_b + w) : 0u;
    }
}

// ---- emit: ordered walk over the maps ----------------------------------------------------------------------
// Word order inside a chunk is (it, tid): word = base + it*256 + tid, so "before" means smaller it, or the same
// it and a smaller thread.  Per it, a block-wide exclusive scan of the words' A and B counts gives each word the
// number of A and B bits before it.
// Optional second round (Algorithm 3 line 10) riding on the emit: with the per-coordinate sums over the workers
// at hand (ssgd_step), the exact sum of each emitted candidate is read here, written to xs[slot] and counted in
// the final selection's first histogram, so no separate gather launch follows.
struct EmitSecondRound {
    const float* xsum;         // [d], or NULL: emit only
    float* xs;                 // [ncand]
    SelBuffers sb;             // final selection: h1 is filled here, its first digit found by the last block
    uint32_t want;             // k
    uint32_t* pending_clear;   // the deferred zero-out's map, emptied here (or NULL)
    int64_t pending_words;
};

static __global__ void __launch_bounds__(SEL_THREADS)
k_map_emit(SparseBuffers sp, int64_t nwords, int64_t nchunks, uint32_t m, int32_t* __restrict__ cand_idx,
           EmitSecondRound E) {
    __shared__ SelShared sh;
    __shared__ uint32_t s_wa[SEL_WARPS], s_wb[SEL_WARPS];
    pdl_trigger();
    if (E.xsum) for (int b = threadIdx.x; b < H1_BINS; b += SEL_THREADS) sh.hist[b] = 0;
    pdl_wait();
    if (E.xsum && E.pending_clear)
        for (int64_t t = (int64_t)blockIdx.x * SEL_THREADS + threadIdx.x; t < E.pending_words; t += (int64_t)gridDim.x * SEL_THREADS)
            E.pending_clear[t] = 0u;
    __syncthreads();
    const uint32_t Q = __ldcg(&sp.state->quota_eq);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    auto emit = [&](uint32_t slot, int64_t coord) {
        if (slot < m) cand_idx[slot] = (int32_t)coord;
    };
    for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
        if (__ldcg(sp.chunk_a + chunk) + __ldcg(sp.chunk_b + chunk) ==
            (chunk + 1 < nchunks ? __ldcg(sp.chunk_a + chunk + 1) + __ldcg(sp.chunk_b + chunk + 1) : 0xFFFFFFFFu))
            continue;                                        // offsets do not move across this chunk: no marks in it
        uint32_t wa[8], wb[8];
        const int64_t base = chunk * MAP_CHUNK_WORDS;
        load_map_words(sp, nwords, base, wa, wb);
        uint32_t run_a = __ldcg(sp.chunk_a + chunk), run_b = __ldcg(sp.chunk_b + chunk);
        const uint32_t slot_lo = run_a + (run_b < Q ? run_b : Q);      // this chunk's candidates fill [slot_lo, slot_hi)
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const uint32_t ca = __popc(wa[it]), cb = __popc(wb[it]);
            uint32_t ia = ca, ib = cb;                       // inclusive over the lanes of this warp
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t oa = __shfl_up_sync(0xFFFFFFFFu, ia, off), ob = __shfl_up_sync(0xFFFFFFFFu, ib, off);
                if (lane >= off) { ia += oa; ib += ob; }
            }
            __syncthreads();                                 // previous iteration's readers are done
            if (lane == 31) { s_wa[warp] = ia; s_wb[warp] = ib; }
            __syncthreads();
            uint32_t a = run_a + ia - ca, b = run_b + ib - cb, ta = 0, tb = 0;
            for (int w = 0; w < SEL_WARPS; ++w) {
                if (w < warp) { a += s_wa[w]; b += s_wb[w]; }
                ta += s_wa[w]; tb += s_wb[w];
            }
            uint32_t bits = wa[it] | wb[it];
            const int64_t w0 = (base + it * SEL_THREADS + threadIdx.x) << 5;
            while (bits) {
                const int bit = __ffs(bits) - 1;
                bits &= bits - 1;
                if ((wa[it] >> bit) & 1u) {
                    emit(a + (b < Q ? b : Q), w0 + bit);
                    ++a;
                } else {
                    if (b < Q) emit(a + b, w0 + bit);
                    ++b;
                }
            }
            run_a += ta;
            run_b += tb;
        }
        if (E.xsum) {
            // second round for this chunk's candidates, all threads of the block in parallel (the loop above hands
            // a thread its candidates one after another: reading the sums there would serialise the latencies)
            uint32_t slot_hi = run_a + (run_b < Q ? run_b : Q);
            if (slot_hi > m) slot_hi = m;
            __syncthreads();                                 // the block's cand_idx stores are visible to the block
            for (uint32_t slot = slot_lo + threadIdx.x; slot < slot_hi; slot += SEL_THREADS) {
                const float x = __ldg(E.xsum + cand_idx[slot]);
                E.xs[slot] = x;
                atomicAdd(&sh.hist[key_of(x) >> H1_SHIFT], 1u);
            }
        }
    }
    if (E.xsum) {
        __syncthreads();
        flush_hist<H1_BINS>(sh.hist, E.sb.h1);
        producer_epilogue(E.sb, E.want, sh);
    }
}

#endif  // __CUDACC__
}  // namespace ssgd
