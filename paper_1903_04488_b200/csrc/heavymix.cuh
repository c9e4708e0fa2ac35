// heavymix.cuh -- Algorithm 1 (HEAVYMIX): the selection rule the paper's convergence theory covers.
//
//   line 1   l2 = median over rows j of sum_b S[j][b]^2          (k_row_sumsq: fp64 partial sums)
//   line 2   est_i = median_j s_j(i) S[j][h_j(i)]                 (the same device code as k_unsketch)
//   line 3   H = { i : est_i^2 >= l2 / k }                        (compared in fp64)
//   line 4   Top_k = H + a random (k - |H|)-subset of the rest    (k_heavymix_keys writes one key per
//            coordinate: 2^30 for heavy ones, else a 30-bit priority mixed from (seed, i) < 2^30; the exact
//            radix select of select.cuh then takes the k largest keys, ties to the smaller index: all of H
//            and the l = k - |H| other coordinates with the largest priorities)
//            |H| > k (outside the paper's guarantee): the k members of H with the largest |est_i|, ties to
//            the smaller index.  k_heavymix_rekey and a second selection, enqueued behind the first, run only
//            in that case (they return at once otherwise): the key becomes the full 31-bit magnitude of a
//            heavy coordinate's estimate and 0 for the others.
//   line 5   exact values of Top_k, summed over the workers       (k_gather)
#pragma once
#include <stdint.h>

#include "estimate.cuh"
#include "hash.cuh"
#include "select.cuh"

namespace ssgd {

struct HeavymixState {          // zeroed before the call
    double rowsum[MAX_R + 1];   // sum of squares per row
    uint32_t nheavy;
    uint32_t pad[3];
};

struct HeavymixArgs {
    const float* table; int64_t c; int64_t d; int32_t r;
    HashParams hp; Bucketizer bk;
    HeavymixState* hm;
    float* keys;                // [d] selection keys stored as fp32 bit patterns, 16-byte aligned
    float* est;                 // [d] the estimates, kept for k_heavymix_rekey, 16-byte aligned
    SelBuffers sb;              // H1 of the keys goes here
    uint32_t k;
    uint64_t fill_seed;
};

#ifdef __CUDACC__

__device__ __forceinline__ uint32_t fill_priority30(uint64_t seed, uint32_t i) {
    uint64_t z = seed + ((uint64_t)i + 1ull) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z ^= z >> 31;
    return (uint32_t)(z >> 34);
}

// sum of squares of every row; grid.y = row, grid.x strides over the columns
static __global__ void __launch_bounds__(256)
k_row_sumsq(const float* __restrict__ table, int64_t c, HeavymixState* __restrict__ hm) {
    __shared__ double s_part[8];
    const int j = blockIdx.y;
    const float* row = table + (int64_t)j * c;
    double acc = 0.0;
    for (int64_t b = (int64_t)blockIdx.x * 256 + threadIdx.x; b < c; b += (int64_t)gridDim.x * 256) {
        const double t = (double)row[b];
        acc = fma(t, t, acc);
    }
    for (int off = 16; off; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < 8; ++w) s += s_part[w];
        atomicAdd(&hm->rowsum[j], s);
    }
}

template <int R, bool POW2>
__global__ void __launch_bounds__(SEL_THREADS)
k_heavymix_keys(const HeavymixArgs A) {
    __shared__ SelShared sh;
    __shared__ double s_thr;
    __shared__ uint32_t s_heavy;
    for (int b = threadIdx.x; b < H1_BINS; b += SEL_THREADS) sh.hist[b] = 0;
    if (threadIdx.x == 0) {
        double rows[MAX_R];
        for (int j = 0; j < R; ++j) rows[j] = A.hm->rowsum[j];
        for (int p = 1; p < R; ++p) {                      // insertion sort; the median is the middle element
            const double key = rows[p];
            int q = p - 1;
            while (q >= 0 && rows[q] > key) { rows[q + 1] = rows[q]; --q; }
            rows[q + 1] = key;
        }
        s_thr = rows[R / 2] / (double)A.k;                 // line 3: l2 / k
        s_heavy = 0;
    }
    __syncthreads();
    const double thr = s_thr;
    const int64_t groups = (A.d + 3) >> 2;
    const int64_t stride = (int64_t)gridDim.x * SEL_THREADS;
    uint32_t my_heavy = 0;
    for (int64_t q = (int64_t)blockIdx.x * SEL_THREADS + threadIdx.x; q < groups; q += stride) {
        const int64_t i0 = q << 2;
        float rowv[4][R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            uint32_t hb[4];
            row_hashes<POW2, 4>(A.hp.row[j], A.bk, (uint32_t)i0, hb);
#pragma unroll
            for (int e = 0; e < 4; ++e)
                rowv[e][j] = apply_sign(table_load(A.table + (int64_t)j * A.c + (hb[e] & P31)), hb[e]);
        }
        uint32_t kv[4];
        float mv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float m = median_of<R>(rowv[e]);
            const bool heavy = (double)m * (double)m >= thr;
            mv[e] = m;
            kv[e] = heavy ? 0x40000000u : fill_priority30(A.fill_seed, (uint32_t)(i0 + e));
            if (heavy && i0 + e < A.d) ++my_heavy;
        }
        if (i0 + 3 < A.d) {
            *reinterpret_cast<uint4*>(A.keys + i0) = make_uint4(kv[0], kv[1], kv[2], kv[3]);
            *reinterpret_cast<float4*>(A.est + i0) = make_float4(mv[0], mv[1], mv[2], mv[3]);
#pragma unroll
            for (int e = 0; e < 4; ++e) atomicAdd(&sh.hist[kv[e] >> H1_SHIFT], 1u);
        } else {
            for (int e = 0; e < 4 && i0 + e < A.d; ++e) {
                A.keys[i0 + e] = __uint_as_float(kv[e]);
                A.est[i0 + e] = mv[e];
                atomicAdd(&sh.hist[kv[e] >> H1_SHIFT], 1u);
            }
        }
    }
    if (my_heavy) atomicAdd(&s_heavy, my_heavy);
    __syncthreads();
    if (threadIdx.x == 0 && s_heavy) atomicAdd(&A.hm->nheavy, s_heavy);
    flush_hist<H1_BINS>(sh.hist, A.sb.h1);
    producer_epilogue(A.sb, A.k, sh);
}

// |H| > k only: keys[i] = magnitude bits of est_i for heavy coordinates, 0 for the others (a heavy coordinate's
// estimate is non-zero unless l2 = 0, and then every coordinate is heavy), and their first histogram.
static __global__ void __launch_bounds__(SEL_THREADS)
k_heavymix_rekey(const HeavymixArgs A, int32_t r, SelBuffers sb2) {
    __shared__ SelShared sh;
    __shared__ double s_thr;
    if (__ldcg(&A.hm->nheavy) <= A.k) return;
    for (int b = threadIdx.x; b < H1_BINS; b += SEL_THREADS) sh.hist[b] = 0;
    if (threadIdx.x == 0) {
        double rows[MAX_R];
        for (int j = 0; j < r; ++j) rows[j] = A.hm->rowsum[j];
        for (int p = 1; p < r; ++p) {
            const double key = rows[p];
            int q = p - 1;
            while (q >= 0 && rows[q] > key) { rows[q + 1] = rows[q]; --q; }
            rows[q + 1] = key;
        }
        s_thr = rows[r / 2] / (double)A.k;
    }
    __syncthreads();
    const double thr = s_thr;
    const int64_t stride = (int64_t)gridDim.x * SEL_THREADS;
    for (int64_t i = (int64_t)blockIdx.x * SEL_THREADS + threadIdx.x; i < A.d; i += stride) {
        const float m = A.est[i];
        const uint32_t kv = (double)m * (double)m >= thr ? key_of(m) : 0u;
        A.keys[i] = __uint_as_float(kv);
        atomicAdd(&sh.hist[kv >> H1_SHIFT], 1u);
    }
    __syncthreads();
    flush_hist<H1_BINS>(sh.hist, sb2.h1);
    producer_epilogue(sb2, A.k, sh);
}

// l2 (median of the row sums) and |H| to caller-provided device words
static __global__ void k_heavymix_report(const HeavymixState* __restrict__ hm, int r, double* __restrict__ l2_out,
                                  int32_t* __restrict__ nheavy_out) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    double rows[MAX_R];
    for (int j = 0; j < r; ++j) rows[j] = hm->rowsum[j];
    for (int p = 1; p < r; ++p) {
        const double key = rows[p];
        int q = p - 1;
        while (q >= 0 && rows[q] > key) { rows[q + 1] = rows[q]; --q; }
        rows[q + 1] = key;
    }
    if (l2_out) *l2_out = rows[r / 2];
    if (nheavy_out) *nheavy_out = (int32_t)hm->nheavy;
}

#endif  // __CUDACC__
}  // namespace ssgd
