// step_kernels.cuh -- kernels of the step that are not in a header of their own: the plain-load
// accumulate+insert (Algorithm 3 lines 5-7), the follow-up row insert for large tables, the merge of
// per-worker tables (line 8) and its 16-bit form, the dense unsketch (line 9), the second-round gather
// (line 10), the emit kernels of the two selections (lines 9, 11), the zero-out (line 13) and the hash dump.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "accum_tma.cuh"
#include "estimate.cuh"
#include "hash.cuh"
#include "select.cuh"

namespace ssgd {

// Every reduction into the merged table carries an L2 evict-last policy (red_add_hint): the table's lines then
// outlive the stream that passes through L2 beside them.  Measured on B200 with it / without (whole step, ms; the
// streamed loads as they were best in each case): 20 MB table, W = 32 2.166 / 2.238; 80 MB 7.11 / 7.24; 5 MB
// W = 256 (bulk-copy kernel) 9.59 / 9.80, W = 32 1.287 / 1.294, W = 16 0.749 / 0.751.
//
// Table bytes one insert kernel may scatter into; larger tables are inserted in row slices.  Measured on B200
// (C4: d = 9e7, W = 16, 5 rows of 4,194,304 = 16 MiB each; whole step, ms): 1 row per kernel 7.11, 2 rows 7.27,
// 3 rows 7.52, 4 rows 8.20, all 5 rows in one kernel 9.20.
constexpr size_t SPLIT_BYTES_DEFAULT = (size_t)24 << 20;
// Table bytes one k_insert_rows pass scatters into: beside it only the per-coordinate sums stream through L2.
// Measured at C4 (whole step, ms; one row in the streaming kernel): passes of 1 row 7.11, 2 rows 7.04, 3 + 1 rows
// 7.02, all 4 remaining rows in one pass 6.93; no row in the streaming kernel and all 5 in one pass 7.32; 2 rows in
// the streaming kernel and 3 in one pass 7.21.
constexpr size_t INSERT_PASS_BYTES = (size_t)64 << 20;
// The plain-load kernel reads g, u, v cached in L2 only (ld.global.cg); the evict-first operator (ld.global.cs)
// can be chosen instead (ssgd_set_stream_loads).  Measured on B200, whole step in ms with .cs / .cg: 5 MB table
// W = 32 1.349 / 1.287, W = 16 0.768 / 0.749, W = 8 0.573 / 0.571; 3.6 MB (W = 4, d = 7.3e7) 2.709 / 2.715; 20 MB
// W = 32 2.235 / 2.166, (W = 4, d = 9e7) 3.449 / 3.442; 80 MB, one row per kernel 7.25 / 7.11.  (Before the
// reductions carried their evict-last policy, .cs was the better choice for tables of 20 MB and more.)
// Blocks per SM of the two unsketch kernels: one resident wave.  Measured on B200 (C2): the dense kernel
// takes 0.222 ms with 4 or 6 blocks per SM in the grid and 0.246 ms with 8 (6 fit: the last third of a
// second wave runs alone); the early-exit kernel 0.205-0.210 ms with 2 or 4, 0.232 ms with 16.
constexpr int PRUNED_GRID = 4;
constexpr int K3_GRID = 4;


// ------------------------------------------------------------------------------------------------
// K1 (plain-load form): momentum + error accumulation + sketch insert.  ssgd_step's default below 64 workers
// (the bulk-copy pipeline of accum_tma.cuh from there on); also the per-worker tables of ssgd_sketch_accumulate and the
// shared-memory table variant.
// ------------------------------------------------------------------------------------------------
enum InsertMode { INS_MERGED_GLOBAL = 0, INS_PER_WORKER = 1, INS_MERGED_SMEM = 2, INS_MERGED_TMA = 3 };

// Measured on B200 (C2, W = 16): 256 threads x 4 workers in flight 4.93 TB/s; 128 x 8 5.38; 128 x 16 5.58;
// 64 x 16 5.56; forcing more resident blocks (fewer registers) or 32 workers in flight is slower.
// The grid has one float4 group per thread on purpose: capping it at 2, 4, 8, 16, 40 blocks per SM (each
// thread then loops over 74 ... 4 groups) took 0.887, 0.860, 0.814, 0.724, 0.654 ms against 0.635 ms, and
// deferring a group's reductions until the next group's loads are issued recovered only part of that (0.805 ms
// at 2 blocks per SM).
constexpr int K1_THREADS = 128;
constexpr int K1_UNROLL = 16;              // workers in flight per thread: 3 x 16 B loads each
constexpr int K1_UNROLL_PW = 4;            // same, for the per-worker-table mode (it also holds 4r hashes)

// UM: workers in flight per thread in the merged modes.  Measured on B200 with 4 workers (d = 7.3e7 / 9e7, r = 5):
// 16 -> 4 brings the kernel from 2.44 / 3.03 ms to 2.18 / 2.69 ms (a third of the registers, more resident blocks
// to cover the stream while the reductions issue); with 8 workers 4, 8 and 16 are equal.
constexpr int K1_UNROLL_FEW = 4;
template <int R, bool POW2, int MODE, int UM = K1_UNROLL>
__global__ void __launch_bounds__(K1_THREADS)
k_accum_insert(const AccumArgs A) {
    extern __shared__ float s_table[];  // MODE == INS_MERGED_SMEM: [R][c]
    const int64_t rc = (int64_t)R * A.c;
    pdl_trigger();
    pdl_wait();
    if (MODE == INS_MERGED_SMEM) {
        for (int64_t t = threadIdx.x; t < rc; t += K1_THREADS) s_table[t] = 0.0f;
        __syncthreads();
    }
    const int64_t groups = (A.d + 3) >> 2;
    const int64_t stride = (int64_t)gridDim.x * K1_THREADS;
    const uint64_t tpol = table_policy();
    for (int64_t q = (int64_t)blockIdx.x * K1_THREADS + threadIdx.x; q < groups; q += stride) {
        const int64_t i0 = q << 2;
        uint32_t hb[R][4];
        if (MODE == INS_PER_WORKER) {
#pragma unroll
            for (int j = 0; j < R; ++j) row_hashes<POW2, 4>(A.hp.row[j], A.bk, (uint32_t)i0, hb[j]);
        }
        // sum over workers of the new v, in fp64 and worker order, rounded once: the value that is sketched and,
        // through xsum, the second round's exact sum (Algorithm 3 line 10) of this coordinate
        double xd[4] = {0., 0., 0., 0.};
        float x[4] = {0.f, 0.f, 0.f, 0.f};
        if (i0 + 3 < A.d) {
            constexpr int U = MODE == INS_PER_WORKER ? K1_UNROLL_PW : UM;
            for (int w0 = 0; w0 < A.W; w0 += U) {
                float4 gg[U], uu[U], vv[U];
                if (A.loads_evict_first) {              // the same for the whole grid
#pragma unroll
                    for (int s = 0; s < U; ++s) {
                        if (w0 + s < A.W) {
                            const int64_t w = w0 + s;
                            gg[s] = __ldcs(reinterpret_cast<const float4*>(A.g + w * A.ld_g + i0));
                            uu[s] = __ldcs(reinterpret_cast<const float4*>(A.u + w * A.ld + i0));
                            vv[s] = __ldcs(reinterpret_cast<const float4*>(A.v + w * A.ld + i0));
                        }
                    }
                } else {
#pragma unroll
                    for (int s = 0; s < U; ++s) {
                        if (w0 + s < A.W) {
                            const int64_t w = w0 + s;
                            gg[s] = __ldcg(reinterpret_cast<const float4*>(A.g + w * A.ld_g + i0));
                            uu[s] = __ldcg(reinterpret_cast<const float4*>(A.u + w * A.ld + i0));
                            vv[s] = __ldcg(reinterpret_cast<const float4*>(A.v + w * A.ld + i0));
                        }
                    }
                }
                const uint32_t pend = pending_bits4(A.pending, i0);   // after the wide loads are on their way
                if (pend) {                              // rare: a coordinate of this group was chosen last step
#pragma unroll
                    for (int s = 0; s < U; ++s) drop_pending(pend, uu[s], vv[s]);
                }
#pragma unroll
                for (int s = 0; s < U; ++s) {
                    if (w0 + s < A.W) {
                        const int64_t w = w0 + s;
                        float4 un, vn;
                        un.x = __fmaf_rn(A.rho, uu[s].x, gg[s].x); vn.x = __fadd_rn(vv[s].x, un.x);
                        un.y = __fmaf_rn(A.rho, uu[s].y, gg[s].y); vn.y = __fadd_rn(vv[s].y, un.y);
                        un.z = __fmaf_rn(A.rho, uu[s].z, gg[s].z); vn.z = __fadd_rn(vv[s].z, un.z);
                        un.w = __fmaf_rn(A.rho, uu[s].w, gg[s].w); vn.w = __fadd_rn(vv[s].w, un.w);
                        __stcs(reinterpret_cast<float4*>(A.u + w * A.ld + i0), un);
                        __stcs(reinterpret_cast<float4*>(A.v + w * A.ld + i0), vn);
                        if (MODE == INS_PER_WORKER) {
                            float* tw = A.table + w * rc;
                            const float vals[4] = {vn.x, vn.y, vn.z, vn.w};
#pragma unroll
                            for (int j = 0; j < R; ++j)
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    if (vals[e] != 0.0f)
                                        red_add(tw + (int64_t)j * A.c + (hb[j][e] & P31), apply_sign(vals[e], hb[j][e]));
                        } else {
                            xd[0] = __dadd_rn(xd[0], (double)vn.x); xd[1] = __dadd_rn(xd[1], (double)vn.y);
                            xd[2] = __dadd_rn(xd[2], (double)vn.z); xd[3] = __dadd_rn(xd[3], (double)vn.w);
                        }
                    }
                }
            }
        } else {
            // ragged last group (d not a multiple of 4): scalar, bounds-checked
            for (int e = 0; e < 4; ++e) {
                const int64_t i = i0 + e;
                if (i >= A.d) break;
                const bool pend = pending_bit(A.pending, i);
                for (int64_t w = 0; w < A.W; ++w) {
                    const float un = __fmaf_rn(A.rho, pend ? 0.f : A.u[w * A.ld + i], A.g[w * A.ld_g + i]);
                    const float vn = __fadd_rn(pend ? 0.f : A.v[w * A.ld + i], un);
                    A.u[w * A.ld + i] = un;
                    A.v[w * A.ld + i] = vn;
                    if (MODE == INS_PER_WORKER) {
#pragma unroll
                        for (int j = 0; j < R; ++j)
                            if (vn != 0.0f)
                                red_add(A.table + w * rc + (int64_t)j * A.c + (hb[j][e] & P31),
                                        apply_sign(vn, hb[j][e]));
                    } else {
                        xd[e] = __dadd_rn(xd[e], (double)vn);
                    }
                }
            }
        }
        if (MODE != INS_PER_WORKER) {
#pragma unroll
            for (int e = 0; e < 4; ++e) x[e] = (float)xd[e];
            if (A.xsum != nullptr) {
                // streaming store: measured 7 us faster at C2 than a store that competes with the table for L2
                if (i0 + 3 < A.d) __stcs(reinterpret_cast<float4*>(A.xsum + i0), make_float4(x[0], x[1], x[2], x[3]));
                else for (int e = 0; e < 4 && i0 + e < A.d; ++e) A.xsum[i0 + e] = x[e];
            }
#pragma unroll
            for (int j = 0; j < R; ++j) {
                if (MODE == INS_MERGED_GLOBAL && j >= A.rows_here) break;
                uint32_t h1[4];
                row_hashes<POW2, 4>(A.hp.row[j], A.bk, (uint32_t)i0, h1);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (i0 + e < A.d && x[e] != 0.0f) {
                        const float sx = apply_sign(x[e], h1[e]);
                        if (MODE == INS_MERGED_SMEM) atomicAdd(&s_table[(int64_t)j * A.c + (h1[e] & P31)], sx);
                        else red_add_hint(A.table + (int64_t)j * A.c + (h1[e] & P31), sx, tpol);
                    }
                }
            }
        }
    }
    if (MODE == INS_MERGED_SMEM) {
        __syncthreads();
        for (int64_t t = threadIdx.x; t < rc; t += K1_THREADS) {
            const float s = s_table[t];
            if (s != 0.0f) red_add(A.table + t, s);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Rows [row_lo, R) of the insert, from the per-coordinate sums written by k_accum_insert.  Used when the
// whole r x c table is too large to stay in L2 next to the stream: the streaming kernel then inserts only as
// many rows as fit, and the rest are inserted here, a few rows (an L2-sized slice of the table) per launch.
// ------------------------------------------------------------------------------------------------
template <int R, bool POW2>
__global__ void __launch_bounds__(256)
k_insert_rows(const float* __restrict__ xsum, int64_t d, float* __restrict__ table, int64_t c, HashParams hp,
              Bucketizer bk, int row_lo, int row_hi) {
    pdl_trigger();
    pdl_wait();
    const int64_t groups = (d + 3) >> 2;
    const int64_t stride = (int64_t)gridDim.x * 256;
    const uint64_t tpol = table_policy();
    for (int64_t q = (int64_t)blockIdx.x * 256 + threadIdx.x; q < groups; q += stride) {
        const int64_t i0 = q << 2;
        float x[4] = {0.f, 0.f, 0.f, 0.f};
        if (i0 + 3 < d) {
            const float4 t = __ldcs(reinterpret_cast<const float4*>(xsum + i0));
            x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
        } else {
            for (int e = 0; e < 4 && i0 + e < d; ++e) x[e] = xsum[i0 + e];
        }
#pragma unroll
        for (int j = 0; j < R; ++j) {
            if (j < row_lo || j >= row_hi) continue;
            uint32_t hb[4];
            row_hashes<POW2, 4>(hp.row[j], bk, (uint32_t)i0, hb);
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (i0 + e < d && x[e] != 0.0f) red_add_hint(table + (int64_t)j * c + (hb[e] & P31), apply_sign(x[e], hb[e]), tpol);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// K2: merge of the per-worker tables, worker order
// ------------------------------------------------------------------------------------------------
static __global__ void __launch_bounds__(256)
k_merge(const float* __restrict__ tables, float* __restrict__ merged, int64_t rc, int32_t W) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if ((rc & 3) == 0) {
        const int64_t n4 = rc >> 2;
        for (int64_t q = t0; q < n4; q += stride) {
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int w0 = 0; w0 < W; w0 += 8) {
                float4 t[8];
#pragma unroll
                for (int s = 0; s < 8; ++s)
                    if (w0 + s < W) t[s] = __ldcs(reinterpret_cast<const float4*>(tables + (int64_t)(w0 + s) * rc) + q);
#pragma unroll
                for (int s = 0; s < 8; ++s)
                    if (w0 + s < W) {
                        acc.x = __fadd_rn(acc.x, t[s].x); acc.y = __fadd_rn(acc.y, t[s].y);
                        acc.z = __fadd_rn(acc.z, t[s].z); acc.w = __fadd_rn(acc.w, t[s].w);
                    }
            }
            reinterpret_cast<float4*>(merged)[q] = acc;
        }
    } else {
        for (int64_t t = t0; t < rc; t += stride) {
            float acc = 0.f;
            for (int w = 0; w < W; ++w) acc = __fadd_rn(acc, tables[(int64_t)w * rc + t]);
            merged[t] = acc;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// 16-bit sketches (Section 6): what a worker would send is its table rounded to binary16 or bfloat16
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint16_t quant16(float x, int fmt) {
    if (fmt == 0) {
        x = fminf(fmaxf(x, -65504.0f), 65504.0f);          // saturate instead of rounding to infinity
        return __half_as_ushort(__float2half_rn(x));
    }
    return __bfloat16_as_ushort(__float2bfloat16_rn(x));
}
__device__ __forceinline__ float dequant16(uint16_t h, int fmt) {
    return fmt == 0 ? __half2float(__ushort_as_half(h)) : __bfloat162float(__ushort_as_bfloat16(h));
}

static __global__ void __launch_bounds__(256)
k_quantize16(const float* __restrict__ x, uint16_t* __restrict__ q, int64_t n, int fmt) {
    const int64_t stride = (int64_t)gridDim.x * 256;
    for (int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x; t < n; t += stride) q[t] = quant16(__ldcs(x + t), fmt);
}

// merged[t] = sum over w = 0..W-1 (that order, fp32) of the decoded q[w][t]
static __global__ void __launch_bounds__(256)
k_merge16(const uint16_t* __restrict__ q, float* __restrict__ merged, int64_t n, int32_t W, int fmt) {
    const int64_t stride = (int64_t)gridDim.x * 256;
    for (int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x; t < n; t += stride) {
        float acc = 0.f;
        for (int w = 0; w < W; ++w) acc = __fadd_rn(acc, dequant16(q[(int64_t)w * n + t], fmt));
        merged[t] = acc;
    }
}

// ------------------------------------------------------------------------------------------------
// K3: estimate of every coordinate (median of r signed buckets) + first histogram of |estimate|
// ------------------------------------------------------------------------------------------------
struct UnsketchArgs {
    const float* table; int64_t c; int64_t d;
    HashParams hp; Bucketizer bk;
    float* est;          // [d], 16-byte aligned
    SelBuffers sb;       // selection buffers of the candidate stage (H1 filled here)
    uint32_t want;       // ncand
};

constexpr int K3_THREADS = 256;
constexpr int K3_NC = 4;  // consecutive coordinates per thread

template <int R, bool POW2>
__global__ void __launch_bounds__(K3_THREADS)
k_unsketch(const UnsketchArgs A) {
    __shared__ SelShared sh;
    uint32_t* s_hist = sh.hist;
    pdl_trigger();
    for (int b = threadIdx.x; b < H1_BINS; b += K3_THREADS) s_hist[b] = 0;
    pdl_wait();
    __syncthreads();
    const int64_t groups = (A.d + K3_NC - 1) / K3_NC;
    const int64_t stride = (int64_t)gridDim.x * K3_THREADS;
    for (int64_t q = (int64_t)blockIdx.x * K3_THREADS + threadIdx.x; q < groups; q += stride) {
        const int64_t i0 = q * K3_NC;
        float rowv[K3_NC][R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            uint32_t hb[K3_NC];
            row_hashes<POW2, K3_NC>(A.hp.row[j], A.bk, (uint32_t)i0, hb);
#pragma unroll
            for (int e = 0; e < K3_NC; ++e)
                rowv[e][j] = apply_sign(table_load(A.table + (int64_t)j * A.c + (hb[e] & P31)), hb[e]);
        }
        float m[K3_NC];
#pragma unroll
        for (int e = 0; e < K3_NC; ++e) m[e] = median_of<R>(rowv[e]);
        if (i0 + K3_NC - 1 < A.d) {
#pragma unroll
            for (int e = 0; e < K3_NC; e += 4)
                *reinterpret_cast<float4*>(A.est + i0 + e) = make_float4(m[e], m[e + 1], m[e + 2], m[e + 3]);
#pragma unroll
            for (int e = 0; e < K3_NC; ++e) atomicAdd(&s_hist[key_of(m[e]) >> H1_SHIFT], 1u);
        } else {
            for (int e = 0; e < K3_NC && i0 + e < A.d; ++e) {
                A.est[i0 + e] = m[e];
                atomicAdd(&s_hist[key_of(m[e]) >> H1_SHIFT], 1u);
            }
        }
    }
    __syncthreads();
    flush_hist<H1_BINS>(s_hist, A.sb.h1);
    producer_epilogue(A.sb, A.want, sh);
}

// ------------------------------------------------------------------------------------------------
// candidate emit (line 9, second half)
// ------------------------------------------------------------------------------------------------
static __global__ void __launch_bounds__(SEL_THREADS)
k_emit_candidates(const float* __restrict__ est, int64_t d, SelBuffers sb, int32_t* __restrict__ cand_idx,
                  float* __restrict__ cand_est, uint32_t cap, int64_t nchunks) {
    sel_emit_chunks<SEL_ITEMS>(est, d, sb, nchunks, [&](uint32_t slot, int64_t i) {
        if (slot >= cap) return;  // cannot happen with consistent histograms; never write past the list
        cand_idx[slot] = (int32_t)i;
        if (cand_est) cand_est[slot] = est[i];
    });
}

// ------------------------------------------------------------------------------------------------
// K5: second round -- xs[m] = sum_w v_w[cand[m]] (fp64, w = 0..W-1), rounded once to fp32
// ------------------------------------------------------------------------------------------------
constexpr int GATHER_UNROLL = 8;   // scattered loads in flight per thread

static __global__ void __launch_bounds__(256)
k_gather(const int32_t* __restrict__ cand, int64_t ncand, const float* __restrict__ v, int64_t ld, int32_t W,
         int64_t d, float* __restrict__ xs, SelBuffers sb, uint32_t want, int32_t* __restrict__ errflag,
         uint32_t* __restrict__ pending_clear, int64_t pending_words) {
    __shared__ SelShared sh;
    uint32_t* s_hist = sh.hist;
    pdl_trigger();
    for (int b = threadIdx.x; b < H1_BINS; b += 256) s_hist[b] = 0;
    pdl_wait();
    __syncthreads();
    const int64_t m = (int64_t)blockIdx.x * 256 + threadIdx.x;
    // the accumulate kernel of this step has applied the pending zero-out: empty the map for k_emit_final
    if (pending_clear)
        for (int64_t t = m; t < pending_words; t += (int64_t)gridDim.x * 256) pending_clear[t] = 0u;
    if (m < ncand) {
        const int64_t i = cand[m];
        float out = 0.0f;
        if (i < 0 || i >= d) {
            atomicExch(errflag, ERR_BAD_INDEX);
        } else {
            double acc = 0.0;
            const float* p = v + i;
            int w = 0;
            for (; w + GATHER_UNROLL <= W; w += GATHER_UNROLL) {
                float t[GATHER_UNROLL];
#pragma unroll
                for (int s = 0; s < GATHER_UNROLL; ++s) t[s] = __ldg(p + (int64_t)(w + s) * ld);
#pragma unroll
                for (int s = 0; s < GATHER_UNROLL; ++s) acc = __dadd_rn(acc, (double)t[s]);
            }
            for (; w < W; ++w) acc = __dadd_rn(acc, (double)__ldg(p + (int64_t)w * ld));
            out = (float)acc;
        }
        xs[m] = out;
        atomicAdd(&s_hist[key_of(out) >> H1_SHIFT], 1u);
    }
    __syncthreads();
    flush_hist<H1_BINS>(s_hist, sb.h1);
    producer_epilogue(sb, want, sh);
}

// Line 10 inside ssgd_step: the accumulate kernel has already summed every coordinate's new v over the workers
// (fp64, worker order, rounded once) on its way to the sketch, so the second round's exact sum of a candidate is
// one read of that array instead of W scattered reads of v.
static __global__ void __launch_bounds__(256)
k_gather_sums(const int32_t* __restrict__ cand, int64_t ncand, const float* __restrict__ xsum, int64_t d,
              float* __restrict__ xs, SelBuffers sb, uint32_t want, int32_t* __restrict__ errflag,
              uint32_t* __restrict__ pending_clear, int64_t pending_words) {
    __shared__ SelShared sh;
    uint32_t* s_hist = sh.hist;
    pdl_trigger();
    for (int b = threadIdx.x; b < H1_BINS; b += 256) s_hist[b] = 0;
    pdl_wait();
    __syncthreads();
    const int64_t m = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (pending_clear)
        for (int64_t t = m; t < pending_words; t += (int64_t)gridDim.x * 256) pending_clear[t] = 0u;
    if (m < ncand) {
        const int64_t i = cand[m];
        float out = 0.0f;
        if (i < 0 || i >= d) atomicExch(errflag, ERR_BAD_INDEX);
        else out = __ldg(xsum + i);
        xs[m] = out;
        atomicAdd(&s_hist[key_of(out) >> H1_SHIFT], 1u);
    }
    __syncthreads();
    flush_hist<H1_BINS>(s_hist, sb.h1);
    producer_epilogue(sb, want, sh);
}

// ------------------------------------------------------------------------------------------------
// final emit (line 11) and zero-out (line 13)
// ------------------------------------------------------------------------------------------------
template <int ITEMS>
__global__ void __launch_bounds__(SEL_THREADS)
k_emit_final(const float* __restrict__ xs, int64_t ncand, SelBuffers sb, const int32_t* __restrict__ cand,
             int32_t* __restrict__ out_idx, float* __restrict__ out_val, uint32_t cap, int64_t nchunks,
             uint32_t* __restrict__ pending) {
    sel_emit_chunks<ITEMS>(xs, ncand, sb, nchunks, [&](uint32_t slot, int64_t m) {
        if (slot >= cap) return;
        const int32_t i = cand[m];
        out_idx[slot] = i;
        out_val[slot] = xs[m];
        if (pending) atomicOr(pending + (i >> 5), 1u << (i & 31));   // deferred line 13: see k_flush_pending
    });
}

// The deferred form of line 13: the chosen coordinates are marked in a d-bit map, and the next step's
// accumulate kernel, which reads every u and v anyway, treats marked coordinates as zero.  This kernel applies
// the map to memory for callers that read u or v in between: one thread per map word.
static __global__ void __launch_bounds__(256)
k_flush_pending(uint32_t* __restrict__ pending, int64_t nwords, float* __restrict__ u, float* __restrict__ v,
                int64_t ld, int32_t W, int64_t d) {
    pdl_trigger();
    pdl_wait();
    const int64_t stride = (int64_t)gridDim.x * 256;
    for (int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x; t < nwords; t += stride) {
        uint32_t bits = pending[t];
        if (bits == 0u) continue;
        pending[t] = 0u;
        while (bits) {
            const int64_t i = t * 32 + (__ffs(bits) - 1);
            bits &= bits - 1;
            if (i < d)
                for (int64_t w = 0; w < W; ++w) { u[w * ld + i] = 0.0f; v[w * ld + i] = 0.0f; }
        }
    }
}

static __global__ void __launch_bounds__(256)
k_zero(const int32_t* __restrict__ out_idx, int64_t k, float* __restrict__ u, float* __restrict__ v,
       int64_t ld, int32_t W, int64_t d) {
    pdl_trigger();
    pdl_wait();
    const int64_t total = k * (int64_t)W;
    const int64_t stride = (int64_t)gridDim.x * 256;
    for (int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x; t < total; t += stride) {
        const int64_t w = t / k, m = t - w * k;   // consecutive threads: consecutive chosen coordinates
        const int64_t i = out_idx[m];
        if (i >= 0 && i < d) {
            u[w * ld + i] = 0.0f;
            v[w * ld + i] = 0.0f;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// hash dump for bit-exactness checks
// ------------------------------------------------------------------------------------------------
template <bool POW2>
__global__ void __launch_bounds__(256)
k_hashes(const int32_t* __restrict__ idx, int64_t n, int32_t r, HashParams hp, Bucketizer bk,
         int32_t* __restrict__ h_out, int32_t* __restrict__ s_out) {
    const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (t >= n) return;
    const uint32_t i = (uint32_t)idx[t];
    for (int j = 0; j < r; ++j) {
        uint32_t hb[1];
        row_hashes<POW2, 1>(hp.row[j], bk, i, hb);
        h_out[(int64_t)j * n + t] = (int32_t)(hb[0] & P31);
        s_out[(int64_t)j * n + t] = (hb[0] >> 31) ? -1 : 1;
    }
}

}  // namespace ssgd
