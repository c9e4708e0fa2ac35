// ssgd.cu -- kernels and C ABI of the Sketched-SGD compression step for sm_100a.
//
// Kernels (Algorithm 3 lines 5-13, Algorithm 4):
//   k_accum_insert      lines 5-7: streams g, u, v once (128-bit loads/stores), updates u and v, and
//                       inserts into the sketch with reductions (red.global.add.f32) -- either the sum
//                       over workers into one merged table (linearity, Section 3), or every worker's
//                       value into its own table, or into a shared-memory table flushed per block.
//   k_merge             line 8: sum of the per-worker tables in worker order.
//   k_unsketch          line 9, first half: median-of-r estimate of every coordinate from the L2-resident
//                       table, plus the first radix histogram of |estimate|.
//   k_sel_*             lines 9 and 11: exact radix select (select.cuh).
//   k_gather            line 10: second-round sums of v over workers at the candidates (fp64, fixed order).
//   k_zero              line 13: u = v = 0 at the chosen coordinates.
// HBM-bound work is the first kernel (20 bytes per worker-coordinate); nothing here is a dense
// contraction, so there are no tensor-core instructions.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <string>

#include "../../include/ssgd.h"
#include "hash.cuh"
#include "select.cuh"
#include "accum_tma.cuh"
#include "accum_ws.cuh"
#include "estimate.cuh"
#include "sparse_select.cuh"
#include "heavymix.cuh"
// Blocks per SM of the two unsketch kernels: one resident wave.  Measured on B200 (C2): the dense kernel
// takes 0.222 ms with 4 or 6 blocks per SM in the grid and 0.246 ms with 8 (6 fit: the last third of a
// second wave runs alone); the early-exit kernel 0.205-0.210 ms with 2 or 4, 0.232 ms with 16.
#ifndef SSGD_SPLIT_BYTES_DEFAULT
// measured on B200 (C4: d = 9e7, W = 16, 5 x 4,194,304 = 80 MB table): unsplit 7.80 ms, 48 MB or 32 MB slices 6.26 ms,
// 16 MB slices 6.44 ms
#define SSGD_SPLIT_BYTES_DEFAULT ((size_t)48 << 20)
#endif
#ifndef SSGD_PRUNED_GRID
#define SSGD_PRUNED_GRID 4
#endif
#ifndef SSGD_K3_GRID
#define SSGD_K3_GRID 4
#endif

namespace ssgd {

// ------------------------------------------------------------------------------------------------
// K1 (plain-load form): momentum + error accumulation + sketch insert.  ssgd_step uses the bulk-copy
// pipeline of accum_tma.cuh; this form serves the per-worker tables of ssgd_sketch_accumulate and the
// shared-memory table variant.
// ------------------------------------------------------------------------------------------------
enum InsertMode { INS_MERGED_GLOBAL = 0, INS_PER_WORKER = 1, INS_MERGED_SMEM = 2, INS_MERGED_TMA = 3, INS_MERGED_WS = 4 };

#ifndef SSGD_K1_UNROLL
#define SSGD_K1_UNROLL 16
#endif
#ifndef SSGD_K1_MINBLOCKS
#define SSGD_K1_MINBLOCKS 1
#endif
// Measured on B200 (C2, W = 16): 256 threads x 4 workers in flight 4.93 TB/s; 128 x 8 5.38; 128 x 16 5.58;
// 64 x 16 5.56; forcing more resident blocks (fewer registers) or 32 workers in flight is slower.
#ifndef SSGD_K1_THREADS
#define SSGD_K1_THREADS 128
#endif
constexpr int K1_THREADS = SSGD_K1_THREADS;
constexpr int K1_UNROLL = SSGD_K1_UNROLL;  // workers in flight per thread: 3 x 16 B loads each
constexpr int K1_UNROLL_PW = 4;            // same, for the per-worker-table mode (it also holds 4r hashes)

template <int R, bool POW2, int MODE>
__global__ void __launch_bounds__(K1_THREADS, SSGD_K1_MINBLOCKS)
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
    for (int64_t q = (int64_t)blockIdx.x * K1_THREADS + threadIdx.x; q < groups; q += stride) {
        const int64_t i0 = q << 2;
        uint32_t hb[R][4];
        if (MODE == INS_PER_WORKER) {
#pragma unroll
            for (int j = 0; j < R; ++j) row_hashes<POW2, 4>(A.hp.row[j], A.bk, (uint32_t)i0, hb[j]);
        }
        float x[4] = {0.f, 0.f, 0.f, 0.f};  // sum over workers of the new v (worker order)
        if (i0 + 3 < A.d) {
            constexpr int U = MODE == INS_PER_WORKER ? K1_UNROLL_PW : K1_UNROLL;
            for (int w0 = 0; w0 < A.W; w0 += U) {
                float4 gg[U], uu[U], vv[U];
#pragma unroll
                for (int s = 0; s < U; ++s) {
                    if (w0 + s < A.W) {
                        const int64_t w = w0 + s;
                        gg[s] = __ldcs(reinterpret_cast<const float4*>(A.g + w * A.ld_g + i0));
                        uu[s] = __ldcs(reinterpret_cast<const float4*>(A.u + w * A.ld + i0));
                        vv[s] = __ldcs(reinterpret_cast<const float4*>(A.v + w * A.ld + i0));
                    }
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
                            x[0] = __fadd_rn(x[0], vn.x); x[1] = __fadd_rn(x[1], vn.y);
                            x[2] = __fadd_rn(x[2], vn.z); x[3] = __fadd_rn(x[3], vn.w);
                        }
                    }
                }
            }
        } else {
            // ragged last group (d not a multiple of 4): scalar, bounds-checked
            for (int e = 0; e < 4; ++e) {
                const int64_t i = i0 + e;
                if (i >= A.d) break;
                for (int64_t w = 0; w < A.W; ++w) {
                    const float un = __fmaf_rn(A.rho, A.u[w * A.ld + i], A.g[w * A.ld_g + i]);
                    const float vn = __fadd_rn(A.v[w * A.ld + i], un);
                    A.u[w * A.ld + i] = un;
                    A.v[w * A.ld + i] = vn;
                    if (MODE == INS_PER_WORKER) {
#pragma unroll
                        for (int j = 0; j < R; ++j)
                            if (vn != 0.0f)
                                red_add(A.table + w * rc + (int64_t)j * A.c + (hb[j][e] & P31),
                                        apply_sign(vn, hb[j][e]));
                    } else {
                        x[e] = __fadd_rn(x[e], vn);
                    }
                }
            }
        }
        if (MODE != INS_PER_WORKER) {
            if (MODE == INS_MERGED_GLOBAL && A.xsum != nullptr) {
                if (i0 + 3 < A.d) *reinterpret_cast<float4*>(A.xsum + i0) = make_float4(x[0], x[1], x[2], x[3]);
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
                        else red_add(A.table + (int64_t)j * A.c + (h1[e] & P31), sx);
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
                if (i0 + e < d && x[e] != 0.0f) red_add(table + (int64_t)j * c + (hb[e] & P31), apply_sign(x[e], hb[e]));
        }
    }
}

// ------------------------------------------------------------------------------------------------
// K2: merge of the per-worker tables, worker order
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
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

__global__ void __launch_bounds__(256)
k_quantize16(const float* __restrict__ x, uint16_t* __restrict__ q, int64_t n, int fmt) {
    const int64_t stride = (int64_t)gridDim.x * 256;
    for (int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x; t < n; t += stride) q[t] = quant16(__ldcs(x + t), fmt);
}

// merged[t] = sum over w = 0..W-1 (that order, fp32) of the decoded q[w][t]
__global__ void __launch_bounds__(256)
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
    if (gate_closed(A.sb.gate)) return;
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
__global__ void __launch_bounds__(SEL_THREADS)
k_emit_candidates(const float* __restrict__ est, int64_t d, SelBuffers sb, int32_t* __restrict__ cand_idx,
                  float* __restrict__ cand_est, uint32_t cap, int64_t nchunks) {
    sel_emit_chunks(est, d, sb, nchunks, [&](uint32_t slot, int64_t i) {
        if (slot >= cap) return;  // cannot happen with consistent histograms; never write past the list
        cand_idx[slot] = (int32_t)i;
        if (cand_est) cand_est[slot] = est[i];
    });
}

// ------------------------------------------------------------------------------------------------
// K5: second round -- xs[m] = sum_w v_w[cand[m]] (fp64, w = 0..W-1), rounded once to fp32
// ------------------------------------------------------------------------------------------------
#ifndef SSGD_GATHER_UNROLL
#define SSGD_GATHER_UNROLL 8
#endif
constexpr int GATHER_UNROLL = SSGD_GATHER_UNROLL;   // scattered loads in flight per thread

__global__ void __launch_bounds__(256)
k_gather(const int32_t* __restrict__ cand, int64_t ncand, const float* __restrict__ v, int64_t ld, int32_t W,
         int64_t d, float* __restrict__ xs, SelBuffers sb, uint32_t want, int32_t* __restrict__ errflag) {
    __shared__ SelShared sh;
    uint32_t* s_hist = sh.hist;
    pdl_trigger();
    for (int b = threadIdx.x; b < H1_BINS; b += 256) s_hist[b] = 0;
    pdl_wait();
    __syncthreads();
    const int64_t m = (int64_t)blockIdx.x * 256 + threadIdx.x;
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

// ------------------------------------------------------------------------------------------------
// final emit (line 11) and zero-out (line 13)
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(SEL_THREADS)
k_emit_final(const float* __restrict__ xs, int64_t ncand, SelBuffers sb, const int32_t* __restrict__ cand,
             int32_t* __restrict__ out_idx, float* __restrict__ out_val, uint32_t cap, int64_t nchunks) {
    sel_emit_chunks(xs, ncand, sb, nchunks, [&](uint32_t slot, int64_t m) {
        if (slot >= cap) return;
        out_idx[slot] = cand[m];
        out_val[slot] = xs[m];
    });
}

__global__ void __launch_bounds__(256)
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

// ==================================================================================================
// host side: context, argument checks, launch plans
// ==================================================================================================
using namespace ssgd;

struct ssgd_ctx {
    int64_t d, c, k;
    int32_t r, W;
    uint64_t seed;
    HashParams hp;
    Bucketizer bk;
    bool pow2;
    int32_t insert_mode;
    // binding
    float* u; float* v; int64_t ld;
    char* ws; size_t ws_bytes; int64_t ncand_max;
    // workspace layout (byte offsets)
    size_t off_table, off_hist_c, off_hist_f, off_state_c, off_state_f, off_err, zero_bytes;
    size_t off_sp_hist, off_sp_state, off_bitmap, off_list_idx, off_list_est;   // sparse candidate path
    int64_t list_cap;
    size_t off_hm;
    int32_t prune_mode;
    size_t persist_bytes;
    size_t split_bytes;     // > 0: ssgd_step inserts at most this many bytes of table rows per kernel   // > 0: launches that touch the table carry an L2 access-policy window of this size
    size_t off_est, off_chunk_c, off_chunk_f, off_cand, off_xs, off_oidx, off_oval, total_bytes;
    int64_t nchunk_c, nchunk_f;
    // device facts
    int device; int sm_count; int max_smem_optin;
    int kt_blocks_per_sm;   // residency of the bulk-copy pipeline kernel (0 = not queried yet)
    int ws_blocks_per_sm;   // same for the warp-specialised kernel
    int64_t launches;
    // optional per-stage timing of ssgd_step (CUDA events on the caller's stream)
    bool timing;
    cudaEvent_t* ev;        // [TIMING_SLOTS][SSGD_NSTAGES + 1]
    int32_t ev_steps;       // steps recorded since the last collection
    std::string last_error;
};

namespace {

constexpr size_t ALIGN = 256;
constexpr int TIMING_SLOTS = 256;
constexpr int EV_PER_STEP = SSGD_NSTAGES + 1;
inline size_t up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

void derive_params(uint64_t seed, int32_t r, HashParams& hp) {
    uint64_t s = seed;
    auto next = [&s]() -> uint64_t {
        s += 0x9E3779B97F4A7C15ull;
        uint64_t z = s;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
        return z ^ (z >> 31);
    };
    const uint64_t p = P31;
    for (int j = 0; j < r; ++j) {
        hp.row[j].a = (uint32_t)(1 + next() % (p - 1));
        hp.row[j].b = (uint32_t)(next() % p);
        hp.row[j].a2 = (uint32_t)(1 + next() % (p - 1));
        hp.row[j].b2 = (uint32_t)(next() % p);
    }
}

void layout(ssgd_ctx* x, int64_t ncand_max) {
    size_t o = 0;
    x->off_table = o;   o += up((size_t)x->r * x->c * 4);
    x->off_hist_c = o;  o += up(SEL_HIST_WORDS * 4);
    x->off_state_c = o; o += up(sizeof(SelState));
    x->off_hist_f = o;  o += up(SEL_HIST_WORDS * 4);
    x->off_state_f = o; o += up(sizeof(SelState));
    x->off_sp_hist = o; o += up(2 * H1_BINS * 4);
    x->off_sp_state = o; o += up(sizeof(SparseState));
    x->off_bitmap = o;  o += up((size_t)((x->d + 31) / 32) * 4);
    x->off_hm = o;      o += up(sizeof(HeavymixState));
    x->off_err = o;     o += up(16);
    x->zero_bytes = o;
    x->nchunk_c = (x->d + SEL_CHUNK - 1) / SEL_CHUNK;
    x->nchunk_f = (ncand_max + SEL_CHUNK - 1) / SEL_CHUNK;
    x->off_est = o;     o += up((size_t)x->d * 4);
    x->off_chunk_c = o; o += up((size_t)x->nchunk_c * 8);
    x->off_chunk_f = o; o += up((size_t)x->nchunk_f * 8);
    x->off_cand = o;    o += up((size_t)ncand_max * 4);
    x->off_xs = o;      o += up((size_t)ncand_max * 4);
    x->list_cap = 4 * ncand_max > 65536 ? 4 * ncand_max : 65536;
    if (x->list_cap > x->d) x->list_cap = x->d;
    x->off_list_idx = o; o += up((size_t)x->list_cap * 4);
    x->off_list_est = o; o += up((size_t)x->list_cap * 4);
    x->off_oidx = o;    o += up((size_t)x->k * 4);
    x->off_oval = o;    o += up((size_t)x->k * 4);
    x->total_bytes = o;
}

SelBuffers sel_buffers(ssgd_ctx* x, bool final_stage) {
    SelBuffers sb{};
    uint32_t* h = reinterpret_cast<uint32_t*>(x->ws + (final_stage ? x->off_hist_f : x->off_hist_c));
    sb.h1 = h; sb.h2 = h + H1_BINS; sb.h3 = h + H1_BINS + H2_BINS;
    sb.state = reinterpret_cast<SelState*>(x->ws + (final_stage ? x->off_state_f : x->off_state_c));
    uint32_t* ch = reinterpret_cast<uint32_t*>(x->ws + (final_stage ? x->off_chunk_f : x->off_chunk_c));
    const int64_t nch = final_stage ? x->nchunk_f : x->nchunk_c;
    sb.chunk_gt = ch; sb.chunk_eq = ch + nch;
    return sb;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int cuda_fail(ssgd_ctx* x, cudaError_t e, const char* what) {
    x->last_error = std::string(what) + ": " + cudaGetErrorString(e);
    return SSGD_ECUDA;
}

#define CU(call, what)                                                   \
    do {                                                                 \
        cudaError_t e_ = (call);                                         \
        if (e_ != cudaSuccess) return cuda_fail(x, e_, what);            \
    } while (0)

#define LAUNCHED(what)                                                   \
    do {                                                                 \
        x->launches++;                                                   \
        cudaError_t e_ = cudaGetLastError();                             \
        if (e_ != cudaSuccess) return cuda_fail(x, e_, what);            \
    } while (0)

int ensure_device(ssgd_ctx* x) {
    if (x->device >= 0) return SSGD_OK;
    int dev = 0;
    CU(cudaGetDevice(&dev), "cudaGetDevice");
    CU(cudaDeviceGetAttribute(&x->sm_count, cudaDevAttrMultiProcessorCount, dev), "sm count");
    CU(cudaDeviceGetAttribute(&x->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev), "smem optin");
    x->device = dev;
    return SSGD_OK;
}

// Launch with programmatic stream serialization: the kernel may become resident while its predecessor
// drains; it orders itself with pdl_wait().  SSGD_NO_PDL=1 in the environment turns the attribute off.
bool pdl_enabled() {
    static const bool on = [] { const char* e = std::getenv("SSGD_NO_PDL"); return !(e && e[0] == '1'); }();
    return on;
}

// An L2 access-policy window for one launch: accesses inside [base, base+bytes) are kept (persisting),
// everything else the kernel touches is treated as streaming.
struct L2Window { const void* base; size_t bytes; };

template <typename... P, typename... A>
cudaError_t launch_pdl_w(cudaStream_t st, L2Window win, void (*kern)(P...), int grid, int block, size_t smem, A... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    int n = 0;
    if (pdl_enabled()) {
        at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (win.base && win.bytes) {
        at[n].id = cudaLaunchAttributeAccessPolicyWindow;
        at[n].val.accessPolicyWindow.base_ptr = const_cast<void*>(win.base);
        at[n].val.accessPolicyWindow.num_bytes = win.bytes;
        at[n].val.accessPolicyWindow.hitRatio = 1.0f;
        at[n].val.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
        at[n].val.accessPolicyWindow.missProp = cudaAccessPropertyStreaming;
        ++n;
    }
    cfg.attrs = at;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kern, P(args)...);
}

template <typename... P, typename... A>
cudaError_t launch_pdl(cudaStream_t st, void (*kern)(P...), int grid, int block, size_t smem, A... args) {
    return launch_pdl_w(st, L2Window{nullptr, 0}, kern, grid, block, smem, args...);
}

inline int grid_for(int64_t items, int threads, int64_t cap) {
    int64_t b = (items + threads - 1) / threads;
    if (b < 1) b = 1;
    if (b > cap) b = cap;
    return (int)b;
}

// ---- K1 dispatch over (R, POW2, MODE) ------------------------------------------------------------
template <int R, bool POW2, int MODE>
int launch_accum_t(ssgd_ctx* x, const AccumArgs& A, cudaStream_t st) {
    const int64_t groups = (A.d + 3) / 4;
    if (MODE == INS_MERGED_SMEM) {
        const size_t smem = (size_t)R * A.c * 4;
        CU(cudaFuncSetAttribute(k_accum_insert<R, POW2, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)smem), "smem attribute");
        const int grid = grid_for(groups, K1_THREADS, x->sm_count);
        k_accum_insert<R, POW2, MODE><<<grid, K1_THREADS, smem, st>>>(A);
    } else {
        const int grid = grid_for(groups, K1_THREADS, (int64_t)1 << 30);
        CU(launch_pdl_w(st, L2Window{MODE == INS_MERGED_GLOBAL ? A.table : nullptr, x->persist_bytes},
                        k_accum_insert<R, POW2, MODE>, grid, K1_THREADS, 0, A), "launch k_accum_insert");
    }
    LAUNCHED("k_accum_insert");
    return SSGD_OK;
}

template <int R, bool POW2>
int launch_accum_m(ssgd_ctx* x, const AccumArgs& A, int mode, cudaStream_t st) {
    switch (mode) {
        case INS_MERGED_GLOBAL: return launch_accum_t<R, POW2, INS_MERGED_GLOBAL>(x, A, st);
        case INS_PER_WORKER: return launch_accum_t<R, POW2, INS_PER_WORKER>(x, A, st);
        default: return launch_accum_t<R, POW2, INS_MERGED_SMEM>(x, A, st);
    }
}

#ifdef SSGD_EXP_ONLY_R5
#define DISPATCH_R(fn, ...)                                                       \
    if (x->r == 5 && x->pow2) return fn<5, true>(__VA_ARGS__);                    \
    return SSGD_EINVAL;
#else
#define DISPATCH_R(fn, ...)                                                       \
    switch (x->r) {                                                               \
        case 1: return x->pow2 ? fn<1, true>(__VA_ARGS__) : fn<1, false>(__VA_ARGS__);    \
        case 3: return x->pow2 ? fn<3, true>(__VA_ARGS__) : fn<3, false>(__VA_ARGS__);    \
        case 5: return x->pow2 ? fn<5, true>(__VA_ARGS__) : fn<5, false>(__VA_ARGS__);    \
        case 7: return x->pow2 ? fn<7, true>(__VA_ARGS__) : fn<7, false>(__VA_ARGS__);    \
        case 9: return x->pow2 ? fn<9, true>(__VA_ARGS__) : fn<9, false>(__VA_ARGS__);    \
        case 11: return x->pow2 ? fn<11, true>(__VA_ARGS__) : fn<11, false>(__VA_ARGS__); \
        case 13: return x->pow2 ? fn<13, true>(__VA_ARGS__) : fn<13, false>(__VA_ARGS__); \
        case 15: return x->pow2 ? fn<15, true>(__VA_ARGS__) : fn<15, false>(__VA_ARGS__); \
        default: return SSGD_EINVAL;                                              \
    }
#endif

int launch_accum(ssgd_ctx* x, const AccumArgs& A, int mode, cudaStream_t st) {
    DISPATCH_R(launch_accum_m, x, A, mode, st)
}

template <int R, bool POW2>
int launch_accum_tma_t(ssgd_ctx* x, const AccumArgs& A, cudaStream_t st) {
    auto kern = k_accum_insert_tma<R, POW2>;
    const size_t smem = sizeof(KtShared);
    if (x->kt_blocks_per_sm == 0) {
        CU(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem), "smem attribute");
        int nb = 0;
        CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kern, KT_THREADS, smem), "occupancy query");
        x->kt_blocks_per_sm = nb < 1 ? 1 : nb;
    }
    const int64_t ntiles = ((A.d & ~(int64_t)3) + KT_TC - 1) / KT_TC;
    const int grid = grid_for(ntiles, 1, (int64_t)x->sm_count * x->kt_blocks_per_sm);
    CU(launch_pdl_w(st, L2Window{A.table, x->persist_bytes}, kern, grid, KT_THREADS, smem, A,
                    reinterpret_cast<int32_t*>(x->ws + x->off_err)), "launch k_accum_insert_tma");
    LAUNCHED("k_accum_insert_tma");
    return SSGD_OK;
}

int launch_accum_tma(ssgd_ctx* x, const AccumArgs& A, cudaStream_t st) {
    DISPATCH_R(launch_accum_tma_t, x, A, st)
}

template <int R, bool POW2>
int launch_insert_rows_t(ssgd_ctx* x, const float* xsum, float* table, int lo, int hi, cudaStream_t st) {
    const int64_t groups = (x->d + 3) / 4;
    CU(launch_pdl(st, k_insert_rows<R, POW2>, grid_for(groups, 256, (int64_t)x->sm_count * 8), 256, 0, xsum, x->d, table, x->c,
                  x->hp, x->bk, lo, hi), "launch k_insert_rows");
    LAUNCHED("k_insert_rows");
    return SSGD_OK;
}

int launch_insert_rows(ssgd_ctx* x, const float* xsum, float* table, int lo, int hi, cudaStream_t st) {
    DISPATCH_R(launch_insert_rows_t, x, xsum, table, lo, hi, st)
}

template <int R, bool POW2>
int launch_accum_ws_t(ssgd_ctx* x, const AccumArgs& A, cudaStream_t st) {
    auto kern = k_accum_insert_ws<R, POW2>;
    const size_t smem = sizeof(WsShared);
    if (x->ws_blocks_per_sm == 0) {
        CU(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem), "smem attribute");
        int nb = 0;
        CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kern, WS_THREADS, smem), "occupancy query");
        x->ws_blocks_per_sm = nb < 1 ? 1 : nb;
    }
    const int64_t ntiles = ((A.d & ~(int64_t)3) + WS_TC - 1) / WS_TC;
    const int grid = grid_for(ntiles, 1, (int64_t)x->sm_count * x->ws_blocks_per_sm);
    CU(launch_pdl_w(st, L2Window{A.table, x->persist_bytes}, kern, grid, WS_THREADS, smem, A,
                    reinterpret_cast<int32_t*>(x->ws + x->off_err)), "launch k_accum_insert_ws");
    LAUNCHED("k_accum_insert_ws");
    return SSGD_OK;
}

int launch_accum_ws(ssgd_ctx* x, const AccumArgs& A, cudaStream_t st) {
    DISPATCH_R(launch_accum_ws_t, x, A, st)
}

template <int R, bool POW2>
int launch_unsketch_t(ssgd_ctx* x, const UnsketchArgs& A, cudaStream_t st) {
    const int64_t groups = (A.d + K3_NC - 1) / K3_NC;
    // a few blocks per SM: each block pays one histogram flush
    const int grid = grid_for(groups, K3_THREADS, (int64_t)x->sm_count * SSGD_K3_GRID);
    CU(launch_pdl(st, k_unsketch<R, POW2>, grid, K3_THREADS, 0, A), "launch k_unsketch");
    LAUNCHED("k_unsketch");
    return SSGD_OK;
}

int launch_unsketch(ssgd_ctx* x, const UnsketchArgs& A, cudaStream_t st) {
    DISPATCH_R(launch_unsketch_t, x, A, st)
}

// Radix-select passes after the producer filled H1: leaves thresholds in sb.state and exclusive
// chunk offsets in sb.chunk_*; the caller launches the emit kernel over `nchunks` blocks.
int launch_select(ssgd_ctx* x, const float* val, int64_t n, const SelBuffers& sb, int64_t nchunks,
                  cudaStream_t st) {
    const int grid = grid_for(n, SEL_THREADS * 8, (int64_t)x->sm_count * 8);
    CU(launch_pdl(st, k_sel_pass2, grid, SEL_THREADS, 0, val, n, sb), "launch k_sel_pass2");
    LAUNCHED("k_sel_pass2");
    CU(launch_pdl(st, k_sel_pass3, grid, SEL_THREADS, 0, val, n, sb), "launch k_sel_pass3");
    LAUNCHED("k_sel_pass3");
    CU(launch_pdl(st, k_sel_count, grid_for(nchunks, 1, (int64_t)x->sm_count * 8), SEL_THREADS, 0, val, n, sb, nchunks),
       "launch k_sel_count");
    LAUNCHED("k_sel_count");
    return SSGD_OK;
}

int check_bound(const ssgd_ctx* x) {
    if (!x) return SSGD_EINVAL;
    if (!x->u || !x->v || !x->ws) return SSGD_ENOTBOUND;
    return SSGD_OK;
}

int check_g(const ssgd_ctx* x, const float* g, int64_t ld_g) {
    if (!g || ld_g < x->d) return SSGD_EINVAL;
    if (!aligned16(g) || (ld_g & 3)) return SSGD_EALIGN;
    return SSGD_OK;
}

// Stage boundary `which` of the step being recorded (no-op unless timing is on and a slot is free).
int mark(ssgd_ctx* x, int which, cudaStream_t st) {
    if (!x->timing || x->ev_steps >= TIMING_SLOTS) return SSGD_OK;
    CU(cudaEventRecord(x->ev[x->ev_steps * EV_PER_STEP + which], st), "event record");
    return SSGD_OK;
}

int unsketch_select(ssgd_ctx* x, const float* merged, int64_t ncand, int32_t* cand_idx, float* cand_est,
                    float* est, cudaStream_t st, bool timed = false, const uint32_t* gate = nullptr) {
    UnsketchArgs A;
    A.table = merged; A.c = x->c; A.d = x->d; A.hp = x->hp; A.bk = x->bk; A.est = est;
    SelBuffers sb = sel_buffers(x, false);
    sb.gate = gate;
    A.sb = sb; A.want = (uint32_t)ncand;
    int e = launch_unsketch(x, A, st);
    if (e) return e;
    if (timed && (e = mark(x, 2, st))) return e;
    if ((e = launch_select(x, est, x->d, sb, x->nchunk_c, st))) return e;
    CU(launch_pdl(st, k_emit_candidates, grid_for(x->nchunk_c, 1, (int64_t)x->sm_count * 8), SEL_THREADS, 0, (const float*)est,
                  x->d, sb, cand_idx, cand_est, (uint32_t)ncand, x->nchunk_c), "launch k_emit_candidates");
    LAUNCHED("k_emit_candidates");
    return SSGD_OK;
}

SparseBuffers sparse_buffers(ssgd_ctx* x) {
    SparseBuffers sp{};
    uint32_t* h = reinterpret_cast<uint32_t*>(x->ws + x->off_sp_hist);
    sp.h1_sample = h; sp.h1 = h + H1_BINS;
    sp.state = reinterpret_cast<SparseState*>(x->ws + x->off_sp_state);
    sp.list_idx = reinterpret_cast<int32_t*>(x->ws + x->off_list_idx);
    sp.list_est = reinterpret_cast<float*>(x->ws + x->off_list_est);
    sp.cap = (uint32_t)x->list_cap;
    sp.bitmap = reinterpret_cast<uint32_t*>(x->ws + x->off_bitmap);
    return sp;
}

// Whether ssgd_step takes the early-exit unsketch + sparse selection (sparse_select.cuh).
bool use_sparse(const ssgd_ctx* x, int64_t ncand) {
    if (x->prune_mode == SSGD_PRUNE_OFF) return false;
    if (x->prune_mode == SSGD_PRUNE_ON) return true;
    // measured at C2's shape: the early exit saves 25-45 us for r = 5, 7, 9 and costs 34 us for r = 3 (only one
    // row can be skipped); at r = 15 with ncand = 1.6e6 the dense kernel is faster (4.78 vs 5.72 ms)
    return x->r >= 5 && x->r <= 9 && x->d >= (1 << 22) && ncand * 8 <= x->d;
}

template <int R, bool POW2>
int launch_sparse_t(ssgd_ctx* x, const SparseArgs& A, cudaStream_t st) {
    const int64_t groups = (A.d + 3) / 4;
    const int64_t windows = (groups + (1 << SPARSE_SAMPLE_SHIFT) - 1) >> SPARSE_SAMPLE_SHIFT;
    CU(launch_pdl(st, k_unsketch_sample<R, POW2>, grid_for(windows, SEL_THREADS, (int64_t)x->sm_count), SEL_THREADS, 0, A),
       "launch k_unsketch_sample");
    LAUNCHED("k_unsketch_sample");
    CU(launch_pdl(st, k_unsketch_pruned<R, POW2>,
                  grid_for((A.d + SSGD_PRUNED_NC - 1) / SSGD_PRUNED_NC, SEL_THREADS, (int64_t)x->sm_count * SSGD_PRUNED_GRID), SEL_THREADS, 0, A),
       "launch k_unsketch_pruned");
    LAUNCHED("k_unsketch_pruned");
    return SSGD_OK;
}

int launch_sparse(ssgd_ctx* x, const SparseArgs& A, cudaStream_t st) {
    DISPATCH_R(launch_sparse_t, x, A, st)
}

int launch_select_sparse(ssgd_ctx* x, const SparseBuffers& sp, int64_t ncand, int32_t* cand_idx, cudaStream_t st) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(SPARSE_CLUSTER);
    cfg.blockDim = dim3(SPARSE_THREADS);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = SPARSE_CLUSTER; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl_enabled() ? 2 : 1;
    CU(cudaLaunchKernelEx(&cfg, k_select_sparse, sp, x->d, (uint32_t)ncand, cand_idx), "launch k_select_sparse");
    LAUNCHED("k_select_sparse");
    return SSGD_OK;
}

// Line 9 with early exit: sample -> pruned unsketch -> cluster selection; the dense path follows, gated.
int unsketch_select_sparse(ssgd_ctx* x, const float* merged, int64_t ncand, int32_t* cand_idx, float* est,
                           cudaStream_t st) {
    SparseArgs A;
    A.table = merged; A.c = x->c; A.d = x->d; A.hp = x->hp; A.bk = x->bk;
    A.sp = sparse_buffers(x);
    A.ncand = (uint32_t)ncand;
    const int64_t groups = (x->d + 3) / 4;
    const int64_t windows = (groups + (1 << SPARSE_SAMPLE_SHIFT) - 1) >> SPARSE_SAMPLE_SHIFT;
    const double mean = (double)ncand * (double)(windows * 4) / (double)x->d;
    A.want_sample = (uint32_t)(mean + 6.0 * std::sqrt(mean) + 16.0 + 1.0);
    int e = launch_sparse(x, A, st);
    if (e) return e;
    if ((e = mark(x, 2, st))) return e;
    if ((e = launch_select_sparse(x, A.sp, ncand, cand_idx, st))) return e;
    return unsketch_select(x, merged, ncand, cand_idx, nullptr, est, st, false, &A.sp.state->fallback);
}

int gather_select_zero(ssgd_ctx* x, const int32_t* cand, int64_t ncand, int32_t* out_idx, float* out_val,
                       cudaStream_t st) {
    float* xs = reinterpret_cast<float*>(x->ws + x->off_xs);
    int32_t* err = reinterpret_cast<int32_t*>(x->ws + x->off_err);
    SelBuffers sb = sel_buffers(x, true);
    const int64_t nch = (ncand + SEL_CHUNK - 1) / SEL_CHUNK;
    CU(launch_pdl(st, k_gather, grid_for(ncand, 256, (int64_t)1 << 30), 256, 0, cand, ncand, (const float*)x->v, x->ld, x->W,
                  x->d, xs, sb, (uint32_t)x->k, err), "launch k_gather");
    LAUNCHED("k_gather");
    int e = launch_select(x, xs, ncand, sb, nch, st);
    if (e) return e;
    CU(launch_pdl(st, k_emit_final, grid_for(nch, 1, (int64_t)x->sm_count * 8), SEL_THREADS, 0, (const float*)xs, ncand, sb,
                  cand, out_idx, out_val, (uint32_t)x->k, nch), "launch k_emit_final");
    LAUNCHED("k_emit_final");
    CU(launch_pdl(st, k_zero, grid_for(x->k * (int64_t)x->W, 256, (int64_t)x->sm_count * 16), 256, 0, (const int32_t*)out_idx,
                  x->k, x->u, x->v, x->ld, x->W, x->d), "launch k_zero");
    LAUNCHED("k_zero");
    return SSGD_OK;
}

int resolve_insert_mode(const ssgd_ctx* x) {
    const size_t table_bytes = (size_t)x->r * x->c * 4;
    const bool fits = table_bytes <= (size_t)200 * 1024 && (int64_t)table_bytes <= x->max_smem_optin;
    if (x->insert_mode == SSGD_INSERT_SMEM) return fits ? INS_MERGED_SMEM : -1;
    if (x->insert_mode == SSGD_INSERT_GLOBAL) return INS_MERGED_GLOBAL;
    if (x->insert_mode == SSGD_INSERT_TMA) return INS_MERGED_TMA;
    if (x->insert_mode == SSGD_INSERT_WS) return INS_MERGED_WS;
    // measured on B200: the bulk-copy pipeline wins once a tile's walk over the workers is long
    // (W = 128: 5.73 vs 5.43 TB/s), plain loads win for short walks (W = 16: 4.93 vs 4.83 TB/s)
    return x->W >= 64 ? INS_MERGED_TMA : INS_MERGED_GLOBAL;
}

template <int R, bool POW2>
int launch_heavymix_keys_t(ssgd_ctx* x, const HeavymixArgs& A, cudaStream_t st) {
    const int64_t groups = (A.d + 3) / 4;
    k_heavymix_keys<R, POW2><<<grid_for(groups, SEL_THREADS, (int64_t)x->sm_count * 4), SEL_THREADS, 0, st>>>(A);
    LAUNCHED("k_heavymix_keys");
    return SSGD_OK;
}

int launch_heavymix_keys(ssgd_ctx* x, const HeavymixArgs& A, cudaStream_t st) {
    DISPATCH_R(launch_heavymix_keys_t, x, A, st)
}

}  // namespace

extern "C" {

int ssgd_create(ssgd_ctx** out, int64_t d, int32_t r, int64_t c, int64_t k, int32_t W, uint64_t seed) {
    if (!out) return SSGD_EINVAL;
    *out = nullptr;
    if (d < 1 || d >= (int64_t)P31) return SSGD_EINVAL;
    if (r < 1 || r > SSGD_MAX_R || (r % 2) == 0) return SSGD_EINVAL;
    if (c < 1 || c >= (int64_t)P31) return SSGD_EINVAL;
    if (k < 1 || k > d || W < 1) return SSGD_EINVAL;
    ssgd_ctx* x = new (std::nothrow) ssgd_ctx();
    if (!x) return SSGD_ENOMEM;
    x->d = d; x->r = r; x->c = c; x->k = k; x->W = W; x->seed = seed;
    std::memset(&x->hp, 0, sizeof(x->hp));
    derive_params(seed, r, x->hp);
    x->bk = make_bucketizer((uint64_t)c);
    x->pow2 = (c & (c - 1)) == 0;
    x->insert_mode = SSGD_INSERT_AUTO;
    x->u = x->v = nullptr; x->ws = nullptr; x->ld = 0; x->ws_bytes = 0; x->ncand_max = 0;
    x->device = -1; x->sm_count = 0; x->max_smem_optin = 0; x->launches = 0; x->kt_blocks_per_sm = 0; x->ws_blocks_per_sm = 0;
    x->timing = false; x->ev = nullptr; x->ev_steps = 0; x->prune_mode = SSGD_PRUNE_AUTO; x->list_cap = 0; x->persist_bytes = 0; x->split_bytes = SSGD_SPLIT_BYTES_DEFAULT;
    *out = x;
    return SSGD_OK;
}

int ssgd_destroy(ssgd_ctx* ctx) {
    if (ctx && ctx->ev) {
        for (int i = 0; i < TIMING_SLOTS * EV_PER_STEP; ++i) cudaEventDestroy(ctx->ev[i]);
        delete[] ctx->ev;
    }
    delete ctx;
    return SSGD_OK;
}

int ssgd_get_hash_params(const ssgd_ctx* x, uint32_t* out4r) {
    if (!x || !out4r) return SSGD_EINVAL;
    for (int j = 0; j < x->r; ++j) {
        out4r[4 * j] = x->hp.row[j].a; out4r[4 * j + 1] = x->hp.row[j].b;
        out4r[4 * j + 2] = x->hp.row[j].a2; out4r[4 * j + 3] = x->hp.row[j].b2;
    }
    return SSGD_OK;
}

int ssgd_set_hash_params(ssgd_ctx* x, const uint32_t* in4r) {
    if (!x || !in4r) return SSGD_EINVAL;
    for (int j = 0; j < x->r; ++j) {
        if (in4r[4 * j] < 1 || in4r[4 * j] >= P31 || in4r[4 * j + 1] >= P31) return SSGD_EINVAL;
        if (in4r[4 * j + 2] < 1 || in4r[4 * j + 2] >= P31 || in4r[4 * j + 3] >= P31) return SSGD_EINVAL;
    }
    for (int j = 0; j < x->r; ++j) {
        x->hp.row[j].a = in4r[4 * j]; x->hp.row[j].b = in4r[4 * j + 1];
        x->hp.row[j].a2 = in4r[4 * j + 2]; x->hp.row[j].b2 = in4r[4 * j + 3];
    }
    return SSGD_OK;
}

int ssgd_set_table_persistence(ssgd_ctx* x, int32_t enable) {
    if (!x) return SSGD_EINVAL;
    x->persist_bytes = 0;
    if (!enable) return SSGD_OK;
    int e = ensure_device(x);
    if (e) return e;
    int max_persist = 0, max_window = 0;
    CU(cudaDeviceGetAttribute(&max_persist, cudaDevAttrMaxPersistingL2CacheSize, x->device), "persisting L2 size");
    CU(cudaDeviceGetAttribute(&max_window, cudaDevAttrMaxAccessPolicyWindowSize, x->device), "access window size");
    size_t want = (size_t)x->r * x->c * 4;
    if (want > (size_t)max_window) want = (size_t)max_window;
    size_t carve = want < (size_t)max_persist ? want : (size_t)max_persist;
    if (carve == 0) return SSGD_OK;
    CU(cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, carve), "set persisting L2 size");
    x->persist_bytes = want;
    return SSGD_OK;
}

int ssgd_set_insert_split(ssgd_ctx* x, int64_t bytes) {
    if (!x || bytes < 0) return SSGD_EINVAL;
    x->split_bytes = (size_t)bytes;
    return SSGD_OK;
}

int ssgd_set_prune_mode(ssgd_ctx* x, int32_t mode) {
    if (!x || mode < SSGD_PRUNE_AUTO || mode > SSGD_PRUNE_ON) return SSGD_EINVAL;
    x->prune_mode = mode;
    return SSGD_OK;
}

int ssgd_step_used_fallback(ssgd_ctx* x, void* stream, int32_t* out) {
    int e = check_bound(x);
    if (e) return e;
    if (!out) return SSGD_EINVAL;
    CU(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)), "stream synchronize");
    SparseState s;
    CU(cudaMemcpy(&s, x->ws + x->off_sp_state, sizeof(s), cudaMemcpyDeviceToHost), "read sparse state");
    out[0] = (int32_t)s.fallback; out[1] = (int32_t)s.n_surv; out[2] = (int32_t)s.bin_lo;
    return SSGD_OK;
}

int ssgd_set_insert_mode(ssgd_ctx* x, int32_t mode) {
    if (!x || mode < SSGD_INSERT_AUTO || mode > SSGD_INSERT_WS) return SSGD_EINVAL;
    x->insert_mode = mode;
    return SSGD_OK;
}

int ssgd_workspace_bytes(const ssgd_ctx* x, int64_t ncand_max, size_t* out_bytes) {
    if (!x || !out_bytes || ncand_max < x->k || ncand_max > x->d) return SSGD_EINVAL;
    ssgd_ctx tmp = *x;
    layout(&tmp, ncand_max);
    *out_bytes = tmp.total_bytes;
    return SSGD_OK;
}

int ssgd_bind(ssgd_ctx* x, float* u, float* v, int64_t ld, void* workspace, size_t workspace_bytes,
              int64_t ncand_max) {
    if (!x || !u || !v || !workspace || ld < x->d) return SSGD_EINVAL;
    if (ncand_max < x->k || ncand_max > x->d) return SSGD_EINVAL;
    if (!aligned16(u) || !aligned16(v) || (ld & 3)) return SSGD_EALIGN;
    if (reinterpret_cast<uintptr_t>(workspace) % ALIGN) return SSGD_EALIGN;
    layout(x, ncand_max);
    if (workspace_bytes < x->total_bytes) return SSGD_EWORKSPACE;
    x->u = u; x->v = v; x->ld = ld;
    x->ws = static_cast<char*>(workspace); x->ws_bytes = workspace_bytes; x->ncand_max = ncand_max;
    int e = ensure_device(x);
    if (e) return e;
    CU(cudaMemset(x->ws + x->off_err, 0, 16), "clear error flag");
    return SSGD_OK;
}

int ssgd_sketch_accumulate(ssgd_ctx* x, const float* g, int64_t ld_g, float rho, float* tables, void* stream) {
    int e = check_bound(x);
    if (e) return e;
    if ((e = check_g(x, g, ld_g))) return e;
    if (!tables) return SSGD_EINVAL;
    if ((e = ensure_device(x))) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CU(cudaMemsetAsync(tables, 0, (size_t)x->W * x->r * x->c * 4, st), "memset tables");
    x->launches++;
    AccumArgs A;
    A.g = g; A.ld_g = ld_g; A.u = x->u; A.v = x->v; A.ld = x->ld; A.W = x->W; A.d = x->d; A.rho = rho;
    A.table = tables; A.c = x->c; A.hp = x->hp; A.bk = x->bk; A.rows_here = x->r; A.xsum = nullptr;
    return launch_accum(x, A, INS_PER_WORKER, st);
}

int ssgd_sketch_merge(ssgd_ctx* x, const float* tables, float* merged, void* stream) {
    if (!x || !tables || !merged) return SSGD_EINVAL;
    const int64_t rc = (int64_t)x->r * x->c;
    if ((rc & 3) == 0 && (!aligned16(tables) || !aligned16(merged))) return SSGD_EALIGN;
    int e = ensure_device(x);
    if (e) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    k_merge<<<grid_for((rc + 3) / 4, 256, (int64_t)x->sm_count * 16), 256, 0, st>>>(tables, merged, rc, x->W);
    LAUNCHED("k_merge");
    return SSGD_OK;
}

int ssgd_sketch_quantize16(ssgd_ctx* x, const float* tables, int32_t fmt, uint16_t* q16, void* stream) {
    if (!x || !tables || !q16 || (fmt != SSGD_FMT_F16 && fmt != SSGD_FMT_BF16)) return SSGD_EINVAL;
    int e = ensure_device(x);
    if (e) return e;
    const int64_t n = (int64_t)x->W * x->r * x->c;
    k_quantize16<<<grid_for(n, 256, (int64_t)x->sm_count * 16), 256, 0, static_cast<cudaStream_t>(stream)>>>(tables, q16, n, fmt);
    LAUNCHED("k_quantize16");
    return SSGD_OK;
}

int ssgd_sketch_merge16(ssgd_ctx* x, const uint16_t* q16, int32_t fmt, float* merged, void* stream) {
    if (!x || !q16 || !merged || (fmt != SSGD_FMT_F16 && fmt != SSGD_FMT_BF16)) return SSGD_EINVAL;
    int e = ensure_device(x);
    if (e) return e;
    const int64_t n = (int64_t)x->r * x->c;
    k_merge16<<<grid_for(n, 256, (int64_t)x->sm_count * 16), 256, 0, static_cast<cudaStream_t>(stream)>>>(q16, merged, n, x->W, fmt);
    LAUNCHED("k_merge16");
    return SSGD_OK;
}

int ssgd_unsketch_candidates(ssgd_ctx* x, const float* merged, int64_t ncand, int32_t* cand_idx,
                             float* cand_est, float* est_all, void* stream) {
    int e = check_bound(x);
    if (e) return e;
    if (!merged || !cand_idx || ncand < x->k || ncand > x->d) return SSGD_EINVAL;
    if (est_all && !aligned16(est_all)) return SSGD_EALIGN;
    if ((e = ensure_device(x))) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CU(cudaMemsetAsync(x->ws + x->off_hist_c, 0, x->off_hist_f - x->off_hist_c, st), "memset hist");
    x->launches++;
    float* est = est_all ? est_all : reinterpret_cast<float*>(x->ws + x->off_est);
    return unsketch_select(x, merged, ncand, cand_idx, cand_est, est, st);
}

int ssgd_exact_topk(ssgd_ctx* x, const int32_t* cand_idx, int64_t ncand, int32_t* out_idx, float* out_val,
                    void* stream) {
    int e = check_bound(x);
    if (e) return e;
    if (!cand_idx || !out_idx || !out_val || ncand < x->k || ncand > x->d) return SSGD_EINVAL;
    if (ncand > x->ncand_max) return SSGD_EWORKSPACE;
    if ((e = ensure_device(x))) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CU(cudaMemsetAsync(x->ws + x->off_hist_f, 0, x->off_err - x->off_hist_f, st), "memset hist");
    x->launches++;
    return gather_select_zero(x, cand_idx, ncand, out_idx, out_val, st);
}

int ssgd_step(ssgd_ctx* x, const float* g, int64_t ld_g, float rho, int64_t ncand, int32_t* out_idx,
              float* out_val, void* stream) {
    int e = check_bound(x);
    if (e) return e;
    if ((e = check_g(x, g, ld_g))) return e;
    if (!out_idx || !out_val || ncand < x->k || ncand > x->d) return SSGD_EINVAL;
    if (ncand > x->ncand_max) return SSGD_EWORKSPACE;
    if ((e = ensure_device(x))) return e;
    const int mode = resolve_insert_mode(x);
    if (mode < 0) return SSGD_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // table, histograms, selection state: one memset (the error flag is sticky until ssgd_status)
    CU(cudaMemsetAsync(x->ws, 0, x->off_err, st), "memset workspace head");
    x->launches++;
    float* merged = reinterpret_cast<float*>(x->ws + x->off_table);
    AccumArgs A;
    A.g = g; A.ld_g = ld_g; A.u = x->u; A.v = x->v; A.ld = x->ld; A.W = x->W; A.d = x->d; A.rho = rho;
    A.table = merged; A.c = x->c; A.hp = x->hp; A.bk = x->bk; A.rows_here = x->r; A.xsum = nullptr;
    // a table that cannot stay in L2 next to the stream is inserted a slice of rows at a time
    const size_t row_bytes = (size_t)x->c * 4;
    const int rows_fit = (int)(x->split_bytes / row_bytes);
    const bool split = mode == INS_MERGED_GLOBAL && x->split_bytes > 0 && rows_fit >= 1 && rows_fit < x->r;
    if (split) { A.rows_here = rows_fit; A.xsum = reinterpret_cast<float*>(x->ws + x->off_est); }
    if ((e = mark(x, 0, st))) return e;
    if ((e = mode == INS_MERGED_TMA ? launch_accum_tma(x, A, st)
             : mode == INS_MERGED_WS ? launch_accum_ws(x, A, st) : launch_accum(x, A, mode, st))) return e;
    if (split)
        for (int lo = rows_fit; lo < x->r; lo += rows_fit)
            if ((e = launch_insert_rows(x, A.xsum, merged, lo, lo + rows_fit < x->r ? lo + rows_fit : x->r, st))) return e;
    if ((e = mark(x, 1, st))) return e;
    int32_t* cand = reinterpret_cast<int32_t*>(x->ws + x->off_cand);
    float* est = reinterpret_cast<float*>(x->ws + x->off_est);
    if (use_sparse(x, ncand)) {
        if ((e = unsketch_select_sparse(x, merged, ncand, cand, est, st))) return e;
    } else {
        if ((e = unsketch_select(x, merged, ncand, cand, nullptr, est, st, true))) return e;
    }
    if ((e = mark(x, 3, st))) return e;
    if ((e = gather_select_zero(x, cand, ncand, out_idx, out_val, st))) return e;
    if ((e = mark(x, 4, st))) return e;
    if (x->timing && x->ev_steps < TIMING_SLOTS) x->ev_steps++;
    return SSGD_OK;
}

int ssgd_set_timing(ssgd_ctx* x, int32_t enable) {
    if (!x) return SSGD_EINVAL;
    if (enable && !x->ev) {
        x->ev = new (std::nothrow) cudaEvent_t[TIMING_SLOTS * EV_PER_STEP];
        if (!x->ev) return SSGD_ENOMEM;
        for (int i = 0; i < TIMING_SLOTS * EV_PER_STEP; ++i) CU(cudaEventCreate(&x->ev[i]), "event create");
    }
    x->timing = enable != 0;
    x->ev_steps = 0;
    return SSGD_OK;
}

int ssgd_get_stage_times(ssgd_ctx* x, void* stream, double* ms_out, int64_t* steps_out) {
    if (!x || !ms_out || !steps_out) return SSGD_EINVAL;
    CU(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)), "stream synchronize");
    for (int sgi = 0; sgi < SSGD_NSTAGES; ++sgi) ms_out[sgi] = 0.0;
    for (int t = 0; t < x->ev_steps; ++t)
        for (int sgi = 0; sgi < SSGD_NSTAGES; ++sgi) {
            float ms = 0.f;
            CU(cudaEventElapsedTime(&ms, x->ev[t * EV_PER_STEP + sgi], x->ev[t * EV_PER_STEP + sgi + 1]), "event elapsed");
            ms_out[sgi] += ms;
        }
    *steps_out = x->ev_steps;
    x->ev_steps = 0;
    return SSGD_OK;
}

int ssgd_heavymix(ssgd_ctx* x, const float* merged, uint64_t fill_seed, int32_t* out_idx, float* out_val,
                  double* l2_out, int32_t* nheavy_out, void* stream) {
    int e = check_bound(x);
    if (e) return e;
    if (!merged || !out_idx || !out_val) return SSGD_EINVAL;
    if ((e = ensure_device(x))) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // histograms + state of the candidate selection, and the HEAVYMIX state
    CU(cudaMemsetAsync(x->ws + x->off_hist_c, 0, x->off_hist_f - x->off_hist_c, st), "memset hist");
    CU(cudaMemsetAsync(x->ws + x->off_hist_f, 0, x->off_sp_hist - x->off_hist_f, st), "memset hist");
    CU(cudaMemsetAsync(x->ws + x->off_hm, 0, sizeof(HeavymixState), st), "memset heavymix state");
    x->launches += 3;
    HeavymixArgs A;
    A.table = merged; A.c = x->c; A.d = x->d; A.r = x->r; A.hp = x->hp; A.bk = x->bk;
    A.hm = reinterpret_cast<HeavymixState*>(x->ws + x->off_hm);
    A.keys = reinterpret_cast<float*>(x->ws + x->off_est);
    A.sb = sel_buffers(x, false);
    A.k = (uint32_t)x->k;
    A.fill_seed = fill_seed;
    dim3 grid((unsigned)grid_for(x->c, 256, x->sm_count * 2), (unsigned)x->r);
    k_row_sumsq<<<grid, 256, 0, st>>>(merged, x->c, A.hm);
    LAUNCHED("k_row_sumsq");
    if ((e = launch_heavymix_keys(x, A, st))) return e;
    if ((e = launch_select(x, A.keys, x->d, A.sb, x->nchunk_c, st))) return e;
    CU(launch_pdl(st, k_emit_candidates, grid_for(x->nchunk_c, 1, (int64_t)x->sm_count * 8), SEL_THREADS, 0, (const float*)A.keys,
                  x->d, A.sb, out_idx, (float*)nullptr, (uint32_t)x->k, x->nchunk_c), "launch k_emit_candidates");
    LAUNCHED("k_emit_candidates");
    // line 5: exact values of the chosen coordinates, summed over the workers
    SelBuffers sf = sel_buffers(x, true);
    CU(launch_pdl(st, k_gather, grid_for(x->k, 256, (int64_t)1 << 30), 256, 0, (const int32_t*)out_idx, x->k, (const float*)x->v,
                  x->ld, x->W, x->d, out_val, sf, (uint32_t)1, reinterpret_cast<int32_t*>(x->ws + x->off_err)),
       "launch k_gather");
    LAUNCHED("k_gather");
    if (l2_out || nheavy_out) {
        // l2 = median of the row sums: computed on the host side of the copy-out by the caller would need a
        // sync; instead one thread writes both results
        k_heavymix_report<<<1, 32, 0, st>>>(A.hm, x->r, l2_out, nheavy_out);
        LAUNCHED("k_heavymix_report");
    }
    return SSGD_OK;
}

int ssgd_step_host(ssgd_ctx* x, const float* g_host, int64_t ld_g, float rho, int64_t ncand, float* g_stage,
                   int32_t* out_idx_host, float* out_val_host, void* stream) {
    int e = check_bound(x);
    if (e) return e;
    if (!g_host || !g_stage || !out_idx_host || !out_val_host) return SSGD_EINVAL;
    if ((e = check_g(x, g_stage, ld_g))) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CU(cudaMemcpyAsync(g_stage, g_host, (size_t)x->W * ld_g * 4, cudaMemcpyHostToDevice, st), "copy g to device");
    int32_t* oidx = reinterpret_cast<int32_t*>(x->ws + x->off_oidx);
    float* oval = reinterpret_cast<float*>(x->ws + x->off_oval);
    if ((e = ssgd_step(x, g_stage, ld_g, rho, ncand, oidx, oval, stream))) return e;
    CU(cudaMemcpyAsync(out_idx_host, oidx, (size_t)x->k * 4, cudaMemcpyDeviceToHost, st), "copy out_idx to host");
    CU(cudaMemcpyAsync(out_val_host, oval, (size_t)x->k * 4, cudaMemcpyDeviceToHost, st), "copy out_val to host");
    CU(cudaStreamSynchronize(st), "stream synchronize");
    return SSGD_OK;
}

int ssgd_step_buffers(const ssgd_ctx* x, const float** merged, const float** est, const int32_t** cand_idx,
                      const float** cand_xs) {
    int e = check_bound(x);
    if (e) return e;
    if (merged) *merged = reinterpret_cast<const float*>(x->ws + x->off_table);
    if (est) *est = reinterpret_cast<const float*>(x->ws + x->off_est);
    if (cand_idx) *cand_idx = reinterpret_cast<const int32_t*>(x->ws + x->off_cand);
    if (cand_xs) *cand_xs = reinterpret_cast<const float*>(x->ws + x->off_xs);
    return SSGD_OK;
}

int ssgd_hashes(ssgd_ctx* x, const int32_t* idx, int64_t n, int32_t* h_out, int32_t* s_out, void* stream) {
    if (!x || n < 0 || (n > 0 && (!idx || !h_out || !s_out))) return SSGD_EINVAL;
    if (n == 0) return SSGD_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int grid = grid_for(n, 256, (int64_t)1 << 30);
    if (x->pow2) k_hashes<true><<<grid, 256, 0, st>>>(idx, n, x->r, x->hp, x->bk, h_out, s_out);
    else k_hashes<false><<<grid, 256, 0, st>>>(idx, n, x->r, x->hp, x->bk, h_out, s_out);
    LAUNCHED("k_hashes");
    return SSGD_OK;
}

int ssgd_launch_count(const ssgd_ctx* x, int64_t* out) {
    if (!x || !out) return SSGD_EINVAL;
    *out = x->launches;
    return SSGD_OK;
}

int ssgd_status(ssgd_ctx* x, void* stream) {
    int e = check_bound(x);
    if (e) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CU(cudaStreamSynchronize(st), "stream synchronize");
    int32_t flag = 0;
    CU(cudaMemcpy(&flag, x->ws + x->off_err, 4, cudaMemcpyDeviceToHost), "read error flag");
    if (flag) {
        CU(cudaMemset(x->ws + x->off_err, 0, 4), "clear error flag");
        return SSGD_EDEVICE;
    }
    return SSGD_OK;
}

// ------------------------------------------------------------------------------------------------
// Second round + final top-k for callers that cannot hand over a workspace (see include/ssgd.h).
// The scratch lives in a fixed device array inside this library; its device address is looked up
// once per device with cudaGetSymbolAddress (in host code the symbol's name is only a stand-in).
// ------------------------------------------------------------------------------------------------
}  // extern "C"

namespace {

constexpr int64_t STATIC_MAX_NCAND = SSGD_STATIC_MAX_NCAND;
constexpr size_t ST_OFF_HIST = 0;                                              // histograms (zeroed per call)
constexpr size_t ST_OFF_STATE = ST_OFF_HIST + SEL_HIST_WORDS * 4;             // selection state (zeroed per call)
constexpr size_t ST_ZERO_BYTES = ST_OFF_STATE + 256;
constexpr size_t ST_OFF_ERR = ST_ZERO_BYTES;                                   // skipped-entry flag
constexpr size_t ST_OFF_CHUNK = ST_OFF_ERR + 256;                              // 2 x nchunks counters
constexpr size_t ST_NCHUNK_MAX = (STATIC_MAX_NCAND + SEL_CHUNK - 1) / SEL_CHUNK;
constexpr size_t ST_OFF_XS = (ST_OFF_CHUNK + 2 * ST_NCHUNK_MAX * 4 + 255) / 256 * 256;   // second-round sums
constexpr size_t ST_BYTES = ST_OFF_XS + (size_t)STATIC_MAX_NCAND * 4;
static_assert(sizeof(SelState) <= 256, "selection state must fit its slot");
static_assert(ST_BYTES <= SSGD_STATIC_SCRATCH_BYTES, "static scratch is smaller than its layout");

static __device__ __align__(256) unsigned char g_static_scratch[SSGD_STATIC_SCRATCH_BYTES];

constexpr int ST_MAX_DEVICES = 64;
struct StaticDevice { unsigned char* scratch; int sm_count; };
StaticDevice g_static_dev[ST_MAX_DEVICES] = {};
std::mutex g_static_mutex;

// Device address of the scratch array on the current device (looked up on the first call per device).
int static_setup(StaticDevice** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= ST_MAX_DEVICES) return SSGD_ECUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDevice& sd = g_static_dev[dev];
    if (!sd.scratch) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return SSGD_ECUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SSGD_ECUDA;
        sd.sm_count = sms;
        sd.scratch = static_cast<unsigned char*>(p);
    }
    *out = &sd;
    return SSGD_OK;
}

}  // namespace

extern "C" {

int ssgd_exact_topk_static(const float* v, int64_t ld, int32_t W, int64_t d, const int32_t* cand_idx,
                           int64_t ncand, int64_t k, int32_t* out_idx, float* out_val, void* stream) {
    if (!v || !cand_idx || !out_idx || !out_val) return SSGD_EINVAL;
    if (d < 1 || d >= (int64_t)P31 || ld < d || W < 1 || k < 1 || k > ncand || ncand > d) return SSGD_EINVAL;
    if (ncand > STATIC_MAX_NCAND) return SSGD_ETOOBIG;
    StaticDevice* sd = nullptr;
    int e = static_setup(&sd);
    if (e) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* base = sd->scratch;
    // the array keeps whatever the previous call left: histograms and selection state start from zero
    if (cudaMemsetAsync(base, 0, ST_ZERO_BYTES, st) != cudaSuccess) return SSGD_ECUDA;
    const int64_t nch = (ncand + SEL_CHUNK - 1) / SEL_CHUNK;
    SelBuffers sb{};
    uint32_t* h = reinterpret_cast<uint32_t*>(base + ST_OFF_HIST);
    sb.h1 = h; sb.h2 = h + H1_BINS; sb.h3 = h + H1_BINS + H2_BINS;
    sb.state = reinterpret_cast<SelState*>(base + ST_OFF_STATE);
    sb.chunk_gt = reinterpret_cast<uint32_t*>(base + ST_OFF_CHUNK);
    sb.chunk_eq = sb.chunk_gt + nch;
    float* xs = reinterpret_cast<float*>(base + ST_OFF_XS);
    int32_t* err = reinterpret_cast<int32_t*>(base + ST_OFF_ERR);
    k_gather<<<grid_for(ncand, 256, (int64_t)1 << 30), 256, 0, st>>>(cand_idx, ncand, v, ld, W, d, xs, sb, (uint32_t)k, err);
    const int grid = grid_for(ncand, SEL_THREADS * 8, (int64_t)sd->sm_count * 8);
    k_sel_pass2<<<grid, SEL_THREADS, 0, st>>>(xs, ncand, sb);
    k_sel_pass3<<<grid, SEL_THREADS, 0, st>>>(xs, ncand, sb);
    k_sel_count<<<(int)nch, SEL_THREADS, 0, st>>>(xs, ncand, sb, nch);
    k_emit_final<<<(int)nch, SEL_THREADS, 0, st>>>(xs, ncand, sb, cand_idx, out_idx, out_val, (uint32_t)k, nch);
    return cudaGetLastError() == cudaSuccess ? SSGD_OK : SSGD_ECUDA;
}

const char* ssgd_strerror(int code) {
    switch (code) {
        case SSGD_OK: return "ok";
        case SSGD_EINVAL: return "invalid argument";
        case SSGD_EALIGN: return "pointer not 16-byte aligned or leading dimension not a multiple of 4";
        case SSGD_ENOTBOUND: return "no state/workspace bound (call ssgd_bind)";
        case SSGD_EWORKSPACE: return "workspace too small for this ncand";
        case SSGD_ECUDA: return "CUDA runtime error (see ssgd_last_error)";
        case SSGD_EDEVICE: return "a kernel reported an error (index out of range, or a bounded wait gave up)";
        case SSGD_ENOMEM: return "out of host memory";
        case SSGD_ETOOBIG: return "size exceeds the fixed capacity of the built-in scratch";
        default: return "unknown error";
    }
}

const char* ssgd_last_error(const ssgd_ctx* x) { return x ? x->last_error.c_str() : ""; }

}  // extern "C"
