// ssgd.cu -- host side of the C ABI (include/ssgd.h): context, argument checks, workspace layout and the
// launch sequences of the Sketched-SGD compression step for sm_100a.
//
// Kernels (Algorithm 3 lines 5-13, Algorithm 4), by header:
//   step_kernels.cuh    k_accum_insert (lines 5-7, plain 128-bit loads; applies the previous step's deferred
//                       line 13), k_insert_rows, k_merge (line 8), k_quantize16 / k_merge16, k_unsketch (line 9,
//                       dense), k_gather (line 10), k_emit_candidates / k_emit_final, k_zero and
//                       k_flush_pending (line 13, eager and deferred), k_hashes
//   accum_tma.cuh       k_accum_insert_tma: lines 5-7 as a bulk-copy (TMA) + mbarrier pipeline
//   filter_unsketch.cuh k_bitmap_build, k_bitmap_fold, k_unsketch_filter: line 9 decided per coordinate on a
//                       one-bit-per-bucket copy of the table in shared memory
//   rowbits_unsketch.cuh k_row_bits, k_rowbits_combine: the same decision when that copy fits shared memory only
//                       one row (or a slice of a row) at a time
//   sparse_select.cuh   k_unsketch_sample, k_unsketch_pruned: the sampled threshold; line 9 with early exit on
//                       the table itself
//   list_select.cuh     k_list_hist, k_list_mark, k_map_emit: exact top-ncand of the survivor list
//   select.cuh          k_sel_pass23 (k_sel_pass2/3), k_sel_count: exact radix select with ordered compaction
//                       (lines 9, 11)
//   small_tail.cuh      k_small_tail: lines 9-13 as one cooperative kernel (small problems)
//   heavymix.cuh        k_row_sumsq, k_heavymix_keys, k_heavymix_rekey: Algorithm 1
//   hash.cuh, estimate.cuh   the hash family and the median-of-r estimate
// The kernels instantiated per (rows, power-of-two columns) are launched from launch_accum.cu,
// launch_unsketch.cu and launch_small.cu; ctx.cuh holds what the units share.
// HBM-bound work is the accumulate+insert kernel (20 bytes per worker-coordinate); nothing here is a dense
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

#include "ctx.cuh"
#include "list_select.cuh"


// ==================================================================================================
// host side: context, argument checks, launch plans
// ==================================================================================================
using namespace ssgd;

namespace {

constexpr size_t ALIGN = 256;
constexpr int TIMING_SLOTS = 256;
// ssgd_sketch_accumulate goes through the workers one launch at a time once all W tables together exceed this
constexpr size_t WORKER_MAJOR_MIN_BYTES = (size_t)32 << 20;
// AUTO takes the one-kernel tail up to this many coordinates (and as many candidates as it can hold).  Measured on
// B200, whole step warm, one kernel / chain of launches: d = 2^20, W = 4, ncand = 2000: 0.097 / 0.128 ms; d = 2^21,
// W = 4, ncand = 4000: 0.156 / 0.210; d = 2e6, W = 16, ncand = 16000: 0.249 / 0.281.  From 2^21 coordinates on the
// chain prunes with the bucket bitmap, which the dense estimates of the one-kernel tail do not beat.
constexpr int64_t SMALL_AUTO_MAX_D = (int64_t)1 << 21;
constexpr int64_t SMALL_INLINE_ZERO_MAX = 65536;            // eager line 13 inside the tail kernel up to this many k*W
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
    // the head, cleared at the start of every step.  What the one-kernel tail of small problems needs cleared comes
    // first (table, its barrier state and counters, H1-H3 and state of the candidate selection), so that its memset
    // stops at zero_small_bytes
    x->off_table = o;   o += up((size_t)x->r * x->c * 4);
    x->off_small = o;   o += up(sizeof(SmallState));
    x->off_hist_c = o;  o += up((size_t)SEL_HIST_WORDS * 4);
    x->off_state_c = o; o += up(sizeof(SelState));
    x->zero_small_bytes = o;
    x->map_bytes = up((size_t)((x->d + 31) / 32) * 4);
    x->off_maps = o;    o += 2 * x->map_bytes;
    x->off_h19_c = o;   o += up((size_t)H19_BINS * 4);
    x->off_hist_f = o;  o += up((size_t)SEL_HIST_WORDS * 4);
    x->off_h19_f = o;   o += up((size_t)H19_BINS * 4);
    x->off_state_f = o; o += up(sizeof(SelState));
    x->off_sp_hist = o; o += up((size_t)(2 * H1_BINS + H2_BINS) * 4);   // its 2^19-bin table is the candidate selection's
    x->off_sp_state = o; o += up(sizeof(SparseState));
    x->nchunk_map = ((x->d + 31) / 32 + MAP_CHUNK_WORDS - 1) / MAP_CHUNK_WORDS;
    x->off_map_chunks = o; o += up((size_t)x->nchunk_map * 8);   // marks per chunk of map words: counted from zero
    x->off_hm = o;      o += up(sizeof(HeavymixState));
    x->off_err = o;     o += up(16);
    x->zero_bytes = o;
    x->nchunk_c = (x->d + SEL_CHUNK - 1) / SEL_CHUNK;
    x->nchunk_f = (ncand_max + SEL_CHUNK_SMALL - 1) / SEL_CHUNK_SMALL;
    x->off_est = o;     o += up((size_t)x->d * 4);
    x->off_xsum = o;    o += up((size_t)x->d * 4);
    x->off_chunk_c = o; o += up((size_t)x->nchunk_c * 8);
    x->off_chunk_f = o; o += up((size_t)x->nchunk_f * 8);
    x->off_cand = o;    o += up((size_t)ncand_max * 4);
    x->off_xs = o;      o += up((size_t)ncand_max * 4);
    x->list_cap = x->d;                                  // the unpruned rerun may list every coordinate
    x->off_list_idx = o; o += up((size_t)x->list_cap * 4);
    x->off_list_est = o; o += up((size_t)x->list_cap * 4);
    x->off_oidx = o;    o += up((size_t)x->k * 4);
    x->off_oval = o;    o += up((size_t)x->k * 4);
    // bit-per-bucket filter: rows padded to 16 bytes; folded by 2^s until r rows fit the shared-memory budget
    auto round4 = [](int64_t w) { return (w + 3) / 4 * 4; };
    const int64_t sf = round4((x->c + 31) / 32);
    int s = 0;
    while (s <= FILTER_MAX_FOLD && x->r * round4((sf + (1 << s) - 1) >> s) > FILTER_MAX_WORDS) ++s;
    x->bm_stride_full = (int32_t)sf;
    x->bm_fold = s <= FILTER_MAX_FOLD ? s : -1;
    x->bm_stride_fold = s <= FILTER_MAX_FOLD ? (int32_t)round4((sf + (1 << s) - 1) >> s) : 0;
    x->off_pending = o; o += x->map_bytes;
    x->off_bm_full = o; o += up((size_t)x->r * sf * 4);
    x->off_bm_fold = o; o += up((size_t)x->r * x->bm_stride_fold * 4);
    // a bitmap that needs folding but whose single row fits shared memory in a few slices is used unfolded, row by row
    x->rb_slices = (int)((sf + FILTER_MAX_WORDS - 1) / FILTER_MAX_WORDS);
    x->rb_slice_words = x->rb_slices > 0 ? (int)(((sf + x->rb_slices - 1) / x->rb_slices + 3) / 4 * 4) : 0;
    x->rowbits = x->bm_fold != 0 && x->rb_slices >= 1 && x->rb_slices <= RB_MAX_SLICES;
    x->off_rowbits = o;
    if (x->rowbits) o += up((size_t)x->rb_slices * x->r * (size_t)((x->d + 31) / 32) * 4);
    x->total_bytes = o;
}

SelBuffers sel_buffers(ssgd_ctx* x, bool final_stage) {
    SelBuffers sb{};
    uint32_t* h = reinterpret_cast<uint32_t*>(x->ws + (final_stage ? x->off_hist_f : x->off_hist_c));
    sb.h1 = h; sb.h2 = h + H1_BINS; sb.h3 = h + H1_BINS + H2_BINS;
    sb.h19 = reinterpret_cast<uint32_t*>(x->ws + (final_stage ? x->off_h19_f : x->off_h19_c));
    sb.state = reinterpret_cast<SelState*>(x->ws + (final_stage ? x->off_state_f : x->off_state_c));
    uint32_t* ch = reinterpret_cast<uint32_t*>(x->ws + (final_stage ? x->off_chunk_f : x->off_chunk_c));
    const int64_t nch = final_stage ? x->nchunk_f : x->nchunk_c;
    sb.chunk_gt = ch; sb.chunk_eq = ch + nch;
    return sb;
}

int ensure_device(ssgd_ctx* x) {
    if (x->device >= 0) return SSGD_OK;
    int dev = 0;
    CU(cudaGetDevice(&dev), "cudaGetDevice");
    CU(cudaDeviceGetAttribute(&x->sm_count, cudaDevAttrMultiProcessorCount, dev), "sm count");
    CU(cudaDeviceGetAttribute(&x->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev), "smem optin");
    x->device = dev;
    return SSGD_OK;
}

// Radix-select passes after the producer filled H1: leaves thresholds in sb.state and exclusive
// chunk offsets in sb.chunk_*; the caller launches the emit kernel over `nchunks` blocks.
int launch_select(ssgd_ctx* x, const float* val, int64_t n, const SelBuffers& sb, int64_t nchunks,
                  cudaStream_t st, bool small_chunks) {
    const int grid = grid_for(n, SEL_THREADS * 8, (int64_t)x->sm_count * 8);
    if (sb.h19) {
        CU(launch_pdl(st, k_sel_pass23, grid, SEL_THREADS, 0, val, n, sb), "launch k_sel_pass23");
        LAUNCHED("k_sel_pass23");
    } else {
        CU(launch_pdl(st, k_sel_pass2, grid, SEL_THREADS, 0, val, n, sb), "launch k_sel_pass2");
        LAUNCHED("k_sel_pass2");
        CU(launch_pdl(st, k_sel_pass3, grid, SEL_THREADS, 0, val, n, sb), "launch k_sel_pass3");
        LAUNCHED("k_sel_pass3");
    }
    if (small_chunks)
        CU(launch_pdl(st, k_sel_count<SEL_ITEMS_SMALL>, grid_for(nchunks, 1, (int64_t)x->sm_count * 8), SEL_THREADS, 0, val, n, sb,
                      nchunks), "launch k_sel_count");
    else
        CU(launch_pdl(st, k_sel_count<SEL_ITEMS>, grid_for(nchunks, 1, (int64_t)x->sm_count * 8), SEL_THREADS, 0, val, n, sb,
                      nchunks), "launch k_sel_count");
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
                    float* est, cudaStream_t st, bool timed = false) {
    UnsketchArgs A;
    A.table = merged; A.c = x->c; A.d = x->d; A.hp = x->hp; A.bk = x->bk; A.est = est;
    SelBuffers sb = sel_buffers(x, false);
    A.sb = sb; A.want = (uint32_t)ncand;
    int e = launch_unsketch(x, A, st);
    if (e) return e;
    if (timed && (e = mark(x, 2, st))) return e;
    if ((e = launch_select(x, est, x->d, sb, x->nchunk_c, st, false))) return e;
    CU(launch_pdl(st, k_emit_candidates, grid_for(x->nchunk_c, 1, (int64_t)x->sm_count * 8), SEL_THREADS, 0, (const float*)est,
                  x->d, sb, cand_idx, cand_est, (uint32_t)ncand, x->nchunk_c), "launch k_emit_candidates");
    LAUNCHED("k_emit_candidates");
    return SSGD_OK;
}

SparseBuffers sparse_buffers(ssgd_ctx* x) {
    SparseBuffers sp{};
    uint32_t* h = reinterpret_cast<uint32_t*>(x->ws + x->off_sp_hist);
    sp.h1_sample = h; sp.h1 = h + H1_BINS; sp.h2 = h + 2 * H1_BINS;
    sp.h19 = reinterpret_cast<uint32_t*>(x->ws + x->off_h19_c);   // never used by both in one step
    sp.state = reinterpret_cast<SparseState*>(x->ws + x->off_sp_state);
    sp.list_idx = reinterpret_cast<int32_t*>(x->ws + x->off_list_idx);
    sp.list_est = reinterpret_cast<float*>(x->ws + x->off_list_est);
    sp.cap = (uint32_t)x->list_cap;
    sp.map_a = reinterpret_cast<uint32_t*>(x->ws + x->off_maps);
    sp.map_b = reinterpret_cast<uint32_t*>(x->ws + x->off_maps + x->map_bytes);
    sp.chunk_a = reinterpret_cast<uint32_t*>(x->ws + x->off_map_chunks);
    sp.chunk_b = sp.chunk_a + x->nchunk_map;
    return sp;
}

// Whether ssgd_step runs lines 9-13 as the one cooperative kernel of small_tail.cuh.  AUTO: up to 2^21 coordinates
// (measured on B200 against the chain of short launches).
bool use_small(const ssgd_ctx* x, int64_t ncand) {
    if (x->prune_mode == SSGD_PRUNE_FUSED) return small_tail_applicable(x, ncand);
    return x->prune_mode == SSGD_PRUNE_AUTO && !x->small_refused && small_tail_applicable(x, ncand) && x->d <= SMALL_AUTO_MAX_D;
}

// Whether ssgd_step takes the pruned first pass + selection on the survivor list (filter_unsketch.cuh,
// sparse_select.cuh, list_select.cuh) instead of the dense unsketch + selection over all d estimates.
bool use_sparse(const ssgd_ctx* x, int64_t ncand) {
    if (x->prune_mode == SSGD_PRUNE_OFF) return false;
    if (x->prune_mode == SSGD_PRUNE_ON || x->prune_mode == SSGD_PRUNE_EARLY_EXIT) return true;
    // measured (W = 16, 5 x 262,144, ncand = d/100): d = 2^20 dense 0.121 ms / pruned 0.125; 2e6 0.241 / 0.233; 4e6 0.408 / 0.357
    if (x->d < (1 << 21) || ncand * 8 > x->d) return false;      // fixed costs outweigh the saving
    // an unfolded bucket bitmap pays for every r; behind a folded one the table kernel may have to run, which was
    // measured to pay for r = 5, 7, 9 only (r = 3: one row can be skipped; r = 15, ncand = 1.6e6: 5.8 vs 4.9 ms)
    return x->bm_fold == 0 || (x->r >= 5 && x->r <= 9);   // (the row-by-row filter hands over to the table kernel the same way)
}


// Line 9 with early exit: sample -> pruned unsketch (-> unpruned rerun if the sample misjudged) -> selection on
// the survivor list (list_select.cuh).
// sums != NULL: the emit kernel also performs the second round (xs, first histogram of the final selection).
int unsketch_select_sparse(ssgd_ctx* x, const float* merged, int64_t ncand, int32_t* cand_idx, cudaStream_t st,
                           const float* sums) {
    SparseArgs A;
    A.table = merged; A.c = x->c; A.d = x->d; A.hp = x->hp; A.bk = x->bk;
    A.sp = sparse_buffers(x);
    A.ncand = (uint32_t)ncand;
    A.rerun = 0;
    A.gated = 0;
    const int64_t groups = (x->d + 3) / 4;
    const int64_t windows = (groups + (1 << SPARSE_SAMPLE_SHIFT) - 1) >> SPARSE_SAMPLE_SHIFT;
    const double mean = (double)ncand * (double)(windows * 4) / (double)x->d;
    A.want_sample = x->sample_rank ? x->sample_rank : (uint32_t)(mean + 6.0 * std::sqrt(mean) + 16.0 + 1.0);
    A.n_sampled_min = windows > 2 ? (uint32_t)(4 * (windows - 2)) : 0u;   // the last window may point past d, the last group may be short
    int e = launch_sparse(x, A, st);
    if (e) return e;
    if ((e = mark(x, 2, st))) return e;
    // the list normally holds 1-2 x ncand entries; the kernels stride over whatever it holds
    const int list_grid = grid_for(4 * ncand, SEL_THREADS * SEL_BATCH, (int64_t)x->sm_count * 8);
    CU(launch_pdl(st, k_list_hist, list_grid, SEL_THREADS, 0, A.sp), "launch k_list_hist");
    LAUNCHED("k_list_hist");
    CU(launch_pdl(st, k_list_mark, list_grid, SEL_THREADS, 0, A.sp, x->nchunk_map), "launch k_list_mark");
    LAUNCHED("k_list_mark");
    const int64_t nwords = (x->d + 31) / 32;
    const int map_grid = grid_for(x->nchunk_map, 1, (int64_t)x->sm_count * 8);
    EmitSecondRound E{};
    if (sums) {
        E.xsum = sums;
        E.xs = reinterpret_cast<float*>(x->ws + x->off_xs);
        E.sb = sel_buffers(x, true);
        E.want = (uint32_t)x->k;
        E.pending_clear = reinterpret_cast<uint32_t*>(x->ws + x->off_pending);
        E.pending_words = nwords;
    }
    CU(launch_pdl(st, k_map_emit, map_grid, SEL_THREADS, 0, A.sp, nwords, x->nchunk_map, (uint32_t)ncand, cand_idx, E),
       "launch k_map_emit");
    LAUNCHED("k_map_emit");
    return SSGD_OK;
}

uint32_t* pending_map(ssgd_ctx* x) { return reinterpret_cast<uint32_t*>(x->ws + x->off_pending); }

// Applies a deferred zero-out to u and v (no-op on an empty map).
int flush_pending(ssgd_ctx* x, cudaStream_t st) {
    const int64_t nwords = (x->d + 31) / 32;
    CU(launch_pdl(st, k_flush_pending, grid_for(nwords, 256, (int64_t)x->sm_count * 16), 256, 0, pending_map(x), nwords,
                  x->u, x->v, x->ld, x->W, x->d), "launch k_flush_pending");
    LAUNCHED("k_flush_pending");
    x->pending_dirty = false;
    return SSGD_OK;
}

// Lines 10, 11, 13.  deferred: the chosen coordinates are marked in the pending map instead of being zeroed now
// (the caller's accumulate kernel has consumed the previous marks; k_gather empties the map before the new ones).
// sums: the accumulate kernel's per-coordinate sums over the workers (ssgd_step), or NULL to read v (stage call).
// xs_ready: the candidate stage has already produced xs and the first histogram (k_map_emit's second round).
int gather_select_zero(ssgd_ctx* x, const int32_t* cand, int64_t ncand, int32_t* out_idx, float* out_val,
                       cudaStream_t st, bool deferred, const float* sums, bool xs_ready = false) {
    float* xs = reinterpret_cast<float*>(x->ws + x->off_xs);
    int32_t* err = reinterpret_cast<int32_t*>(x->ws + x->off_err);
    SelBuffers sb = sel_buffers(x, true);
    const int64_t nch = (ncand + SEL_CHUNK_SMALL - 1) / SEL_CHUNK_SMALL;
    uint32_t* pend = pending_map(x);                     // whatever the accumulate kernel consumed is cleared here
    if (xs_ready) {
    } else if (sums) {
        CU(launch_pdl(st, k_gather_sums, grid_for(ncand, 256, (int64_t)1 << 30), 256, 0, cand, ncand, sums, x->d, xs, sb,
                      (uint32_t)x->k, err, pend, (int64_t)((x->d + 31) / 32)), "launch k_gather_sums");
        LAUNCHED("k_gather_sums");
    } else {
        CU(launch_pdl(st, k_gather, grid_for(ncand, 256, (int64_t)1 << 30), 256, 0, cand, ncand, (const float*)x->v, x->ld, x->W,
                      x->d, xs, sb, (uint32_t)x->k, err, pend, (int64_t)((x->d + 31) / 32)), "launch k_gather");
        LAUNCHED("k_gather");
    }
    int e = launch_select(x, xs, ncand, sb, nch, st, true);
    if (e) return e;
    CU(launch_pdl(st, k_emit_final<SEL_ITEMS_SMALL>, grid_for(nch, 1, (int64_t)x->sm_count * 8), SEL_THREADS, 0, (const float*)xs, ncand, sb,
                  cand, out_idx, out_val, (uint32_t)x->k, nch, deferred ? pending_map(x) : (uint32_t*)nullptr), "launch k_emit_final");
    LAUNCHED("k_emit_final");
    if (deferred) {
        x->pending_dirty = true;
    } else {
        CU(launch_pdl(st, k_zero, grid_for(x->k * (int64_t)x->W, 256, (int64_t)x->sm_count * 16), 256, 0, (const int32_t*)out_idx,
                      x->k, x->u, x->v, x->ld, x->W, x->d), "launch k_zero");
        LAUNCHED("k_zero");
    }
    return SSGD_OK;
}

int resolve_insert_mode(const ssgd_ctx* x) {
    const size_t table_bytes = (size_t)x->r * x->c * 4;
    const bool fits = table_bytes <= (size_t)200 * 1024 && (int64_t)table_bytes <= x->max_smem_optin;
    if (x->insert_mode == SSGD_INSERT_SMEM) return fits ? INS_MERGED_SMEM : -1;
    if (x->insert_mode == SSGD_INSERT_GLOBAL) return INS_MERGED_GLOBAL;
    if (x->insert_mode == SSGD_INSERT_TMA) return INS_MERGED_TMA;
    // measured on B200 at d = 11,173,962 (plain loads / bulk-copy pipeline, TB/s): W = 32 6.06 / 5.58; 48 5.97 / 5.83;
    // 64 5.88 / 5.91; 96 5.82 / 6.01; 128 5.75 / 6.06; 256 5.42 / 6.13 -- the plain kernel's threads loop over the
    // workers 16 at a time, and loop less well than they start.  Those figures are for evict-first loads in the plain
    // kernel; reading with .cg (its default) it holds out longer (ms per step, plain / bulk-copy): W = 128
    // 4.88 / 4.91; 160 6.11 / 6.08; 256 9.86 / 9.59
    const bool plain_reads_cg = x->stream_loads != SSGD_STREAM_EVICT_FIRST;
    return x->W >= (plain_reads_cg ? 144 : 64) ? INS_MERGED_TMA : INS_MERGED_GLOBAL;
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
    x->device = -1; x->sm_count = 0; x->max_smem_optin = 0; x->launches = 0; x->kt_blocks_per_sm = 0;
    x->small_grid = 0; x->small_refused = false; x->wait_ns = 2000000000ull; x->withhold = 0;
    x->timing = false; x->ev = nullptr; x->ev_steps = 0; x->prune_mode = SSGD_PRUNE_AUTO; x->list_cap = 0; x->sample_rank = 0; x->filter_ready = false; x->rowbits = false; x->rowbits_ready = false; x->bm_fold = -1; x->zero_mode = SSGD_ZERO_DEFERRED; x->pending_dirty = false; x->sched_mode = SSGD_SCHED_AUTO; x->persist_bytes = 0; x->split_bytes = SPLIT_BYTES_DEFAULT; x->stream_loads = SSGD_STREAM_AUTO;
    *out = x;
    return SSGD_OK;
}

int ssgd_destroy(ssgd_ctx* ctx) {
    if (ctx && ctx->pending_dirty) return SSGD_EPENDING;   // Algorithm 3 line 13 of the last step exists only as marks
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

int ssgd_set_prune_sample_rank(ssgd_ctx* x, int64_t rank) {
    if (!x || rank < 0 || rank > 0x7FFFFFFF) return SSGD_EINVAL;
    x->sample_rank = (uint32_t)rank;
    return SSGD_OK;
}

int ssgd_set_stream_loads(ssgd_ctx* x, int32_t mode) {
    if (!x || mode < SSGD_STREAM_AUTO || mode > SSGD_STREAM_L2_ONLY) return SSGD_EINVAL;
    x->stream_loads = mode;
    return SSGD_OK;
}

int ssgd_set_insert_split(ssgd_ctx* x, int64_t bytes) {
    if (!x || bytes < 0) return SSGD_EINVAL;
    x->split_bytes = (size_t)bytes;
    return SSGD_OK;
}

int ssgd_set_accumulate_schedule(ssgd_ctx* x, int32_t mode) {
    if (!x || mode < SSGD_SCHED_AUTO || mode > SSGD_SCHED_WORKER_MAJOR) return SSGD_EINVAL;
    x->sched_mode = mode;
    return SSGD_OK;
}

int ssgd_set_prune_mode(ssgd_ctx* x, int32_t mode) {
    if (!x || mode < SSGD_PRUNE_AUTO || mode > SSGD_PRUNE_FUSED) return SSGD_EINVAL;
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
    out[3] = (int32_t)s.use_table; out[4] = (int32_t)s.fold_ones;
    return SSGD_OK;
}

int ssgd_set_insert_mode(ssgd_ctx* x, int32_t mode) {
    if (!x || mode < SSGD_INSERT_AUTO || mode > SSGD_INSERT_TMA) return SSGD_EINVAL;
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
    if (x->pending_dirty) return SSGD_EPENDING;
    layout(x, ncand_max);
    if (workspace_bytes < x->total_bytes) return SSGD_EWORKSPACE;
    x->u = u; x->v = v; x->ld = ld;
    x->ws = static_cast<char*>(workspace); x->ws_bytes = workspace_bytes; x->ncand_max = ncand_max;
    int e = ensure_device(x);
    if (e) return e;
    CU(cudaMemset(x->ws + x->off_err, 0, 16), "clear error flag");
    CU(cudaMemset(x->ws + x->off_pending, 0, x->map_bytes), "clear pending map");   // nothing awaits its zero-out
    x->pending_dirty = false;
    return SSGD_OK;
}

int ssgd_unbind(ssgd_ctx* x) {
    if (!x) return SSGD_EINVAL;
    x->u = x->v = nullptr; x->ws = nullptr; x->ld = 0; x->ws_bytes = 0; x->ncand_max = 0;
    x->pending_dirty = false;
    return SSGD_OK;
}

int ssgd_sketch_accumulate(ssgd_ctx* x, const float* g, int64_t ld_g, float rho, float* tables, void* stream) {
    int e = check_bound(x);
    if (e) return e;
    if ((e = check_g(x, g, ld_g))) return e;
    if (!tables) return SSGD_EINVAL;
    if ((e = ensure_device(x))) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (x->pending_dirty && (e = flush_pending(x, st))) return e;
    CU(cudaMemsetAsync(tables, 0, (size_t)x->W * x->r * x->c * 4, st), "memset tables");
    x->launches++;
    AccumArgs A;
    A.g = g; A.ld_g = ld_g; A.u = x->u; A.v = x->v; A.ld = x->ld; A.W = x->W; A.d = x->d; A.rho = rho;
    A.table = tables; A.c = x->c; A.hp = x->hp; A.bk = x->bk; A.rows_here = x->r; A.xsum = nullptr; A.pending = nullptr;
    A.loads_evict_first = 1;
    A.wait_ns = x->wait_ns; A.withhold = 0;
    const size_t all_tables = (size_t)x->W * x->r * x->c * 4;
    const bool worker_major = x->sched_mode == SSGD_SCHED_WORKER_MAJOR ||
                              (x->sched_mode == SSGD_SCHED_AUTO && x->W > 1 && all_tables > WORKER_MAJOR_MIN_BYTES);
    if (!worker_major) return launch_accum(x, A, INS_PER_WORKER, st);
    // one worker per launch: its g, u, v stream past once and the reductions go to its own r x c table only, which
    // stays L2-resident for the whole launch (a single worker's sketch is the merged-table kernel with W = 1)
    const int64_t rc = (int64_t)x->r * x->c;
    for (int w = 0; w < x->W; ++w) {
        AccumArgs B = A;
        B.W = 1;
        B.g = g + (int64_t)w * ld_g; B.u = x->u + (int64_t)w * x->ld; B.v = x->v + (int64_t)w * x->ld;
        B.table = tables + (int64_t)w * rc;
        if ((e = launch_accum(x, B, INS_MERGED_GLOBAL, st))) return e;
    }
    return SSGD_OK;
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
    CU(cudaMemsetAsync(x->ws + x->off_hist_c, 0, x->zero_small_bytes - x->off_hist_c, st), "memset hist");   // H1-H3, state
    CU(cudaMemsetAsync(x->ws + x->off_h19_c, 0, x->off_hist_f - x->off_h19_c, st), "memset hist");           // 2^19-bin table
    x->launches += 2;
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
    if (x->pending_dirty && (e = flush_pending(x, st))) return e;
    CU(cudaMemsetAsync(x->ws + x->off_hist_f, 0, x->off_err - x->off_hist_f, st), "memset hist");
    x->launches++;
    return gather_select_zero(x, cand_idx, ncand, out_idx, out_val, st, false, nullptr);
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
    const bool small = use_small(x, ncand);
    if (x->prune_mode == SSGD_PRUNE_FUSED && !small) return SSGD_EINVAL;
    // table, histograms, selection state: one memset (the error flag is sticky until ssgd_status)
    CU(cudaMemsetAsync(x->ws, 0, small ? x->zero_small_bytes : x->off_err, st), "memset workspace head");
    x->launches++;
    float* merged = reinterpret_cast<float*>(x->ws + x->off_table);
    AccumArgs A;
    A.g = g; A.ld_g = ld_g; A.u = x->u; A.v = x->v; A.ld = x->ld; A.W = x->W; A.d = x->d; A.rho = rho;
    A.table = merged; A.c = x->c; A.hp = x->hp; A.bk = x->bk; A.rows_here = x->r; A.xsum = nullptr;
    A.loads_evict_first = x->stream_loads == SSGD_STREAM_EVICT_FIRST ? 1 : 0;
    A.pending = pending_map(x);      // the previous step's deferred zero-out, applied while u and v stream past
    A.wait_ns = x->wait_ns; A.withhold = x->withhold;
    // a table that cannot stay in L2 next to the stream is inserted a slice of rows at a time
    const size_t row_bytes = (size_t)x->c * 4;
    const int rows_fit = (int)(x->split_bytes / row_bytes);
    const bool split = mode == INS_MERGED_GLOBAL && x->split_bytes > 0 && rows_fit >= 1 && rows_fit < x->r;
    A.xsum = reinterpret_cast<float*>(x->ws + x->off_xsum);   // the second round reads these instead of W values of v
    if (split) A.rows_here = rows_fit;
    if ((e = mark(x, 0, st))) return e;
    if ((e = mode == INS_MERGED_TMA ? launch_accum_tma(x, A, st) : launch_accum(x, A, mode, st))) return e;
    if (split) {
        // the follow-up passes have only the per-coordinate sums streaming beside the table: more rows per pass
        const int pass_rows = (int)(INSERT_PASS_BYTES / row_bytes) > rows_fit ? (int)(INSERT_PASS_BYTES / row_bytes) : rows_fit;
        for (int lo = rows_fit; lo < x->r; lo += pass_rows)
            if ((e = launch_insert_rows(x, A.xsum, merged, lo, lo + pass_rows < x->r ? lo + pass_rows : x->r, st))) return e;
    }
    if ((e = mark(x, 1, st))) return e;
    int32_t* cand = reinterpret_cast<int32_t*>(x->ws + x->off_cand);
    float* est = reinterpret_cast<float*>(x->ws + x->off_est);
    if (small) {
        // lines 9-13 in one cooperative kernel
        SmallArgs T{};
        T.table = merged; T.c = x->c; T.d = x->d; T.hp = x->hp; T.bk = x->bk; T.est = est;
        SelBuffers sb = sel_buffers(x, false);
        T.h1 = sb.h1; T.h2 = sb.h2; T.h3 = sb.h3;
        T.st = reinterpret_cast<SmallState*>(x->ws + x->off_small);
        T.map_a = reinterpret_cast<uint32_t*>(x->ws + x->off_maps);
        T.map_b = reinterpret_cast<uint32_t*>(x->ws + x->off_maps + x->map_bytes);
        T.xsum = A.xsum; T.cand_idx = cand; T.xs = reinterpret_cast<float*>(x->ws + x->off_xs);
        T.ncand = (uint32_t)ncand; T.k = (uint32_t)x->k; T.out_idx = out_idx; T.out_val = out_val;
        const bool deferred = x->zero_mode == SSGD_ZERO_DEFERRED;
        T.pending = pending_map(x); T.pending_words = (x->d + 31) / 32; T.mark_pending = deferred ? 1 : 0;
        T.u = x->u; T.v = x->v; T.ld = x->ld; T.W = x->W;
        T.zero_inline = (!deferred && x->k * (int64_t)x->W <= SMALL_INLINE_ZERO_MAX) ? 1 : 0;
        T.wait_ns = x->wait_ns; T.withhold = x->withhold;
        T.errflag = reinterpret_cast<int32_t*>(x->ws + x->off_err);
        e = launch_small_tail(x, T, st);
        if (e == SMALL_TAIL_REFUSED) {
            if (x->prune_mode == SSGD_PRUNE_FUSED) { x->last_error = "cooperative launch refused: the device cannot hold one block per SM at once"; return SSGD_ECUDA; }
            x->small_refused = true;                       // AUTO: this step and the following ones take the chain
            CU(cudaMemsetAsync(x->ws + x->zero_small_bytes, 0, x->off_err - x->zero_small_bytes, st), "memset workspace head");
            x->launches++;
            goto chain;
        }
        if (e) return e;
        if ((e = mark(x, 2, st)) || (e = mark(x, 3, st))) return e;
        if (deferred) {
            x->pending_dirty = true;
        } else if (!T.zero_inline) {
            CU(launch_pdl(st, k_zero, grid_for(x->k * (int64_t)x->W, 256, (int64_t)x->sm_count * 16), 256, 0, (const int32_t*)out_idx,
                          x->k, x->u, x->v, x->ld, x->W, x->d), "launch k_zero");
            LAUNCHED("k_zero");
        }
        if ((e = mark(x, 4, st))) return e;
        if (x->timing && x->ev_steps < TIMING_SLOTS) x->ev_steps++;
        return SSGD_OK;
    }
chain:
    const bool sparse = use_sparse(x, ncand);
    if (sparse) {
        if ((e = unsketch_select_sparse(x, merged, ncand, cand, st, A.xsum))) return e;
    } else {
        if ((e = unsketch_select(x, merged, ncand, cand, nullptr, est, st, true))) return e;
    }
    if ((e = mark(x, 3, st))) return e;
    if ((e = gather_select_zero(x, cand, ncand, out_idx, out_val, st, x->zero_mode == SSGD_ZERO_DEFERRED, A.xsum, sparse))) return e;
    if ((e = mark(x, 4, st))) return e;
    if (x->timing && x->ev_steps < TIMING_SLOTS) x->ev_steps++;
    return SSGD_OK;
}

int ssgd_tail_trace(ssgd_ctx* x, void* stream, int64_t* out12) {
    int e = check_bound(x);
    if (e) return e;
    if (!out12) return SSGD_EINVAL;
    CU(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)), "stream synchronize");
    SmallState s;
    CU(cudaMemcpy(&s, x->ws + x->off_small, sizeof(s), cudaMemcpyDeviceToHost), "read tail state");
    for (int t = 0; t < 12; ++t) out12[t] = s.trace[t] ? (int64_t)(s.trace[t] - s.trace[0]) : -1;
    return SSGD_OK;
}

int ssgd_set_wait_limit_ns(ssgd_ctx* x, int64_t ns) {
    if (!x || ns < 1000) return SSGD_EINVAL;
    x->wait_ns = (uint64_t)ns;
    return SSGD_OK;
}

int ssgd_test_withhold_block(ssgd_ctx* x, int32_t block_plus_one) {
    if (!x || block_plus_one < -1) return SSGD_EINVAL;
    x->withhold = block_plus_one;
    return SSGD_OK;
}

int ssgd_set_zero_mode(ssgd_ctx* x, int32_t mode) {
    if (!x || (mode != SSGD_ZERO_DEFERRED && mode != SSGD_ZERO_EAGER)) return SSGD_EINVAL;
    x->zero_mode = mode;
    return SSGD_OK;
}

int ssgd_flush(ssgd_ctx* x, void* stream) {
    int e = check_bound(x);
    if (e) return e;
    if ((e = ensure_device(x))) return e;
    return flush_pending(x, static_cast<cudaStream_t>(stream));
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
    if (x->pending_dirty && (e = flush_pending(x, st))) return e;   // line 5 reads v
    // histograms + state of the candidate selection, and the HEAVYMIX state
    CU(cudaMemsetAsync(x->ws + x->off_hist_c, 0, x->zero_small_bytes - x->off_hist_c, st), "memset hist");   // H1-H3, state
    CU(cudaMemsetAsync(x->ws + x->off_h19_c, 0, x->off_hist_f - x->off_h19_c, st), "memset hist");           // 2^19-bin table
    CU(cudaMemsetAsync(x->ws + x->off_hist_f, 0, x->off_sp_hist - x->off_hist_f, st), "memset hist");
    CU(cudaMemsetAsync(x->ws + x->off_hm, 0, sizeof(HeavymixState), st), "memset heavymix state");
    x->launches += 4;
    HeavymixArgs A;
    A.table = merged; A.c = x->c; A.d = x->d; A.r = x->r; A.hp = x->hp; A.bk = x->bk;
    A.hm = reinterpret_cast<HeavymixState*>(x->ws + x->off_hm);
    A.keys = reinterpret_cast<float*>(x->ws + x->off_est);
    A.est = reinterpret_cast<float*>(x->ws + x->off_list_est);   // the survivor list's room: d floats
    A.sb = sel_buffers(x, false);
    A.k = (uint32_t)x->k;
    A.fill_seed = fill_seed;
    dim3 grid((unsigned)grid_for(x->c, 256, x->sm_count * 2), (unsigned)x->r);
    k_row_sumsq<<<grid, 256, 0, st>>>(merged, x->c, A.hm);
    LAUNCHED("k_row_sumsq");
    if ((e = launch_heavymix_keys(x, A, st))) return e;
    if ((e = launch_select(x, A.keys, x->d, A.sb, x->nchunk_c, st, false))) return e;
    CU(launch_pdl(st, k_emit_candidates, grid_for(x->nchunk_c, 1, (int64_t)x->sm_count * 8), SEL_THREADS, 0, (const float*)A.keys,
                  x->d, A.sb, out_idx, (float*)nullptr, (uint32_t)x->k, x->nchunk_c), "launch k_emit_candidates");
    LAUNCHED("k_emit_candidates");
    // |H| > k (decided on the device): a second selection among the heavy coordinates on their full magnitudes
    // overwrites out_idx; its kernels return at once otherwise.  It uses the final stage's histograms and state
    // and, once the first selection is done with them, the candidate stage's chunk counters.
    SelBuffers sb2 = sel_buffers(x, true);
    sb2.chunk_gt = A.sb.chunk_gt; sb2.chunk_eq = A.sb.chunk_eq;
    sb2.gate = &A.hm->nheavy; sb2.gate_above = (uint32_t)x->k;
    k_heavymix_rekey<<<grid_for(x->d, SEL_THREADS * 4, (int64_t)x->sm_count * 8), SEL_THREADS, 0, st>>>(A, x->r, sb2);
    LAUNCHED("k_heavymix_rekey");
    if ((e = launch_select(x, A.keys, x->d, sb2, x->nchunk_c, st, false))) return e;
    CU(launch_pdl(st, k_emit_candidates, grid_for(x->nchunk_c, 1, (int64_t)x->sm_count * 8), SEL_THREADS, 0, (const float*)A.keys,
                  x->d, sb2, out_idx, (float*)nullptr, (uint32_t)x->k, x->nchunk_c), "launch k_emit_candidates");
    LAUNCHED("k_emit_candidates");
    // line 5: exact values of the chosen coordinates, summed over the workers
    SelBuffers sf = sel_buffers(x, true);
    CU(launch_pdl(st, k_gather, grid_for(x->k, 256, (int64_t)1 << 30), 256, 0, (const int32_t*)out_idx, x->k, (const float*)x->v,
                  x->ld, x->W, x->d, out_val, sf, (uint32_t)1, reinterpret_cast<int32_t*>(x->ws + x->off_err),
                  (uint32_t*)nullptr, (int64_t)0), "launch k_gather");
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
    k_gather<<<grid_for(ncand, 256, (int64_t)1 << 30), 256, 0, st>>>(cand_idx, ncand, v, ld, W, d, xs, sb, (uint32_t)k, err, nullptr, 0);
    const int grid = grid_for(ncand, SEL_THREADS * 8, (int64_t)sd->sm_count * 8);
    k_sel_pass2<<<grid, SEL_THREADS, 0, st>>>(xs, ncand, sb);
    k_sel_pass3<<<grid, SEL_THREADS, 0, st>>>(xs, ncand, sb);
    k_sel_count<SEL_ITEMS><<<(int)nch, SEL_THREADS, 0, st>>>(xs, ncand, sb, nch);
    k_emit_final<SEL_ITEMS><<<(int)nch, SEL_THREADS, 0, st>>>(xs, ncand, sb, cand_idx, out_idx, out_val, (uint32_t)k, nch, nullptr);
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
        case SSGD_EPENDING: return "a deferred zero-out is pending: call ssgd_flush first (or ssgd_unbind to discard it)";
        default: return "unknown error";
    }
}

const char* ssgd_last_error(const ssgd_ctx* x) { return x ? x->last_error.c_str() : ""; }

}  // extern "C"
