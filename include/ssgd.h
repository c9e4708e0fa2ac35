/*
 * ssgd.h -- C ABI of the Sketched-SGD compression step for NVIDIA B200 (sm_100a).
 *
 * One step of the paper's empirical training procedure (Algorithm 3, lines 5-13) over W workers
 * whose state lives, batched, on ONE GPU:
 *
 *   line 5   momentum                 u_w <- rho*u_w + g_w
 *   line 6   error accumulation       v_w <- v_w + u_w                       (the new u_w)
 *   line 7   Count Sketch of v_w      S_w[j][h_j(i)] += s_j(i) * v_w[i]      (Algorithm 4, update)
 *   line 8   aggregate                S = sum_w S_w                           (plain sum, see below)
 *   line 9   top-ncand by |estimate|  est[i] = median_j s_j(i)*S[j][h_j(i)]   (Algorithm 4, estimate)
 *   line 10  second round             xs[m] = sum_w v_w[cand[m]]
 *   line 11  k-sparse update          the k candidates with the largest |xs|
 *   line 13  masking / error reset    u_w[i] = v_w[i] = 0 at those k coordinates, every worker
 *
 * Conventions
 *  - Every call returns an int status: SSGD_OK (0) or a negative SSGD_E* code.  Nothing throws,
 *    aborts or traps.  Arguments are checked on the host before anything is launched.
 *  - "device" pointers are CUDA device pointers of the current device, owned by the caller.  The
 *    library allocates no device memory: all scratch is the caller's workspace (ssgd_bind).
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Stage calls and
 *    ssgd_step only enqueue work; they never synchronise.  Results are valid once the stream
 *    has reached that point.
 *  - Worker-major layout: g, u, v are [W][ld] fp32, row w at base + w*ld, only the first d entries
 *    of a row are read or written.  Bases must be 16-byte aligned and ld a multiple of 4
 *    (SSGD_EALIGN otherwise), ld >= d.
 *  - Hash family (fixed by the problem statement; Algorithm 4 line 2 leaves it open), p = 2^31-1:
 *        h_j(i) = ((a_j*i  + b_j ) mod p) mod c
 *        s_j(i) = 2*(((a'_j*i + b'_j) mod p) & 1) - 1
 *    with i the 0-based coordinate and j the 0-based row.  a_j, b_j, a'_j, b'_j come from `seed`:
 *    a 64-bit state s starts at seed; each draw does s += 0x9E3779B97F4A7C15, z = s,
 *    z = (z^(z>>30))*0xBF58476D1CE4E5B9, z = (z^(z>>27))*0x94D049BB133111EB, out = z^(z>>31);
 *    row j takes four draws in the order a, b, a', b' with a = 1 + out mod (p-1), b = out mod p.
 *  - The aggregate is the SUM of the workers' sketches and out_val is the SUM of the workers'
 *    values (Algorithm 3 line 10 stores the sum; the 1/W of line 8 does not change any selection).
 *  - Selections use the total order "larger magnitude first (fp32 bit pattern of |x|), then smaller
 *    coordinate index first", so they are unique given their inputs.
 *  - Inputs must be finite.  fp32 throughout; the only fused multiply-add is the momentum line.
 */
#ifndef SSGD_H
#define SSGD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SSGD_OK          0
#define SSGD_EINVAL     -1  /* bad shape, size, NULL pointer, ld < d, k > ncand, ncand > d, even r ... */
#define SSGD_EALIGN     -2  /* base pointer not 16-byte aligned, or ld not a multiple of 4             */
#define SSGD_ENOTBOUND  -3  /* ssgd_bind has not been called                                           */
#define SSGD_EWORKSPACE -4  /* workspace too small for the requested ncand                             */
#define SSGD_ECUDA      -5  /* a CUDA runtime call failed; ssgd_last_error gives its text              */
#define SSGD_EDEVICE    -6  /* a kernel recorded an error: bad index in a caller's list, or a wait gave up */
#define SSGD_ENOMEM     -7  /* host allocation failed                                                  */
#define SSGD_ETOOBIG    -8  /* size beyond the fixed capacity of ssgd_exact_topk_static                */
#define SSGD_EPENDING   -9  /* a deferred zero-out has not been applied yet: ssgd_flush first (or ssgd_unbind) */

#define SSGD_MAX_R 15

/* Insert variants of ssgd_step (ssgd_set_insert_mode) */
#define SSGD_INSERT_AUTO   0  /* SSGD_INSERT_TMA when W >= 144, else SSGD_INSERT_GLOBAL (measured)           */
#define SSGD_INSERT_GLOBAL 1  /* plain 128-bit loads; reductions straight into the L2-resident table    */
#define SSGD_INSERT_SMEM   2  /* per-block table in shared memory, flushed once; needs r*c*4 <= 200 KiB */
#define SSGD_INSERT_TMA    3  /* bulk-copy (TMA) + mbarrier pipeline; reductions into the L2 table      */

/* How ssgd_step evaluates Algorithm 3 line 9 (ssgd_set_prune_mode).  A median of r values reaches a magnitude
 * only if (r+1)/2 of them do, so with a threshold taken from a sample of the estimates most coordinates can be
 * ruled out from "is this bucket's magnitude above the threshold" alone.  ON: that test is precomputed as one bit
 * per bucket and kept in shared memory: all r*c bits at once if they fit; else one row (or one of up to four
 * slices of a row) per thread block, the r bits of every coordinate being combined afterwards; else OR-folded up
 * to 32 buckets per bit; otherwise as EARLY_EXIT.  EARLY_EXIT: the test is applied to the table values themselves and a coordinate stops reading
 * rows once it cannot pass.  OFF: every coordinate reads all r rows.  The candidates are identical in all modes.
 * AUTO is ON when d >= 2^21, ncand <= d/8 (below that the fixed costs outweigh the saving) and either the bitmap
 * fits as a whole or 5 <= r <= 9; else OFF.  Unless the bitmap fits as a whole, ON measures its density each step
 * and runs the EARLY_EXIT kernel instead when its bits would rule out too few coordinates. */
#define SSGD_PRUNE_AUTO 0
#define SSGD_PRUNE_OFF  1
#define SSGD_PRUNE_ON   2
#define SSGD_PRUNE_EARLY_EXIT 3
/* FUSED: lines 9-13 run as ONE cooperative kernel (dense estimates, exact radix select and ordered candidate emit
 * behind grid barriers, the second round where a candidate is emitted, the final top-k and line 13 by the last
 * block), for problems so small that a chain of short
 * launches costs more than the work: needs d <= 2^22 and ncand <= 16384 (SSGD_EINVAL from ssgd_step otherwise).
 * AUTO takes this path for d <= 2^21 when it applies.  The results are those of the other modes. */
#define SSGD_PRUNE_FUSED 4

typedef struct ssgd_ctx ssgd_ctx; /* opaque host object; holds no device memory */

/* Algorithm 4 init(r, c) plus the shape of Algorithm 3: d coordinates, r rows (odd, 1..15), c columns,
 * k final sparsity, W workers; 1 <= d < 2^31-1, 1 <= c < 2^31-1, 1 <= k <= d, W >= 1.  Host only. */
int ssgd_create(ssgd_ctx** out, int64_t d, int32_t r, int64_t c, int64_t k, int32_t W, uint64_t seed);
/* Frees the host object.  While a deferred zero-out of the last ssgd_step is still pending (see
 * ssgd_set_zero_mode) the bound u and v do not hold Algorithm 3 line 13's zeros yet and the marks live only in
 * the workspace, so the call refuses with SSGD_EPENDING and leaves the context alive: call ssgd_flush first, or
 * ssgd_unbind to give the marks up on purpose.  (It does not write the zeros itself because it cannot know
 * that the caller's buffers still exist.) */
int ssgd_destroy(ssgd_ctx* ctx);

/* The 4r hash parameters, row j at out4r[4j..4j+3] = a_j, b_j, a'_j, b'_j (host memory). */
int ssgd_get_hash_params(const ssgd_ctx* ctx, uint32_t* out4r);
/* Replace them (for tests): a, a' in [1, p-1], b, b' in [0, p-1]. */
int ssgd_set_hash_params(ssgd_ctx* ctx, const uint32_t* in4r);
int ssgd_set_insert_mode(ssgd_ctx* ctx, int32_t mode);
int ssgd_set_prune_mode(ssgd_ctx* ctx, int32_t mode);
/* When ssgd_step applies Algorithm 3 line 13 (u, v <- 0 at the k chosen coordinates).
 * DEFERRED (default): ssgd_step only marks the chosen coordinates in a d-bit map inside the workspace; the NEXT
 * ssgd_step reads marked coordinates of u and v as +0 inside the kernel that streams all of u and v anyway, so
 * the zero-out costs no scattered writes.  Until then the memory of u and v still holds the old values at those
 * coordinates: call ssgd_flush before reading u or v yourself.  The library's own entry points that read u or v
 * (ssgd_sketch_accumulate, ssgd_exact_topk, ssgd_heavymix) flush first; ssgd_exact_topk_static has no context
 * and cannot.  Every result (chosen coordinates, values, the state after a flush) is identical in both modes.
 * The pending marks are state of the method that lives in the workspace: to checkpoint, call ssgd_flush and
 * save u and v; ssgd_bind and ssgd_destroy refuse (SSGD_EPENDING) while marks are pending.
 * EAGER: ssgd_step writes the zeros before it returns control to the stream's next operation. */
#define SSGD_ZERO_DEFERRED 0
#define SSGD_ZERO_EAGER    1
int ssgd_set_zero_mode(ssgd_ctx* ctx, int32_t mode);
/* Limit, in nanoseconds (>= 1000; default 2e9), of every wait inside a kernel: the grid barriers of the FUSED tail
 * and the pipeline barriers of the bulk-copy insert kernel.  A wait that runs out makes its kernel record an
 * error and return; ssgd_status then reports SSGD_EDEVICE once, results of that step are undefined, and the
 * context stays usable. */
int ssgd_set_wait_limit_ns(ssgd_ctx* ctx, int64_t ns);
/* Test hook: thread block (block_plus_one - 1) of those kernels leaves without ever arriving at its barriers, so
 * that the others' waits run out (nothing hangs, nothing faults); 0 switches the hook off.  -1: ssgd_step behaves as
 * if the device had refused the cooperative launch of the FUSED tail (which happens when it cannot hold one thread
 * block per SM at once, e.g. with SMs taken by another context): under SSGD_PRUNE_AUTO the step then takes the chain
 * of ordinary launches, and so do the following steps; under SSGD_PRUNE_FUSED it returns SSGD_ECUDA. */
int ssgd_test_withhold_block(ssgd_ctx* ctx, int32_t block_plus_one);
/* Applies a deferred zero-out to u and v now (device pointers bound by ssgd_bind), on `stream`.  Cheap when
 * nothing is pending (one pass over d/8 bytes).  It always launches: the marks may come from a replayed CUDA
 * graph, which the host side of the context does not see. */
int ssgd_flush(ssgd_ctx* ctx, void* stream);
/* For tables too large to stay in L2 next to the streamed g, u, v: let the streaming kernel insert only as
 * many rows as fit in `bytes` and insert the remaining rows from the per-coordinate sums in follow-up
 * launches of at most `bytes` of table each (plain-load insert variant only; 0 = never split; default 24 MiB,
 * which leaves tables up to that size untouched). */
int ssgd_set_insert_split(ssgd_ctx* ctx, int64_t bytes);
/* Cache operator of the plain-load accumulate+insert kernel's reads of g, u, v (ssgd_step with
 * SSGD_INSERT_GLOBAL).  AUTO = L2_ONLY (ld.global.cg: not kept in L1, normal priority in L2; the table's lines are
 * protected by the evict-last policy of the reductions).  EVICT_FIRST: ld.global.cs.  The result of a step does
 * not depend on it. */
#define SSGD_STREAM_AUTO        0
#define SSGD_STREAM_EVICT_FIRST 1
#define SSGD_STREAM_L2_ONLY     2
int ssgd_set_stream_loads(ssgd_ctx* ctx, int32_t mode);
/* Opt-in: reserve part of L2 for the sketch table while the accumulate+insert kernel streams g, u, v past it
 * (cudaLimitPersistingL2CacheSize of this process's CUDA context is raised to the table size, capped by the
 * device; the launches then carry an access-policy window over the table).  Off by default because the limit
 * is shared with everything else the process runs on that device.  enable = 0 stops attaching the window. */
int ssgd_set_table_persistence(ssgd_ctx* ctx, int32_t enable);
/* Diagnostics of the last ssgd_step's pruned path (waits for the stream), five values: out[0] != 0 if the
 * sampled threshold kept fewer than ncand coordinates and the pass was redone without pruning, out[1] = number
 * of coordinates on the survivor list, out[2] = the prune threshold as a histogram-bin index (0: nothing
 * pruned), out[3] = 1 if the bucket bitmap was too dense and the first pass read the table instead,
 * out[4] = set bits of the bitmap that was measured (the unfolded one if it is used row by row, else the folded
 * one; 0 if the bitmap fits shared memory as a whole and is not measured). */
int ssgd_step_used_fallback(ssgd_ctx* ctx, void* stream, int32_t* out5);
/* Diagnostics of the last ssgd_step that took the FUSED tail (waits for the stream): nanoseconds since the tail
 * kernel's first thread block started, at 12 points -- [0] start, [1] table rows copied to shared memory (if any),
 * [2] its estimates done, [3]-[5] past the first three grid barriers (the digits of the threshold), [11] past the
 * fourth (segment counts complete), all of thread block 0; of the block that finishes the step alone: [6] it knows
 * it is the last (candidates and their sums are in place), [7], [8] candidates loaded, [9] final threshold known,
 * [10] end.  -1 where no stamp was taken. */
int ssgd_tail_trace(ssgd_ctx* ctx, void* stream, int64_t* out12);
/* For tests and diagnostics: the rank (from the top) in the sample's histogram that sets the prune threshold;
 * 0 = derive it from ncand (mean + 6 sigma + 16).  A rank of 1 puts the threshold at the largest sampled
 * estimate, which forces the unpruned rerun. */
int ssgd_set_prune_sample_rank(ssgd_ctx* ctx, int64_t rank);

/* Bytes of device scratch needed to run steps with up to ncand_max candidates (host only). */
int ssgd_workspace_bytes(const ssgd_ctx* ctx, int64_t ncand_max, size_t* out_bytes);

/* Attach the caller-owned worker state u, v ([W][ld] fp32, device; Algorithm 3 line 1 wants them
 * zero before the first step) and the caller-owned workspace (device, 256-byte aligned, at least
 * ssgd_workspace_bytes(ncand_max)).  The buffers must stay valid while the context uses them.  Rebinding a
 * context whose last step's zero-out is still pending is refused with SSGD_EPENDING (see ssgd_destroy). */
int ssgd_bind(ssgd_ctx* ctx, float* u, float* v, int64_t ld, void* workspace, size_t workspace_bytes,
              int64_t ncand_max);
/* Detaches u, v and the workspace.  A pending deferred zero-out is DISCARDED (the previously bound u and v keep
 * their old values at the last step's k coordinates): the explicit way out of SSGD_EPENDING for a caller who no
 * longer wants that state.  Touches no device memory. */
int ssgd_unbind(ssgd_ctx* ctx);

/* Algorithm 3 lines 5-7 (Algorithm 4 update): updates the bound u, v from g ([W][ld_g] fp32, device,
 * read only) and writes each worker's own sketch to tables[w] ([W][r][c] fp32, device; zeroed by the
 * call, then filled with reductions, so bucket sums are order-dependent in the last bits). */
int ssgd_sketch_accumulate(ssgd_ctx* ctx, const float* g, int64_t ld_g, float rho, float* tables,
                           void* stream);

/* How ssgd_sketch_accumulate walks the W x d worker-coordinates.  COORDINATE_MAJOR: one launch, a thread owns a
 * group of coordinates and visits every worker (hashes computed once per coordinate; reductions scatter over all
 * W tables at once).  WORKER_MAJOR: one launch per worker, so that only that worker's r x c table receives
 * reductions and stays L2-resident meanwhile (hashes recomputed per worker).  AUTO: WORKER_MAJOR once the W
 * tables together exceed 32 MiB.  The results are the same up to the order of the reductions. */
#define SSGD_SCHED_AUTO             0
#define SSGD_SCHED_COORDINATE_MAJOR 1
#define SSGD_SCHED_WORKER_MAJOR     2
int ssgd_set_accumulate_schedule(ssgd_ctx* ctx, int32_t mode);

/* Algorithm 3 line 8 (mergeability, Section 3): merged[j][b] = sum over w = 0..W-1, in that order,
 * of tables[w][j][b].  merged is [r][c] fp32, device. */
int ssgd_sketch_merge(ssgd_ctx* ctx, const float* tables, float* merged, void* stream);

/* 16-bit sketches (Section 6: quantising sketches to 16 bits).  ssgd_sketch_quantize16 rounds the W per-worker
 * tables ([W][r][c] fp32, device) to a 16-bit format, round-to-nearest-even -- SSGD_FMT_F16: IEEE binary16,
 * magnitudes beyond 65504 saturate; SSGD_FMT_BF16: bfloat16 -- into q16 ([W][r][c] uint16, device): what each
 * worker would transmit.  ssgd_sketch_merge16 is the server side: merged[j][b] = sum over w = 0..W-1, in that
 * order, in fp32, of the decoded q16[w][j][b].  The rest of the pipeline runs on `merged` unchanged. */
#define SSGD_FMT_F16  0
#define SSGD_FMT_BF16 1
int ssgd_sketch_quantize16(ssgd_ctx* ctx, const float* tables, int32_t fmt, uint16_t* q16, void* stream);
int ssgd_sketch_merge16(ssgd_ctx* ctx, const uint16_t* q16, int32_t fmt, float* merged, void* stream);

/* Algorithm 3 line 9 (Algorithm 4 estimate for every coordinate, Section 5.2): computes est[i] for
 * all i < d from merged ([r][c] fp32, device) and writes the ncand coordinates with the largest
 * |est| to cand_idx ([ncand] int32, device), in ASCENDING coordinate order.  cand_est ([ncand] fp32)
 * and est_all ([d] fp32, 16-byte aligned) are optional device outputs (NULL to skip).  k <= ncand <= d. */
int ssgd_unsketch_candidates(ssgd_ctx* ctx, const float* merged, int64_t ncand, int32_t* cand_idx,
                             float* cand_est, float* est_all, void* stream);

/* Algorithm 3 lines 10, 11 and 13: sums the bound v over workers at each candidate (fp64, w = 0..W-1),
 * keeps the k largest by |sum| (ties: earlier position in cand_idx, which is the smaller coordinate
 * when cand_idx is ascending), writes them to out_idx/out_val ([k], device, in cand_idx order), and
 * then sets u and v to +0.0f at those k coordinates in every worker.  Entries of cand_idx must be
 * distinct and in [0, d); an out-of-range entry is skipped and reported by ssgd_status. */
int ssgd_exact_topk(ssgd_ctx* ctx, const int32_t* cand_idx, int64_t ncand, int32_t* out_idx,
                    float* out_val, void* stream);

/* Algorithm 3 lines 5-13 in one call: the stages above, with the workers' values summed before the
 * insert (sum_w S(v_w) = S(sum_w v_w), Section 3), so no per-worker table is materialised.
 * The same kernel keeps each coordinate's sum over the workers (fp64, worker order, rounded once), so line 10
 * reads one number per candidate instead of W values of v; the result is bit-identical to ssgd_exact_topk's.
 * out_idx/out_val: [k] device outputs, ascending coordinate order.  Line 13 is applied as ssgd_set_zero_mode
 * says: by default it is deferred into the next ssgd_step (or ssgd_flush). */
int ssgd_step(ssgd_ctx* ctx, const float* g, int64_t ld_g, float rho, int64_t ncand,
              int32_t* out_idx, float* out_val, void* stream);

/* Algorithm 1 (HEAVYMIX), the selection rule of the paper's analysis, on a merged [r][c] table (device):
 *   line 1  l2 = median over rows of the row's sum of squared counters (fp64)
 *   line 3  H = { i : est_i^2 >= l2 / k }, est the median-of-r estimate, compared in fp64
 *   line 4  Top_k = H plus a uniformly random (k - |H|)-subset of the other coordinates: every coordinate has
 *           a 30-bit priority mixed from (fill_seed, i) -- z = fill_seed + (i+1)*0x9E3779B97F4A7C15,
 *           z = (z^(z>>30))*0xBF58476D1CE4E5B9, z = (z^(z>>27))*0x94D049BB133111EB, z ^= z>>31, priority = z>>34
 *           -- and the non-heavy coordinates with the largest priorities are taken (ties: smaller index).
 *           Should more than k coordinates be heavy (outside the paper's guarantee), the k heavy coordinates
 *           with the largest |est| are kept (fp32 bit pattern of the magnitude, ties: smaller index) and
 *           nothing else.
 *   line 5  out_val[t] = sum over the workers of the bound v at out_idx[t] (fp64, worker order).
 * out_idx / out_val: [k] device outputs, ascending coordinate order.  l2_out (device double) and nheavy_out
 * (device int32) are optional.  The bound state is read, not modified (a deferred zero-out is applied first).
 * Asynchronous on `stream`. */
int ssgd_heavymix(ssgd_ctx* ctx, const float* merged, uint64_t fill_seed, int32_t* out_idx, float* out_val,
                  double* l2_out, int32_t* nheavy_out, void* stream);

/* The same step for a caller whose gradients and results live in HOST memory: copies g_host
 * ([W][ld_g] fp32; pinned memory makes the copy asynchronous) into g_stage (device, [W][ld_g]),
 * runs ssgd_step, copies the k results back to out_idx_host/out_val_host and waits for the stream. */
int ssgd_step_host(ssgd_ctx* ctx, const float* g_host, int64_t ld_g, float rho, int64_t ncand,
                   float* g_stage, int32_t* out_idx_host, float* out_val_host, void* stream);

/* Device pointers into the workspace holding, after ssgd_step, the merged [r][c] table, est[d] and
 * the candidate list [ncand] (for tests and diagnostics).  Any of the outputs may be NULL.  est[d] is
 * only filled when the step ran without pruning (or fell back to the dense path). */
int ssgd_step_buffers(const ssgd_ctx* ctx, const float** merged, const float** est,
                      const int32_t** cand_idx, const float** cand_xs);

/* h_j(i), s_j(i) for n coordinates idx[n] (device int32) -> h_out, s_out ([r][n] int32, device).
 * The same device functions the step uses (Algorithm 4 lines 2, 6, 11); for bit-exactness checks. */
int ssgd_hashes(ssgd_ctx* ctx, const int32_t* idx, int64_t n, int32_t* h_out, int32_t* s_out,
                void* stream);

/* Second round and final top-k WITHOUT a workspace.  (The paper has no counterpart: this exists for
 * the way the library gets embedded, not for the method.)
 *
 * Who needs it: code that is handed gradient and state buffers but may not allocate device memory
 * itself -- a compression hook called from inside a trainer whose caching allocator owns the whole
 * GPU (a raw cudaMalloc there can fail, and it stalls every stream of the device while it runs), or a
 * caller on a latency-critical path that must not trigger allocation at all.  Such a caller cannot
 * provide the workspace that ssgd_bind asks for, so this entry point keeps its scratch (second-round
 * sums, radix histograms, chunk counters) in a fixed array of SSGD_STATIC_SCRATCH_BYTES (1.06 MiB)
 * that is part of the library image: every GPU that loads the library holds that much until the
 * process exits.  The call itself allocates nothing, on the host or on the device.
 *
 * What it computes: Algorithm 3 lines 10-11 exactly as ssgd_exact_topk does -- xs[m] = sum over
 * w = 0..W-1 of v[w][cand_idx[m]] (fp64, that order), then the k entries with the largest |xs|, ties
 * to the earlier position -- written to out_idx/out_val ([k], device) in cand_idx order.  It does NOT
 * zero any state (line 13 stays with the caller) and needs no context: v ([W][ld] fp32, device),
 * cand_idx ([ncand] int32, device, distinct, in [0, d); out-of-range entries count as zero) and the
 * sizes are passed directly.  k <= ncand <= min(d, SSGD_STATIC_MAX_NCAND); a larger ncand is refused
 * with SSGD_ETOOBIG before anything is launched.
 *
 * Sharing: all calls on one GPU use the same array, and it still holds the previous call's data.
 * Each call first clears the parts that must start at zero, in stream order.  Two calls whose work
 * can overlap on the GPU (different streams without an ordering between them, or different host
 * threads doing so) race on the array and give wrong results: keep calls on one device ordered.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that
 * device current); make that first call before starting any stream capture.  Asynchronous on
 * `stream` like the other stage calls. */
#define SSGD_STATIC_MAX_NCAND     262144
#define SSGD_STATIC_SCRATCH_BYTES 1114112
int ssgd_exact_topk_static(const float* v, int64_t ld, int32_t W, int64_t d, const int32_t* cand_idx,
                           int64_t ncand, int64_t k, int32_t* out_idx, float* out_val, void* stream);

/* Optional per-stage timing of ssgd_step with CUDA events recorded on the caller's stream (up to 256
 * steps between collections).  Stages: 0 = the accumulate+insert kernel, 1 = the unsketch kernel,
 * 2 = candidate selection, 3 = second round + final top-k + zero-out.  ssgd_get_stage_times waits for
 * the stream, writes the summed milliseconds per stage to ms_out[SSGD_NSTAGES] and the number of steps
 * they cover to steps_out (host memory), and starts a new collection. */
#define SSGD_NSTAGES 4
int ssgd_set_timing(ssgd_ctx* ctx, int32_t enable);
int ssgd_get_stage_times(ssgd_ctx* ctx, void* stream, double* ms_out, int64_t* steps_out);

/* Number of kernels (and memset nodes) the library has launched through this context so far. */
int ssgd_launch_count(const ssgd_ctx* ctx, int64_t* out);

/* Waits for the stream, then returns SSGD_EDEVICE if a kernel recorded an error since the last call
 * (the flag is cleared), SSGD_ECUDA if the stream reports a CUDA error, else SSGD_OK. */
int ssgd_status(ssgd_ctx* ctx, void* stream);

const char* ssgd_strerror(int code);
const char* ssgd_last_error(const ssgd_ctx* ctx); /* text of the last CUDA error seen, or "" */

#ifdef __cplusplus
}
#endif
#endif
