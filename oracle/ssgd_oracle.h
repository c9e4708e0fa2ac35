/*
 * ssgd_oracle.h -- plain, slow, single-threaded CPU statement of one Sketched-SGD
 * compression step (Algorithm 3 "Empirical Training", lines 5-13, with the Count
 * Sketch of Algorithm 4), and of the HEAVYMIX selection rule (Algorithm 1).
 *
 * THIS IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be checked
 * against something written directly from the paper.  It shares no code with the
 * CUDA library, is never linked into it, and nothing on the product path may call
 * it.  All pointers are HOST pointers.  Every function returns 0 on success and a
 * negative value on invalid arguments.
 *
 * Precision.  The worker state u, v and the gradients g are fp32, as stored by the
 * method.  Every sum whose order a parallel implementation cannot reproduce (the
 * sketch counters, the second-round sums) is accumulated in fp64 here.  Decisions
 * that turn floating point into an index (which coordinates are the largest) are
 * taken on fp32 values, the precision the state is kept in: the fp64 counters are
 * rounded once to fp32 before the median, the fp64 second-round sums once before
 * the final top-k.
 *
 * Parity status.  Every function below is pinned by the CPU test-suite
 * (tests/test_oracle_pins.py) against closed forms, brute force, library routines
 * and invariants, except one property it cannot pin: the constants of the paper's
 * epsilon-guarantee for the estimate (Section 3; the Count Sketch theorem of Appendix B) are not
 * given, so the *statistical quality* of the hash family is "parity unpinned"
 * (only its variance law for pairwise-independent hashing is checked).
 */
#ifndef SSGD_ORACLE_H
#define SSGD_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SSGD_ORACLE_MAX_R 15

typedef struct ssgd_oracle_ctx ssgd_oracle_ctx;

/* Hash parameters from a seed: for row j = 0..r-1, out[4j..4j+3] = a_j, b_j, a'_j, b'_j.
 * Generator: 64-bit counter s (initially seed); each draw does s += 0x9E3779B97F4A7C15,
 * z = s, z = (z ^ (z>>30)) * 0xBF58476D1CE4E5B9, z = (z ^ (z>>27)) * 0x94D049BB133111EB,
 * value = z ^ (z>>31).  Four draws per row, in the order a, b, a', b':
 * a = 1 + value mod (p-1), b = value mod p, with p = 2^31 - 1.
 * (Algorithm 4 line 2 only says "init sign hashes and bucket hashes".) */
int ssgd_oracle_derive_params(uint64_t seed, int32_t r, uint32_t* out4r);

/* Problem shape of Algorithm 3 / Algorithm 4 init(r, c): d coordinates, r rows (odd,
 * 1..15), c columns, k final sparsity, W workers.  Requires 1 <= d < 2^31 - 1,
 * 1 <= c < 2^31 - 1, 1 <= k <= d, W >= 1. */
int ssgd_oracle_create(ssgd_oracle_ctx** out, int64_t d, int32_t r, int64_t c, int64_t k,
                       int32_t W, uint64_t seed);
void ssgd_oracle_destroy(ssgd_oracle_ctx* ctx);
int ssgd_oracle_get_params(const ssgd_oracle_ctx* ctx, uint32_t* out4r);
/* Replace the hash parameters (tests inject a=1, b=0 etc.). a, a' in [1, p-1]; b, b' in [0, p-1]. */
int ssgd_oracle_set_params(ssgd_oracle_ctx* ctx, const uint32_t* in4r);

/* h_j(i) = ((a_j*i + b_j) mod p) mod c and s_j(i) = 2*(((a'_j*i + b'_j) mod p) & 1) - 1 for the
 * n coordinates idx[0..n-1]; h_out and s_out are [r][n] row-major.  (Algorithm 4 lines 2, 6, 11.) */
int ssgd_oracle_hashes(const ssgd_oracle_ctx* ctx, int64_t n, const int64_t* idx,
                       int32_t* h_out, int32_t* s_out);

/* Algorithm 3 lines 5-6 for every worker: u <- fma(rho, u, g) (one rounding), v <- v + u
 * (the new u).  g is [W][ld_g], u and v are [W][ld]; only the first d entries of a row are used. */
int ssgd_oracle_accumulate(const ssgd_oracle_ctx* ctx, const float* g, int64_t ld_g, float rho,
                           float* u, float* v, int64_t ld);

/* Algorithm 4 update(i, x_i) for i = 0..d-1: T[j][h_j(i)] += s_j(i) * x_i.  T is [r][c] fp64 and
 * is ADDED to (caller zeroes it).  If M is not NULL, M[j][h_j(i)] += |x_i| (the L1 mass of each
 * bucket, used by tests to scale tolerances; not part of the method). */
int ssgd_oracle_sketch_f32(const ssgd_oracle_ctx* ctx, const float* x, double* T, double* M);
int ssgd_oracle_sketch_f64(const ssgd_oracle_ctx* ctx, const double* x, double* T, double* M);

/* Algorithm 3 lines 7-8: sketch every worker's v into its own table, then T = sum over workers
 * in the order w = 0..W-1 (the plain sum, not the mean: the selection does not depend on the
 * positive factor 1/W, and line 10 stores a sum).  T, M are [r][c] outputs (overwritten; M may be
 * NULL).  Tw, if not NULL, receives the W per-worker tables, [W][r][c]. */
int ssgd_oracle_sketch_workers(const ssgd_oracle_ctx* ctx, const float* v, int64_t ld,
                               double* T, double* M, double* Tw);

/* Algorithm 4 estimate(i) for every i: est[i] = median_j( s_j(i) * Tf[j][h_j(i)] ), the middle
 * element of the r sorted values (r is odd).  Tf is the [r][c] table in fp32. */
int ssgd_oracle_estimate(const ssgd_oracle_ctx* ctx, const float* Tf, float* est);

/* The m best of n items under the total order "larger |val| first (compared on the fp32 bit
 * pattern of |val|, so -0 == +0), then smaller id first".  ids may be NULL (id = position).
 * out_pos[0..m-1] receives POSITIONS into val/ids, best first.  (Algorithm 3 lines 9 and 11.) */
int ssgd_oracle_select(int64_t n, const float* val, const int32_t* ids, int64_t m, int32_t* out_pos);

/* Algorithm 3 line 10: xs[t] = sum over w = 0..W-1 (in that order, fp64) of v_w[cand[t]]. */
int ssgd_oracle_second_round(const ssgd_oracle_ctx* ctx, const float* v, int64_t ld,
                             const int32_t* cand, int64_t ncand, double* xs);

/* Algorithm 3 line 13: u_w[i] = v_w[i] = +0.0f for every listed coordinate i and every worker. */
int ssgd_oracle_zero(const ssgd_oracle_ctx* ctx, float* u, float* v, int64_t ld,
                     const int32_t* idx, int64_t n);

/* One whole step, Algorithm 3 lines 5-13, calling the functions above in the paper's order.
 * Required outputs: out_idx[k], out_val[k] (best first).  Optional outputs (NULL to skip):
 * T_out, M_out [r][c] fp64; est_out [d] fp32; cand_out [ncand] (best first); xs_out [ncand] fp64
 * (aligned with cand_out).  If zero_state is 0 the final zeroing (line 13) is skipped so that a
 * test can apply another admissible selection with ssgd_oracle_zero. */
int ssgd_oracle_step(const ssgd_oracle_ctx* ctx, const float* g, int64_t ld_g, float rho,
                     float* u, float* v, int64_t ld, int64_t ncand,
                     int32_t* out_idx, float* out_val,
                     double* T_out, double* M_out, float* est_out,
                     int32_t* cand_out, double* xs_out, int32_t zero_state);

/* ---- Algorithm 1 (HEAVYMIX): the selection rule the paper's theory covers ---------------------------
 *
 * Per-coordinate priority of the random fill: a 64-bit mix of (seed, i),
 *   z = seed + (i+1)*0x9E3779B97F4A7C15;  z = (z^(z>>30))*0xBF58476D1CE4E5B9;
 *   z = (z^(z>>27))*0x94D049BB133111EB;   z ^= z>>31;   priority = upper 30 bits of z.
 * The l coordinates of NH with the largest priority (ties: smaller index) are a uniformly random
 * l-subset of NH for a random seed: that is the reading of "rand_l(NH)" taken here. */
int ssgd_oracle_fill_priority(uint64_t seed, int64_t n, const int64_t* idx, uint32_t* out);

/* Line 1: the squared-norm estimate of the sketched vector, median over rows j of sum_b Tf[j][b]^2
 * (each row is an AMS-type estimator, Appendix B), accumulated in fp64 in bucket order. */
int ssgd_oracle_l2_estimate(const ssgd_oracle_ctx* ctx, const float* Tf, double* l2_out);

/* Lines 1-5 on an fp32 [r][c] table Tf:
 *   l2 = ssgd_oracle_l2_estimate;  est = ssgd_oracle_estimate;
 *   H  = { i : (double)est_i^2 >= l2/k }           (line 3, read with the square its proof uses)
 *   NH = the other coordinates
 *   Top = H + rand_l(NH), l = k - |H|               (line 4): the l members of NH with the largest fill
 *         priority, ties to the smaller index.
 *         |H| > k lies outside the paper's guarantee and its line 4 (l would be negative); the reading taken
 *         then is "the k members of H with the largest |est|" under the method's usual total order
 *         (fp32 bit pattern of the magnitude, ties to the smaller index), and nothing from NH.
 *   out_val[t] = (float) sum over w = 0..W-1 of v_w[out_idx[t]]   (line 5, fp64 in worker order)
 * out_idx is ascending.  nheavy_out receives |H|.  The state is not modified. */
int ssgd_oracle_heavymix(const ssgd_oracle_ctx* ctx, const float* Tf, const float* v, int64_t ld,
                         uint64_t fill_seed, int32_t* out_idx, float* out_val, double* l2_out,
                         int64_t* nheavy_out);

/* ---- 16-bit sketches (Section 6: "quantizing sketches to 16 bits") ------------------------------------
 * What a worker would transmit: its fp32 sketch rounded to a 16-bit format, round-to-nearest-even.
 * fmt 0: IEEE binary16 (values beyond +-65504 saturate to +-65504); fmt 1: bfloat16 (upper 16 bits of fp32).
 * q16 receives the n encodings.  Inputs must be finite. */
int ssgd_oracle_quantize16(int64_t n, const float* x, int32_t fmt, uint16_t* q16);
/* The server's merge of W quantised sketches: out[t] = sum over w = 0..W-1, in that order, in fp32, of the
 * decoded q16[w][t]; q16 is [W][n]. */
int ssgd_oracle_merge16(int32_t W, int64_t n, const uint16_t* q16, int32_t fmt, float* out);

#ifdef __cplusplus
}
#endif
#endif
