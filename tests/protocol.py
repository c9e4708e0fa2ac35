"""Staged parity protocol: one ssgd_step of the CUDA library against the CPU oracle.

Both sides get the same g and start from bit-identical u, v.  Because reductions into the sketch
happen in an unspecified order on the GPU, later stages are compared *conditionally*:

  1. u, v after momentum/error accumulation ........ bit-exact (outside the zeroed coordinates)
  2. merged table .................................. |S_gpu - T| <= 1e-5 * M per bucket, M = L1 mass of the bucket
     estimates ..................................... |est_gpu - est| <= tau_i = 1e-5 * max_j M[j][h_j(i)]
  3. candidates .................................... exactly the top-ncand of the GPU's own estimates
                                                     (total order), and admissible w.r.t. the oracle:
                                                     contains every i with |est_i| - tau_i above the highest
                                                     possible threshold, none with |est_i| + tau_i below the lowest
  4. final k ....................................... the oracle's lines 10-11 applied to the GPU's candidates:
                                                     identical index set, identical values
  5. zero-out ...................................... exactly the GPU's k coordinates, every worker, u and v, +0.0f
  6. lock step ..................................... the oracle adopts the GPU's (admissible) selection, so both
                                                     sides enter the next step with bit-identical state.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import select as oracle_select
from paper_1903_04488_b200 import ssgd as S

TABLE_RTOL = 1e-5   # relative to the L1 mass hashed into the bucket


def bucket_tau(orc, M, idx=None, chunk=1 << 20):
    """tau_i = TABLE_RTOL * max_j M[j][h_j(i)] for the listed coordinates (all if idx is None)."""
    if idx is None:
        idx = np.arange(orc.d, dtype=np.int64)
    tau = np.zeros(idx.size)
    for s in range(0, idx.size, chunk):
        h, _ = orc.hashes(idx[s:s + chunk])
        m = np.zeros(h.shape[1])
        for j in range(orc.r):
            m = np.maximum(m, M[j, h[j]])
        tau[s:s + chunk] = TABLE_RTOL * m
    return tau


def oracle_intermediates(orc, g_h, rho, u_o, v_o, ncand, by_linearity):
    """T, M (fp64 [r][c]), est (fp32 [d]), cand (best first) of the oracle for this step; u_o, v_o are
    advanced by the momentum/error accumulation (not zeroed).

    by_linearity=False: the oracle's own step (every worker sketched on its own, then summed).
    by_linearity=True: for sizes where W separate sketches take minutes -- the oracle's accumulate, then
    ONE oracle sketch of the fp64 sum over workers (sum_w S(v_w) = S(sum_w v_w), a pinned property of the
    oracle) and one of sum_w |v_w| for the bucket masses, then the oracle's estimate and selection."""
    if not by_linearity:
        o = orc.step(g_h, rho, u_o, v_o, ncand, zero_state=False, full=True)
        return o["T"], o["M"], o["est"], o["cand"], o["out_idx"]
    orc.accumulate(g_h, rho, u_o, v_o)
    d = orc.d
    x64 = np.zeros(d)
    a64 = np.zeros(d)
    for w in range(orc.W):                      # worker order, fp64
        x64 += v_o[w, :d]
        a64 += np.abs(v_o[w, :d])
    T = orc.sketch(x64)
    M = orc.sketch(a64, with_mass=True)[1]
    est = orc.estimate(T.astype(np.float32))
    cand = oracle_select(est, ncand)
    return T, M, est, cand, None


def check_step(orc, eng, g_dev, rho, ncand, u_o, v_o, *, check_est=True, report=None, by_linearity=False,
               flush=False):
    """Runs eng.step on g_dev and the oracle on the same g; asserts the protocol; adopts.

    orc: oracle.Oracle; eng: bound Ssgd; u_o, v_o: the oracle's numpy state, bit-identical to the
    engine's bound state on entry and again on exit (with flush=True: the state in memory after ssgd_flush;
    otherwise, in the deferred zero mode, the state with the pending zero-out applied on the host copy).
    Returns (out_idx, out_val) as numpy arrays."""
    d, W, k = orc.d, orc.W, orc.k
    dev = g_dev.device
    out_idx = torch.empty(k, dtype=torch.int32, device=dev)
    out_val = torch.empty(k, dtype=torch.float32, device=dev)
    eng.step(g_dev, rho, ncand, out_idx, out_val)
    assert eng.status() == 0
    u_g, v_g, _ = eng._keep
    merged_t, _, cand_t, xs_t = eng.step_buffers(ncand)
    merged_g, cand_g, xs_g = merged_t.cpu().numpy(), cand_t.cpu().numpy(), xs_t.cpu().numpy()
    # the step may have skipped estimates that provably cannot matter (early exit); the dense stage call
    # on the step's own table gives the estimate of EVERY coordinate, and must pick the same candidates
    est_t = torch.empty(d + 4, dtype=torch.float32, device=dev)[:d]
    cand_dense = torch.empty(ncand, dtype=torch.int32, device=dev)
    eng.unsketch_candidates(merged_t, ncand, cand_dense, None, est_t)
    est_g = est_t.cpu().numpy()
    assert (cand_dense.cpu().numpy() == cand_g).all(), "step and dense stage call disagree on the candidates"
    out_idx_g, out_val_g = out_idx.cpu().numpy(), out_val.cpu().numpy()
    if flush:
        eng.flush()
    u_g_h, v_g_h = u_g.cpu().numpy(), v_g.cpu().numpy()
    pending = eng.zero_mode == S.ZERO_DEFERRED and not flush

    # oracle, without its own zero-out
    g_h = g_dev.cpu().numpy()
    T, M, est_o, cand_o, out_idx_o = oracle_intermediates(orc, g_h, rho, u_o, v_o, ncand, by_linearity)
    del g_h

    # 5 + 1: the k chosen coordinates are distinct, ascending, in range (the bit-exact comparison of u and
    # v -- zeros exactly there, the oracle's accumulation everywhere else -- follows the adoption below)
    assert len(np.unique(out_idx_g)) == k and out_idx_g.min() >= 0 and out_idx_g.max() < d
    assert (np.diff(out_idx_g) > 0).all(), "out_idx must be ascending"

    # 2: table and estimates
    err = np.abs(merged_g.astype(np.float64) - T)
    assert (err <= TABLE_RTOL * M).all(), f"table: worst error/mass {np.max(err / np.maximum(M, 1e-300)):.3e}"
    tau = None
    if check_est:
        tau = bucket_tau(orc, M)
        e_err = np.abs(est_g.astype(np.float64) - est_o.astype(np.float64))
        assert (e_err <= tau).all(), "estimates outside tolerance"

    # 3: candidates -- exact given the GPU's own estimates, admissible against the oracle's
    assert (np.diff(cand_g) > 0).all(), "cand_idx must be ascending and distinct"
    want_c = np.sort(oracle_select(est_g, ncand))
    assert (cand_g == want_c).all(), "candidates are not the top-ncand of the GPU's estimates"
    if check_est and ncand < d:
        a = np.abs(est_o.astype(np.float64))
        hi = np.partition(a + tau, d - ncand)[d - ncand]   # ncand-th largest upper bound
        lo = np.partition(a - tau, d - ncand)[d - ncand]   # ncand-th largest lower bound
        inc = np.zeros(d, bool)
        inc[cand_g] = True
        assert inc[(a - tau) > hi].all(), "a coordinate surely above the threshold is missing"
        assert not inc[(a + tau) < lo].any(), "a coordinate surely below the threshold was selected"
    if report is not None:
        report.append(dict(cand_sym_diff=int(np.setxor1d(cand_g, cand_o).size)))

    # 4: final top-k -- the oracle's second round and top-k on the GPU's candidates
    xs = orc.second_round(v_o, cand_g)
    assert (xs_g == xs.astype(np.float32)).all(), "second-round sums differ"
    want_idx, want_val = orc.final_topk(cand_g, xs)
    order = np.argsort(want_idx)
    assert (out_idx_g == want_idx[order]).all(), "final k-set differs from the oracle's on the same candidates"
    assert (out_val_g.view(np.uint32) == want_val[order].view(np.uint32)).all(), "out_val differs"
    if report is not None and out_idx_o is not None:
        report[-1]["final_sym_diff_vs_unadopted"] = int(np.setxor1d(out_idx_g, out_idx_o).size)

    # 5 + 6: adopt the GPU's selection (the oracle zeroes u, v there, every worker); then the whole state
    # must agree bit for bit: +0.0f at the chosen coordinates, the oracle's accumulation everywhere else.
    # In the deferred zero mode without a flush, line 13 is still pending on the GPU side: its memory must then
    # equal the oracle's state BEFORE the zero-out, bit for bit and everywhere (nothing but the accumulation has
    # touched it); that the engine has marked exactly the chosen coordinates shows in the next step's comparison
    # (a missing or extra mark changes u and v there) and in the flushed comparisons.
    if not pending:
        orc.zero(u_o, v_o, out_idx_g)
    for name, got, want in (("u", u_g_h, u_o), ("v", v_g_h, v_o)):
        for w in range(W):
            assert (got[w].view(np.uint32) == want[w].view(np.uint32)).all(), \
                f"{name}[{w}]: state differs from the oracle's (accumulation or zero-out mask)"
    if pending:
        orc.zero(u_o, v_o, out_idx_g)
    return out_idx_g, out_val_g
