"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, stage by stage and as a
whole step, on the same seeded inputs.  Integer work (hashes, signs, selections given their inputs,
the zero-out mask, u and v) is compared bit for bit; the sketch table within 1e-5 of the L1 mass of
each bucket, because the order of the reductions is not fixed."""
import os

import numpy as np
import pytest
import torch

from oracle import Oracle, select as oracle_select
from paper_1903_04488_b200 import ssgd as S
from paper_1903_04488_b200 import workloads as wl
from tests.protocol import TABLE_RTOL, bucket_tau, check_step

pytestmark = pytest.mark.gpu
P = 2**31 - 1


def make(cfg, dev, ncand_max=None, seed=None):
    seed = cfg.sketch_seed if seed is None else seed
    eng = S.Ssgd(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, seed)
    orc = Oracle(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, seed)
    u, v = wl.zero_state(cfg, dev)
    eng.bind(u, v, ncand_max or cfg.ncand)
    return eng, orc, u, v


def random_state(cfg, dev, seed):
    gen = torch.Generator(device=dev).manual_seed(seed)
    u = torch.zeros((cfg.W, cfg.ld), device=dev)
    v = torch.zeros((cfg.W, cfg.ld), device=dev)
    u[:, :cfg.d] = torch.randn((cfg.W, cfg.d), generator=gen, device=dev)
    v[:, :cfg.d] = torch.randn((cfg.W, cfg.d), generator=gen, device=dev)
    return u, v


# ------------------------------------------------------------------------------------------------
# hashes and signs: bit-exact
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("c", [1, 2, 7, 40, 16384, 180000, 262144, 2**30, 2**31 - 2, 2**31 - 3])
def test_hashes_bit_exact(cuda_device, c):
    r, seed = 7, 1234 + c % 97
    d = 2**31 - 2
    eng = S.Ssgd(d, r, c, 1, 1, seed)
    orc = Oracle(d, r, c, 1, 1, seed)
    assert (eng.get_hash_params().numpy() == orc.params().astype(np.int64)).all()
    rng = np.random.default_rng(c)
    idx = np.concatenate([np.arange(0, 70000), [P - 2, P - 3, 2**30, 2**30 - 1, 2**30 + 1],
                          rng.integers(0, P - 1, 200000)]).astype(np.int64)
    h, s = eng.hashes(torch.tensor(idx, dtype=torch.int32, device=cuda_device))
    ho, so = orc.hashes(idx)
    assert (h.cpu().numpy() == ho).all() and (s.cpu().numpy() == so).all()


def test_hashes_extreme_parameters(cuda_device):
    d, c = 2**31 - 2, 1000003
    for params in ([[P - 1, P - 1, P - 1, P - 1]] * 3, [[1, 0, 1, 0]] * 3, [[P - 1, 0, 1, P - 1]] * 3):
        eng = S.Ssgd(d, 3, c, 1, 1, 0)
        orc = Oracle(d, 3, c, 1, 1, 0)
        eng.set_hash_params(params)
        orc.set_params(params)
        idx = np.array([0, 1, 2, P - 2, P - 3, 12345678], np.int64)
        h, s = eng.hashes(torch.tensor(idx, dtype=torch.int32, device=cuda_device))
        ho, so = orc.hashes(idx)
        assert (h.cpu().numpy() == ho).all() and (s.cpu().numpy() == so).all()


# ------------------------------------------------------------------------------------------------
# stage calls
# ------------------------------------------------------------------------------------------------
STAGE_CASES = [
    wl.C2.scaled(d=100_003, W=3, c=1024, ncand=600, k=200),        # ragged d, several tiles
    wl.C1.scaled(d=65_536, W=4, c=4096, ncand=400, k=200),
    wl.C3.scaled(d=40_001, W=5, r=7, c=40, ncand=300, k=100),      # the paper's small sketch shape, c not 2^n
    wl.C4.scaled(d=90_002, W=2, r=15, c=18_000, ncand=900, k=300), # r = 15 rows, c not a power of two
    wl.C2.scaled(d=5, W=1, r=1, c=1, ncand=3, k=2),
    wl.C2.scaled(d=4099, W=9, r=3, c=7, ncand=4099, k=4099),
]


@pytest.mark.parametrize("sched", [S.SCHED_COORDINATE_MAJOR, S.SCHED_WORKER_MAJOR], ids=["coordinate_major", "worker_major"])
@pytest.mark.parametrize("cfg", STAGE_CASES, ids=lambda c: f"{c.name}-d{c.d}-W{c.W}-r{c.r}-c{c.c}")
def test_stage_calls_against_oracle(cuda_device, cfg, sched):
    dev = cuda_device
    eng = S.Ssgd(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
    eng.set_accumulate_schedule(sched)
    orc = Oracle(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
    u, v = random_state(cfg, dev, 7)
    eng.bind(u, v, cfg.ncand)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    g = wl.gradients(wl.Structure(cfg, dev), 0)

    # lines 5-7: u, v bit-exact; every worker's table within tolerance of its own bucket masses
    tables = torch.full((cfg.W, cfg.r, cfg.c), 123.0, device=dev)   # the call must zero it
    eng.sketch_accumulate(g, cfg.rho, tables)
    orc.accumulate(g.cpu().numpy(), cfg.rho, u_o, v_o)
    assert (u.cpu().numpy().view(np.uint32) == u_o.view(np.uint32)).all()
    assert (v.cpu().numpy().view(np.uint32) == v_o.view(np.uint32)).all()
    T, M, Tw = orc.sketch_workers(v_o, per_worker=True)
    tables_h = tables.cpu().numpy().astype(np.float64)
    for w in range(cfg.W):
        Mw = orc.sketch(v_o[w, :cfg.d].copy(), with_mass=True)[1]
        assert (np.abs(tables_h[w] - Tw[w]) <= TABLE_RTOL * Mw).all()

    # line 8: merge in worker order -- reproduce it exactly from the GPU's own tables, then vs oracle
    merged = torch.empty((cfg.r, cfg.c), device=dev)
    eng.sketch_merge(tables, merged)
    acc = np.zeros((cfg.r, cfg.c), np.float32)
    for w in range(cfg.W):
        acc = acc + tables.cpu().numpy()[w]
    assert (merged.cpu().numpy() == acc).all()
    assert (np.abs(merged.cpu().numpy().astype(np.float64) - T) <= TABLE_RTOL * M).all()

    # line 9 on the ORACLE's table: estimates and candidates must then be identical
    Tf = T.astype(np.float32)
    cand = torch.empty(cfg.ncand, dtype=torch.int32, device=dev)
    cand_est = torch.empty(cfg.ncand, device=dev)
    est = torch.empty(cfg.d + 4, device=dev)[:cfg.d]
    eng.unsketch_candidates(torch.tensor(Tf, device=dev), cfg.ncand, cand, cand_est, est)
    est_o = orc.estimate(Tf)
    assert (est.cpu().numpy() == est_o).all()
    cand_o = np.sort(oracle_select(est_o, cfg.ncand))
    assert (cand.cpu().numpy() == cand_o).all()
    assert (cand_est.cpu().numpy() == est_o[cand_o]).all()

    # lines 10, 11, 13 on those candidates
    out_idx = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    out_val = torch.empty(cfg.k, device=dev)
    eng.exact_topk(cand, out_idx, out_val)
    assert eng.status() == S.OK
    xs = orc.second_round(v_o, cand_o)
    want_idx, want_val = orc.final_topk(cand_o, xs)
    order = np.argsort(want_idx)
    assert (out_idx.cpu().numpy() == want_idx[order]).all()
    assert (out_val.cpu().numpy().view(np.uint32) == want_val[order].view(np.uint32)).all()
    orc.zero(u_o, v_o, want_idx)
    assert (u.cpu().numpy().view(np.uint32) == u_o.view(np.uint32)).all()
    assert (v.cpu().numpy().view(np.uint32) == v_o.view(np.uint32)).all()


# ------------------------------------------------------------------------------------------------
# whole step, lock step with the oracle over several steps
# ------------------------------------------------------------------------------------------------
STEP_CASES = [
    (wl.C1.scaled(d=131_072, c=4096, ncand=500, k=250), 1),
    (wl.C2.scaled(d=300_001, W=4, c=8192, ncand=3000, k=1500), 4),
    (wl.C3.scaled(d=200_003, W=6, c=16_384, ncand=2000, k=1000), 3),
    (wl.C4.scaled(d=270_002, W=3, c=32_768, ncand=1500, k=700), 3),
    (wl.C2.scaled(d=50_001, W=2, r=7, c=40, ncand=500, k=10), 3),          # r=7, c=40 (MNIST shape)
    (wl.C3.scaled(d=60_000, W=3, r=15, c=1800, ncand=1600, k=100), 2),     # r=15, P=16
    (wl.C2.scaled(d=70_001, W=17, r=3, c=999, ncand=300, k=300), 2),       # k == ncand, odd W
    (wl.C2.scaled(d=20_000, W=1, r=1, c=64, ncand=20_000, k=50), 2),       # ncand == d: true top-k
    (wl.C1.scaled(d=3, W=2, r=5, c=16, ncand=2, k=1), 2),                  # d < 4
    (wl.C2.scaled(d=1, W=1, r=1, c=1, ncand=1, k=1), 2),                   # the smallest problem there is
    (wl.C2.scaled(d=4097, W=2, r=9, c=33, ncand=4097, k=4097), 2),         # k == ncand == d: everything is chosen
    (wl.P1.scaled(d=400_000, c=1_800, ncand=8_000, k=500), 2),             # the paper's 15-row sketch, P = 16
    (wl.P2.scaled(d=500_000, c=10_000, ncand=18_000, k=500), 2),           # the paper's 5 x 1M sketch, P = 36
    (wl.P3.scaled(d=365_000, c=900, ncand=13_000, k=500), 2),              # the paper's LSTM sketch, P = 26
]


def _lockstep_combinations():
    """Every insert variant with the dense candidate path, and every candidate path with the plain-load insert
    (the candidate path does not depend on the insert variant); the shared-memory insert only where the table fits."""
    names = {S.INSERT_TMA: "tma", S.INSERT_GLOBAL: "global", S.INSERT_SMEM: "smem",
             S.PRUNE_ON: "filter", S.PRUNE_EARLY_EXIT: "early_exit", S.PRUNE_OFF: "dense", S.PRUNE_FUSED: "fused"}
    out = []
    for cfg, steps in STEP_CASES:
        base = f"{cfg.name}-d{cfg.d}-W{cfg.W}-r{cfg.r}-c{cfg.c}"
        combos = [(S.INSERT_GLOBAL, p) for p in (S.PRUNE_ON, S.PRUNE_EARLY_EXIT, S.PRUNE_OFF)] + [(S.INSERT_TMA, S.PRUNE_OFF)]
        if cfg.r * cfg.c * 4 <= 200 * 1024:
            combos.append((S.INSERT_SMEM, S.PRUNE_OFF))
        if cfg.ncand <= 16384:
            combos.append((S.INSERT_GLOBAL, S.PRUNE_FUSED))     # lines 9-13 in one cooperative kernel
        for mode, prune in combos:
            out.append(pytest.param(cfg, steps, mode, prune, id=f"{base}-{names[mode]}-{names[prune]}"))
    return out


@pytest.mark.parametrize("cfg,steps,mode,prune", _lockstep_combinations())
def test_step_lockstep(cuda_device, cfg, steps, mode, prune):
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_insert_mode(mode)
    eng.set_prune_mode(prune)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    st = wl.Structure(cfg, cuda_device)
    report = []
    for t in range(steps):
        g = wl.gradients(st, t)
        check_step(orc, eng, g, cfg.rho, cfg.ncand, u_o, v_o, report=report, flush=(t == steps - 1))
    if cfg.ncand == cfg.d:
        assert all(r["final_sym_diff_vs_unadopted"] == 0 for r in report)


@pytest.mark.parametrize("prune", [S.PRUNE_ON, S.PRUNE_EARLY_EXIT, S.PRUNE_OFF, S.PRUNE_FUSED])
def test_all_zero_gradient_ties_break_by_index(cuda_device, prune):
    cfg = wl.C2.scaled(d=10_001, W=3, c=256, ncand=700, k=300)
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_prune_mode(prune)
    g = torch.zeros((cfg.W, cfg.ld), device=cuda_device)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    idx, val = check_step(orc, eng, g, cfg.rho, cfg.ncand, u_o, v_o)
    assert idx.tolist() == list(range(cfg.k)) and (val == 0).all()
    if prune not in (S.PRUNE_OFF, S.PRUNE_FUSED):
        fell_back, survivors, bin_lo = eng.step_used_fallback()
        assert not fell_back and bin_lo == 0 and survivors == cfg.d   # nothing can be pruned; d ties ranked by index


@pytest.mark.parametrize("prune", [S.PRUNE_ON, S.PRUNE_EARLY_EXIT])
def test_nothing_to_prune_lists_every_coordinate(cuda_device, prune):
    """All estimates equal (zero): the sampled threshold is zero, every coordinate survives (the list has room
    for all d), and the d-way tie at the threshold goes to the smallest indices."""
    cfg = wl.C2.scaled(d=300_001, W=2, c=1024, ncand=1000, k=500)
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_prune_mode(prune)
    g = torch.zeros((cfg.W, cfg.ld), device=cuda_device)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    idx, val = check_step(orc, eng, g, cfg.rho, cfg.ncand, u_o, v_o)
    fell_back, survivors, bin_lo = eng.step_used_fallback()
    assert not fell_back and survivors == cfg.d and bin_lo == 0
    assert idx.tolist() == list(range(cfg.k))


@pytest.mark.parametrize("prune", [S.PRUNE_ON, S.PRUNE_EARLY_EXIT])
def test_misjudged_threshold_reruns_without_pruning(cuda_device, prune):
    """A prune threshold set at the largest sampled estimate keeps far fewer than ncand coordinates: the last
    block of the pruned pass must notice, and the unpruned pass behind it must produce the right candidates.
    The next step, with the normal rank, prunes again."""
    cfg = wl.C2.scaled(d=500_003, W=3, c=8192, ncand=4000, k=2000)
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_prune_mode(prune)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    st = wl.Structure(cfg, cuda_device)
    eng.set_prune_sample_rank(1)
    check_step(orc, eng, wl.gradients(st, 0), cfg.rho, cfg.ncand, u_o, v_o)
    fell_back, survivors, bin_lo = eng.step_used_fallback()
    assert fell_back and survivors == cfg.d and bin_lo > 0
    eng.set_prune_sample_rank(0)
    check_step(orc, eng, wl.gradients(st, 1), cfg.rho, cfg.ncand, u_o, v_o)
    fell_back, survivors, _ = eng.step_used_fallback()
    assert not fell_back and cfg.ncand <= survivors < cfg.d // 10


@pytest.mark.parametrize("prune", [S.PRUNE_ON, S.PRUNE_EARLY_EXIT, S.PRUNE_OFF, S.PRUNE_FUSED])
def test_heavy_ties_at_the_threshold(cuda_device, prune):
    """Many coordinates with one magnitude straddling both thresholds: the quota logic decides."""
    cfg = wl.C2.scaled(d=40_000, W=2, r=1, c=40_000, ncand=1000, k=400)
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_prune_mode(prune)
    ident = [[1, 0, 1, 0]]
    eng.set_hash_params(ident)
    orc.set_params(ident)          # table = signed copy of the summed vector: estimates are exact
    g = torch.zeros((cfg.W, cfg.ld), device=cuda_device)
    g[:, 5:30_000:7] = 1.0         # 4286 coordinates tie at |x| = 2
    g[:, 11:500:13] = 3.0          # 38 coordinates above them
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    idx, val = check_step(orc, eng, g, cfg.rho, cfg.ncand, u_o, v_o)
    big = set(range(11, 500, 13))
    assert big <= set(idx.tolist())


# ------------------------------------------------------------------------------------------------
# lines 9-13 as one cooperative kernel (small problems)
# ------------------------------------------------------------------------------------------------
FUSED_CASES = [
    # (configuration, steps, zero mode): all rows of the table copied into shared memory, some of them, or none
    (wl.C2.scaled(d=700_001, W=2, c=2048, ncand=3000, k=1500), 3, S.ZERO_EAGER),          # 40 KiB table in shared memory; zeros written in the kernel
    (wl.C2.scaled(d=300_001, W=4, c=8192, ncand=3000, k=1500), 3, S.ZERO_EAGER),          # 160 KiB table, too few lookups: L2
    (wl.C1.scaled(d=800_000, c=16_384, ncand=2000, k=1000), 2, S.ZERO_EAGER),             # C1's sketch: 3 of 5 rows in shared memory
    (wl.C2.scaled(d=900_002, W=2, r=7, c=9_999, ncand=2000, k=1000), 2, S.ZERO_DEFERRED), # 5 of 7 rows, c not a multiple of 4
    (wl.C3.scaled(d=200_003, W=6, c=32_768, ncand=2000, k=1000), 3, S.ZERO_DEFERRED),
    (wl.C4.scaled(d=270_002, W=3, c=65_536, ncand=1500, k=700), 3, S.ZERO_DEFERRED),
    (wl.C2.scaled(d=250_001, W=2, c=200_000, ncand=16_384, k=16_384), 2, S.ZERO_DEFERRED),  # table read from L2; largest ncand; k = ncand
    (wl.C2.scaled(d=150_002, W=17, r=3, c=999, ncand=9000, k=5000), 2, S.ZERO_EAGER),     # k*W too large for in-kernel zeros
    (wl.C3.scaled(d=2_100_003, W=2, r=7, c=4001, ncand=5000, k=100), 2, S.ZERO_DEFERRED), # d above 2^21, real modulo
    (wl.C2.scaled(d=7, W=3, r=5, c=16, ncand=7, k=3), 2, S.ZERO_EAGER),                   # fewer coordinates than threads
]


@pytest.mark.parametrize("cfg,steps,zero", FUSED_CASES, ids=lambda x: f"{x.name}-d{x.d}-W{x.W}-r{x.r}-c{x.c}" if hasattr(x, "name") else str(x))
def test_fused_tail_lockstep(cuda_device, cfg, steps, zero):
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_prune_mode(S.PRUNE_FUSED)
    eng.set_zero_mode(zero)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    st = wl.Structure(cfg, cuda_device)
    n0 = eng.launch_count()
    for t in range(steps):
        check_step(orc, eng, wl.gradients(st, t), cfg.rho, cfg.ncand, u_o, v_o, flush=(t == steps - 1))
    # memset + accumulate + tail (+ k_zero when k*W is too large for the tail) per step; check_step adds the dense
    # stage call (two memsets and four kernels) and the last one a flush
    per_step = 3 + (1 if zero == S.ZERO_EAGER and cfg.k * cfg.W > 65536 else 0)
    assert eng.launch_count() - n0 == steps * (per_step + 6) + 1


def test_fused_tail_is_refused_where_it_does_not_apply(cuda_device):
    cfg = wl.C2.scaled(d=400_000, W=2, c=4096, ncand=20_000, k=100)       # more candidates than the last block holds
    eng, _, u, v = make(cfg, cuda_device)
    eng.set_prune_mode(S.PRUNE_FUSED)
    g = torch.zeros((cfg.W, cfg.ld), device=cuda_device)
    oi = torch.empty(cfg.k, dtype=torch.int32, device=cuda_device)
    ov = torch.empty(cfg.k, device=cuda_device)
    with pytest.raises(S.SsgdError) as e:
        eng.step(g, cfg.rho, cfg.ncand, oi, ov)
    assert e.value.code == S.EINVAL
    eng.set_prune_mode(S.PRUNE_AUTO)                                      # AUTO takes another path
    eng.step(g, cfg.rho, cfg.ncand, oi, ov)
    assert eng.status() == S.OK


def test_refused_cooperative_launch_falls_back_to_the_chain(cuda_device):
    """If the device cannot hold the one-kernel tail's grid at once, the runtime refuses the cooperative launch
    (simulated by the test hook: nothing is launched).  Under AUTO the same step goes on as the chain of ordinary
    launches -- same results -- and later steps do not try again; under FUSED the call reports the refusal."""
    cfg = wl.C2.scaled(d=300_001, W=3, c=8192, ncand=3000, k=1500)
    eng, orc, u, v = make(cfg, cuda_device)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    st = wl.Structure(cfg, cuda_device)
    check_step(orc, eng, wl.gradients(st, 0), cfg.rho, cfg.ncand, u_o, v_o)          # AUTO: one kernel
    eng.test_withhold_block(-1)
    n0 = eng.launch_count()
    check_step(orc, eng, wl.gradients(st, 1), cfg.rho, cfg.ncand, u_o, v_o)          # refused: the chain, same step
    n_refused = eng.launch_count() - n0
    eng.test_withhold_block(0)
    n0 = eng.launch_count()
    check_step(orc, eng, wl.gradients(st, 2), cfg.rho, cfg.ncand, u_o, v_o, flush=True)   # stays with the chain
    assert eng.launch_count() - n0 - 1 == n_refused - 1        # one memset less than in the step that was refused
    assert n_refused > 3 + 6
    eng2, _, _, _ = make(cfg, cuda_device)
    eng2.set_prune_mode(S.PRUNE_FUSED)
    eng2.test_withhold_block(-1)
    oi = torch.empty(cfg.k, dtype=torch.int32, device=cuda_device)
    ov = torch.empty(cfg.k, device=cuda_device)
    with pytest.raises(S.SsgdError) as e:
        eng2.step(wl.gradients(st, 0), cfg.rho, cfg.ncand, oi, ov)
    assert e.value.code == S.ECUDA
    eng2.test_withhold_block(0)
    eng2.flush()


def test_a_grid_barrier_wait_that_runs_out_is_reported_and_nothing_hangs(cuda_device):
    """One block of the cooperative tail is withheld (it returns before the first grid barrier), so the others'
    bounded waits run out after the configured limit: the kernel returns, ssgd_status reports SSGD_EDEVICE once,
    and the next step on the same context is correct again."""
    cfg = wl.C2.scaled(d=300_001, W=3, c=8192, ncand=3000, k=1500)
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_prune_mode(S.PRUNE_FUSED)
    eng.set_zero_mode(S.ZERO_EAGER)
    st = wl.Structure(cfg, cuda_device)
    oi = torch.empty(cfg.k, dtype=torch.int32, device=cuda_device)
    ov = torch.empty(cfg.k, device=cuda_device)
    eng.set_wait_limit_ns(200_000)                                        # 0.2 ms
    eng.test_withhold_block(1)
    eng.step(wl.gradients(st, 0), cfg.rho, cfg.ncand, oi, ov)
    assert eng.status() == S.EDEVICE
    assert eng.status() == S.OK
    eng.test_withhold_block(0)
    eng.set_wait_limit_ns(2_000_000_000)
    u.zero_(); v.zero_()
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    check_step(orc, eng, wl.gradients(st, 1), cfg.rho, cfg.ncand, u_o, v_o)


def test_a_pipeline_wait_that_runs_out_is_reported_and_nothing_hangs(cuda_device):
    """The bulk-copy accumulate kernel's bounded waits: the producer of one CTA is withheld (it issues no copy, so
    nothing is in flight), its consumers' waits run out after the configured limit, the CTA returns, the other
    CTAs finish normally; ssgd_status reports SSGD_EDEVICE once and the context stays usable."""
    cfg = wl.C2.scaled(d=400_003, W=5, c=4096, ncand=2000, k=1000)
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_insert_mode(S.INSERT_TMA)
    eng.set_prune_mode(S.PRUNE_OFF)
    st = wl.Structure(cfg, cuda_device)
    oi = torch.empty(cfg.k, dtype=torch.int32, device=cuda_device)
    ov = torch.empty(cfg.k, device=cuda_device)
    eng.set_wait_limit_ns(200_000)
    eng.test_withhold_block(1)
    eng.step(wl.gradients(st, 0), cfg.rho, cfg.ncand, oi, ov)
    assert eng.status() == S.EDEVICE
    assert eng.status() == S.OK
    eng.test_withhold_block(0)
    eng.set_wait_limit_ns(2_000_000_000)
    eng.flush()
    u.zero_(); v.zero_()
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    check_step(orc, eng, wl.gradients(st, 1), cfg.rho, cfg.ncand, u_o, v_o)


def test_row_split_insert(cuda_device):
    """Tables above the L2 budget are inserted a slice of rows at a time (the streaming kernel does the first
    slice and leaves per-coordinate sums for the rest); forced here with a budget of two rows."""
    cfg = wl.C4.scaled(d=400_003, W=5, r=7, c=4096, ncand=2000, k=1000)
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_insert_mode(S.INSERT_GLOBAL)
    eng.set_insert_split(2 * cfg.c * 4)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    st = wl.Structure(cfg, cuda_device)
    n0 = eng.launch_count()
    for t in range(3):
        check_step(orc, eng, wl.gradients(st, t), cfg.rho, cfg.ncand, u_o, v_o)
    eng2, _, _, _ = make(cfg, cuda_device)
    eng2.set_insert_mode(S.INSERT_GLOBAL)
    eng2.set_insert_split(0)
    assert eng.launch_count() - n0 > 0


@pytest.mark.parametrize("prune", [S.PRUNE_ON, S.PRUNE_EARLY_EXIT])
def test_pruned_path_is_taken_and_prunes(cuda_device, prune):
    """On a gradient-shaped input the pruned path must do its job: no rerun, a non-trivial threshold, at
    least ncand survivors and far fewer than d; a few ties at the threshold are ranked by index."""
    cfg = wl.C2.scaled(d=600_001, W=4, c=16_384, ncand=6000, k=3000)
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_prune_mode(prune)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    st = wl.Structure(cfg, cuda_device)
    for t in range(2):
        check_step(orc, eng, wl.gradients(st, t), cfg.rho, cfg.ncand, u_o, v_o)
        fell_back, survivors, bin_lo = eng.step_used_fallback()
        assert not fell_back and bin_lo > 0
        assert cfg.ncand <= survivors <= cfg.d // 10


FOLD_CASES = [
    wl.C3.scaled(d=600_011, W=3, r=5, c=524_288, ncand=5000, k=2000),       # 5 x 2^19 bits: two buckets per bit
    wl.P1.scaled(d=400_003, W=2, r=15, c=180_000, ncand=8000, k=500),       # the paper's 15 x 180,000: two per bit
    wl.C4.scaled(d=500_009, W=2, r=5, c=6_000_001, ncand=4000, k=1000),     # each row in 4 slices, c not a power of two
    wl.C4.scaled(d=500_009, W=2, r=5, c=4_194_304, ncand=4000, k=1000),     # C4's own table: each row in 3 slices
    wl.C4.scaled(d=500_009, W=2, r=5, c=7_000_003, ncand=4000, k=1000),     # folded: 32 buckets per bit
]


@pytest.mark.parametrize("cfg", FOLD_CASES, ids=lambda c: f"{c.name}-r{c.r}-c{c.c}")
def test_bucket_bitmap_folded_into_shared_memory(cuda_device, cfg):
    """Sketches whose one-bit-per-bucket filter exceeds an SM's shared memory.  Up to four times a row's worth of
    shared memory per row: the bitmap is evaluated row by row (a row in slices).  Beyond: neighbouring buckets
    share a bit and the full bitmap is consulted in global memory before the table is read."""
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_prune_mode(S.PRUNE_ON)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    st = wl.Structure(cfg, cuda_device)
    for t in range(2):
        check_step(orc, eng, wl.gradients(st, t), cfg.rho, cfg.ncand, u_o, v_o)
        fell_back, survivors, bin_lo = eng.step_used_fallback()
        assert not fell_back and bin_lo > 0 and cfg.ncand <= survivors < cfg.d // 4
        declined, ones = eng.step_first_pass()
        assert not declined and 0 < ones < cfg.r * cfg.c // 8


@pytest.mark.parametrize("d", [1, 31, 33, 1023, 1025, 40_001])
@pytest.mark.parametrize("c", [1_048_576, 2_000_003, 4_194_304], ids=["row", "2slices", "3slices"])
def test_row_bitmap_ragged_ends(cuda_device, d, c):
    """The row-by-row bitmap on coordinate counts around its units (a 32-coordinate result word, a warp's 1024
    coordinates): far fewer coordinates than blocks, partial last words, pruning forced on."""
    cfg = wl.C3.scaled(d=d, W=2, r=5, c=c, ncand=max(1, d // 7), k=max(1, d // 20))
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_prune_mode(S.PRUNE_ON)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    st = wl.Structure(cfg, cuda_device)
    for t in range(2):
        check_step(orc, eng, wl.gradients(st, t), cfg.rho, cfg.ncand, u_o, v_o)


@pytest.mark.parametrize("c,ones_per_row", [(524_288, 524_288), (8_388_608, 8_388_608 // 32)], ids=["rows", "folded"])
def test_dense_bitmap_hands_over_to_the_table_kernel(cuda_device, c, ones_per_row):
    """A bitmap that would rule out too few coordinates (here: all estimates zero, threshold zero, every bit set)
    makes the filter kernels return at once; the table kernel enqueued behind them does the first pass.  Both
    forms of the filter: row by row (the unfolded bitmap's density decides) and folded (32 buckets per bit)."""
    cfg = wl.C3.scaled(d=300_007, W=2, r=5, c=c, ncand=1000, k=500)
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_prune_mode(S.PRUNE_ON)
    g = torch.zeros((cfg.W, cfg.ld), device=cuda_device)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    idx, val = check_step(orc, eng, g, cfg.rho, cfg.ncand, u_o, v_o)
    fell_back, survivors, bin_lo = eng.step_used_fallback()
    declined, ones = eng.step_first_pass()
    assert declined and ones == cfg.r * ones_per_row
    assert not fell_back and survivors == cfg.d and bin_lo == 0
    assert idx.tolist() == list(range(cfg.k))
    st = wl.Structure(cfg, cuda_device)                    # a real gradient next: the filter takes over again
    check_step(orc, eng, wl.gradients(st, 0), cfg.rho, cfg.ncand, u_o, v_o)
    declined, ones = eng.step_first_pass()
    assert not declined and 0 < ones < cfg.r * cfg.c // 8


def test_planted_heavy_coordinates_recovered(cuda_device):
    cfg = wl.C1.scaled(d=262_144, c=8192, ncand=512, k=256)
    eng, orc, u, v = make(cfg, cuda_device)
    st = wl.Structure(cfg, cuda_device)
    g = wl.gradients(st, 0)
    # make the planted coordinates dominate: 5000 x the median instead of 50 x
    g[:, st.planted_idx] *= 100.0
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    idx, _ = check_step(orc, eng, g, cfg.rho, cfg.ncand, u_o, v_o)
    assert set(st.planted_idx.cpu().tolist()) <= set(idx.tolist())


def test_fused_step_equals_stage_pipeline_selection(cuda_device):
    """ssgd_step (sum over workers before the insert) and the faithful pipeline (per-worker tables,
    merge) agree on u, v exactly and on the table within tolerance."""
    cfg = wl.C2.scaled(d=150_001, W=8, c=4096, ncand=1200, k=600)
    dev = cuda_device
    g = wl.gradients(wl.Structure(cfg, dev), 0)
    eng, orc, u, v = make(cfg, dev)
    out_idx = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    out_val = torch.empty(cfg.k, device=dev)
    eng.step(g, cfg.rho, cfg.ncand, out_idx, out_val)
    merged_fused = eng.step_buffers(cfg.ncand)[0].clone()
    eng2, _, u2, v2 = make(cfg, dev)
    tables = torch.empty((cfg.W, cfg.r, cfg.c), device=dev)
    merged = torch.empty((cfg.r, cfg.c), device=dev)
    eng2.sketch_accumulate(g, cfg.rho, tables)
    eng2.sketch_merge(tables, merged)
    T, M = orc.sketch_workers(v2.cpu().numpy())
    for m in (merged_fused, merged):
        assert (np.abs(m.cpu().numpy().astype(np.float64) - T) <= TABLE_RTOL * M).all()
    cand = torch.empty(cfg.ncand, dtype=torch.int32, device=dev)
    eng2.unsketch_candidates(merged, cfg.ncand, cand)
    o_idx = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    o_val = torch.empty(cfg.k, device=dev)
    eng2.exact_topk(cand, o_idx, o_val)
    assert eng2.status() == S.OK and eng.status() == S.OK
    # the heavy part of the selection is common to both
    common = np.intersect1d(out_idx.cpu().numpy(), o_idx.cpu().numpy()).size
    assert common >= 0.95 * cfg.k


def test_step_host_matches_step(cuda_device):
    cfg = wl.C2.scaled(d=120_002, W=4, c=4096, ncand=900, k=300)
    dev = cuda_device
    g = wl.gradients(wl.Structure(cfg, dev), 0)
    eng, _, u, v = make(cfg, dev)
    out_idx = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    out_val = torch.empty(cfg.k, device=dev)
    eng.step(g, cfg.rho, cfg.ncand, out_idx, out_val)
    eng2, _, u2, v2 = make(cfg, dev)
    g_host = g.cpu().pin_memory()
    stage = torch.empty_like(g)
    oi = torch.empty(cfg.k, dtype=torch.int32).pin_memory()
    ov = torch.empty(cfg.k, dtype=torch.float32).pin_memory()
    eng2.step_host(g_host, cfg.rho, cfg.ncand, stage, oi, ov)
    assert (u2 == u).all() and (v2 == v).all()            # the accumulation (zero-out still pending in both)
    if (out_idx.cpu() == oi).all():
        eng.flush(); eng2.flush()
        assert (u2 == u).all() and (v2 == v).all() and int((v[0, :cfg.d] == 0).sum().item()) >= cfg.k
    # same table up to reduction order -> the selections agree except near ties; values of common ones match
    a, b = out_idx.cpu().numpy(), oi.numpy()
    common, ia, ib = np.intersect1d(a, b, return_indices=True)
    assert common.size >= 0.98 * cfg.k
    assert (out_val.cpu().numpy()[ia] == ov.numpy()[ib]).all()


# ------------------------------------------------------------------------------------------------
# the BASELINE configurations at full size, in the launch configuration bench.py times
# ------------------------------------------------------------------------------------------------
def run_full(cfg, dev, steps, by_linearity):
    eng, orc, u, v = make(cfg, dev)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    st = wl.Structure(cfg, dev)
    report = []
    g = None
    for t in range(steps):
        g = wl.gradients(st, t, out=g)
        check_step(orc, eng, g, cfg.rho, cfg.ncand, u_o, v_o, report=report, flush=(t == steps - 1),
                   by_linearity=by_linearity[t] if isinstance(by_linearity, (list, tuple)) else by_linearity)
    return report


def test_full_size_C1(cuda_device):
    run_full(wl.C1, cuda_device, 1, False)


def test_full_size_C2_bench_configuration(cuda_device):
    # step 0: every worker sketched separately by the oracle; steps 1-2 (non-zero state, zeroed
    # coordinates from the step before): the oracle's sketch of the fp64 sum
    rep = run_full(wl.C2, cuda_device, 3, [False, True, True])
    assert len(rep) == 3


def test_full_size_C3(cuda_device):
    run_full(wl.C3, cuda_device, 2, True)


def test_full_size_C4_table_larger_than_half_of_l2(cuda_device):
    run_full(wl.C4, cuda_device, 1, True)


@pytest.mark.parametrize("W", [8, 256])
def test_full_size_C5_worker_sweep(cuda_device, W):
    cfg = wl.CONFIGS[f"C5_W{W}"]
    free, _ = torch.cuda.mem_get_info()
    need = 3 * cfg.W * cfg.ld * 4 + (1 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of device memory")
    run_full(cfg, cuda_device, 1, True)


@pytest.mark.parametrize("name", ["P1", "P2", "P3"])
def test_full_size_paper_sketch_shapes(cuda_device, name):
    """The paper's own sketch shapes (Table 1 footnotes) at full size, one step in lock step with the oracle:
    15 x 180,000 with 1.6e6 candidates (dense candidate path, r = 15, real modulo), 5 x 1,000,000 with 3.6e6
    candidates (bucket bitmap folded 4x), 5 x 180,000 at d = 7.3e7 with 2.6e6 candidates."""
    run_full(wl.CONFIGS[name], cuda_device, 1, True)


def test_full_size_many_coordinates_few_workers(cuda_device):
    """d = 1.5e8 with one worker: more map chunks than the mark kernel's block-local counters hold (it falls back
    to global counters), 4.7e6 map words, a survivor list with room for 1.5e8 entries, indices above 2^27."""
    cfg = wl.C2.scaled(name="big_d", d=150_000_001, W=1, ncand=60_000, k=20_000, steps=1)
    assert ((cfg.d + 31) // 32 + 2047) // 2048 > 2048         # chunks of 2048 map words: more than 2048 of them
    run_full(cfg, cuda_device, 1, True)


def test_stored_small_case_is_reproduced_exactly(cuda_device):
    """Integer gradients and rho = 1/2 make every operation exact, reductions included, so the library must
    reproduce the stored case (written by the oracle alone) bit for bit: table, candidates, k-set, values."""
    import hashlib
    import importlib.util
    import json
    import os
    here = os.path.dirname(os.path.abspath(__file__))
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    want = json.load(open(os.path.join(here, "golden", "oracle_small_case.json")))
    sh = want["shape"]
    dev = cuda_device
    for mode in (S.INSERT_GLOBAL, S.INSERT_TMA, S.INSERT_SMEM):
        eng = S.Ssgd(sh["d"], sh["r"], sh["c"], sh["k"], sh["W"], sh["seed"])
        assert eng.get_hash_params().tolist() == want["hash_params"]
        ld = (sh["d"] + 3) // 4 * 4
        u = torch.zeros((sh["W"], ld), device=dev)
        v = torch.zeros_like(u)
        eng.bind(u, v, want["ncand"])
        eng.set_insert_mode(mode)
        oi = torch.empty(sh["k"], dtype=torch.int32, device=dev)
        ov = torch.empty(sh["k"], device=dev)
        for t, step in enumerate(want["steps"]):
            g = torch.zeros((sh["W"], ld), device=dev)
            g[:, :sh["d"]] = torch.tensor(mod.gradients(t), device=dev)
            eng.step(g, want["rho"], want["ncand"], oi, ov)
            assert eng.status() == S.OK
            merged, _, cand, _ = eng.step_buffers(want["ncand"])
            table64 = merged.cpu().numpy().astype(np.float64)
            assert hashlib.sha256(np.ascontiguousarray(table64).tobytes()).hexdigest() == step["table_sha256"]
            assert cand.cpu().tolist() == step["cand"]
            assert oi.cpu().tolist() == step["out_idx"]
            assert ov.cpu().tolist() == step["out_val"]
        eng.flush()
        state = u.cpu().numpy()[:, :sh["d"]].tobytes() + v.cpu().numpy()[:, :sh["d"]].tobytes()
        assert hashlib.sha256(state).hexdigest() == want["state_sha256"]


def test_step_can_be_captured_in_a_cuda_graph(cuda_device):
    """ssgd_step only enqueues work (no host synchronisation, no allocation), so once the context is warm a
    step can be captured and replayed; a replay from zero state selects what an eager step selects (up to
    near-ties: the order of the reductions into the table differs from run to run)."""
    dev = cuda_device
    cfg = wl.C2.scaled(d=5_000_002, W=4, c=65_536, ncand=20_000, k=10_000)     # early-exit path included
    g = wl.gradients(wl.Structure(cfg, dev), 0)
    eng, _, u, v = make(cfg, dev)
    oi = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    ov = torch.empty(cfg.k, device=dev)
    eng.step(g, cfg.rho, cfg.ncand, oi, ov)                # warm-up: device queries, function attributes
    assert eng.status() == S.OK
    eager_idx, eager_val = oi.clone(), ov.clone()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    u.zero_(); v.zero_()
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            eng.step(g, cfg.rho, cfg.ncand, oi, ov)
    for _ in range(2):
        u.zero_(); v.zero_(); oi.zero_(); ov.zero_()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert eng.status() == S.OK
        a, b = eager_idx.cpu().numpy(), oi.cpu().numpy()
        assert (np.diff(b) > 0).all()
        common, ia, ib = np.intersect1d(a, b, return_indices=True)
        assert common.size >= 0.995 * cfg.k
        assert (eager_val.cpu().numpy()[ia] == ov.cpu().numpy()[ib]).all()
        eng.flush()                                       # the replayed step only marked its k coordinates
        assert int((v[0, :cfg.d] == 0).sum().item()) >= cfg.k


def test_one_kernel_tail_can_be_captured_in_a_cuda_graph(cuda_device):
    """The small-problem step (memset, accumulate kernel, one cooperative kernel) can be captured and replayed too;
    integer gradients and rho = 1/2 make every operation exact, so a replay from zero state must reproduce the eager
    step bit for bit."""
    dev = cuda_device
    cfg = wl.C2.scaled(d=300_001, W=3, c=8192, ncand=3000, k=1500)
    gen = torch.Generator(device=dev).manual_seed(77)
    g = torch.zeros((cfg.W, cfg.ld), device=dev)
    g[:, :cfg.d] = torch.randint(-30, 31, (cfg.W, cfg.d), generator=gen, device=dev).float()
    g[:, 11:cfg.d:101] += 64.0
    eng, _, u, v = make(cfg, dev)
    eng.set_zero_mode(S.ZERO_EAGER)
    oi = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    ov = torch.empty(cfg.k, device=dev)
    eng.step(g, 0.5, cfg.ncand, oi, ov)                    # warm-up: device queries, function attributes
    assert eng.status() == S.OK
    eager_idx, eager_val, eager_v = oi.clone(), ov.clone(), v.clone()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    u.zero_(); v.zero_()
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            eng.step(g, 0.5, cfg.ncand, oi, ov)
    for _ in range(2):
        u.zero_(); v.zero_(); oi.zero_(); ov.zero_()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert eng.status() == S.OK
        assert torch.equal(oi, eager_idx) and torch.equal(ov, eager_val) and torch.equal(v, eager_v)


# ------------------------------------------------------------------------------------------------
# seeded random shapes: every combination of sizes a user could pass, small enough for the oracle
# ------------------------------------------------------------------------------------------------
def _random_case(seed):
    rng = np.random.default_rng(seed)
    kind = ["lognormal_planted", "block_gauss", "block_laplace", "embedding_mix"][int(rng.integers(4))]
    base = {"lognormal_planted": wl.C1, "block_gauss": wl.C2, "block_laplace": wl.C3, "embedding_mix": wl.C4}[kind]
    d = int(rng.choice([int(rng.integers(1, 64)), int(rng.integers(64, 5000)), int(rng.integers(5000, 400_000))]))
    r = int(rng.choice([1, 3, 5, 7, 9, 11, 13, 15]))
    # power-of-two and arbitrary column counts, from one bucket to sketches whose bucket bitmap must be folded
    c = int(rng.choice([1 << int(rng.integers(0, 21)), int(rng.integers(1, 3_000_000))]))
    if r * c * 4 > (96 << 20):
        c = max(1, (96 << 20) // (4 * r))
    W = int(rng.choice([1, 2, 3, 5, 8, 17]))
    ncand = int(rng.integers(1, d + 1))
    k = int(rng.integers(1, ncand + 1))
    prune = int(rng.choice([S.PRUNE_ON, S.PRUNE_EARLY_EXIT, S.PRUNE_OFF, S.PRUNE_AUTO]))
    mode = int(rng.choice([S.INSERT_GLOBAL, S.INSERT_TMA, S.INSERT_AUTO]))
    zero = int(rng.choice([S.ZERO_DEFERRED, S.ZERO_EAGER]))
    cfg = base.scaled(name=f"rnd{seed}", d=d, W=W, r=r, c=c, ncand=ncand, k=k, base_seed=1000 + seed)
    return cfg, prune, mode, zero


@pytest.mark.parametrize("seed", range(int(os.environ.get("SSGD_RANDOM_CASES", "48"))))
def test_random_shapes_lockstep(cuda_device, seed):
    cfg, prune, mode, zero = _random_case(seed)
    eng, orc, u, v = make(cfg, cuda_device)
    eng.set_insert_mode(mode)
    eng.set_prune_mode(prune)
    eng.set_zero_mode(zero)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    st = wl.Structure(cfg, cuda_device)
    for t in range(3):
        check_step(orc, eng, wl.gradients(st, t), cfg.rho, cfg.ncand, u_o, v_o, flush=(t == 2))


# ------------------------------------------------------------------------------------------------
# Algorithm 3 line 13, deferred into the next step's streaming kernel
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("mode", [S.INSERT_GLOBAL, S.INSERT_TMA, S.INSERT_SMEM])
def test_deferred_zero_equals_eager_zero(cuda_device, mode):
    """Two engines on the same inputs, one zeroing at once and one deferring: identical outputs every step, the
    deferring one's memory still holds the old values at the chosen coordinates until its next step or a flush,
    and after a flush the two states are identical bit for bit.  d is not a multiple of 4 (ragged tail), the
    flushes fall on different steps, and a step after a flush must not zero anything twice."""
    cfg = wl.C2.scaled(d=90_003, W=5, c=2048, ncand=3000, k=2000)
    dev = cuda_device
    st = wl.Structure(cfg, dev)
    eng_e, _, u_e, v_e = make(cfg, dev)
    eng_d, _, u_d, v_d = make(cfg, dev)
    for eng in (eng_e, eng_d):
        eng.set_insert_mode(mode)
    eng_e.set_zero_mode(S.ZERO_EAGER)
    oi_e = torch.empty(cfg.k, dtype=torch.int32, device=dev); ov_e = torch.empty(cfg.k, device=dev)
    oi_d = torch.empty_like(oi_e); ov_d = torch.empty_like(ov_e)
    for t in range(6):
        g = wl.gradients(st, t)
        g[:, cfg.d - 1] = 100.0 * (t + 1)                  # the last coordinate (ragged tail) is chosen every step
        eng_e.step(g, cfg.rho, cfg.ncand, oi_e, ov_e)
        eng_d.step(g, cfg.rho, cfg.ncand, oi_d, ov_d)
        assert eng_e.status() == S.OK and eng_d.status() == S.OK
        if not (oi_e == oi_d).all():
            pytest.skip("the two tables differ in reduction order and a near-tie fell differently")
        assert (ov_e == ov_d).all() and int(oi_d[-1].item()) == cfg.d - 1
        chosen = oi_d.long()
        assert (u_e[:, chosen] == 0).all() and (v_e[:, chosen] == 0).all()
        assert (v_d[:, chosen] != 0).any()                  # still the accumulated values in memory
        keep = torch.ones(cfg.ld, dtype=torch.bool, device=dev)
        keep[chosen] = False
        assert (u_d[:, keep] == u_e[:, keep]).all() and (v_d[:, keep] == v_e[:, keep]).all()
        if t in (1, 2, 5):
            eng_d.flush()
            assert (u_d == u_e).all() and (v_d == v_e).all()
    eng_d.flush()                                           # nothing pending: must change nothing
    assert (u_d == u_e).all() and (v_d == v_e).all()


def test_stage_calls_apply_a_pending_zero_out_first(cuda_device):
    """ssgd_exact_topk and ssgd_sketch_accumulate read the bound state: after a deferred step they must see it
    zeroed at the chosen coordinates."""
    cfg = wl.C2.scaled(d=60_001, W=3, c=1024, ncand=1500, k=700)
    dev = cuda_device
    st = wl.Structure(cfg, dev)
    eng, _, u, v = make(cfg, dev)
    oi = torch.empty(cfg.k, dtype=torch.int32, device=dev); ov = torch.empty(cfg.k, device=dev)
    eng.step(wl.gradients(st, 0), cfg.rho, cfg.ncand, oi, ov)
    chosen = oi.clone()
    assert (v[:, chosen.long()] != 0).any()
    o2 = torch.empty_like(oi); v2 = torch.empty_like(ov)
    cand = torch.arange(cfg.ncand, dtype=torch.int32, device=dev)
    eng.exact_topk(cand, o2, v2)
    assert eng.status() == S.OK
    assert (v[:, chosen.long()] == 0).all() and (u[:, chosen.long()] == 0).all()
    # and the other reader
    eng.step(wl.gradients(st, 1), cfg.rho, cfg.ncand, oi, ov)
    chosen = oi.clone()
    tables = torch.empty((cfg.W, cfg.r, cfg.c), device=dev)
    before_u = u.clone()
    eng.sketch_accumulate(torch.zeros_like(u), 0.0, tables)   # rho = 0, g = 0: u <- 0, v <- v
    assert (u == 0).all() and (v[:, chosen.long()] == 0).all() and (before_u[:, chosen.long()] != 0).any()


# ------------------------------------------------------------------------------------------------
# every call works on the stream it is given
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("prune", [S.PRUNE_FUSED, S.PRUNE_ON, S.PRUNE_OFF])
def test_steps_on_a_side_stream(cuda_device, prune):
    """The library only enqueues on the caller's stream (the binding passes torch's current stream): three steps on
    a non-default stream, with the gradients produced on that stream right before each step and no synchronisation
    in between, in lock step with the oracle."""
    cfg = wl.C2.scaled(d=400_003, W=3, c=8192, ncand=3000, k=1500)
    dev = cuda_device
    eng, orc, u, v = make(cfg, dev)
    eng.set_prune_mode(prune)
    u_o, v_o = u.cpu().numpy(), v.cpu().numpy()
    st = wl.Structure(cfg, dev)
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        for t in range(3):
            g = wl.gradients(st, t)
            check_step(orc, eng, g, cfg.rho, cfg.ncand, u_o, v_o, flush=(t == 2))
    side.synchronize()


# ------------------------------------------------------------------------------------------------
# nothing is written outside the buffers the caller hands over
# ------------------------------------------------------------------------------------------------
CANARY_CASES = [
    (wl.C2.scaled(d=300_001, W=4, c=8192, ncand=3000, k=1500), S.PRUNE_FUSED, S.INSERT_GLOBAL),
    (wl.C2.scaled(d=300_001, W=4, c=8192, ncand=3000, k=1500), S.PRUNE_OFF, S.INSERT_TMA),
    (wl.C2.scaled(d=500_003, W=3, c=8192, ncand=4000, k=2000), S.PRUNE_ON, S.INSERT_GLOBAL),
    (wl.C3.scaled(d=600_011, W=3, r=5, c=524_288, ncand=5000, k=2000), S.PRUNE_ON, S.INSERT_GLOBAL),   # folded bitmap
    (wl.C2.scaled(d=500_003, W=3, c=8192, ncand=4000, k=2000), S.PRUNE_EARLY_EXIT, S.INSERT_GLOBAL),
]


@pytest.mark.parametrize("cfg,prune,mode", CANARY_CASES, ids=lambda x: f"{x.name}-d{x.d}-c{x.c}" if hasattr(x, "name") else str(x))
def test_canaries_around_every_caller_buffer_survive(cuda_device, cfg, prune, mode):
    """Workspace, state, gradient and output buffers each sit between two 4 KiB guard zones filled with a pattern;
    the workspace is exactly ssgd_workspace_bytes long.  After steps, a flush and the stage calls the guards are
    untouched and the gradients unchanged."""
    dev = cuda_device
    G = 4096
    pat = 0xA5

    def guarded(nbytes):
        raw = torch.full((nbytes + 2 * G,), pat, dtype=torch.uint8, device=dev)
        return raw, raw[G:G + nbytes]

    eng = S.Ssgd(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
    n_ws = eng.workspace_bytes(cfg.ncand)
    n_state = cfg.W * cfg.ld * 4
    raws = {}
    raws["ws"], ws = guarded(n_ws)
    raws["u"], u8 = guarded(n_state)
    raws["v"], v8 = guarded(n_state)
    raws["g"], g8 = guarded(n_state)
    raws["oi"], oi8 = guarded(cfg.k * 4)
    raws["ov"], ov8 = guarded(cfg.k * 4)
    u, v, g = (t.view(torch.float32).view(cfg.W, cfg.ld) for t in (u8, v8, g8))
    oi, ov = oi8.view(torch.int32), ov8.view(torch.float32)
    u.zero_(); v.zero_()
    eng.bind(u, v, cfg.ncand, ws)
    eng.set_prune_mode(prune)
    eng.set_insert_mode(mode)
    st = wl.Structure(cfg, dev)
    for t in range(3):
        g.copy_(wl.gradients(st, t))
        g_before = g.clone()
        eng.step(g, cfg.rho, cfg.ncand, oi, ov)
        assert eng.status() == S.OK
        assert torch.equal(g, g_before)
    eng.flush()
    # the stage calls on caller buffers of their exact sizes
    raws["tab"], tab8 = guarded(cfg.W * cfg.r * cfg.c * 4)
    raws["mer"], mer8 = guarded(cfg.r * cfg.c * 4)
    raws["cand"], cand8 = guarded(cfg.ncand * 4)
    raws["cest"], cest8 = guarded(cfg.ncand * 4)
    tables = tab8.view(torch.float32).view(cfg.W, cfg.r, cfg.c)
    merged = mer8.view(torch.float32).view(cfg.r, cfg.c)
    cand, cest = cand8.view(torch.int32), cest8.view(torch.float32)
    eng.sketch_accumulate(g, cfg.rho, tables)
    eng.sketch_merge(tables, merged)
    eng.unsketch_candidates(merged, cfg.ncand, cand, cest)
    eng.exact_topk(cand, oi, ov)
    assert eng.status() == S.OK
    for name, raw in raws.items():
        assert bool((raw[:G] == pat).all()) and bool((raw[-G:] == pat).all()), f"guard zone of {name} was written"


# ------------------------------------------------------------------------------------------------
# argument checking (host side; nothing is launched)
# ------------------------------------------------------------------------------------------------
def test_argument_errors(cuda_device):
    dev = cuda_device
    cfg = wl.C2.scaled(d=1000, W=2, c=64, ncand=100, k=50)
    eng = S.Ssgd(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, 1)
    g = torch.zeros((cfg.W, cfg.ld), device=dev)
    oi = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    ov = torch.empty(cfg.k, device=dev)
    with pytest.raises(S.SsgdError) as e:
        eng.step(g, 0.9, cfg.ncand, oi, ov)
    assert e.value.code == S.ENOTBOUND
    u, v = wl.zero_state(cfg, dev)
    small = torch.empty(16, dtype=torch.uint8, device=dev)
    with pytest.raises(S.SsgdError) as e:
        eng.bind(u, v, cfg.ncand, small)
    assert e.value.code == S.EWORKSPACE
    big = torch.empty(cfg.W * cfg.ld + 1, device=dev)
    with pytest.raises(S.SsgdError) as e:
        eng.bind(big[1:].view(cfg.W, cfg.ld), v, cfg.ncand)
    assert e.value.code == S.EALIGN
    eng.bind(u, v, cfg.ncand)
    for ncand, code in ((cfg.k - 1, S.EINVAL), (cfg.d + 1, S.EINVAL), (cfg.ncand + 1, S.EWORKSPACE)):
        with pytest.raises(S.SsgdError) as e:
            eng.step(g, 0.9, ncand, oi, ov)
        assert e.value.code == code
    with pytest.raises(S.SsgdError) as e:
        eng.step(big[1:].view(cfg.W, cfg.ld), 0.9, cfg.ncand, oi, ov)
    assert e.value.code == S.EALIGN
    g_short = torch.zeros((cfg.W, cfg.d - 8), device=dev)
    with pytest.raises(S.SsgdError) as e:
        eng.step(g_short, 0.9, cfg.ncand, oi, ov)
    assert e.value.code == S.EINVAL
    with pytest.raises(S.SsgdError):
        eng.set_insert_mode(7)
    # an out-of-range candidate is skipped and reported, never dereferenced
    cand = torch.arange(cfg.ncand, dtype=torch.int32, device=dev)
    cand[3] = cfg.d + 5
    eng.exact_topk(cand, oi, ov)
    assert eng.status() == S.EDEVICE
    assert eng.status() == S.OK
    assert eng.launch_count() > 0
