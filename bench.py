#!/usr/bin/env python
"""Benchmark of the Sketched-SGD compression step (ssgd_step) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload C2]

A "step" is one pass of the whole hot path (momentum + error accumulation + sketch insert, unsketch,
candidate selection, second round, final top-k, zero-out) over one batch of synthetic worker
gradients.  Workload at N = 1: configuration C2 (d = 11,173,962, W = 16, 5 x 262,144 sketch,
100,000 candidates, k = 50,000, rho = 0.9), ten resident gradient sets used in rotation.

The path does not shard (one GPU holds all simulated workers; no collectives), so --gpus N runs N
independent replicas, one process per GPU, and the value is the sum over replicas (weak scaling).

One JSON line on stdout (rank 0).  --impl reference times the CPU oracle instead, on a bounded
sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "ssgd_step coordinates/s (W*d per step)"
UNIT = "coordinates/s"
FALLBACK_HBM_GBS = 6650.0          # earlier measurement on this machine, used only if no peaks file exists
ORACLE_COORDS_PER_S = 4.0e6        # conservative single-thread estimate used to size oracle samples
# DRAM bytes per launch of k_accum_insert from an ncu capture (dram__bytes_read.sum + dram__bytes_write.sum),
# keyed by workload (None where no capture exists).
NCU_TRAFFIC_BYTES = {"C2": 3.550e9}   # 1906.1 MB at d = 6,000,002 scaled in proportion to d (profiles/k_accum_insert_C2_d6M.md)


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Polls SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.005):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            "hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
            "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
            "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
            "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap,
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if mask & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            pass
    return local_rank


def oracle_sample(cfg, budget_coords: float):
    """A bounded sample of the workload for the CPU oracle: fewer workers first, then fewer coordinates
    (sketch width, candidates and k shrink in proportion, so d/c and ncand/d are kept)."""
    W = max(1, min(cfg.W, int(budget_coords // cfg.d)))
    if W * cfg.d <= budget_coords:
        return cfg.scaled(W=W), f"first {W} of {cfg.W} workers of {cfg.name}, all d={cfg.d} coordinates, 1 step from zero state"
    f = max(budget_coords / cfg.d, 1e-3)
    d = max(4096, int(cfg.d * f))
    c = max(64, 1 << int(round((cfg.c * d / cfg.d)).bit_length() - 1))
    k = max(1, int(cfg.k * d / cfg.d))
    ncand = max(k, int(cfg.ncand * d / cfg.d))
    s = cfg.scaled(W=1, d=d, c=c, k=k, ncand=ncand)
    return s, (f"1 of {cfg.W} workers of {cfg.name}, d={d} of {cfg.d} coordinates with c={c}, ncand={ncand}, k={k} "
               f"scaled in proportion, 1 step from zero state")


def time_oracle(sample_cfg, g_host, steps: int):
    """Seconds per step of the oracle as it stands (single thread), state re-zeroed before each step."""
    import numpy as np
    from oracle import Oracle
    orc = Oracle(sample_cfg.d, sample_cfg.r, sample_cfg.c, sample_cfg.k, sample_cfg.W, sample_cfg.sketch_seed)
    times = []
    for _ in range(steps):
        u = np.zeros_like(g_host)
        v = np.zeros_like(g_host)
        t0 = time.perf_counter()
        orc.step(g_host, sample_cfg.rho, u, v, sample_cfg.ncand)
        times.append(time.perf_counter() - t0)
    return times


def run_reference(args, cfg):
    """The reference arm: the CPU oracle, timed on the host cores on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from paper_1903_04488_b200 import workloads as wl
    total = max(1, args.steps + args.warmup)
    budget = min(ORACLE_COORDS_PER_S * 150.0 / total, 8.0 * cfg.d)
    scfg, what = oracle_sample(cfg, budget)
    torch.manual_seed(0)
    g = wl.gradients(wl.Structure(scfg, "cpu"), 0).numpy()
    time_oracle(scfg, g, args.warmup)
    times = time_oracle(scfg, g, args.steps)
    sec = sum(times) / len(times)
    value = scfg.W * scfg.d / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(cfg, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def communication(cfg):
    """What one worker sends and receives per step, in values (Section 5.1: P*k + |S| + k), and the
    compression factor 2d / (|S| + P*k + k) of Section 5.3 -- a property of the configuration, printed as context."""
    sketch = cfg.r * cfg.c
    per_worker = sketch + cfg.ncand + cfg.k
    return {"sketch_values": sketch, "second_round_values": cfg.ncand, "update_values": cfg.k,
            "per_worker_values": per_worker, "compression_vs_dense": 2.0 * cfg.d / per_worker}


def workload_config(cfg, args):
    return {
        "mode": getattr(args, "mode", "fused"),
        "communication": communication(cfg),
        "workload": f"{cfg.name}: d={cfg.d}, W={cfg.W}, r={cfg.r}, c={cfg.c}, ncand={cfg.ncand}, k={cfg.k}, "
                    f"rho={cfg.rho}, {cfg.steps} resident gradient sets in rotation",
        "l2": "inputs larger than L2: every step streams 20*W*d bytes of g, u, v",
        "zero_out": "deferred (library default): a step marks its k coordinates, the next step's accumulate kernel "
                    "reads them as zero; the last step's marks are applied by ssgd_flush inside the timed region",
        "parallelism": "replicas only" if args.gpus > 1 else "single GPU",
    }


def run_ours(args, cfg):
    import torch
    from paper_1903_04488_b200 import ssgd as S
    from paper_1903_04488_b200 import workloads as wl
    from paper_1903_04488_b200.replicas import Replicas

    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    rep = Replicas("nccl", dev)
    rank, world, barrier = rep.rank, rep.world, rep.barrier
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch with torch.distributed.run")

    # replicas differ only in their seeds
    rcfg = cfg.scaled(base_seed=cfg.base_seed + rep.replica_seed_offset())
    st = wl.Structure(rcfg, dev)
    n_sets = args.sets or cfg.steps
    g_sets = [wl.gradients(st, t) for t in range(n_sets)]
    u, v = wl.zero_state(cfg, dev)
    eng = S.Ssgd(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
    eng.bind(u, v, cfg.ncand)
    eng.set_prune_mode({"auto": S.PRUNE_AUTO, "off": S.PRUNE_OFF, "on": S.PRUNE_ON, "early_exit": S.PRUNE_EARLY_EXIT}[args.prune])
    out_idx = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    out_val = torch.empty(cfg.k, dtype=torch.float32, device=dev)

    if args.mode == "faithful":
        # what the paper transmits: every worker's own sketch is materialised, then merged (Algorithm 3 lines 7-8)
        tables = torch.empty((cfg.W, cfg.r, cfg.c), dtype=torch.float32, device=dev)
        merged = torch.empty((cfg.r, cfg.c), dtype=torch.float32, device=dev)
        cand = torch.empty(cfg.ncand, dtype=torch.int32, device=dev)

        def one_step(g):
            eng.sketch_accumulate(g, cfg.rho, tables)
            eng.sketch_merge(tables, merged)
            eng.unsketch_candidates(merged, cfg.ncand, cand)
            eng.exact_topk(cand, out_idx, out_val)
    else:
        def one_step(g):
            eng.step(g, cfg.rho, cfg.ncand, out_idx, out_val)

    for t in range(max(3, args.warmup)):
        one_step(g_sets[t % n_sets])
    assert eng.status() == S.OK
    eng.flush()
    u.zero_(); v.zero_()
    torch.cuda.synchronize()

    # ---- timed region: K steps, inputs resident in HBM ------------------------------------------
    sampler = ClockSampler(physical_gpu_index(local_rank))
    eng.set_timing(True)
    launches0 = eng.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(); torch.cuda.synchronize()
    sampler.start()
    ev0.record()
    for t in range(args.steps):
        one_step(g_sets[t % n_sets])
    eng.flush()         # the last step's zero-out (deferred into the next step's kernel) is paid inside the region
    ev1.record()
    torch.cuda.synchronize(); barrier()
    clocks = sampler.stop()
    ms_total = ev0.elapsed_time(ev1)
    launches = eng.launch_count() - launches0
    stage_ms, stage_n = eng.get_stage_times()
    eng.set_timing(False)
    assert eng.status() == S.OK
    value, ms_step = rep.whole_job_value(cfg.W * cfg.d, ms_total / args.steps)

    # ---- end to end: host gradients in, host results out, through ssgd_step_host ------------------
    e2e_steps = 0 if (args.no_e2e or args.mode != "fused") else max(1, min(args.steps, 20))
    g_host = [g_sets[i % n_sets].cpu().pin_memory() for i in range(2 if e2e_steps else 0)]
    g_stage = torch.empty_like(g_sets[0])
    oi_h = torch.empty(cfg.k, dtype=torch.int32).pin_memory()
    ov_h = torch.empty(cfg.k, dtype=torch.float32).pin_memory()
    u.zero_(); v.zero_()
    for t in range(2 if e2e_steps else 0):
        eng.step_host(g_host[t % 2], cfg.rho, cfg.ncand, g_stage, oi_h, ov_h)
    eng.flush()
    u.zero_(); v.zero_()
    barrier(); torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(e2e_steps):
        eng.step_host(g_host[t % 2], cfg.rho, cfg.ncand, g_stage, oi_h, ov_h)
    eng.flush()
    e1.record()
    torch.cuda.synchronize(); barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = rep.max_over_ranks(e2e_ms)
    e2e_value = world * cfg.W * cfg.d / (e2e_ms / e2e_steps * 1e-3) if e2e_steps else None

    # ---- roofline of the dominant kernel and of the whole step -----------------------------------
    peak, peak_kind = peaks()
    split = stage_n > 0         # stage calls are not instrumented: no per-kernel split in faithful mode
    k1_ms = stage_ms[0] / stage_n if split else None
    k1_bytes = 20.0 * cfg.W * cfg.d                       # g read; u, v read and written
    k1_gbs = k1_bytes / (k1_ms * 1e-3) / 1e9 if split else None
    step_bytes = (20.0 * cfg.W * cfg.d + 8.0 * cfg.r * cfg.c + 8.0 * cfg.d + 4.0 * cfg.W * cfg.ncand
                  + 8.0 * cfg.W * cfg.k + 8.0 * cfg.k)
    step_gbs = step_bytes / (ms_step * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "kernel": "k_accum_insert", "achieved": k1_gbs, "peak": peak, "unit": "GB/s",
        "frac": k1_gbs / peak if split else None, "peak_source": f"of {peak_kind}", "traffic": NCU_TRAFFIC_BYTES.get(cfg.name),
        "algorithmic_bytes_per_launch": k1_bytes, "ms_per_launch": k1_ms, "launches_timed": stage_n,
    }
    breakdown = {n: (ms / stage_n if split else None) for n, ms in
                 zip(("accumulate_insert_ms", "unsketch_ms", "select_candidates_ms", "second_round_topk_zero_ms"), stage_ms)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(cfg, args),
        "clocks": clocks, "gpu_launches": launches,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": cfg.W * cfg.ld * 4,
                "d2h_bytes_per_step": 8 * cfg.k, "steps": e2e_steps, "ms_per_step": e2e_ms / max(1, e2e_steps)},
        "roofline": roofline,
        "step_hbm": {"algorithmic_bytes_per_step": step_bytes, "achieved": step_gbs, "peak": peak, "unit": "GB/s",
                     "frac": step_gbs / peak, "peak_source": f"of {peak_kind}", "frac_of_8000_nominal": step_gbs / 8000.0},
        "stage_ms": breakdown,
    }

    # ---- the oracle beside it (rank 0, N = 1 only): a bounded sample of the same inputs ----------
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        scfg, what = oracle_sample(cfg, 8.0 * cfg.d)
        g_h = g_sets[0][: scfg.W].cpu().numpy()
        del g_sets
        sec = time_oracle(scfg, g_h, 1)[0]
        line["cpu_baseline"] = {"value": scfg.W * scfg.d / sec, "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": what, "seconds": sec}
    if rank == 0:
        print(json.dumps(line), flush=True)
    rep.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="C2")
    ap.add_argument("--mode", choices=["fused", "faithful"], default="fused",
                    help="fused: ssgd_step; faithful: per-worker sketches materialised and merged (stage calls)")
    ap.add_argument("--prune", choices=["auto", "off", "on", "early_exit"], default="auto",
                    help="how Algorithm 3 line 9 is evaluated (profiling runs; the default is what a user gets)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--d", type=int, default=0, help="override the number of coordinates (small profiling cases)")
    ap.add_argument("--sets", type=int, default=0, help="resident gradient sets (default: the workload's steps)")
    args = ap.parse_args()
    from paper_1903_04488_b200 import workloads as wl
    cfg = wl.CONFIGS[args.workload]
    if args.d:
        cfg = cfg.scaled(name=f"{cfg.name}[d={args.d}]", d=args.d)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
