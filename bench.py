#!/usr/bin/env python
"""Benchmark of the Sketched-SGD compression step (ssgd_step) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload all|C1|C2|...]

A "step" is one pass of the whole hot path (momentum + error accumulation + sketch insert, unsketch,
candidate selection, second round, final top-k, zero-out) over one batch of synthetic worker gradients.

With no --workload the run covers every configuration of the benchmark spec, one after the other on one
GPU -- C1 (cold L2), C2, C3, C4 and the worker sweep C5 at W = 8, 32, 128, 256 -- and reports each under
`per_config` (median and minimum over >= 5 repetitions of the configuration's own step sequence, every
repetition from re-zeroed state; per-stage times from a separate pass).  The top-level `value`,
`ms_per_step`, `roofline` and `e2e` belong to the HEADLINE workload, the largest single-GPU configuration
(C5 at W = 256: 57.5 GB of algorithmic traffic per step): W warm-up steps, then exactly K steps in one timed
region.  --workload NAME runs that one configuration as the headline (profiling runs).

The path does not shard (one GPU holds all simulated workers; no collectives), so --gpus N runs N
independent replicas, one process per GPU, and the value is the sum over replicas (weak scaling); the
per-configuration sweep is done at N = 1 only.

One JSON line on stdout (rank 0).  --impl reference times the CPU oracle instead, on a bounded sample of
the headline workload.
"""
from __future__ import annotations

import argparse
import json
import os
import platform
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
HEADLINE = "C5_W256"
SWEEP = ("C1", "C2", "C3", "C4", "C5_W8", "C5_W32", "C5_W128", "C5_W256")
PAPER_SHAPES = ("P1", "P2", "P3")  # the paper's own sketch shapes (Table 1 footnotes), timed after the sweep
L2_FLUSH_BYTES = 512 << 20         # written between repetitions of configurations whose working set fits in L2
COLD_SETS = 8                      # independent (g, u, v, workspace) sets rotated through for such configurations
# DRAM bytes per launch of the accumulate+insert kernel from ncu captures (dram__bytes_read.sum +
# dram__bytes_write.sum on a small case, scaled in proportion to W*d), keyed by kernel: bytes per worker-coordinate
NCU_TRAFFIC_BYTES_PER_UNIT = {
    "k_accum_insert": 1906.1e6 / (16 * 6_000_002),       # profiles/k_accum_insert_C2_d6M.md
    "k_accum_insert_tma": 5.11767e9 / (256 * 1_000_002),  # profiles/k_accum_insert_tma_C5_W256_d1M.md
}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def host_facts():
    model = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except Exception:
        pass
    try:
        usable = len(os.sched_getaffinity(0))
    except Exception:
        usable = os.cpu_count() or 1
    return {"nproc": os.cpu_count() or 1, "usable_cores": usable, "cpu_model": model or platform.processor()}


def host_memory_available() -> int:
    """Bytes of host memory this process may still take: the smaller of MemAvailable and the cgroup's headroom."""
    avail = 1 << 62
    try:
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemAvailable:"):
                    avail = int(line.split()[1]) * 1024
    except Exception:
        pass
    try:
        with open("/sys/fs/cgroup/memory.max") as f:
            lim = f.read().strip()
        with open("/sys/fs/cgroup/memory.current") as f:
            cur = int(f.read().strip())
        if lim != "max":
            avail = min(avail, int(lim) - cur)
    except Exception:
        pass
    return avail


class ClockSampler:
    """Polls SM clock and throttle reasons of one GPU through NVML while a timed region runs."""

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
        return self

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


# ---------------------------------------------------------------------------------------------------
# the CPU oracle beside it
# ---------------------------------------------------------------------------------------------------
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


def time_oracle_threaded(cfg, g_host, threads: int):
    """Seconds for one step with the oracle's own plain functions called from `threads` host threads: Algorithm 3
    lines 5-7 (accumulate, per-worker sketch) run one worker per task (ctypes releases the interpreter lock), the
    sum over workers in worker order, and lines 9-13 on one thread as the oracle states them.  Nothing under
    oracle/ is changed for this; the result is that of the single-threaded step."""
    import concurrent.futures
    import numpy as np
    from oracle import Oracle, select as oracle_select
    one = [Oracle(cfg.d, cfg.r, cfg.c, cfg.k, 1, cfg.sketch_seed) for _ in range(cfg.W)]   # same seed: same hashes
    allw = Oracle(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
    u = np.zeros_like(g_host)
    v = np.zeros_like(g_host)
    t0 = time.perf_counter()

    def worker(w):
        one[w].accumulate(g_host[w:w + 1], cfg.rho, u[w:w + 1], v[w:w + 1])
        return one[w].sketch(v[w, :cfg.d])

    with concurrent.futures.ThreadPoolExecutor(max_workers=threads) as pool:
        tables = list(pool.map(worker, range(cfg.W)))
    T = np.zeros_like(tables[0])
    for Tw in tables:                              # worker order
        T += Tw
    est = allw.estimate(T.astype(np.float32))
    cand = oracle_select(est, cfg.ncand)
    xs = allw.second_round(v, cand)
    idx, _ = allw.final_topk(cand, xs)
    allw.zero(u, v, idx)
    return time.perf_counter() - t0


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
        "cpu_baseline": dict({"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": what}, **host_facts()),
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------------
# configuration facts
# ---------------------------------------------------------------------------------------------------
def communication(cfg):
    """What one worker sends and receives per step, in values (Section 5.1: P*k + |S| + k), and the
    compression factor 2d / (|S| + P*k + k) of Section 5.3 -- a property of the configuration, printed as context."""
    sketch = cfg.r * cfg.c
    per_worker = sketch + cfg.ncand + cfg.k
    return {"sketch_values": sketch, "second_round_values": cfg.ncand, "update_values": cfg.k,
            "per_worker_values": per_worker, "compression_vs_dense": 2.0 * cfg.d / per_worker}


def fits_in_l2(cfg) -> bool:
    return 3 * cfg.W * cfg.ld * 4 < (126 << 20)


def workload_config(cfg, args):
    cold = fits_in_l2(cfg)
    return {
        "mode": getattr(args, "mode", "fused"),
        "communication": communication(cfg),
        "workload": f"{cfg.name}: d={cfg.d}, W={cfg.W}, r={cfg.r}, c={cfg.c}, ncand={cfg.ncand}, k={cfg.k}, "
                    f"rho={cfg.rho}, {cfg.steps} resident gradient set(s) in rotation",
        "l2": (f"working set smaller than L2: {COLD_SETS} independent (g, u, v, workspace) sets in rotation and a "
               f"{L2_FLUSH_BYTES >> 20} MiB buffer overwritten before each timed repetition") if cold else
              "inputs larger than L2: every step streams 20*W*d bytes of g, u, v",
        "zero_out": ("eager (single-step configuration: there is no next step to defer into)" if cfg.steps == 1 else
                     "deferred (library default): a step marks its k coordinates, the next step's accumulate kernel "
                     "reads them as zero; the last step's marks are applied by ssgd_flush inside the timed region"),
        "parallelism": "replicas only" if args.gpus > 1 else "single GPU",
    }


def step_bytes(cfg) -> float:
    return (20.0 * cfg.W * cfg.d + 8.0 * cfg.r * cfg.c + 8.0 * cfg.d + 4.0 * cfg.W * cfg.ncand
            + 8.0 * cfg.W * cfg.k + 8.0 * cfg.k)


def dominant_kernel(cfg) -> str:
    return "k_accum_insert_tma" if cfg.W >= 144 else "k_accum_insert"


# ---------------------------------------------------------------------------------------------------
# one configuration on one GPU
# ---------------------------------------------------------------------------------------------------
class Bench:
    """Everything resident for one configuration: gradient sets, state, engine(s), outputs."""

    def __init__(self, cfg, dev, args, n_sets, seed_offset=0):
        import torch
        from paper_1903_04488_b200 import ssgd as S
        from paper_1903_04488_b200 import workloads as wl
        self.cfg, self.dev, self.S, self.torch = cfg, dev, S, torch
        rcfg = cfg.scaled(base_seed=cfg.base_seed + seed_offset)
        st = wl.Structure(rcfg, dev)
        self.g_sets = [wl.gradients(st, t) for t in range(n_sets)]
        self.cold = fits_in_l2(cfg)
        n_eng = COLD_SETS if self.cold else 1
        self.engines, self.states = [], []
        for _ in range(n_eng):
            u, v = wl.zero_state(cfg, dev)
            eng = S.Ssgd(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
            eng.bind(u, v, cfg.ncand)
            eng.set_prune_mode({"auto": S.PRUNE_AUTO, "off": S.PRUNE_OFF, "on": S.PRUNE_ON,
                                "early_exit": S.PRUNE_EARLY_EXIT}[args.prune])
            if cfg.steps == 1:
                eng.set_zero_mode(S.ZERO_EAGER)
            self.engines.append(eng)
            self.states.append((u, v))
        if self.cold:                                     # every engine streams its own copy of the gradients
            self.g_cold = [self.g_sets[0]] + [self.g_sets[0].clone() for _ in range(n_eng - 1)]
            self.flush_buf = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
        self.out_idx = torch.empty(cfg.k, dtype=torch.int32, device=dev)
        self.out_val = torch.empty(cfg.k, dtype=torch.float32, device=dev)
        self.mode = args.mode
        if self.mode == "faithful":
            # what the paper transmits: every worker's own sketch is materialised, then merged (Algorithm 3 lines 7-8)
            self.tables = torch.empty((cfg.W, cfg.r, cfg.c), dtype=torch.float32, device=dev)
            self.merged = torch.empty((cfg.r, cfg.c), dtype=torch.float32, device=dev)
            self.cand = torch.empty(cfg.ncand, dtype=torch.int32, device=dev)

    @property
    def eng(self):
        return self.engines[0]

    def one_step(self, t, e=0):
        cfg, eng = self.cfg, self.engines[e]
        g = self.g_cold[e] if self.cold else self.g_sets[t % len(self.g_sets)]
        if self.mode == "faithful":
            eng.sketch_accumulate(g, cfg.rho, self.tables)
            eng.sketch_merge(self.tables, self.merged)
            eng.unsketch_candidates(self.merged, cfg.ncand, self.cand)
            eng.exact_topk(self.cand, self.out_idx, self.out_val)
        else:
            eng.step(g, cfg.rho, cfg.ncand, self.out_idx, self.out_val)

    def flush(self, eng):
        """Applies the last step's zero-out where it is deferred (eager engines have written their zeros already)."""
        if eng.zero_mode == self.S.ZERO_DEFERRED:
            eng.flush()

    def zero_state(self):
        for eng in self.engines:
            eng.flush()
        for u, v in self.states:
            u.zero_(); v.zero_()

    def sequence(self):
        """The configuration's own step sequence, with the last step's zero-out applied: cfg.steps steps (on every
        one of the rotating sets when the working set fits in L2).  Returns the number of steps enqueued."""
        if self.cold:
            for e in range(len(self.engines)):
                for t in range(self.cfg.steps):
                    self.one_step(t, e)
                self.flush(self.engines[e])
            return len(self.engines) * self.cfg.steps
        for t in range(self.cfg.steps):
            self.one_step(t)
        self.flush(self.eng)
        return self.cfg.steps

    def timed_sequence(self):
        """ms per step of one sequence from re-zeroed state (state reset and L2 flush outside the timed region)."""
        torch = self.torch
        self.zero_state()
        if self.cold:
            self.flush_buf.fill_(1)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        n = self.sequence()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    def warm_sequence(self, n):
        """ms per step of n back-to-back steps on ONE set (its g, u, v stay in L2 if they fit): labelled warm."""
        torch = self.torch
        self.zero_state()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for t in range(n):
            self.one_step(t)
        self.flush(self.eng)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    def stage_pass(self):
        """Per-stage milliseconds per step from one sequence with the library's stage events on."""
        if self.mode != "fused":
            return None, 0
        self.zero_state()
        for eng in self.engines:
            eng.set_timing(True)
        self.sequence()
        tot, n = [0.0] * 4, 0
        for eng in self.engines:
            ms, k = eng.get_stage_times()
            tot = [a + b for a, b in zip(tot, ms)]
            n += k
            eng.set_timing(False)
        names = ("accumulate_insert_ms", "unsketch_ms", "select_candidates_ms", "second_round_topk_zero_ms")
        return ({nm: (x / n if n else None) for nm, x in zip(names, tot)}, n)

    def status_ok(self):
        return all(eng.status() == self.S.OK for eng in self.engines)


def measure_config(cfg, dev, args, gpu_index, reps):
    """The per_config record of one configuration (N = 1)."""
    import torch
    b = Bench(cfg, dev, args, n_sets=args.sets or cfg.steps)
    for _ in range(max(1, -(-3 // b.cfg.steps))):            # at least 3 warm-up steps
        b.sequence()
    assert b.status_ok()
    sampler = ClockSampler(gpu_index, period_s=0.002).start()
    times = [b.timed_sequence() for _ in range(reps)]
    clocks = sampler.stop()
    stage, stage_n = b.stage_pass()
    assert b.status_ok()
    peak, peak_kind = peaks()
    med, mn = statistics.median(times), min(times)
    sb = step_bytes(cfg)
    rec = {
        "workload": workload_config(cfg, args)["workload"],
        "l2": workload_config(cfg, args)["l2"],
        "repetitions": reps, "steps_per_repetition": (COLD_SETS if b.cold else 1) * cfg.steps,
        "ms_per_step_median": med, "ms_per_step_min": mn,
        "coordinates_per_s": cfg.W * cfg.d / (med * 1e-3),
        "step_hbm": {"algorithmic_bytes_per_step": sb, "achieved": sb / (med * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                     "frac": sb / (med * 1e-3) / 1e9 / peak, "peak_source": f"of {peak_kind}",
                     "frac_of_8000_nominal": sb / (med * 1e-3) / 1e9 / 8000.0},
        "stage_ms": stage,
        "clocks": clocks,
    }
    if stage and stage.get("accumulate_insert_ms"):
        k1 = 20.0 * cfg.W * cfg.d / (stage["accumulate_insert_ms"] * 1e-3) / 1e9
        rec["roofline"] = {"bound": "hbm", "kernel": dominant_kernel(cfg), "achieved": k1, "peak": peak, "unit": "GB/s",
                           "frac": k1 / peak, "peak_source": f"of {peak_kind}"}
        # the operation-rate bound of the accumulate+insert kernel (measured across shapes): a reduction into the L2-resident
        # table costs the L2 about what a 32-byte sector of the stream costs; 2.6e11 such operations per second
        ops = 20.0 * cfg.W * cfg.d / 32.0 + float(cfg.d) * cfg.r
        t_ops = ops / 2.6e11 * 1e3
        t_hbm = 20.0 * cfg.W * cfg.d / (peak * 1e9) * 1e3
        rec["roofline"]["operation_rate_bound_ms"] = t_ops
        rec["roofline"]["frac_of_binding_bound"] = max(t_ops, t_hbm) / stage["accumulate_insert_ms"]
    if b.cold:
        rec["ms_per_step_warm_l2"] = b.warm_sequence(20)
    if b.mode == "faithful":
        rec["sketch16"] = time_sketch16(b)
        rec["heavymix"] = time_heavymix(b)
    del b
    torch.cuda.empty_cache()
    return rec


def time_sketch16(b):
    """16-bit sketches (Section 6) on the per-worker tables of the faithful pipeline: what quantising them and
    merging the 16-bit encodings costs beside the fp32 merge, with the bytes each kernel moves."""
    torch, S, cfg = b.torch, b.S, b.cfg
    q16 = torch.empty((cfg.W, cfg.r, cfg.c), dtype=torch.int16, device=b.dev)
    rc = cfg.r * cfg.c

    def timed(fn, n=20):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    out = {"merge_fp32_ms": timed(lambda: b.eng.sketch_merge(b.tables, b.merged)),
           "merge_fp32_bytes": 4 * rc * (cfg.W + 1)}
    for name, fmt in (("f16", S.FMT_F16), ("bf16", S.FMT_BF16)):
        out[f"quantize_{name}_ms"] = timed(lambda: b.eng.sketch_quantize16(b.tables, fmt, q16))
        out[f"merge_{name}_ms"] = timed(lambda: b.eng.sketch_merge16(q16, fmt, b.merged))
    out["quantize_bytes"] = 6 * rc * cfg.W
    out["merge16_bytes"] = 2 * rc * cfg.W + 4 * rc
    out["note"] = "working set (W tables) may fit in L2: these are warm figures"
    return out


def time_heavymix(b):
    """Algorithm 1 (HEAVYMIX) on the merged table the faithful pipeline left behind: the other way from a sketch to k
    coordinates (norm estimate, heavy set, seeded random fill, exact values of the chosen ones)."""
    torch, cfg = b.torch, b.cfg
    oi = torch.empty(cfg.k, dtype=torch.int32, device=b.dev)
    ov = torch.empty(cfg.k, dtype=torch.float32, device=b.dev)
    l2 = torch.empty(1, dtype=torch.float64, device=b.dev)
    nh = torch.empty(1, dtype=torch.int32, device=b.dev)
    for _ in range(3):
        b.eng.heavymix(b.merged, 12345, oi, ov, l2, nh)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    n = 10
    for _ in range(n):
        b.eng.heavymix(b.merged, 12345, oi, ov, l2, nh)
    e1.record()
    torch.cuda.synchronize()
    return {"ms": e0.elapsed_time(e1) / n, "heavy": int(nh.item()), "k": cfg.k,
            "note": "one call of ssgd_heavymix on the merged table (L2-warm), d*r table reads + selection over d keys"}


def run_ours(args):
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
    gpu_index = physical_gpu_index(local_rank)
    peak, peak_kind = peaks()

    sweep_all = args.workload == "all"
    head_name = HEADLINE if sweep_all else args.workload
    cfg = wl.CONFIGS[head_name]
    if args.d:
        cfg = cfg.scaled(name=f"{cfg.name}[d={args.d}]", d=args.d)
    free, _ = torch.cuda.mem_get_info()
    n_sets = args.sets or cfg.steps
    need = (n_sets + 3) * cfg.W * cfg.ld * 4 + (4 << 30)
    notes = []
    if sweep_all and free < need:                          # the largest configuration does not fit this device
        notes.append(f"{head_name} needs {need >> 30} GiB of device memory, {free >> 30} GiB free: headline on C4")
        head_name = "C4"
        cfg = wl.CONFIGS[head_name]
        n_sets = args.sets or cfg.steps

    # ---- per-configuration sweep (N = 1 only; the headline configuration comes last and stays resident) ----
    per_config = {}
    if sweep_all and world == 1:
        reps = max(5, args.reps)
        for name in SWEEP:
            c = wl.CONFIGS[name]
            f, _ = torch.cuda.mem_get_info()
            if f < (c.steps + 2) * c.W * c.ld * 4 + (4 << 30):
                per_config[name] = {"skipped": f"needs more device memory than the {f >> 30} GiB free"}
                continue
            per_config[name] = measure_config(c, dev, args, gpu_index, reps)
        for name in PAPER_SHAPES:
            c = wl.CONFIGS[name]
            f, _ = torch.cuda.mem_get_info()
            if f >= (c.steps + 2) * c.W * c.ld * 4 + (4 << 30):
                per_config[name] = measure_config(c, dev, args, gpu_index, reps)
        if args.faithful_c2:
            fargs = argparse.Namespace(**dict(vars(args), mode="faithful"))
            per_config["C2_faithful"] = measure_config(wl.CONFIGS["C2"], dev, fargs, gpu_index, reps)

    # ---- headline: W warm-up steps, then exactly K steps in one timed region, inputs resident in HBM -----------
    b = Bench(cfg, dev, args, n_sets=n_sets, seed_offset=rep.replica_seed_offset())
    warm = max(3, args.warmup)
    if b.cold:
        for _ in range(-(-warm // (len(b.engines) * cfg.steps))):
            b.sequence()
    else:
        for t in range(warm):
            b.one_step(t)
    assert b.status_ok()
    b.zero_state()
    if b.cold:
        b.flush_buf.fill_(1)
    torch.cuda.synchronize()
    sampler = ClockSampler(gpu_index)
    launches0 = sum(e.launch_count() for e in b.engines)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(); torch.cuda.synchronize()
    sampler.start()
    ev0.record()
    if b.cold:
        for t in range(args.steps):                        # one step (and its zero-out) per set, sets in rotation
            e = t % len(b.engines)
            b.one_step(0, e)
            b.flush(b.engines[e])
    else:
        for t in range(args.steps):
            b.one_step(t)
        b.flush(b.eng)  # the last step's zero-out (deferred into the next step's kernel) is paid inside the region
    ev1.record()
    torch.cuda.synchronize(); barrier()
    clocks = sampler.stop()
    ms_total = ev0.elapsed_time(ev1)
    launches = sum(e.launch_count() for e in b.engines) - launches0
    assert b.status_ok()
    value, ms_step = rep.whole_job_value(cfg.W * cfg.d, ms_total / args.steps)
    stage, stage_n = b.stage_pass()                        # separate pass: stage events stay out of the headline timing
    assert b.status_ok()

    # ---- end to end: host gradients in, host results out, through ssgd_step_host ---------------------------------
    e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": cfg.W * cfg.ld * 4, "d2h_bytes_per_step": 8 * cfg.k}
    g_bytes = cfg.W * cfg.ld * 4
    e2e_steps = 0 if (args.no_e2e or args.mode != "fused") else max(1, min(args.steps, 20 if g_bytes < (2 << 30) else 3))
    if e2e_steps and host_memory_available() < 3 * g_bytes + (8 << 30):
        notes.append(f"end-to-end leg skipped: a pinned host copy of one gradient set ({g_bytes >> 20} MiB) does not "
                     f"fit the host memory this process may take")
        e2e_steps = 0
    if e2e_steps:
        eng = b.eng
        g_host = b.g_sets[0].cpu().pin_memory()
        g_stage = torch.empty_like(b.g_sets[0])
        oi_h = torch.empty(cfg.k, dtype=torch.int32).pin_memory()
        ov_h = torch.empty(cfg.k, dtype=torch.float32).pin_memory()
        b.zero_state()
        eng.step_host(g_host, cfg.rho, cfg.ncand, g_stage, oi_h, ov_h)
        b.zero_state()
        # the plain host-to-device rate of the same buffer, for context
        torch.cuda.synchronize()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record(); g_stage.copy_(g_host, non_blocking=True); c1.record()
        torch.cuda.synchronize()
        h2d_gbs = g_bytes / (c0.elapsed_time(c1) * 1e-3) / 1e9
        barrier(); torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for t in range(e2e_steps):
            eng.step_host(g_host, cfg.rho, cfg.ncand, g_stage, oi_h, ov_h)
        eng.flush()
        e1.record()
        torch.cuda.synchronize(); barrier()
        e2e_ms = rep.max_over_ranks(e0.elapsed_time(e1)) / e2e_steps
        e2e.update({"value": world * cfg.W * cfg.d / (e2e_ms * 1e-3), "steps": e2e_steps, "ms_per_step": e2e_ms,
                    "h2d_gbs_plain_copy": h2d_gbs, "frac_of_plain_copy_rate": (g_bytes / (e2e_ms * 1e-3) / 1e9) / h2d_gbs})
        del g_host, g_stage

    # ---- roofline of the dominant kernel and of the whole step ------------------------------------------------------
    kern = dominant_kernel(cfg)
    k1_ms = stage["accumulate_insert_ms"] if stage else None
    k1_bytes = 20.0 * cfg.W * cfg.d                       # g read; u, v read and written
    k1_gbs = k1_bytes / (k1_ms * 1e-3) / 1e9 if k1_ms else None
    per_unit = NCU_TRAFFIC_BYTES_PER_UNIT.get(kern)
    sb = step_bytes(cfg)
    step_gbs = sb / (ms_step * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "kernel": kern, "achieved": k1_gbs, "peak": peak, "unit": "GB/s",
        "frac": k1_gbs / peak if k1_gbs else None, "peak_source": f"of {peak_kind}",
        "traffic": per_unit * cfg.W * cfg.d if per_unit else None,
        "algorithmic_bytes_per_launch": k1_bytes, "ms_per_launch": k1_ms, "launches_timed": stage_n,
    }
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(cfg, args),
        "clocks": clocks, "gpu_launches": launches, "e2e": e2e, "roofline": roofline,
        "step_hbm": {"algorithmic_bytes_per_step": sb, "achieved": step_gbs, "peak": peak, "unit": "GB/s",
                     "frac": step_gbs / peak, "peak_source": f"of {peak_kind}", "frac_of_8000_nominal": step_gbs / 8000.0},
        "stage_ms": stage,
    }
    if per_config:
        line["per_config"] = per_config
    if notes:
        line["notes"] = notes

    # ---- the oracle beside it (rank 0, N = 1 only): one whole step of C2, every worker, from zero state ---------
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        del b
        torch.cuda.empty_cache()
        ocfg = wl.CONFIGS["C2"] if sweep_all else cfg
        facts = host_facts()
        if ocfg.W * ocfg.d > 2.5e8:                        # keep the leg near 10-30 s of CPU work
            scfg, what = oracle_sample(ocfg, 1.8e8)
        else:
            scfg, what = ocfg, f"the whole {ocfg.name} step: all {ocfg.W} workers, all d={ocfg.d} coordinates, 1 step from zero state"
        g_h = wl.gradients(wl.Structure(scfg, dev), 0).cpu().numpy()
        sec = time_oracle(scfg, g_h, 1)[0]
        cb = {"value": scfg.W * scfg.d / sec, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": what, "seconds": sec}
        cb.update(facts)
        threads = max(1, min(scfg.W, facts["usable_cores"]))
        if threads > 1:
            sec_t = time_oracle_threaded(scfg, g_h, threads)
            cb["threaded_over_workers"] = {
                "value": scfg.W * scfg.d / sec_t, "seconds": sec_t, "cores": threads,
                "what": "Algorithm 3 lines 5-7 one worker per thread (the oracle's plain functions called from "
                        "bench.py's threads), lines 8-13 on one thread"}
        line["cpu_baseline"] = cb
    if rank == 0:
        print(json.dumps(line), flush=True)
    rep.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="all",
                    help="all (default): every configuration, headline on the largest; or one configuration's name")
    ap.add_argument("--reps", type=int, default=5, help="repetitions of each configuration's step sequence (>= 5)")
    ap.add_argument("--mode", choices=["fused", "faithful"], default="fused",
                    help="fused: ssgd_step; faithful: per-worker sketches materialised and merged (stage calls)")
    ap.add_argument("--faithful-c2", action="store_true", default=True,
                    help="also time the faithful pipeline at C2 in the sweep")
    ap.add_argument("--prune", choices=["auto", "off", "on", "early_exit"], default="auto",
                    help="how Algorithm 3 line 9 is evaluated (profiling runs; the default is what a user gets)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--d", type=int, default=0, help="override the number of coordinates (small profiling cases)")
    ap.add_argument("--sets", type=int, default=0, help="resident gradient sets (default: the workload's steps)")
    args = ap.parse_args()
    if args.impl == "reference":
        from paper_1903_04488_b200 import workloads as wl
        cfg = wl.CONFIGS[HEADLINE if args.workload == "all" else args.workload]
        if args.d:
            cfg = cfg.scaled(name=f"{cfg.name}[d={args.d}]", d=args.d)
        run_reference(args, cfg)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
