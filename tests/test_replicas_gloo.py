"""The N > 1 path of the benchmark (independent replicas, barrier, max-over-ranks timing, whole-job
value) exercised with two CPU processes over gloo."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_1903_04488_b200.replicas import Replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    rep = Replicas("gloo")
    rep.barrier()
    local_ms = 2.0 + rank            # rank 1 is the slow one
    value, ms = rep.whole_job_value(1000.0, local_ms)
    rep.barrier()
    out.put((rank, rep.world, value, ms, rep.max_over_ranks(float(rank)), rep.replica_seed_offset()))
    rep.close()


def test_two_replicas_over_gloo():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, w, value, ms, mx, off in got:
        assert w == 2 and ms == 3.0 and mx == 1.0
        assert abs(value - 2 * 1000.0 / 3.0e-3) < 1e-6      # both replicas' units over the slowest time
        assert off == 100 * rank


def test_single_process_needs_no_group():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    rep = Replicas("gloo")
    assert rep.world == 1 and rep.max_over_ranks(5.0) == 5.0
    value, ms = rep.whole_job_value(10.0, 2.0)
    assert ms == 2.0 and value == 5000.0
    rep.barrier()
    rep.close()
    assert not torch.distributed.is_initialized()
