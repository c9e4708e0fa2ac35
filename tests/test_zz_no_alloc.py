"""The workspace-free second round + top-k (ssgd_exact_topk_static) against ssgd_exact_topk and the CPU oracle.

Some users of this library are not allowed to allocate device memory: a gradient-compression hook
that runs inside a trainer whose own allocator holds all of the GPU's memory gets buffers handed in
and nothing else, and an allocation on a latency-critical path would stall the whole device anyway.
They cannot give ssgd_bind a workspace, so ssgd_exact_topk_static keeps its scratch in a fixed array
inside the library.  That array is shared by every call and keeps the previous call's contents, which
is why this test calls the entry point twice in a row, on different inputs, and wants both results to
match the workspace-based entry point exactly (the work is integer selection on identically computed
sums, so the comparison is bit for bit, as in the other parity tests) -- and, because the two entry points
share kernels, the oracle's own second round and final top-k (Algorithm 3 lines 10-11) as well.

Collected last on purpose (file name): if it fails, a run that stops at the first failure has already
run every other test.  It does not depend on them: it passes alone in a fresh process too.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_1903_04488_b200 import ssgd as S
from paper_1903_04488_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def reference_topk(cfg, v, cand, dev):
    """out_idx, out_val of the existing entry point, run on copies so that its zero-out touches nothing."""
    eng = S.Ssgd(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
    u2, v2 = torch.zeros_like(v), v.clone()
    eng.bind(u2, v2, cand.numel())
    out_idx = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    out_val = torch.empty(cfg.k, dtype=torch.float32, device=dev)
    eng.exact_topk(cand, out_idx, out_val)
    assert eng.status() == S.OK
    return out_idx, out_val


def test_static_entry_point_matches_workspace_entry_point_twice(cuda_device):
    dev = cuda_device
    cfg = wl.C2.scaled(d=400_003, W=6, c=8192, ncand=9000, k=3000)
    st = wl.Structure(cfg, dev)
    gen = torch.Generator(device=dev).manual_seed(99)
    for call in range(2):
        # a different state and a different, larger-then-smaller candidate list each time: stale
        # histogram, counter or sum contents from the first call would change the second result
        v = wl.gradients(st, call) * (1.0 + call)
        ncand = cfg.ncand if call == 0 else cfg.ncand // 2 + 1
        cand = torch.randperm(cfg.d, generator=gen, device=dev)[:ncand].sort().values.to(torch.int32)
        v_before = v.clone()
        out_idx = torch.full((cfg.k,), -1, dtype=torch.int32, device=dev)
        out_val = torch.full((cfg.k,), float("nan"), dtype=torch.float32, device=dev)
        S.exact_topk_static(v, cfg.d, cand, cfg.k, out_idx, out_val)
        torch.cuda.synchronize()
        want_idx, want_val = reference_topk(cfg, v, cand, dev)
        assert torch.equal(out_idx, want_idx)
        assert torch.equal(out_val.view(torch.int32), want_val.view(torch.int32))
        assert torch.equal(v, v_before)          # this entry point never writes the state
        # Algorithm 3 lines 10-11 as the oracle states them, on the same v and candidates
        orc = Oracle(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
        cand_h = cand.cpu().numpy()
        xs = orc.second_round(v.cpu().numpy(), cand_h)
        o_idx, o_val = orc.final_topk(cand_h, xs)
        order = np.argsort(o_idx)
        assert (out_idx.cpu().numpy() == o_idx[order]).all()
        assert (out_val.cpu().numpy().view(np.uint32) == o_val[order].view(np.uint32)).all()


def test_static_entry_point_counts_an_out_of_range_candidate_as_zero(cuda_device):
    """A candidate outside [0, d) is never dereferenced: its sum counts as 0, the rest is unchanged."""
    dev = cuda_device
    cfg = wl.C2.scaled(d=50_001, W=3, c=1024, ncand=600, k=100)
    v = wl.gradients(wl.Structure(cfg, dev), 0)
    cand = torch.arange(0, 3 * cfg.ncand, 3, dtype=torch.int32, device=dev)
    bad = cand.clone()
    bad[7] = cfg.d + 123
    bad[8] = -5
    out = []
    for c in (cand, bad):
        oi = torch.empty(cfg.k, dtype=torch.int32, device=dev)
        ov = torch.empty(cfg.k, device=dev)
        S.exact_topk_static(v, cfg.d, c, cfg.k, oi, ov)
        torch.cuda.synchronize()
        out.append((oi.cpu().numpy(), ov.cpu().numpy()))
    orc = Oracle(cfg.d, cfg.r, cfg.c, cfg.k, cfg.W, cfg.sketch_seed)
    xs = orc.second_round(v.cpu().numpy(), cand.cpu().numpy())
    xs_bad = xs.copy()
    xs_bad[[7, 8]] = 0.0
    for (gi, gv), x, c in zip(out, (xs, xs_bad), (cand, bad)):
        o_idx, o_val = orc.final_topk(c.cpu().numpy(), x)
        pos = {int(i): n for n, i in enumerate(c.cpu().numpy())}
        order = np.argsort([pos[int(i)] for i in o_idx])     # outputs come in cand_idx order
        assert (gi == o_idx[order]).all() and (gv.view(np.uint32) == o_val[order].view(np.uint32)).all()


def test_static_entry_point_rejects_what_it_cannot_hold(cuda_device):
    dev = cuda_device
    lib = S.lib()
    d, W = S.STATIC_MAX_NCAND + 10, 1
    v = torch.zeros((W, d + 2), device=dev)
    cand = torch.arange(d, dtype=torch.int32, device=dev)
    oi = torch.empty(4, dtype=torch.int32, device=dev)
    ov = torch.empty(4, device=dev)
    with pytest.raises(S.SsgdError) as e:
        S.exact_topk_static(v, d, cand, 4, oi, ov)                       # ncand beyond the fixed capacity
    assert e.value.code == S.ETOOBIG
    assert b"capacity" in lib.ssgd_strerror(S.ETOOBIG)
    small = cand[:100].contiguous()
    args = lambda **kw: dict(dict(v=v.data_ptr(), ld=d + 2, W=W, d=d, cand=small.data_ptr(), ncand=100, k=4,
                                  oi=oi.data_ptr(), ov=ov.data_ptr()), **kw)
    for bad in (dict(v=None), dict(cand=None), dict(oi=None), dict(k=0), dict(k=101), dict(ld=d - 1), dict(W=0),
                dict(ncand=d + 1)):
        a = args(**bad)
        code = lib.ssgd_exact_topk_static(a["v"], a["ld"], a["W"], a["d"], a["cand"], a["ncand"], a["k"], a["oi"],
                                          a["ov"], None)
        assert code == S.EINVAL
    # at the capacity limit itself the call is accepted and selects the planted maxima
    n = S.STATIC_MAX_NCAND
    v.zero_()
    v[0, 5] = 3.0
    v[0, n - 1] = -7.0
    cand_full = torch.arange(n, dtype=torch.int32, device=dev)
    oi2 = torch.empty(2, dtype=torch.int32, device=dev)
    ov2 = torch.empty(2, device=dev)
    S.exact_topk_static(v, d, cand_full, 2, oi2, ov2)
    torch.cuda.synchronize()
    assert oi2.tolist() == [5, n - 1] and ov2.tolist() == [3.0, -7.0]
